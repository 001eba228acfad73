"""CPU oracle for the MoQAE inference hot path.  TEST INFRASTRUCTURE ONLY.

This module is the slow, plain reference that the CUDA library is checked
against.  It is written from the paper's definitions (Section 3.1 overview,
Section 3.2 Eq. 1 and Eq. 2, Section 3.4 routing freezing / routing sharing,
and the Limitations section's "dequantise, then attend in high precision") and
from the storage format fixed in this repository.  It shares no code with the
CUDA path and must never be imported by the product package: only the tests,
the smoke check and the benchmark's CPU-baseline leg may call it.

Arithmetic: the router and attention are evaluated in float64 from the exact
values of the 16-bit inputs.  The quantiser follows a fixed sequence of
single IEEE binary32 operations (stated in `quantize_groups`) so that integer
codes and packed words have exactly one correct value.

Parity pins (see tests, all CPU-only):
  * attention   - pinned (textbook softmax attention, library SDPA, invariants)
  * quantiser   - pinned (error bound, brute force over fp16 pairs, lossless
                  integer case, constant groups)
  * packing     - pinned (closed-form sizes, independent bit-position check,
                  round trip)
  * router      - pinned (hand-built score matrices with every tie pattern,
                  brute force, library GEMV in linear mode); the paper prints
                  no worked example, so beyond these definitional pins the
                  router and quantiser are "parity unpinned by the paper".

Input convention: 16-bit tensors arrive as numpy uint16 bit patterns plus a
dtype flag (0 = IEEE fp16, 1 = bfloat16), because numpy has no bfloat16.
"""
from __future__ import annotations

import numpy as np

EXPERT_BITS = (2, 4, 8, 16)      # expert index -> bit width (ascending)
N_EXPERTS = 4
HEAD_DIM = 128
GROUP = 32                        # quantisation group length
TILE_TOKENS = 32                  # tokens per storage tile (= one key group)
META_BYTES = 1024                 # per quantised tile
DT_FP16 = 0
DT_BF16 = 1


# ----------------------------------------------------------------------------
# exact conversions
# ----------------------------------------------------------------------------
def to_f32(u16: np.ndarray, dtype: int) -> np.ndarray:
    """Exact value of fp16 / bf16 bit patterns as float32."""
    u16 = np.ascontiguousarray(u16, dtype=np.uint16)
    if dtype == DT_FP16:
        return u16.view(np.float16).astype(np.float32)
    if dtype == DT_BF16:
        return (u16.astype(np.uint32) << np.uint32(16)).view(np.float32)
    raise ValueError("dtype must be 0 (fp16) or 1 (bf16)")


def to_f64(u16: np.ndarray, dtype: int) -> np.ndarray:
    return to_f32(u16, dtype).astype(np.float64)


def fp16_round_down(x32: np.ndarray) -> np.ndarray:
    """Largest fp16 value <= x (x float32)."""
    x32 = np.asarray(x32, dtype=np.float32)
    with np.errstate(over="ignore"):
        h = x32.astype(np.float16)                      # round to nearest even
    too_big = h.astype(np.float32) > x32
    return np.where(too_big, np.nextafter(h, np.float16(-np.inf)), h).astype(np.float16)


def fp16_round_up(x32: np.ndarray) -> np.ndarray:
    """Smallest fp16 value >= x (x float32)."""
    x32 = np.asarray(x32, dtype=np.float32)
    with np.errstate(over="ignore"):
        h = x32.astype(np.float16)
    too_small = h.astype(np.float32) < x32
    return np.where(too_small, np.nextafter(h, np.float16(np.inf)), h).astype(np.float16)


# ----------------------------------------------------------------------------
# Router: Eq. 1, Eq. 2, routing freezing, routing sharing
# ----------------------------------------------------------------------------
def router_logits(x64: np.ndarray, W1: np.ndarray, W2=None, W3=None, bias=None) -> np.ndarray:
    """Eq. 1 per token, float64.

    x64 [n, D]; W1, W2 [D, M]; W3 [M, M]; bias [M] (all float64).
    Gated form (W2 and W3 given):  P = f((x W1) * (x W2)) W3 + bias with
    f = SiLU applied AFTER the element-wise product, as Eq. 1 is written.
    Linear form (W2 = W3 = None):  P = x W1 + bias.
    No softmax: argmax over probabilities equals argmax over logits.
    """
    u = x64 @ W1
    if W2 is None:
        if W3 is not None:
            raise ValueError("W3 without W2")
        P = u
    else:
        a = u * (x64 @ W2)
        h = a / (1.0 + np.exp(-a))          # SiLU(a) = a * sigmoid(a)
        P = h @ W3
    if bias is not None:
        P = P + np.asarray(bias, dtype=np.float64)
    return P


def token_experts(P: np.ndarray) -> np.ndarray:
    """Per-token top-1 (Section 3.2): first index of the row maximum."""
    return np.argmax(P, axis=1).astype(np.int64)    # numpy argmax = first occurrence


def chunk_vote(e: np.ndarray, n_experts: int = N_EXPERTS):
    """Eq. 2 for one chunk: histogram of token choices, winner = first maximum."""
    votes = np.zeros(n_experts, dtype=np.int32)
    for k in e:
        votes[int(k)] += 1
    return votes, int(np.argmax(votes))


def route(hidden_u16: np.ndarray, dtype: int, chunk: int, W1_u16, W2_u16=None, W3=None,
          bias=None, rf_first_chunk: bool = True):
    """Bit-width map of one routing-sharing group.

    hidden_u16 [B, T, D_in]; W1_u16/W2_u16 [D_in, M] in the same 16-bit dtype;
    W3 [M, M] and bias [M] float32.
    Returns dict(map uint8 [B, C], votes int32 [B, C, M], token_expert [B, C*N],
    margin float64 [B, C*N] (top-1 minus top-2 logit), pmax float64 [B, C*N]).
    C = T // chunk; the T mod chunk trailing tokens are never routed (they stay
    in the 16-bit tail, Section 3.2).  With routing freezing the first chunk
    is fixed to the 16-bit expert without consulting the router (Section 3.4);
    its votes row is all zero.
    """
    B, T, D = hidden_u16.shape
    C = T // chunk
    W1 = to_f64(W1_u16, dtype)
    W2 = None if W2_u16 is None else to_f64(W2_u16, dtype)
    W3_ = None if W3 is None else np.asarray(W3, dtype=np.float32).astype(np.float64)
    b_ = None if bias is None else np.asarray(bias, dtype=np.float32).astype(np.float64)
    M = W1.shape[1]
    bmap = np.zeros((B, C), dtype=np.uint8)
    votes = np.zeros((B, C, M), dtype=np.int32)
    tok = np.full((B, C * chunk), -1, dtype=np.int64)
    margin = np.full((B, C * chunk), np.inf)
    pmax = np.zeros((B, C * chunk))
    for b in range(B):
        for c in range(C):
            if c == 0 and rf_first_chunk:
                bmap[b, c] = M - 1          # the 16-bit expert is the last one
                continue
            x = to_f64(hidden_u16[b, c * chunk:(c + 1) * chunk], dtype)
            P = router_logits(x, W1, W2, W3_, b_)
            e = token_experts(P)
            v, r = chunk_vote(e, M)
            bmap[b, c] = r
            votes[b, c] = v
            tok[b, c * chunk:(c + 1) * chunk] = e
            srt = np.sort(P, axis=1)
            margin[b, c * chunk:(c + 1) * chunk] = srt[:, -1] - srt[:, -2]
            pmax[b, c * chunk:(c + 1) * chunk] = np.max(np.abs(P), axis=1)
    return dict(map=bmap, votes=votes, token_expert=tok, margin=margin, pmax=pmax)


def reachable_winners(votes_row: np.ndarray, fragile_tokens_experts, fragile_alt):
    """Winners a chunk can reach when each fragile token may flip to its runner-up.

    votes_row [M]; fragile_tokens_experts / fragile_alt: lists of the current and
    the runner-up expert of each fragile token.  Exact for any number of tokens:
    the set of reachable vote vectors is grown token by token (a token either keeps
    its expert or moves its vote to the runner-up), and every vector's winner under
    the tie rule of Eq. 2 (first maximum) is collected.
    """
    states = {tuple(int(v) for v in votes_row)}
    for cur, alt in zip(fragile_tokens_experts, fragile_alt):
        moved = set()
        for v in states:
            w = list(v)
            w[cur] -= 1
            w[alt] += 1
            moved.add(tuple(w))
        states |= moved
    return {int(np.argmax(np.asarray(v))) for v in states}


def layer_group(layer: int, rs_group: int) -> int:
    """Routing sharing (Section 3.4): blocks are partitioned into runs of
    rs_group consecutive blocks; every block of a run uses the map of the run's
    first block.  A short last run is allowed."""
    return layer // rs_group


def n_groups(n_layers: int, rs_group: int) -> int:
    return (n_layers + rs_group - 1) // rs_group


def assign_slots(bmap: np.ndarray, n_experts: int = N_EXPERTS):
    """Chunk index table: slot of chunk c = number of earlier chunks of the same
    sequence with the same width.  bmap [B, C] -> slot int32 [B, C], count [B, M]."""
    B, C = bmap.shape
    slot = np.zeros((B, C), dtype=np.int32)
    count = np.zeros((B, n_experts), dtype=np.int32)
    for b in range(B):
        for c in range(C):
            w = int(bmap[b, c])
            slot[b, c] = count[b, w]
            count[b, w] += 1
    return slot, count


# ----------------------------------------------------------------------------
# Quantiser (group-wise asymmetric min-max, group 32)
# ----------------------------------------------------------------------------
def quantize_groups(x32: np.ndarray, bits: int):
    """Quantise along the LAST axis (one group: 32 elements, or the 8 / 16 tokens of a
    short chunk for key groups, see `quantize_tile`).

    Canonical sequence; "binary32" steps are single IEEE operations rounded to
    nearest even unless a direction is stated:
        mn, mx   exact minimum / maximum of the group
        z  = largest fp16 <= mn, with -0 stored as +0        (stored zero)
        r  = mx - float(z)                                    (binary32)
        s  = smallest fp16 >= r / (2^bits - 1)                (binary32 division; stored scale)
        if s == 0: every code is 0
        inv = 1 / float(s)                                    (binary32)
        d   = x - float(z)                                    (binary32)
        code = min(2^bits - 1, max(0, rint(d * inv)))
    where d * inv is the EXACT product of the two binary32 numbers (it has at most
    48 significant bits, so float64 holds it exactly) and rint rounds it to the
    nearest integer, halves to even.  Returns (scale fp16, zero fp16, codes uint8).
    Dequantised value (defined, not computed here): code * s + z.
    """
    x32 = np.asarray(x32, dtype=np.float32)
    assert 1 <= x32.shape[-1] <= GROUP        # key groups of chunks shorter than 32 tokens are shorter
    qmax = np.float32((1 << bits) - 1)
    mn = x32.min(axis=-1)
    mx = x32.max(axis=-1)
    z = fp16_round_down(mn)
    z = np.where(z == 0, np.float16(0.0), z).astype(np.float16)     # -0 -> +0
    zf = z.astype(np.float32)
    r = (mx - zf).astype(np.float32)
    s = fp16_round_up((r / qmax).astype(np.float32))
    sf = s.astype(np.float32)
    with np.errstate(divide="ignore", invalid="ignore", over="ignore"):
        inv = (np.float32(1.0) / sf).astype(np.float32)
        d = (x32 - zf[..., None]).astype(np.float32)
        t = d.astype(np.float64) * inv[..., None].astype(np.float64)   # exact
        c = np.rint(t)
    c = np.minimum(np.float64(qmax), np.maximum(0.0, c))
    c = np.where((sf == 0)[..., None], 0.0, c)
    return s, z, c.astype(np.uint8)


def quantize_tile(K32: np.ndarray, V32: np.ndarray, bits: int):
    """One tile: K32, V32 float32 [32 tokens, 128 channels].

    Keys: one group per channel over the tile's 32 tokens (per-channel inside
    the chunk).  Values: one group per token over 32 consecutive channels.
    Returns dict with k_scale/k_zero fp16 [128], k_codes uint8 [32,128],
    v_scale/v_zero fp16 [4, 32] ([channel group, token]), v_codes uint8 [32,128].
    """
    n = K32.shape[0]
    assert K32.shape == (n, HEAD_DIM) and V32.shape == (n, HEAD_DIM) and n in (8, 16, TILE_TOKENS)
    ks, kz, kc = quantize_groups(K32.T, bits)                   # [128, n] groups over the tile's tokens
    vg = V32.reshape(n, HEAD_DIM // GROUP, GROUP)               # [n, 4, 32]
    vs, vz, vc = quantize_groups(vg, bits)                      # vs [n, 4]
    t = dict(k_scale=ks, k_zero=kz, k_codes=np.ascontiguousarray(kc.T),
             v_scale=np.ascontiguousarray(vs.T), v_zero=np.ascontiguousarray(vz.T),
             v_codes=vc.reshape(n, HEAD_DIM))
    if n < TILE_TOKENS:
        # A chunk of 8 or 16 tokens (the small chunk sizes of the paper's chunk-size ablation) is
        # one tile whose remaining token positions are padding: codes 0, value scale / zero 0.
        # Its key groups are the chunk's own tokens of one channel ("per channel within the
        # chunk" with fewer than 32 tokens to group).
        pad = TILE_TOKENS - n
        t["k_codes"] = np.concatenate([t["k_codes"], np.zeros((pad, HEAD_DIM), np.uint8)])
        t["v_codes"] = np.concatenate([t["v_codes"], np.zeros((pad, HEAD_DIM), np.uint8)])
        t["v_scale"] = np.concatenate([t["v_scale"], np.zeros((HEAD_DIM // GROUP, pad), np.float16)], axis=1)
        t["v_zero"] = np.concatenate([t["v_zero"], np.zeros((HEAD_DIM // GROUP, pad), np.float16)], axis=1)
    return t


def tile_tokens(chunk: int) -> int:
    """Token positions of a tile that hold tokens: 32, or the whole chunk if it is shorter."""
    return min(chunk, TILE_TOKENS)


def tiles_per_chunk(chunk: int) -> int:
    return max(1, chunk // TILE_TOKENS)


def dequantize_tile(t: dict):
    """float64 K̂, V̂ [32, 128] of a quantised tile: code * scale + zero."""
    Kh = t["k_codes"].astype(np.float64) * t["k_scale"].astype(np.float64)[None, :] \
        + t["k_zero"].astype(np.float64)[None, :]
    vs = np.repeat(t["v_scale"].astype(np.float64).T, GROUP, axis=1)   # [32 tok, 128]
    vz = np.repeat(t["v_zero"].astype(np.float64).T, GROUP, axis=1)
    Vh = t["v_codes"].astype(np.float64) * vs + vz
    return Kh, Vh


# ----------------------------------------------------------------------------
# Storage format
# ----------------------------------------------------------------------------
# A quantised tile (32 tokens x 128 channels of one kv head, b = 2, 4 or 8 bits)
# is 1024 + 1024*b bytes:
#   [   0,  256)  key scale    fp16 x 128
#   [ 256,  512)  key zero     fp16 x 128
#   [ 512,  768)  value scale  fp16 x 128   (4 channel groups x 32 tokens)
#   [ 768, 1024)  value zero   fp16 x 128
#   [1024, 1024 + 512 b)            key payload
#   [1024 + 512 b, 1024 + 1024 b)   value payload
# Inside each part the order is the one in which the decode kernel's 32 lanes
# consume the data; the functions below state it element by element.
def tile_bytes(bits: int) -> int:
    """Bytes of one 32-token tile of one kv head (K and V together)."""
    return 16384 if bits == 16 else META_BYTES + 2 * TILE_TOKENS * 16 * bits


def slot_bytes(bits: int, chunk: int) -> int:
    """A chunk of 32 j tokens is j tiles; a chunk of 8 or 16 tokens is one (padded) tile."""
    return max(1, chunk // TILE_TOKENS) * tile_bytes(bits)


def key_code_location(t: int, c: int, bits: int):
    """(byte offset inside the key payload, bit offset inside that byte) of the
    code of token row t, channel c.

    Token t = 16*blk + 8*hh + g, channel c = 32*q + cc.  The 32 codes of one
    (t, q) form a piece of 4*bits bytes, code cc at bits [bits*cc, bits*cc+bits)
    of the piece taken as a little-endian bit string.  Pieces live in 16-byte
    units, unit index:
        bits 2:  32*blk + 4*g + q,                     hh selects bytes [8hh, 8hh+8)
        bits 4:  32*(2*blk + hh) + 4*g + q
        bits 8:  32*(2*(2*blk + hh) + j) + 4*g + q,    j = which 16 bytes of the piece
    """
    blk, hh, g = t >> 4, (t >> 3) & 1, t & 7
    q, cc = c >> 5, c & 31
    byte_in_piece, bit = (cc * bits) >> 3, (cc * bits) & 7
    if bits == 2:
        return (32 * blk + 4 * g + q) * 16 + 8 * hh + byte_in_piece, bit
    if bits == 4:
        return (32 * (2 * blk + hh) + 4 * g + q) * 16 + byte_in_piece, bit
    if bits == 8:
        return (32 * (2 * (2 * blk + hh) + (byte_in_piece >> 4)) + 4 * g + q) * 16 + (byte_in_piece & 15), bit
    raise ValueError("bits")


def value_code_location(t: int, c: int, bits: int):
    """(byte offset of the little-endian 32-bit word inside the value payload,
    bit offset inside that word) of the code of token row t, channel c.

    Token t = 16*blk + 8*half + 2*t4 + e, channel c = 32*cg + 4*g + r4.
    Lane ln = 4*g + t4 owns, per blk, the 16 channel rows R = 4*cg + r4; row R
    sits in word w = R*bits/8 of the lane at slot R mod (8/bits); the code is at
    bit  bits*slot + 8*half + 16*e.  Words are grouped in 16-byte units per lane:
    byte offset = ((blk*(bits/2) + w/4)*32 + ln)*16 + (w mod 4)*4.
    """
    blk, half, t4, e = t >> 4, (t >> 3) & 1, (t >> 1) & 3, t & 1
    cg, g, r4 = c >> 5, (c >> 2) & 7, c & 3
    R = 4 * cg + r4
    w, slot = (R * bits) >> 3, R % (8 // bits)
    ln = 4 * g + t4
    return ((blk * (bits // 2) + (w >> 2)) * 32 + ln) * 16 + (w & 3) * 4, bits * slot + 8 * half + 16 * e


def key_meta_index(c: int, bits: int) -> int:
    """Halfword index of channel c in the key scale (and key zero) array.

    With n = 32/bits codes per 32-bit payload word, channel c = 32*q + cc sits in
    word j = cc / n at position i = cc mod n.  Positions i and i + n/2 share a
    register of the decode kernel (low / high half); of the n/2 registers of a
    word the first n/4 come from the word itself, the others from the word
    shifted right by 8 bits.  Register number r = j*(n/2) + s*(n/4) + m with
    i mod (n/2) = s*(n/4) + m; index = ((r/4)*4 + q)*8 + (r mod 4)*2 + (i >= n/2).
    """
    n = 32 // bits
    q, cc = c >> 5, c & 31
    j, i = cc // n, cc % n
    hi, i2 = int(i >= n // 2), i % (n // 2)
    s_, m = i2 // (n // 4), i2 % (n // 4)
    r = j * (n // 2) + s_ * (n // 4) + m
    return ((r >> 2) * 4 + q) * 8 + (r & 3) * 2 + hi


def key_zero_index(c: int, bits: int) -> int:
    """Halfword index of channel c in the key zero array: as `key_meta_index`, but
    inside each group of four registers the registers are stored in the order
    0, 2, 1, 3 (so that registers r and r + 2 are neighbours)."""
    i = key_meta_index(c, bits)
    r4 = (i >> 1) & 3
    return (i & ~6) | ((0, 2, 1, 3)[r4] << 1)


def value_scale_index(cg: int, t: int) -> int:
    """Halfword index of (channel group cg, token t) in the value scale array;
    t = 16*blk + 8*half + 2*t4 + e."""
    blk, half, t4, e = t >> 4, (t >> 3) & 1, (t >> 1) & 3, t & 1
    return ((((blk * 2 + (cg >> 1)) * 4 + t4) * 4 + (cg & 1) * 2 + half) * 2) + e


def value_zero_index(cg: int, t: int) -> int:
    """Halfword index of (channel group cg, token t) in the value zero array."""
    blk, half, t4, e = t >> 4, (t >> 3) & 1, (t >> 1) & 3, t & 1
    return ((((blk * 4 + cg) * 4 + t4) * 2 + half) * 2) + e


def raw_location(c: int, t: int) -> int:
    """Byte offset of channel c in a 256-byte raw (16-bit) row of token row t:
    16-byte unit U = c // 8 stored at (U & 8) | ((U xor t) & 7)."""
    U = c >> 3
    Up = (U & 8) | ((U ^ t) & 7)
    return Up * 16 + (c & 7) * 2


_TABLES = {}


def _tables(bits: int):
    """Index tables built from the location functions, cached (pure bookkeeping):
    32-bit word index and shift of every key / value code, halfword index of
    every metadata entry."""
    if bits in _TABLES:
        return _TABLES[bits]
    kw = np.zeros((TILE_TOKENS, HEAD_DIM), dtype=np.int64)
    ks = np.zeros((TILE_TOKENS, HEAD_DIM), dtype=np.uint32)
    vw = np.zeros((TILE_TOKENS, HEAD_DIM), dtype=np.int64)
    vs = np.zeros((TILE_TOKENS, HEAD_DIM), dtype=np.uint32)
    for t in range(TILE_TOKENS):
        for c in range(HEAD_DIM):
            byte, bit = key_code_location(t, c, bits)
            kw[t, c], ks[t, c] = byte // 4, 8 * (byte % 4) + bit
            byte, bit = value_code_location(t, c, bits)
            vw[t, c], vs[t, c] = byte // 4, bit
    km = np.array([key_meta_index(c, bits) for c in range(HEAD_DIM)], dtype=np.int64)
    kz = np.array([key_zero_index(c, bits) for c in range(HEAD_DIM)], dtype=np.int64)
    vsi = np.array([[value_scale_index(cg, t) for t in range(TILE_TOKENS)] for cg in range(4)], dtype=np.int64)
    vzi = np.array([[value_zero_index(cg, t) for t in range(TILE_TOKENS)] for cg in range(4)], dtype=np.int64)
    _TABLES[bits] = (kw, ks, vw, vs, km, kz, vsi, vzi)
    return _TABLES[bits]


def _raw_table():
    if "raw" not in _TABLES:
        off = np.zeros((TILE_TOKENS, HEAD_DIM), dtype=np.int64)
        for t in range(TILE_TOKENS):
            for c in range(HEAD_DIM):
                off[t, c] = (t * 256 + raw_location(c, t)) // 2
        _TABLES["raw"] = off
    return _TABLES["raw"]


def _pack_payload(codes: np.ndarray, word: np.ndarray, shift: np.ndarray, bits: int) -> np.ndarray:
    out = np.zeros(TILE_TOKENS * 4 * bits, dtype=np.uint32)
    np.bitwise_or.at(out, word.ravel(), (codes.astype(np.uint32) << shift).ravel())
    return out.view(np.uint8)


def _unpack_payload(payload_u8: np.ndarray, word: np.ndarray, shift: np.ndarray, bits: int) -> np.ndarray:
    w = np.ascontiguousarray(payload_u8).view(np.uint32)
    return ((w[word] >> shift) & np.uint32((1 << bits) - 1)).astype(np.uint8)


def pack_tile(t: dict, bits: int) -> np.ndarray:
    """Quantised tile (as returned by `quantize_tile`) -> bytes in the storage format."""
    kw, ks, vw, vs, km, kz, vsi, vzi = _tables(bits)
    out = np.zeros(tile_bytes(bits), dtype=np.uint8)
    h = out[:META_BYTES].view(np.uint16)
    h[0 + km] = np.asarray(t["k_scale"], dtype=np.float16).view(np.uint16)
    h[128 + kz] = np.asarray(t["k_zero"], dtype=np.float16).view(np.uint16)
    h[256 + vsi] = np.ascontiguousarray(t["v_scale"], dtype=np.float16).view(np.uint16)
    h[384 + vzi] = np.ascontiguousarray(t["v_zero"], dtype=np.float16).view(np.uint16)
    pb = TILE_TOKENS * 16 * bits
    out[1024:1024 + pb] = _pack_payload(t["k_codes"], kw, ks, bits)
    out[1024 + pb:1024 + 2 * pb] = _pack_payload(t["v_codes"], vw, vs, bits)
    return out


def unpack_tile(buf: np.ndarray, bits: int) -> dict:
    kw, ks, vw, vs, km, kz, vsi, vzi = _tables(bits)
    buf = np.ascontiguousarray(buf, dtype=np.uint8)
    pb = TILE_TOKENS * 16 * bits
    h = buf[:META_BYTES].view(np.uint16)
    return dict(k_scale=h[0 + km].view(np.float16).copy(), k_zero=h[128 + kz].view(np.float16).copy(),
                v_scale=h[256 + vsi].view(np.float16).copy(), v_zero=h[384 + vzi].view(np.float16).copy(),
                k_codes=_unpack_payload(buf[1024:1024 + pb], kw, ks, bits),
                v_codes=_unpack_payload(buf[1024 + pb:1024 + 2 * pb], vw, vs, bits))


def pack_raw_tile(K_u16: np.ndarray, V_u16: np.ndarray) -> np.ndarray:
    """16-bit tile: K rows then V rows, input bit patterns, swizzled units."""
    off = _raw_table()
    out = np.zeros(16384 // 2, dtype=np.uint16)
    out[off.ravel()] = K_u16.ravel()
    out[4096 + off.ravel()] = V_u16.ravel()
    return out.view(np.uint8)


def unpack_raw_tile(buf: np.ndarray):
    off = _raw_table()
    w = np.ascontiguousarray(buf, dtype=np.uint8).view(np.uint16)
    return w[off], w[4096 + off]


# ----------------------------------------------------------------------------
# Cache construction (prefill): quantise + pack into per-width pools
# ----------------------------------------------------------------------------
def quantize_kv(K_u16: np.ndarray, V_u16: np.ndarray, dtype: int, chunk: int,
                bmap: np.ndarray, capacity=None):
    """K_u16, V_u16 [B, T, H_kv, 128]; bmap uint8 [B, C] (expert index per chunk).

    Returns dict(pools=[4 x uint8 [B, H_kv, capacity_w, slot_bytes_w]],
    slot [B, C], count [B, 4], tail_k/tail_v uint16 [B, H_kv, r, 128], tail_len r).
    Chunk c of sequence b goes to pool[w] slot slot[b, c] for every kv head;
    trailing T mod chunk tokens are kept as raw 16-bit rows (Section 3.2).
    """
    B, T, H, d = K_u16.shape
    assert d == HEAD_DIM and (chunk % TILE_TOKENS == 0 or chunk in (8, 16))
    C = T // chunk
    assert bmap.shape == (B, C)
    slot, count = assign_slots(bmap)
    if capacity is None:
        capacity = [max(1, int(count[:, w].max())) for w in range(N_EXPERTS)]
    pools = [np.zeros((B, H, capacity[w], slot_bytes(EXPERT_BITS[w], chunk)), dtype=np.uint8)
             for w in range(N_EXPERTS)]
    tpc, nt = tiles_per_chunk(chunk), tile_tokens(chunk)
    for b in range(B):
        for c in range(C):
            w = int(bmap[b, c])
            bits = EXPERT_BITS[w]
            tb = tile_bytes(bits)
            for h in range(H):
                for j in range(tpc):
                    t0 = c * chunk + j * TILE_TOKENS
                    Kt = K_u16[b, t0:t0 + nt, h]
                    Vt = V_u16[b, t0:t0 + nt, h]
                    if bits == 16:
                        if nt < TILE_TOKENS:                   # short chunk: zero rows fill the tile
                            zr = np.zeros((TILE_TOKENS - nt, HEAD_DIM), np.uint16)
                            Kt, Vt = np.concatenate([Kt, zr]), np.concatenate([Vt, zr])
                        blob = pack_raw_tile(Kt, Vt)
                    else:
                        blob = pack_tile(quantize_tile(to_f32(Kt, dtype), to_f32(Vt, dtype), bits), bits)
                    pools[w][b, h, slot[b, c], j * tb:(j + 1) * tb] = blob
    r = T - C * chunk
    tail_k = np.ascontiguousarray(np.transpose(K_u16[:, C * chunk:], (0, 2, 1, 3)))
    tail_v = np.ascontiguousarray(np.transpose(V_u16[:, C * chunk:], (0, 2, 1, 3)))
    return dict(pools=pools, slot=slot, count=count, capacity=list(capacity), map=np.array(bmap, dtype=np.uint8),
                tail_k=tail_k, tail_v=tail_v, tail_len=r)


def uniform_quantize_reference(X_u16: np.ndarray, dtype: int, bits: int, per_channel: bool, chunk: int):
    """Stand-alone uniform quantiser over a whole [T, 128] tensor, chunk by chunk,
    used to pin "all chunks routed to one width == uniform quantisation".
    Returns the dequantised float64 tensor for the T//chunk*chunk leading tokens."""
    X = to_f32(X_u16, dtype)
    T = (X.shape[0] // chunk) * chunk
    out = np.zeros((T, HEAD_DIM))
    for t0 in range(0, T, GROUP):
        blk = X[t0:t0 + GROUP]
        if per_channel:
            s, z, c = quantize_groups(blk.T, bits)
            out[t0:t0 + GROUP] = (c.astype(np.float64) * s.astype(np.float64)[:, None]
                                  + z.astype(np.float64)[:, None]).T
        else:
            g = blk.reshape(GROUP, HEAD_DIM // GROUP, GROUP)
            s, z, c = quantize_groups(g, bits)
            out[t0:t0 + GROUP] = (c.astype(np.float64) * s.astype(np.float64)[..., None]
                                  + z.astype(np.float64)[..., None]).reshape(GROUP, HEAD_DIM)
    return out


# ----------------------------------------------------------------------------
# Decode attention over the mixed-precision cache
# ----------------------------------------------------------------------------
def cache_kv_rows(cache: dict, dtype: int, chunk: int, b: int, h: int):
    """All cached rows of (sequence b, kv head h) as float64 K̂, V̂ [n, 128],
    pool by pool then the tail (softmax attention does not depend on key order)."""
    Ks, Vs = [], []
    tpc, nt = tiles_per_chunk(chunk), tile_tokens(chunk)
    for w in range(N_EXPERTS):
        bits = EXPERT_BITS[w]
        tb = tile_bytes(bits)
        for s in range(int(cache["count"][b, w])):
            blob = cache["pools"][w][b, h, s]
            for j in range(tpc):
                tile = blob[j * tb:(j + 1) * tb]
                if bits == 16:
                    Ku, Vu = unpack_raw_tile(tile)
                    Ks.append(to_f64(Ku[:nt], dtype))
                    Vs.append(to_f64(Vu[:nt], dtype))
                else:
                    Kh, Vh = dequantize_tile(unpack_tile(tile, bits))
                    Ks.append(Kh[:nt])
                    Vs.append(Vh[:nt])
    if cache["tail_len"] > 0:
        Ks.append(to_f64(cache["tail_k"][b, h, :cache["tail_len"]], dtype))
        Vs.append(to_f64(cache["tail_v"][b, h, :cache["tail_len"]], dtype))
    if not Ks:
        return np.zeros((0, HEAD_DIM)), np.zeros((0, HEAD_DIM))
    return np.concatenate(Ks, axis=0), np.concatenate(Vs, axis=0)


def softmax_attention(q64: np.ndarray, K64: np.ndarray, V64: np.ndarray, scale: float) -> np.ndarray:
    """out = softmax(scale * K q) V for one query (no mask: a decode query sees
    every cached token).  An empty cache gives zeros."""
    if K64.shape[0] == 0:
        return np.zeros(V64.shape[1])
    s = (K64 @ q64) * scale
    p = np.exp(s - s.max())
    return (p @ V64) / p.sum()


def decode_attn(q_u16: np.ndarray, dtype: int, cache: dict, chunk: int, scale=None) -> np.ndarray:
    """q_u16 [B, H_q, 128] -> float64 out [B, H_q, 128].  Query head h reads kv
    head h // (H_q / H_kv).  Keys are dequantised, then scores, softmax and the
    weighted sum are taken in float64 (Limitations section: dequantise before
    the product with the query)."""
    B, Hq, d = q_u16.shape
    Hkv = cache["pools"][0].shape[1]
    G = Hq // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    q = to_f64(q_u16, dtype)
    out = np.zeros((B, Hq, d))
    for b in range(B):
        for h in range(Hkv):
            K64, V64 = cache_kv_rows(cache, dtype, chunk, b, h)
            for g in range(G):
                out[b, h * G + g] = softmax_attention(q[b, h * G + g], K64, V64, scale)
    return out


def round_to_16bit(x64: np.ndarray, dtype: int) -> np.ndarray:
    """float64 -> bit patterns (uint16) of the nearest fp16 / bf16 value, ties to even, in ONE
    rounding: the value is divided by the spacing of the target format at its magnitude (a power
    of two, so the division is exact), rounded to an integer with rint, and multiplied back."""
    x64 = np.asarray(x64, dtype=np.float64)
    sig, emin = (11, -14) if dtype == DT_FP16 else (8, -126)          # significant bits, smallest normal exponent
    _, e = np.frexp(x64)                                              # |x| = m * 2^e, m in [0.5, 1)
    quantum = np.ldexp(1.0, np.maximum(e, emin + 1) - sig)
    y = np.rint(x64 / quantum) * quantum                              # exactly representable in the target format
    if dtype == DT_FP16:
        return y.astype(np.float16).view(np.uint16)
    return (y.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)


def project_kv(hidden_u16: np.ndarray, Wk_u16: np.ndarray, Wv_u16: np.ndarray, dtype: int, n_kv_heads: int):
    """The key / value projections that feed the quantiser (Section 3.1: the chunks a block
    quantises are its own keys and values): K = hidden Wk^T, V = hidden Wv^T from the exact
    values of the 16-bit inputs in float64, then one rounding to the 16-bit dtype.
    hidden [B, T, D]; Wk, Wv [H_kv * 128, D] -> K_u16, V_u16 [B, T, H_kv, 128]."""
    x = to_f64(hidden_u16, dtype)
    B, T, _ = x.shape
    K64 = x @ to_f64(Wk_u16, dtype).T
    V64 = x @ to_f64(Wv_u16, dtype).T
    shape = (B, T, n_kv_heads, HEAD_DIM)
    return (round_to_16bit(K64, dtype).reshape(shape), round_to_16bit(V64, dtype).reshape(shape),
            K64.reshape(shape), V64.reshape(shape))


def cache_bytes(count: np.ndarray, chunk: int, n_kv_heads: int, tail_len: int) -> int:
    """Closed form of the bytes a cache holds: sum_w count_w * slot_bytes_w per head,
    plus 512 bytes per tail token per head."""
    total = 0
    for b in range(count.shape[0]):
        for w in range(N_EXPERTS):
            total += int(count[b, w]) * slot_bytes(EXPERT_BITS[w], chunk) * n_kv_heads
        total += tail_len * n_kv_heads * 2 * HEAD_DIM * 2
    return total


# ----------------------------------------------------------------------------
# Prefill attention over the quantised chunks (causal)
# ----------------------------------------------------------------------------
def cache_kv_rows_in_order(cache: dict, dtype: int, chunk: int, b: int, h: int):
    """Cached rows of (sequence b, kv head h) in TOKEN order as float64 K̂, V̂ [T, 128]:
    chunk c comes from pool map[b, c], slot slot[b, c]; the tail follows."""
    Ks, Vs = [], []
    tpc, nt = tiles_per_chunk(chunk), tile_tokens(chunk)
    C = cache["map"].shape[1]
    for c in range(C):
        w = int(cache["map"][b, c])
        bits = EXPERT_BITS[w]
        tb = tile_bytes(bits)
        blob = cache["pools"][w][b, h, int(cache["slot"][b, c])]
        for j in range(tpc):
            tile = blob[j * tb:(j + 1) * tb]
            if bits == 16:
                Ku, Vu = unpack_raw_tile(tile)
                Ks.append(to_f64(Ku[:nt], dtype))
                Vs.append(to_f64(Vu[:nt], dtype))
            else:
                Kh, Vh = dequantize_tile(unpack_tile(tile, bits))
                Ks.append(Kh[:nt])
                Vs.append(Vh[:nt])
    if cache["tail_len"] > 0:
        Ks.append(to_f64(cache["tail_k"][b, h, :cache["tail_len"]], dtype))
        Vs.append(to_f64(cache["tail_v"][b, h, :cache["tail_len"]], dtype))
    if not Ks:
        return np.zeros((0, HEAD_DIM)), np.zeros((0, HEAD_DIM))
    return np.concatenate(Ks, axis=0), np.concatenate(Vs, axis=0)


def prefill_attn(q_u16: np.ndarray, dtype: int, cache: dict, chunk: int, scale=None) -> np.ndarray:
    """Causal attention of every prompt position over the cache built from the same prompt
    (Section 3.1: the block quantises its chunks, then "proceeds with the formal calculation";
    Limitations section: keys are dequantised before the product with the query).
    q_u16 [B, T, H_q, 128] -> float64 out [B, T, H_q, 128]; position t sees the dequantised
    rows 0..t of kv head h // (H_q / H_kv)."""
    B, T, Hq, d = q_u16.shape
    Hkv = cache["pools"][0].shape[1]
    G = Hq // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    q = to_f64(q_u16, dtype)
    out = np.zeros((B, T, Hq, d))
    for b in range(B):
        for h in range(Hkv):
            K64, V64 = cache_kv_rows_in_order(cache, dtype, chunk, b, h)
            assert K64.shape[0] == T
            for g in range(G):
                s = (q[b, :, h * G + g] @ K64.T) * scale                       # [T, T]
                s = np.where(np.tri(T, dtype=bool), s, -np.inf)
                p = np.exp(s - s.max(axis=1, keepdims=True))
                out[b, :, h * G + g] = (p @ V64) / p.sum(axis=1, keepdims=True)
    return out
