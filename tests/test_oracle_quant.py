"""Pins for the oracle's quantiser and storage format."""
import numpy as np
import pytest

from oracle import moqae_oracle as O

RS = np.random.RandomState
BITS = (2, 4, 8)


def test_directed_fp16_rounding():
    rs = RS(0)
    x = (rs.randn(20000) * np.exp(rs.randn(20000) * 3)).astype(np.float32)
    dn = O.fp16_round_down(x).astype(np.float32)
    up = O.fp16_round_up(x).astype(np.float32)
    assert (dn <= x).all() and (up >= x).all()
    # tight: the next fp16 towards x overshoots
    assert (np.nextafter(O.fp16_round_down(x), np.float16(np.inf)).astype(np.float32) > x).all()
    assert (np.nextafter(O.fp16_round_up(x), np.float16(-np.inf)).astype(np.float32) < x).all()
    exact = np.float16(1.5)
    assert O.fp16_round_down(np.float32(exact)) == exact and O.fp16_round_up(np.float32(exact)) == exact


@pytest.mark.parametrize("bits", BITS)
@pytest.mark.parametrize("dtype", [0, 1])
def test_error_bound_half_scale(bits, dtype):
    rs = RS(bits * 7 + dtype)
    x = rs.randn(500, 32) * np.exp(rs.randn(500, 1))
    x[::7] *= 10
    if dtype == 0:
        u = x.astype(np.float16).view(np.uint16)
    else:
        u = (x.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    x32 = O.to_f32(u, dtype)
    s, z, c = O.quantize_groups(x32, bits)
    xh = c.astype(np.float64) * s.astype(np.float64)[:, None] + z.astype(np.float64)[:, None]
    err = np.abs(xh - x32.astype(np.float64))
    slack = 4 * np.spacing(np.abs(x32).max(axis=1).astype(np.float32)).astype(np.float64)
    assert (err <= s.astype(np.float64)[:, None] / 2 + slack[:, None]).all()
    qmax = (1 << bits) - 1
    assert c.max() <= qmax
    imin, imax = x32.argmin(1), x32.argmax(1)
    rows = np.arange(len(x32))
    assert (c[rows, imin] == 0).all()
    assert (c[rows, imax] >= qmax - 1).all()
    # covering property: z <= min and z + qmax*s >= max (nothing is clamped away)
    assert (z.astype(np.float32) <= x32.min(1)).all()
    top = z.astype(np.float64) + qmax * s.astype(np.float64)
    assert (top >= x32.max(1).astype(np.float64) - slack).all()


@pytest.mark.parametrize("bits", BITS)
def test_constant_group_exact(bits):
    x = np.full((3, 32), np.float16(-2.75), dtype=np.float32)
    s, z, c = O.quantize_groups(x, bits)
    assert (s == 0).all() and (c == 0).all() and (z == np.float16(-2.75)).all()


def test_eight_bit_lossless_on_integers():
    rs = RS(3)
    x = rs.randint(0, 256, size=(64, 32)).astype(np.float32)
    x[:, 0], x[:, 1] = 0, 255
    s, z, c = O.quantize_groups(x, 8)
    assert (s == 1).all() and (z == 0).all() and (c == x.astype(np.uint8)).all()


def test_two_bit_levels_by_hand():
    # min 0, max 3 -> scale 1, codes are the values; 1.5 rounds to even (2), 0.5 -> 0, 2.5 -> 2
    x = np.zeros((1, 32), np.float32)
    x[0, :6] = [0, 3, 1.5, 0.5, 2.5, 1.0]
    s, z, c = O.quantize_groups(x, 2)
    assert s[0] == 1 and z[0] == 0 and list(c[0, :6]) == [0, 3, 2, 0, 2, 1]


def test_brute_force_two_value_groups_over_fp16_range():
    # groups that hold only two distinct fp16 values (a < b): the low value must get code 0,
    # the high one 2^bits - 1 (or one less after the scale was rounded up), for a dense sweep
    # of fp16 bit patterns including subnormals and large magnitudes.
    pats = np.arange(0, 0x7800, 37, dtype=np.uint16)            # positive finite, < 32768
    vals = np.concatenate([pats.view(np.float16), -pats.view(np.float16)]).astype(np.float32)
    rs = RS(9)
    a = rs.choice(vals, 4000)
    b = rs.choice(vals, 4000)
    lo, hi = np.minimum(a, b), np.maximum(a, b)
    keep = hi > lo
    lo, hi = lo[keep], hi[keep]
    g = np.repeat(lo[:, None], 32, 1)
    g[:, 16:] = hi[:, None]
    for bits in BITS:
        s, z, c = O.quantize_groups(g, bits)
        qmax = (1 << bits) - 1
        assert (z.astype(np.float32) == lo).all()               # fp16 inputs: zero is exact
        assert (c[:, :16] == 0).all()
        normal = s.astype(np.float32) >= 2.0 ** -14       # a subnormal fp16 scale is coarser
        assert (c[normal, 16:] >= qmax - 1).all() and (c[:, 16:] <= qmax).all()
        rec = c[:, 16].astype(np.float64) * s.astype(np.float64) + z.astype(np.float64)
        assert (np.abs(rec - hi) <= s.astype(np.float64) / 2 + 1e-30).all()


def test_scalar_reimplementation_agrees():
    # element-by-element restatement with Python scalars and numpy scalar float32 ops
    rs = RS(11)
    x = (rs.randn(8, 32) * 3).astype(np.float16).astype(np.float32)
    for bits in BITS:
        s, z, c = O.quantize_groups(x, bits)
        for r in range(8):
            mn, mx = min(x[r]), max(x[r])
            zz = np.float16(mn)
            if np.float32(zz) > mn:
                zz = np.nextafter(zz, np.float16(-np.inf))
            q = np.float32(np.float32(mx) - np.float32(zz)) / np.float32((1 << bits) - 1)
            ss = np.float16(q)
            if np.float32(ss) < q:
                ss = np.nextafter(ss, np.float16(np.inf))
            assert ss == s[r] and zz == z[r]
            inv = np.float32(1) / np.float32(ss)
            for i in range(32):
                from fractions import Fraction
                prod = Fraction(float(np.float32(x[r, i] - np.float32(zz)))) * Fraction(float(inv))   # exact
                lo = prod.numerator // prod.denominator
                frac = prod - lo
                code = lo + (1 if frac > Fraction(1, 2) or (frac == Fraction(1, 2) and lo % 2 == 1) else 0)
                code = int(min((1 << bits) - 1, max(0, code)))
                assert code == c[r, i]


def test_negative_zero_minimum_is_stored_as_plus_zero():
    x = np.zeros((1, 32), np.float32)
    x[0, 0] = -0.0
    x[0, 1] = 1.0
    for bits in BITS:
        s_, z, c = O.quantize_groups(x, bits)
        assert z.view(np.uint16)[0] == 0x0000 and c[0, 1] == (1 << bits) - 1 and c[0, 0] == 0


@pytest.mark.parametrize("bits", BITS)
def test_codes_never_need_the_clamp(bits):
    """z <= min and s >= (max - z)/(2^b - 1) up to one binary32 rounding, so the rounded
    product already lies in [0, 2^b - 1]: the clamp of the definition is never active on
    finite inputs (checked on wide-range random groups and on groups built to sit at the edge)."""
    rs = RS(40 + bits)
    qmax = (1 << bits) - 1
    x = np.clip(rs.randn(4000, 32) * np.exp(rs.randn(4000, 1) * 4), -32000, 32000).astype(np.float16).astype(np.float32)
    edge = np.zeros((2000, 32), np.float32)
    step = np.clip(np.exp(rs.randn(2000) * 3), 1e-7, 60.0).astype(np.float16).astype(np.float32)
    edge[:, 1] = step * qmax                   # max exactly qmax steps above the minimum
    edge[:, 2:] = (rs.randint(0, 2 * qmax + 1, (2000, 30)) * 0.5).astype(np.float32) * step[:, None]
    for g in (x, edge, -edge):
        s_, z, c = O.quantize_groups(g, bits)
        zf, sf = z.astype(np.float32), s_.astype(np.float32)
        ok = sf > 0
        inv = (np.float32(1) / sf[ok]).astype(np.float32)
        d = (g[ok] - zf[ok, None]).astype(np.float32)
        raw = np.rint(d.astype(np.float64) * inv[:, None].astype(np.float64))
        assert raw.min() >= 0 and raw.max() <= qmax
        assert (raw == c[ok]).all()


def test_tile_group_orientation():
    # keys: groups run over tokens for a fixed channel; values: over 32 channels of a token
    K = np.zeros((32, 128), np.float32)
    V = np.zeros((32, 128), np.float32)
    K[:, 5] = np.arange(32)                 # only channel 5 varies over tokens
    V[7, 64:96] = np.arange(32)             # only token 7, channel group 2 varies
    t = O.quantize_tile(K, V, 8)
    assert t["k_scale"].shape == (128,) and t["v_scale"].shape == (4, 32)
    assert np.count_nonzero(t["k_scale"]) == 1 and t["k_scale"][5] > 0
    assert np.count_nonzero(t["v_scale"]) == 1 and t["v_scale"][2, 7] > 0
    Kh, Vh = O.dequantize_tile(t)
    assert np.abs(Kh - K).max() <= float(t["k_scale"][5]) / 2 + 1e-6
    assert np.abs(Vh - V).max() <= float(t["v_scale"][2, 7]) / 2 + 1e-6


@pytest.mark.parametrize("bits", BITS)
def test_pack_round_trip_and_sizes(bits):
    rs = RS(bits)
    t = dict(k_scale=rs.rand(128).astype(np.float16), k_zero=rs.randn(128).astype(np.float16),
             v_scale=rs.rand(4, 32).astype(np.float16), v_zero=rs.randn(4, 32).astype(np.float16),
             k_codes=rs.randint(0, 1 << bits, (32, 128)).astype(np.uint8),
             v_codes=rs.randint(0, 1 << bits, (32, 128)).astype(np.uint8))
    blob = O.pack_tile(t, bits)
    assert blob.size == O.tile_bytes(bits) == 32 * {2: 96, 4: 160, 8: 288}[bits]
    u = O.unpack_tile(blob, bits)
    for k in t:
        assert (u[k] == t[k]).all(), k


def _random_tile(rs, bits):
    return dict(k_scale=rs.rand(128).astype(np.float16), k_zero=rs.randn(128).astype(np.float16),
                v_scale=rs.rand(4, 32).astype(np.float16), v_zero=rs.randn(4, 32).astype(np.float16),
                k_codes=rs.randint(0, 1 << bits, (32, 128)).astype(np.uint8),
                v_codes=rs.randint(0, 1 << bits, (32, 128)).astype(np.uint8))


@pytest.mark.parametrize("bits", BITS)
def test_pack_layout_seen_from_the_consuming_lanes(bits):
    """Independent statement of the format (tests/lane_reader.py): reading a packed tile the way
    the 32 lanes of the decode kernel do finds every code and every scale / zero where the
    tensor-core fragments need it.  The reader uses none of the oracle's location functions."""
    from tests.lane_reader import read_tile_as_lanes
    rs = RS(100 + bits)
    t = _random_tile(rs, bits)
    got = read_tile_as_lanes(O.pack_tile(t, bits), bits)
    for k in t:
        assert (got[k].view(np.uint16 if got[k].dtype == np.float16 else np.uint8) ==
                t[k].view(np.uint16 if t[k].dtype == np.float16 else np.uint8)).all(), k


@pytest.mark.parametrize("bits", BITS)
def test_locations_are_bijections(bits):
    kb = {O.key_code_location(t, c, bits) for t in range(32) for c in range(128)}
    vb = {O.value_code_location(t, c, bits) for t in range(32) for c in range(128)}
    assert len(kb) == len(vb) == 4096
    assert max(b for b, _ in kb) < 512 * bits and max(b for b, _ in vb) <= 512 * bits - 4
    assert sorted(O.key_meta_index(c, bits) for c in range(128)) == list(range(128))
    assert sorted(O.key_zero_index(c, bits) for c in range(128)) == list(range(128))
    assert sorted(O.value_scale_index(cg, t) for cg in range(4) for t in range(32)) == list(range(128))
    assert sorted(O.value_zero_index(cg, t) for cg in range(4) for t in range(32)) == list(range(128))


def test_raw_tile_round_trip_and_swizzle():
    rs = RS(4)
    K = rs.randint(0, 65536, (32, 128)).astype(np.uint16)
    V = rs.randint(0, 65536, (32, 128)).astype(np.uint16)
    blob = O.pack_raw_tile(K, V)
    assert blob.size == O.tile_bytes(16) == 32 * 512
    K2, V2 = O.unpack_raw_tile(blob)
    assert (K2 == K).all() and (V2 == V).all()
    w = blob.view(np.uint16)
    for tok, ch in [(0, 0), (1, 0), (9, 77), (31, 127), (13, 64)]:
        unit = ch // 8
        phys = (unit & 8) | ((unit ^ tok) & 7)
        assert w[tok * 128 + phys * 8 + ch % 8] == K[tok, ch]
        assert w[4096 + tok * 128 + phys * 8 + ch % 8] == V[tok, ch]


def test_slot_and_cache_bytes_closed_form():
    for chunk in (32, 64, 128, 256, 512):
        assert [O.slot_bytes(b, chunk) for b in (2, 4, 8, 16)] == [chunk * x for x in (96, 160, 288, 512)]
    cnt = np.array([[3, 2, 1, 1]])
    assert O.cache_bytes(cnt, 128, 8, 5) == 8 * (128 * (3 * 96 + 2 * 160 + 288 + 512) + 5 * 512)
    mix = np.array([0.1, 0.4, 0.4, 0.1])
    assert abs((mix * np.array(O.EXPERT_BITS)).sum() - 6.6) < 1e-12     # average-bits notion


def _small_kv(B=2, T=200, H=2, seed=0, dtype=0):
    rs = RS(seed)
    K = rs.randn(B, T, H, 128)
    K[..., 3] *= 10
    V = rs.randn(B, T, H, 128)
    if dtype == 0:
        return K.astype(np.float16).view(np.uint16), V.astype(np.float16).view(np.uint16)
    f = lambda a: (a.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    return f(K), f(V)


@pytest.mark.parametrize("w", [0, 1, 2])
def test_uniform_map_equals_standalone_uniform_quantiser(w):
    K, V = _small_kv()
    chunk = 64
    bmap = np.full((2, 200 // chunk), w, np.uint8)
    cache = O.quantize_kv(K, V, 0, chunk, bmap)
    assert cache["tail_len"] == 200 % chunk
    for b in range(2):
        for h in range(2):
            Kh, Vh = O.cache_kv_rows(cache, 0, chunk, b, h)
            n = (200 // chunk) * chunk
            refK = O.uniform_quantize_reference(K[b, :, h], 0, O.EXPERT_BITS[w], True, chunk)
            refV = O.uniform_quantize_reference(V[b, :, h], 0, O.EXPERT_BITS[w], False, chunk)
            assert (Kh[:n] == refK).all() and (Vh[:n] == refV).all()
            assert (Kh[n:] == O.to_f64(K[b, n:, h], 0)).all()           # tail stays exact


def test_mixed_map_places_chunks_in_pools():
    K, V = _small_kv(T=256 + 17, dtype=1)
    chunk = 64
    bmap = np.array([[3, 0, 1, 0], [3, 2, 2, 1]], np.uint8)
    cache = O.quantize_kv(K, V, 1, chunk, bmap)
    assert cache["count"].tolist() == [[2, 1, 0, 1], [0, 1, 2, 1]]
    assert cache["slot"].tolist() == [[0, 0, 0, 1], [0, 0, 1, 0]]
    assert cache["tail_len"] == 17 and cache["tail_k"].shape == (2, 2, 17, 128)
    # 16-bit chunks reproduce their rows exactly
    Ku, Vu = O.unpack_raw_tile(cache["pools"][3][1, 1, 0][:16384])
    assert (Ku == K[1, 0:32, 1]).all() and (Vu == V[1, 0:32, 1]).all()
    # sequence 0 chunk 3 (2-bit, second 2-bit chunk) sits in slot 1 of pool 0
    t = O.unpack_tile(cache["pools"][0][0, 0, 1][:O.tile_bytes(2)], 2)
    ref = O.quantize_tile(O.to_f32(K[0, 192:224, 0], 1), O.to_f32(V[0, 192:224, 0], 1), 2)
    for k in ref:
        assert (t[k] == ref[k]).all()


# ---- chunks shorter than a tile (8 and 16 tokens, the small sizes of the chunk-size ablation) ----
@pytest.mark.parametrize("chunk", [8, 16])
@pytest.mark.parametrize("bits", BITS)
def test_short_chunk_tile_groups_are_the_chunks_own_tokens(chunk, bits):
    rs = RS(300 + chunk + bits)
    K = (rs.randn(chunk, 128) * np.exp(rs.randn(1, 128))).astype(np.float16).astype(np.float32)
    V = rs.randn(chunk, 128).astype(np.float16).astype(np.float32)
    t = O.quantize_tile(K, V, bits)
    assert t["k_codes"].shape == (32, 128) and t["v_scale"].shape == (4, 32)
    # padding positions carry nothing
    assert (t["k_codes"][chunk:] == 0).all() and (t["v_codes"][chunk:] == 0).all()
    assert (t["v_scale"][:, chunk:] == 0).all() and (t["v_zero"][:, chunk:] == 0).all()
    # the key group of a channel is its `chunk` tokens: zero = its minimum, and the s/2 bound holds
    assert (t["k_zero"].astype(np.float32) == K.min(0)).all()
    Kh, Vh = O.dequantize_tile(t)
    assert (np.abs(Kh[:chunk] - K) <= t["k_scale"].astype(np.float64)[None, :] / 2 * (1 + 2e-7) + 1e-12).all()
    vs = np.repeat(t["v_scale"].astype(np.float64).T[:chunk], 32, axis=1)
    assert (np.abs(Vh[:chunk] - V) <= vs / 2 * (1 + 2e-7) + 1e-12).all()
    # the group maximum reaches the top code (or one below), the minimum code 0
    kc = t["k_codes"][:chunk]
    nonconst = t["k_scale"] > 0
    assert (kc.min(0) == 0).all() and (kc.max(0)[nonconst] >= (1 << bits) - 2).all()
    # a value group is 32 channels of one token, exactly as in a full tile
    full = O.quantize_tile(np.concatenate([K, K, K, K])[:32], np.concatenate([V, V, V, V])[:32], bits)
    assert (full["v_codes"][:chunk] == t["v_codes"][:chunk]).all()
    assert (full["v_scale"][:, :chunk] == t["v_scale"][:, :chunk]).all()
    # pack / unpack keeps everything, padding included
    u = O.unpack_tile(O.pack_tile(t, bits), bits)
    for k in t:
        assert (u[k] == t[k]).all(), k


@pytest.mark.parametrize("chunk", [8, 16])
def test_short_chunks_cache_sizes_rows_and_sixteen_bit_exactness(chunk):
    K, V = _small_kv(T=chunk * 9 + 3, dtype=1)
    B, T, H, _ = K.shape
    C = T // chunk
    bmap = RS(chunk).randint(0, 4, size=(B, C)).astype(np.uint8)
    cache = O.quantize_kv(K, V, 1, chunk, bmap)
    # one (padded) tile per chunk: slot bytes are those of a single tile
    for w, bits in enumerate(O.EXPERT_BITS):
        assert cache["pools"][w].shape[-1] == O.tile_bytes(bits) == O.slot_bytes(bits, chunk)
    assert cache["tail_len"] == 3
    for b in range(B):
        for h in range(H):
            Kh, Vh = O.cache_kv_rows_in_order(cache, 1, chunk, b, h)
            assert Kh.shape == (T, 128)                       # padding positions are not tokens
            for c in range(C):
                sl = slice(c * chunk, (c + 1) * chunk)
                if bmap[b, c] == 3:                           # 16-bit chunks are exact
                    assert (Kh[sl] == O.to_f64(K[b, sl, h], 1)).all() and (Vh[sl] == O.to_f64(V[b, sl, h], 1)).all()
                else:                                         # others within half a scale of the chunk's own range
                    x = O.to_f64(K[b, sl, h], 1)
                    rng = x.max(0) - x.min(0)
                    bits = O.EXPERT_BITS[bmap[b, c]]
                    assert (np.abs(Kh[sl] - x) <= rng[None, :] / ((1 << bits) - 1) / 2 * 1.01 + 1e-3 * np.abs(x).max()).all()
            assert (Kh[C * chunk:] == O.to_f64(K[b, C * chunk:, h], 1)).all()
            # the pool-by-pool walk sees the same multiset of rows
            Kp, _ = O.cache_kv_rows(cache, 1, chunk, b, h)
            assert Kp.shape == Kh.shape and np.allclose(np.sort(Kp.sum(1)), np.sort(Kh.sum(1)))


def test_short_chunks_all_sixteen_bit_attention_equals_plain_attention():
    K, V = _small_kv(T=8 * 11 + 5, dtype=0)
    B, T, H, _ = K.shape
    bmap = np.full((B, T // 8), 3, np.uint8)
    cache = O.quantize_kv(K, V, 0, 8, bmap)
    q = RS(3).randn(B, H, 128).astype(np.float16)
    out = O.decode_attn(q.view(np.uint16), 0, cache, 8)
    for b in range(B):
        for h in range(H):
            ref = O.softmax_attention(q[b, h].astype(np.float64), O.to_f64(K[b, :, h], 0), O.to_f64(V[b, :, h], 0), 1 / np.sqrt(128))
            assert np.abs(out[b, h] - ref).max() < 1e-12
