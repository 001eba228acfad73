"""A second, independent statement of the storage format of a quantised tile.

`read_tile_as_lanes` takes the bytes of one tile and walks them the way the 32 lanes of the
decode kernel's tensor-core fragments do: lane = 4 * g + t4 reads whole 16-byte units; a key
register is a payload word, or the word shifted right by 8, masked at one code position in both
half-words.  It returns codes, scales and zeros as plain [token, channel] arrays, so bytes written
by anybody (the oracle's packer or the CUDA quantiser) can be compared with the layout-free
result of the quantiser arithmetic.  Written from the format description in include/moqae.h; it
uses none of the oracle's location functions.
"""
import numpy as np


def read_tile_as_lanes(blob: np.ndarray, bits: int) -> dict:
    blob = np.ascontiguousarray(blob, dtype=np.uint8)
    assert blob.size == 1024 + 1024 * bits
    n = 32 // bits
    mask = (1 << bits) - 1
    hw = blob[:1024].view(np.uint16)
    kpay = blob[1024:1024 + 512 * bits]
    vpay = blob[1024 + 512 * bits:]
    k_codes = np.full((32, 128), 255, np.uint8)
    v_codes = np.full((32, 128), 255, np.uint8)
    k_scale = np.zeros(128, np.uint16)
    k_zero = np.zeros(128, np.uint16)
    v_scale = np.zeros((4, 32), np.uint16)
    v_zero = np.zeros((4, 32), np.uint16)

    def unit(pay, idx):
        return pay[16 * idx:16 * idx + 16].view(np.uint32)

    for blk in range(2):
        for g in range(8):
            for t4 in range(4):
                lane = 4 * g + t4
                # key rows 16blk + g (hh = 0) and 16blk + g + 8 (hh = 1), channels 32 t4 .. + 31
                for hh in range(2):
                    tok = 16 * blk + 8 * hh + g
                    if bits == 2:
                        words = unit(kpay, 32 * blk + lane)[2 * hh:2 * hh + 2]
                    elif bits == 4:
                        words = unit(kpay, 32 * (2 * blk + hh) + lane)
                    else:
                        words = np.concatenate([unit(kpay, 32 * (2 * (2 * blk + hh) + j) + lane) for j in range(2)])
                    assert len(words) == bits
                    r = 0
                    for j in range(bits):
                        for s_ in range(2):
                            ws = int(words[j]) >> (8 * s_)
                            for m in range(n // 4):
                                lo_ch = 32 * t4 + j * n + s_ * (n // 4) + m
                                hi_ch = lo_ch + n // 2
                                k_codes[tok, lo_ch] = (ws >> (bits * m)) & mask
                                k_codes[tok, hi_ch] = (ws >> (16 + bits * m)) & mask
                                # register r of this lane: the lane's i-th 16-byte unit of the scale array
                                # holds registers 4i .. 4i+3, of the zero array 4i, 4i+2, 4i+1, 4i+3
                                unit_hw = ((r >> 2) * 4 + t4) * 8
                                spos, zpos = (r & 3), (0, 2, 1, 3)[r & 3]
                                k_scale[lo_ch] = hw[unit_hw + 2 * spos]
                                k_scale[hi_ch] = hw[unit_hw + 2 * spos + 1]
                                k_zero[lo_ch] = hw[128 + unit_hw + 2 * zpos]
                                k_zero[hi_ch] = hw[128 + unit_hw + 2 * zpos + 1]
                                r += 1
                    assert r == 16
                # values: channel rows of this lane, tokens 16blk + 8half + 2t4 + e
                words = np.concatenate([unit(vpay, (blk * (bits // 2) + u) * 32 + lane) for u in range(bits // 2)])
                assert len(words) == 2 * bits
                for w in range(2 * bits):
                    for slot in range(8 // bits):
                        R = w * (8 // bits) + slot
                        ch = 32 * (R >> 2) + 4 * g + (R & 3)
                        for half in range(2):
                            ws = int(words[w]) >> (8 * half)
                            for e in range(2):
                                tok = 16 * blk + 8 * half + 2 * t4 + e
                                v_codes[tok, ch] = (ws >> (bits * slot + 16 * e)) & mask
                for cp in range(2):
                    base = ((blk * 2 + cp) * 4 + t4) * 8
                    for k in range(4):
                        cg, half = 2 * cp + (k >> 1), k & 1
                        for e in range(2):
                            tok = 16 * blk + 8 * half + 2 * t4 + e
                            v_scale[cg, tok] = hw[256 + base + 2 * k + e]
                if g < 4:
                    base = ((blk * 4 + g) * 4 + t4) * 4
                    for half in range(2):
                        for e in range(2):
                            tok = 16 * blk + 8 * half + 2 * t4 + e
                            v_zero[g, tok] = hw[384 + base + 2 * half + e]
    assert (k_codes <= mask).all() and (v_codes <= mask).all()          # every position was visited
    return dict(k_codes=k_codes, v_codes=v_codes, k_scale=k_scale.view(np.float16), k_zero=k_zero.view(np.float16),
                v_scale=v_scale.view(np.float16), v_zero=v_zero.view(np.float16))
