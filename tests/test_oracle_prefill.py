"""Pins for the oracle's causal prefill attention over the quantised chunks."""
import numpy as np
import torch

from oracle import moqae_oracle as O

RS = np.random.RandomState


def _inputs(B=2, T=32 * 5 + 7, Hq=4, Hkv=2, seed=0):
    rs = RS(seed)
    f = lambda a: a.astype(np.float16).view(np.uint16)
    K = rs.randn(B, T, Hkv, 128)
    K[..., 9] *= 10
    return f(rs.randn(B, T, Hq, 128)), f(K), f(rs.randn(B, T, Hkv, 128))


def test_all_16_bit_map_equals_library_causal_attention():
    q, K, V = _inputs()
    B, T, Hq, _ = q.shape
    chunk = 32
    cache = O.quantize_kv(K, V, 0, chunk, np.full((B, T // chunk), 3, np.uint8))
    got = O.prefill_attn(q, 0, cache, chunk)
    tq = torch.from_numpy(O.to_f64(q, 0)).permute(0, 2, 1, 3)
    tk = torch.from_numpy(O.to_f64(K, 0)).permute(0, 2, 1, 3).repeat_interleave(2, dim=1)
    tv = torch.from_numpy(O.to_f64(V, 0)).permute(0, 2, 1, 3).repeat_interleave(2, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True).permute(0, 2, 1, 3).numpy()
    assert np.abs(got - ref).max() < 1e-12


def test_rows_against_first_principles_and_the_decode_oracle():
    q, K, V = _inputs(seed=1)
    B, T, Hq, _ = q.shape
    chunk = 64
    bmap = RS(2).randint(0, 4, size=(B, T // chunk)).astype(np.uint8)
    cache = O.quantize_kv(K, V, 0, chunk, bmap)
    got = O.prefill_attn(q, 0, cache, chunk)
    # position 0 sees only itself: the output is the dequantised value row 0 of its kv head
    for b in range(B):
        for h in range(Hq):
            _, V64 = O.cache_kv_rows_in_order(cache, 0, chunk, b, h // 2)
            assert np.abs(got[b, 0, h] - V64[0]).max() < 1e-12
    # the last position sees the whole cache: it equals the decode oracle for the same query
    dec = O.decode_attn(q[:, T - 1], 0, cache, chunk)
    assert np.abs(got[:, T - 1] - dec).max() < 1e-12
    # token order of the in-order walk: 16-bit chunks reproduce their input rows in place
    for b in range(B):
        K64, _ = O.cache_kv_rows_in_order(cache, 0, chunk, b, 1)
        for c in range(T // chunk):
            if bmap[b, c] == 3:
                assert (K64[c * chunk:(c + 1) * chunk] == O.to_f64(K[b, c * chunk:(c + 1) * chunk, 1], 0)).all()
        assert (K64[(T // chunk) * chunk:] == O.to_f64(K[b, (T // chunk) * chunk:, 1], 0)).all()
