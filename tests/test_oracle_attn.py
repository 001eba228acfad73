"""Pins for the oracle's decode attention."""
import numpy as np
import pytest
import torch

from oracle import moqae_oracle as O

RS = np.random.RandomState


def f16(a):
    return np.asarray(a).astype(np.float16).view(np.uint16)


def bf16(a):
    return (np.asarray(a).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)


def _inputs(B=2, T=160, Hkv=2, Hq=4, seed=0, conv=f16):
    rs = RS(seed)
    K = rs.randn(B, T, Hkv, 128)
    V = rs.randn(B, T, Hkv, 128)
    q = rs.randn(B, Hq, 128)
    return conv(K), conv(V), conv(q)


@pytest.mark.parametrize("dtype,conv", [(0, f16), (1, bf16)])
def test_all_16bit_map_is_textbook_attention(dtype, conv):
    K, V, q = _inputs(conv=conv, T=150)
    chunk = 32
    bmap = np.full((2, 150 // chunk), 3, np.uint8)
    cache = O.quantize_kv(K, V, dtype, chunk, bmap)
    out = O.decode_attn(q, dtype, cache, chunk)
    Kf, Vf, qf = O.to_f64(K, dtype), O.to_f64(V, dtype), O.to_f64(q, dtype)
    # direct float64 evaluation of softmax(q K^T / sqrt(d)) V, GQA group of 2
    for b in range(2):
        for h in range(4):
            kv = h // 2
            s = Kf[b, :, kv] @ qf[b, h] / np.sqrt(128.0)
            p = np.exp(s - s.max())
            p /= p.sum()
            assert np.allclose(out[b, h], p @ Vf[b, :, kv], rtol=1e-12, atol=1e-14)
    # independent library check: torch SDPA on the same values (float64, CPU)
    tq = torch.from_numpy(qf).unsqueeze(2)                              # [B, Hq, 1, d]
    tk = torch.from_numpy(Kf).permute(0, 2, 1, 3).repeat_interleave(2, dim=1)
    tv = torch.from_numpy(Vf).permute(0, 2, 1, 3).repeat_interleave(2, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv).squeeze(2).numpy()
    assert np.allclose(out, ref, rtol=1e-10, atol=1e-12)


def test_invariants_mixed_cache():
    K, V, q = _inputs(T=32 * 6 + 5, seed=2)
    chunk = 32
    bmap = np.array([[3, 0, 1, 2, 0, 1], [3, 2, 2, 0, 1, 0]], np.uint8)
    cache = O.quantize_kv(K, V, 0, chunk, bmap)
    out = O.decode_attn(q, 0, cache, chunk)
    for b in range(2):
        for h in range(4):
            Kh, Vh = O.cache_kv_rows(cache, 0, chunk, b, h // 2)
            assert Kh.shape[0] == 32 * 6 + 5
            # a convex combination of the dequantised value rows
            assert (out[b, h] <= Vh.max(0) + 1e-12).all() and (out[b, h] >= Vh.min(0) - 1e-12).all()
            # order of the keys does not matter
            perm = RS(h).permutation(Kh.shape[0])
            o2 = O.softmax_attention(O.to_f64(q, 0)[b, h], Kh[perm], Vh[perm], 1 / np.sqrt(128.0))
            assert np.allclose(o2, out[b, h], rtol=1e-12, atol=1e-14)
            # split evaluation merged with the log-sum-exp rule gives the same result
            qv = O.to_f64(q, 0)[b, h]
            parts = []
            for lo, hi in [(0, 50), (50, 51), (51, Kh.shape[0])]:
                s = Kh[lo:hi] @ qv / np.sqrt(128.0)
                m = s.max()
                p = np.exp(s - m)
                parts.append((m, p.sum(), p @ Vh[lo:hi]))
            M = max(m for m, _, _ in parts)
            l = sum(l_ * np.exp(m - M) for m, l_, _ in parts)
            o = sum(o_ * np.exp(m - M) for m, _, o_ in parts) / l
            assert np.allclose(o, out[b, h], rtol=1e-12, atol=1e-14)


def test_quantised_attention_close_to_exact_and_ordered_by_width():
    K, V, q = _inputs(T=256, seed=4)
    errs = []
    exact = O.decode_attn(q, 0, O.quantize_kv(K, V, 0, 64, np.full((2, 4), 3, np.uint8)), 64)
    for w in (0, 1, 2):
        out = O.decode_attn(q, 0, O.quantize_kv(K, V, 0, 64, np.full((2, 4), w, np.uint8)), 64)
        errs.append(np.abs(out - exact).max())
    assert errs[0] > errs[1] > errs[2] and errs[2] < errs[0] / 20, errs


def test_single_token_and_uniform_scores():
    # one cached token: the output is that token's value row whatever the query
    K, V, q = _inputs(B=1, T=1, Hkv=1, Hq=1, seed=5)
    cache = O.quantize_kv(K, V, 0, 32, np.zeros((1, 0), np.uint8))
    out = O.decode_attn(q, 0, cache, 32)
    assert np.allclose(out[0, 0], O.to_f64(V, 0)[0, 0, 0], atol=1e-15)
    # zero query: uniform weights, output is the mean of the dequantised values
    K, V, q = _inputs(B=1, T=96, Hkv=1, Hq=1, seed=6)
    q[:] = 0
    cache = O.quantize_kv(K, V, 0, 32, np.array([[3, 1, 0]], np.uint8))
    out = O.decode_attn(q, 0, cache, 32)
    _, Vh = O.cache_kv_rows(cache, 0, 32, 0, 0)
    assert np.allclose(out[0, 0], Vh.mean(0), rtol=1e-12, atol=1e-14)


def test_empty_cache_gives_zero():
    K, V, q = _inputs(B=1, T=0, Hkv=1, Hq=1)
    cache = O.quantize_kv(K, V, 0, 32, np.zeros((1, 0), np.uint8))
    assert (O.decode_attn(q, 0, cache, 32) == 0).all()
