"""GPU parity: moqae_project_quantize_kv (K/V projection on the tensor cores with the quantiser as
its epilogue) against the oracle.

  * the rounded K/V rows the kernel hands back are within one unit in the last place of the
    16-bit dtype of the oracle's float64 product, plus the worst-case error of a float32
    accumulation of d_in products in any order (d_in * 2^-24 * sum |h_i w_i|, which matters only for
    results that cancel to almost nothing); a value next to a rounding boundary may land on
    either side;
  * the packed pools, tables and tail are byte for byte what the oracle's quantiser + packer make
    of THOSE rows (the kernel's own rounded K/V), so the epilogue is held to the same bit-exact
    standard as the stand-alone quantise kernel;
  * decode attention over the resulting cache matches the oracle.
"""
import numpy as np
import pytest
import torch

from oracle import moqae_oracle as O
from paper_2506_07533_b200 import binding as mq
from paper_2506_07533_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def ulp_of(x64, dtype):
    sig, emin = (11, -14) if dtype == 0 else (8, -126)
    _, e = np.frexp(x64)
    return np.ldexp(1.0, np.maximum(e, emin + 1) - sig)


def project_case(B, T, Hkv, D, chunk, dtype, bmap, seed, check_decode=True):
    hid = synth.normal((B, T, D), dtype, seed, "cpu")
    Wk = synth.normal((Hkv * 128, D), dtype, seed + 1, "cpu", std=1.0 / np.sqrt(D))
    Wv = synth.normal((Hkv * 128, D), dtype, seed + 2, "cpu", std=1.0 / np.sqrt(D))
    Wk[5] *= 10.0                                       # an outlier key channel
    cfg = mq.make_config(n_layers=2, n_q_heads=Hkv, n_kv_heads=Hkv, chunk=chunk, dtype=dtype, d_in=D,
                         max_tokens=max(T, chunk), batch=B)
    cap = [max(1, int((bmap == w).sum(1).max())) if bmap.size else 1 for w in range(4)]
    cache = mq.moqae_cache_bind(cfg, cap, zero_pools=True)
    tdt = synth.torch_dtype(dtype)
    k_r = torch.zeros((B, T, Hkv, 128), dtype=tdt, device="cuda")
    v_r = torch.zeros((B, T, Hkv, 128), dtype=tdt, device="cuda")
    fm = torch.from_numpy(bmap).cuda() if bmap.size else None
    layer = 1
    mq.moqae_project_quantize_kv(cfg, hid.cuda(), Wk.cuda(), Wv.cuda(), T, layer, cache, forced_map=fm,
                                 k_rounded=k_r, v_rounded=v_r)
    torch.cuda.synchronize()
    assert mq.moqae_poll_status(cache) == 0
    K16, V16, K64, V64 = O.project_kv(synth.to_u16(hid), synth.to_u16(Wk), synth.to_u16(Wv), dtype, Hkv)
    if T:
        absh = np.abs(O.to_f64(synth.to_u16(hid), dtype))
        for got, x64, Wm in ((k_r, K64, Wk), (v_r, V64, Wv)):
            g = O.to_f64(synth.to_u16(got), dtype)
            acc = D * 2.0 ** -24 * (absh @ np.abs(O.to_f64(synth.to_u16(Wm), dtype)).T).reshape(x64.shape)
            assert (np.abs(g - x64) <= ulp_of(x64, dtype) * 1.001 + acc).all()
        frac_equal = float((synth.to_u16(k_r) == K16).mean())
        assert frac_equal > 0.99                        # nearly every value rounds the same way
    # bytes: the oracle quantises the kernel's own rounded rows
    ocache = O.quantize_kv(synth.to_u16(k_r), synth.to_u16(v_r), dtype, chunk, bmap)
    H.compare_pools(cache, ocache, layer)
    if check_decode and T:
        q = synth.normal((B, Hkv, 128), dtype, seed + 3, "cpu")
        ws = torch.zeros(mq.moqae_decode_attn_workspace(cfg), dtype=torch.uint8, device="cuda")
        out = torch.full((B, Hkv, 128), float("nan"), dtype=torch.float32, device="cuda")
        mq.moqae_decode_attn(cfg, q.cuda(), layer, cache, out, ws)
        torch.cuda.synchronize()
        ok, e_abs, e_rel = H.attn_tolerance_ok(out.cpu().numpy(), O.decode_attn(synth.to_u16(q), dtype, ocache, chunk))
        assert ok, (e_abs, e_rel)


@pytest.mark.parametrize("dtype", [0, 1])
def test_mixed_map_ragged_tail(dtype):
    B, T, chunk = 2, 64 * 5 + 21, 64                  # 3 units of 128 tokens per sequence, the last one ragged
    bmap = np.array([[3, 0, 1, 2, 0], [2, 1, 0, 3, 1]], np.uint8)
    project_case(B, T, 2, 128, chunk, dtype, bmap, 900 + dtype)


def test_long_reduction_many_heads():
    # d_in 1024 = 16 ring stages per unit (every stage reused several times), 8 kv heads, chunk 128
    B, T, chunk = 1, 128 * 3 + 77, 128
    bmap = np.array([[0, 2, 1]], np.uint8)
    project_case(B, T, 8, 1024, chunk, 1, bmap, 910)


def test_more_units_than_sms_wrap_around():
    # 5 sequences x 10 units x 4 heads = 200 units on 148 persistent CTAs: some run two units, which
    # exercises both accumulator buffers and the reuse of the epilogue's staging memory
    B, T, chunk = 5, 32 * 39 + 3, 32
    bmap = np.random.RandomState(4).randint(0, 4, size=(B, T // chunk)).astype(np.uint8)
    project_case(B, T, 4, 64, chunk, 1, bmap, 920, check_decode=False)


def test_short_and_empty_contexts():
    project_case(1, 20, 2, 64, 32, 0, np.zeros((1, 0), np.uint8), 930)          # tail only
    project_case(2, 128, 1, 64, 128, 1, np.array([[1], [3]], np.uint8), 931)    # exactly one unit, no tail
    project_case(1, 0, 1, 64, 32, 1, np.zeros((1, 0), np.uint8), 932)           # nothing at all


def test_argument_errors():
    cfg = mq.make_config(n_layers=1, n_q_heads=2, n_kv_heads=2, chunk=32, dtype=1, d_in=96, max_tokens=64, batch=1)
    cache = mq.moqae_cache_bind(cfg, [1, 1, 1, 1])
    hid = torch.zeros((1, 64, 96), dtype=torch.bfloat16, device="cuda")
    W = torch.zeros((256, 96), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(mq.MoqaeError) as e:
        mq.moqae_project_quantize_kv(cfg, hid, W, W, 64, 0, cache)
    assert e.value.code == mq.ERR_UNSUPPORTED                                   # d_in not a multiple of 64
