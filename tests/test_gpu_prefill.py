"""GPU parity: moqae_prefill_attn (causal attention of the prompt over its quantised cache) against
the oracle on the same packed cache.  The kernel rounds three things to fp16 before its
tensor-core products: the dequantised keys (which perturbs the scores), the softmax weights P
and the dequantised values.  Each rounding is at most 2^-11 relative, and a row whose softmax
is dominated by one token passes them on undamped, so the bound is
|err| <= 3 * 2^-11 * max|V| and, per (sequence, position, head) row, max|err| / max|ref| <= 1e-2."""
import numpy as np
import pytest
import torch

from oracle import moqae_oracle as O
from paper_2506_07533_b200 import binding as mq
from paper_2506_07533_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def prefill_case(B, T, Hq, Hkv, chunk, dtype, bmap, seed):
    K, V = H.make_kv(B, T, Hkv, dtype, seed)
    q = synth.normal((B, T, Hq, 128), dtype, seed + 1, "cpu")
    ocache = O.quantize_kv(synth.to_u16(K), synth.to_u16(V), dtype, chunk, bmap)
    ref = O.prefill_attn(synth.to_u16(q), dtype, ocache, chunk)
    cfg = mq.make_config(n_layers=2, n_q_heads=Hq, n_kv_heads=Hkv, chunk=chunk, dtype=dtype, d_in=64,
                         max_tokens=max(T, chunk), batch=B)
    cap = [max(1, int(ocache["count"][:, w].max())) if bmap.size else 1 for w in range(4)]
    cache = mq.moqae_cache_bind(cfg, cap, zero_pools=True)
    fm = torch.from_numpy(bmap).cuda() if bmap.size else None
    mq.moqae_quantize_kv(cfg, K.cuda(), V.cuda(), T, 1, cache, forced_map=fm)
    abs_tol = 3 * 2.0 ** -11 * float(V.float().abs().max())
    # both ways of feeding the products: every CTA expanding the packed tiles itself (no
    # workspace), and the layer expanded once into an fp16 workspace that the CTAs fetch from
    ws = torch.full((mq.moqae_prefill_attn_workspace(cfg, T),), 0xFF, dtype=torch.uint8, device="cuda")
    for workspace in (None, ws):
        out = torch.full((B, T, Hq, 128), float("nan"), dtype=torch.float32, device="cuda")
        mq.moqae_prefill_attn(cfg, q.cuda(), T, 1, cache, out, workspace=workspace)
        torch.cuda.synchronize()
        assert mq.moqae_poll_status(cache) == 0
        got = out.cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all()
        ok, e_abs, e_rel = H.attn_tolerance_ok(got.reshape(1, -1, 128), ref.reshape(1, -1, 128), abs_tol=abs_tol, rel_tol=1e-2)
        assert ok, (workspace is not None, e_abs, e_rel)
    return e_abs, e_rel


@pytest.mark.parametrize("w", [0, 1, 2, 3])
def test_uniform_width(w):
    B, T, chunk = 1, 128 * 2, 64
    prefill_case(B, T, 2, 2, chunk, 0, np.full((B, T // chunk), w, np.uint8), 700 + w)


@pytest.mark.parametrize("dtype", [0, 1])
def test_mixed_map_gqa_ragged(dtype):
    B, T, chunk = 2, 32 * 13 + 21, 32                  # several 128-token blocks, a ragged tail
    bmap = np.random.RandomState(5 + dtype).randint(0, 4, size=(B, T // chunk)).astype(np.uint8)
    prefill_case(B, T, 4, 2, chunk, dtype, bmap, 710 + dtype)


def test_longer_prompt_many_blocks_wide_gqa():
    # 9 blocks of 128 tokens (every operand stage is reused several times, five CTAs per head of
    # different lengths), 8 query heads on 2 kv heads, chunk 128, a tail of 77 tokens
    B, T, chunk = 1, 128 * 8 + 77, 128
    bmap = np.random.RandomState(9).randint(0, 4, size=(B, T // chunk)).astype(np.uint8)
    prefill_case(B, T, 8, 2, chunk, 1, bmap, 730)


def test_short_prompts():
    prefill_case(1, 7, 2, 1, 32, 0, np.zeros((1, 0), np.uint8), 720)          # tail only
    prefill_case(1, 128, 1, 1, 128, 1, np.array([[1]], np.uint8), 721)        # exactly one block
    prefill_case(2, 129, 2, 2, 64, 1, np.array([[3, 0], [2, 1]], np.uint8), 722)


def test_workspace_size_and_rejection():
    cfg = mq.make_config(n_layers=1, n_q_heads=4, n_kv_heads=2, chunk=64, dtype=1, d_in=64, max_tokens=300, batch=3)
    assert mq.moqae_prefill_attn_workspace(cfg, 300) == 2 * 3 * 2 * 384 * 256      # 300 tokens -> 3 blocks of 128
    assert mq.moqae_prefill_attn_workspace(cfg, 0) == 0
    cache = mq.moqae_cache_bind(cfg, [1, 1, 1, 1], zero_pools=True)
    q = torch.zeros(3, 300, 4, 128, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(3, 300, 4, 128, dtype=torch.float32, device="cuda")
    small = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(RuntimeError):
        mq.moqae_prefill_attn(cfg, q, 300, 0, cache, out, workspace=small)
