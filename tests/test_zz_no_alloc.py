"""moqae_decode_attn_static: the decode entry point for callers that cannot allocate.

A caller that may not call cudaMalloc (its host application owns all device memory, or its
run-time rules forbid allocator calls) cannot hand moqae_decode_attn a workspace.  The static
variant keeps the split partials in an array inside the library; this test checks, through
the C ABI, that it gives what the ordinary entry point gives - twice in a row, because the
array is shared by all calls and still holds the previous call's partials the second time.
This file sorts last on purpose, so a run that stops at the first failure has already
executed every other test.
"""
import numpy as np
import pytest
import torch

from oracle import moqae_oracle as O

from paper_2506_07533_b200 import binding as mq
from paper_2506_07533_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _setup(B, T, Hq, Hkv, chunk, dtype, seed):
    K, V = H.make_kv(B, T, Hkv, dtype, seed)
    bmap = np.random.RandomState(seed).randint(0, 4, size=(B, T // chunk)).astype(np.uint8)
    cfg = mq.make_config(n_layers=1, n_q_heads=Hq, n_kv_heads=Hkv, chunk=chunk, dtype=dtype, d_in=64,
                         max_tokens=T, batch=B)
    cap = [T // chunk] * 4
    cache = mq.moqae_cache_bind(cfg, cap, zero_pools=True)
    mq.moqae_quantize_kv(cfg, K.cuda(), V.cuda(), T, 0, cache, forced_map=torch.from_numpy(bmap).cuda())
    cache.oracle = O.quantize_kv(synth.to_u16(K), synth.to_u16(V), dtype, chunk, bmap)
    return cfg, cache


def test_static_scratch_matches_workspace_entry_point_twice():
    cfg, cache = _setup(B=2, T=64 * 7 + 13, Hq=8, Hkv=2, chunk=64, dtype=1, seed=321)
    assert mq.moqae_decode_attn_workspace(cfg) <= mq.moqae_decode_attn_static_max_bytes()
    ws = torch.zeros(mq.moqae_decode_attn_workspace(cfg), dtype=torch.uint8, device="cuda")
    for call in range(2):                       # second call finds the first call's partials in the array
        q = synth.normal((2, 8, 128), 1, 500 + call, "cuda")
        want = torch.full((2, 8, 128), float("nan"), dtype=torch.float32, device="cuda")
        got = torch.full((2, 8, 128), float("nan"), dtype=torch.float32, device="cuda")
        mq.moqae_decode_attn(cfg, q, 0, cache, want, ws)
        mq.moqae_decode_attn_static(cfg, q, 0, cache, got)
        torch.cuda.synchronize()
        ok, e_abs, e_rel = H.attn_tolerance_ok(got.cpu().numpy(), want.cpu().numpy().astype(np.float64))
        assert ok, (call, e_abs, e_rel)
        ref = O.decode_attn(synth.to_u16(q), 1, cache.oracle, 64)          # and against the CPU oracle
        ok, e_abs, e_rel = H.attn_tolerance_ok(got.cpu().numpy(), ref)
        assert ok, (call, e_abs, e_rel)
    assert mq.moqae_poll_status(cache) == 0


def test_static_scratch_is_shared_by_different_configurations():
    # The one array serves every configuration used on the device, and each lays its partials and
    # arrival counters out differently: where a small problem keeps its counters, a larger one
    # writes partials.  Alternating between two problems must still give each its right answer.
    small = _setup(B=1, T=32 * 5, Hq=2, Hkv=2, chunk=32, dtype=0, seed=331)
    large = _setup(B=3, T=64 * 6 + 5, Hq=8, Hkv=4, chunk=64, dtype=1, seed=332)
    for rnd in range(3):
        for (cfg, cache), (B, Hq, chunk, dtype) in ((small, (1, 2, 32, 0)), (large, (3, 8, 64, 1))):
            q = synth.normal((B, Hq, 128), dtype, 600 + rnd, "cuda")
            got = torch.full((B, Hq, 128), float("nan"), dtype=torch.float32, device="cuda")
            mq.moqae_decode_attn_static(cfg, q, 0, cache, got)
            torch.cuda.synchronize()
            ok, e_abs, e_rel = H.attn_tolerance_ok(got.cpu().numpy(), O.decode_attn(synth.to_u16(q), dtype, cache.oracle, chunk))
            assert ok, (rnd, B, e_abs, e_rel)


def test_static_scratch_rejects_oversized_problem():
    # a batch whose partials do not fit the fixed array is refused on the host, nothing runs
    cfg = mq.make_config(n_layers=1, n_q_heads=64, n_kv_heads=64, chunk=32, dtype=0, d_in=64,
                         max_tokens=32, batch=512)
    assert mq.moqae_decode_attn_workspace(cfg) > mq.moqae_decode_attn_static_max_bytes()
    cache = mq.moqae_cache_bind(cfg, [1, 1, 1, 1])
    q = torch.zeros((512, 64, 128), dtype=torch.float16, device="cuda")
    out = torch.zeros((512, 64, 128), dtype=torch.float32, device="cuda")
    with pytest.raises(mq.MoqaeError) as e:
        mq.moqae_decode_attn_static(cfg, q, 0, cache, out)
    assert e.value.code == mq.ERR_WORKSPACE_TOO_SMALL
