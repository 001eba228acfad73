"""GPU parity: moqae_quantize_kv against the oracle, byte for byte."""
import numpy as np
import pytest
import torch

from oracle import moqae_oracle as O
from paper_2506_07533_b200 import binding as mq
from paper_2506_07533_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


# largest 16-bit values below 32752, the edge of the documented input domain (|x| < 32752 keeps the
# span of every group, max - zero, below the largest finite fp16)
TOP = {0: 32736.0, 1: 32640.0}


def run_case(B, T, Hkv, chunk, dtype, bmap, seed, n_layers=1, layer=0, rs_group=1, scale=1.0):
    K, V = H.make_kv(B, T, Hkv, dtype, seed)
    if scale != 1.0:                        # scaled-up values saturate at the edge of the domain
        K = (K.float() * scale).clamp(-TOP[dtype], TOP[dtype]).to(K.dtype)
        V = (V.float() * scale).clamp(-TOP[dtype], TOP[dtype]).to(V.dtype)
    ocache = O.quantize_kv(synth.to_u16(K), synth.to_u16(V), dtype, chunk, bmap)
    cfg = mq.make_config(n_layers=n_layers, n_q_heads=Hkv, n_kv_heads=Hkv, chunk=chunk, dtype=dtype,
                         d_in=64, max_tokens=max(T, chunk), batch=B, rs_group=rs_group)
    cap = [max(1, int(ocache["count"][:, w].max())) if bmap.size else 1 for w in range(4)]
    cache = mq.moqae_cache_bind(cfg, cap, zero_pools=True)
    fm = torch.from_numpy(bmap).cuda() if bmap.size else None
    mq.moqae_quantize_kv(cfg, K.cuda(), V.cuda(), T, layer, cache, forced_map=fm)
    assert mq.moqae_poll_status(cache) == 0
    H.compare_pools(cache, ocache, layer)
    return cache, ocache


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("chunk", [32, 128])
def test_mixed_map_small(dtype, chunk):
    B, T, Hkv = 2, chunk * 7 + 13, 3
    rs = np.random.RandomState(chunk + dtype)
    bmap = rs.randint(0, 4, size=(B, T // chunk)).astype(np.uint8)
    run_case(B, T, Hkv, chunk, dtype, bmap, seed=11 + chunk + dtype)


@pytest.mark.parametrize("w", [0, 1, 2, 3])
def test_uniform_maps_config1_shape(w):
    # config 1: batch 1, 8 kv heads, context 4096, chunk 128, fp16, outlier key channels
    bmap = np.full((1, 32), w, np.uint8)
    run_case(1, 4096, 8, 128, 0, bmap, seed=1)


@pytest.mark.parametrize("chunk", [64, 256, 512])
def test_chunk_sizes(chunk):
    B, T = 1, chunk * 3
    bmap = np.array([[3, 0, 1]], np.uint8) if chunk != 256 else np.array([[2, 0, 1]], np.uint8)
    run_case(B, T, 2, chunk, 1, bmap, seed=chunk)


def test_edge_cases():
    # tail only (context shorter than a chunk), and an exactly empty context
    run_case(2, 20, 2, 32, 0, np.zeros((2, 0), np.uint8), seed=3)
    run_case(1, 0, 1, 32, 1, np.zeros((1, 0), np.uint8), seed=4)
    # tiny and huge magnitudes (subnormal fp16 scales; values near the top of the domain)
    bmap = np.array([[0, 1, 2, 3]], np.uint8)
    run_case(1, 128, 2, 32, 0, bmap, seed=5, scale=1e-4)
    run_case(1, 128, 2, 32, 1, bmap, seed=6, scale=1e-6)
    run_case(1, 128, 2, 32, 1, bmap, seed=7, scale=2000.0)
    run_case(1, 128, 2, 32, 0, bmap, seed=8, scale=2.0e4)      # most values AT the edge of the domain


@pytest.mark.parametrize("dtype", [0, 1])
def test_values_at_the_edge_of_the_domain(dtype):
    # groups that span the whole domain [-TOP, TOP] (scale = 65472 / (2^b - 1) at fp16), groups pinned
    # at one edge, and edge values next to tiny ones
    B, T, Hkv, chunk = 1, 128, 2, 32
    rs = np.random.RandomState(77 + dtype)
    top = TOP[dtype]
    K = rs.choice([-top, top, 0.0, 1e-3, -top / 2, 7.0], size=(B, T, Hkv, 128)).astype(np.float32)
    V = rs.choice([-top, top, 0.0, 1e-3, top / 3, -5.0], size=(B, T, Hkv, 128)).astype(np.float32)
    K[:, :, :, 3] = top                      # constant column at the edge
    V[:, 9] = -top                           # constant row at the other edge
    K[:, :32, 0, 4] = np.linspace(-top, top, 32)
    tdt = synth.torch_dtype(dtype)
    K, V = torch.from_numpy(K).to(tdt), torch.from_numpy(V).to(tdt)
    bmap = np.array([[0, 1, 2, 3]], np.uint8)
    ocache = O.quantize_kv(synth.to_u16(K), synth.to_u16(V), dtype, chunk, bmap)
    cfg = mq.make_config(n_layers=1, n_q_heads=Hkv, n_kv_heads=Hkv, chunk=chunk, dtype=dtype, d_in=64,
                         max_tokens=T, batch=B)
    cache = mq.moqae_cache_bind(cfg, [1, 1, 1, 1], zero_pools=True)
    mq.moqae_quantize_kv(cfg, K.cuda(), V.cuda(), T, 0, cache, forced_map=torch.from_numpy(bmap).cuda())
    assert mq.moqae_poll_status(cache) == 0
    H.compare_pools(cache, ocache, 0)
    # and the decode kernel stays finite and accurate on such a cache (outputs are of the order of top)
    q = synth.normal((B, Hkv, 128), dtype, 5, "cpu", std=0.01)
    ref = O.decode_attn(synth.to_u16(q), dtype, ocache, chunk)
    ws = torch.zeros(mq.moqae_decode_attn_workspace(cfg), dtype=torch.uint8, device="cuda")
    out = torch.full((B, Hkv, 128), float("nan"), dtype=torch.float32, device="cuda")
    mq.moqae_decode_attn(cfg, q.cuda(), 0, cache, out, ws)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    assert np.isfinite(got).all()
    err = np.abs(got - ref)
    assert (err.max(-1) / np.abs(ref).max(-1)).max() <= 1e-2


@pytest.mark.parametrize("dtype", [0, 1])
def test_gpu_bytes_read_lane_by_lane_equal_the_layout_free_quantiser(dtype):
    # Layout-independent check: the bytes the GPU wrote are taken apart by tests/lane_reader.py (the
    # format as the decode lanes see it, none of the oracle's location functions) and compared with
    # the oracle's quantiser arithmetic on the raw tile, which knows nothing about any layout.
    from tests.lane_reader import read_tile_as_lanes
    B, T, Hkv, chunk = 2, 64 * 3, 2, 64
    K, V = H.make_kv(B, T, Hkv, dtype, 131 + dtype)
    bmap = np.array([[0, 1, 2], [2, 0, 1]], np.uint8)
    cfg = mq.make_config(n_layers=1, n_q_heads=Hkv, n_kv_heads=Hkv, chunk=chunk, dtype=dtype, d_in=64,
                         max_tokens=T, batch=B)
    cache = mq.moqae_cache_bind(cfg, [1, 1, 1, 1], zero_pools=True)
    mq.moqae_quantize_kv(cfg, K.cuda(), V.cuda(), T, 0, cache, forced_map=torch.from_numpy(bmap).cuda())
    torch.cuda.synchronize()
    K32, V32 = O.to_f32(synth.to_u16(K), dtype), O.to_f32(synth.to_u16(V), dtype)
    for b in range(B):
        for c in range(T // chunk):
            w = int(bmap[b, c])
            bits = (2, 4, 8)[w]
            for h in range(Hkv):
                slot = cache.pool(w)[0, b, h, 0].cpu().numpy()          # each width occurs once per sequence
                for ti in range(chunk // 32):
                    t0 = c * chunk + 32 * ti
                    blob = slot[ti * O.tile_bytes(bits):(ti + 1) * O.tile_bytes(bits)]
                    got = read_tile_as_lanes(blob, bits)
                    want = O.quantize_tile(K32[b, t0:t0 + 32, h], V32[b, t0:t0 + 32, h], bits)
                    for k in want:
                        a, e = got[k], want[k]
                        if a.dtype == np.float16:
                            a, e = a.view(np.uint16), e.view(np.uint16)
                        assert (a == e).all(), (b, c, h, ti, k)


def test_constant_groups_and_ties():
    B, T, Hkv, chunk = 1, 96, 1, 32
    K = torch.zeros(B, T, Hkv, 128, dtype=torch.float16)
    V = torch.zeros(B, T, Hkv, 128, dtype=torch.float16)
    K[:, :, :, 1] = 3.25                     # constant column -> scale 0
    K[:, ::2, :, 2] = 1.0                    # two-level column
    V[:, :, :, 40:44] = torch.tensor([0.5, 1.5, 2.5, 3.0])   # exact halves -> round to even
    V[:, 5] = -7.0                           # constant row
    bmap = np.array([[0, 1, 2]], np.uint8)
    ocache = O.quantize_kv(synth.to_u16(K), synth.to_u16(V), 0, chunk, bmap)
    cfg = mq.make_config(n_layers=1, n_q_heads=1, n_kv_heads=1, chunk=chunk, dtype=0, d_in=64,
                         max_tokens=T, batch=B)
    cache = mq.moqae_cache_bind(cfg, [1, 1, 1, 1], zero_pools=True)
    mq.moqae_quantize_kv(cfg, K.cuda(), V.cuda(), T, 0, cache, forced_map=torch.from_numpy(bmap).cuda())
    H.compare_pools(cache, ocache, 0)


def test_layers_of_a_sharing_group_use_one_map():
    # routing sharing: layers 0 and 1 (group of 2) are packed with the same map and slots
    B, T, Hkv, chunk = 1, 32 * 5, 2, 32
    bmap = np.array([[3, 0, 2, 0, 1]], np.uint8)
    K, V = H.make_kv(B, T, Hkv, 1, 21)
    K2, V2 = H.make_kv(B, T, Hkv, 1, 22)
    cfg = mq.make_config(n_layers=3, n_q_heads=Hkv, n_kv_heads=Hkv, chunk=chunk, dtype=1, d_in=64,
                         max_tokens=T, batch=B, rs_group=2)
    cache = mq.moqae_cache_bind(cfg, [2, 2, 2, 2], zero_pools=True)
    mq.moqae_quantize_kv(cfg, K.cuda(), V.cuda(), T, 0, cache, forced_map=torch.from_numpy(bmap).cuda())
    mq.moqae_quantize_kv(cfg, K2.cuda(), V2.cuda(), T, 1, cache)          # no map given: the group's
    assert (cache.map[0, 0, :5].cpu().numpy() == bmap[0]).all()
    H.compare_pools(cache, O.quantize_kv(synth.to_u16(K), synth.to_u16(V), 1, chunk, bmap), 0)
    H.compare_pools(cache, O.quantize_kv(synth.to_u16(K2), synth.to_u16(V2), 1, chunk, bmap), 1)


def test_pool_full_is_reported_not_written():
    B, T, Hkv, chunk = 1, 32 * 4, 1, 32
    bmap = np.array([[0, 0, 0, 1]], np.uint8)
    K, V = H.make_kv(B, T, Hkv, 0, 31)
    cfg = mq.make_config(n_layers=1, n_q_heads=1, n_kv_heads=1, chunk=chunk, dtype=0, d_in=64,
                         max_tokens=T, batch=B)
    cache = mq.moqae_cache_bind(cfg, [2, 1, 1, 1], zero_pools=True)       # three 2-bit chunks, room for two
    guard = cache.buffers[0].clone()
    mq.moqae_quantize_kv(cfg, K.cuda(), V.cuda(), T, 0, cache, forced_map=torch.from_numpy(bmap).cuda())
    assert mq.moqae_poll_status(cache) == mq.ERR_POOL_FULL
    used = 2 * 32 * 96
    assert (cache.buffers[0][used:] == guard[used:]).all()               # nothing beyond the pool's end
