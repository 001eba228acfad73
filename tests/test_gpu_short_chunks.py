"""GPU parity for chunks of 8 and 16 tokens (the small sizes of the paper's chunk-size ablation):
router votes per chunk, packed bytes of the one-tile slots (padding included), decode attention
that must not attend to the padding, appends and a tail flush - all against the oracle."""
import numpy as np
import pytest
import torch

from oracle import moqae_oracle as O
from paper_2506_07533_b200 import binding as mq
from paper_2506_07533_b200 import synth
from tests import helpers as H
from tests.test_gpu_route import check_route

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("chunk", [8, 16])
@pytest.mark.parametrize("rf", [True, False])
def test_route(chunk, rf):
    # odd and even numbers of routed chunks, a tail, gated and linear routers
    check_route(2, chunk * 13 + 5, 128, chunk, 1, True, rf, seed=40 + chunk, w_std=0.1)
    check_route(1, chunk * 6, 64, chunk, 0, False, rf, seed=41 + chunk, w_std=0.1)
    check_route(1, chunk, 64, chunk, 0, True, rf, seed=42)


@pytest.mark.parametrize("chunk", [8, 16])
@pytest.mark.parametrize("dtype", [0, 1])
def test_quantize_and_decode(chunk, dtype):
    B, T, Hq, Hkv = 2, chunk * 21 + 5, 4, 2
    K, V = H.make_kv(B, T, Hkv, dtype, 600 + chunk + dtype)
    bmap = np.random.RandomState(chunk + dtype).randint(0, 4, size=(B, T // chunk)).astype(np.uint8)
    ocache = O.quantize_kv(synth.to_u16(K), synth.to_u16(V), dtype, chunk, bmap)
    cfg = mq.make_config(n_layers=1, n_q_heads=Hq, n_kv_heads=Hkv, chunk=chunk, dtype=dtype, d_in=64,
                         max_tokens=T, batch=B)
    cap = [max(1, int(ocache["count"][:, w].max())) for w in range(4)]
    cache = mq.moqae_cache_bind(cfg, cap, zero_pools=True)
    # poison the pools: the quantiser must write the padding itself
    for w in range(4):
        cache.buffers[w].fill_(0xEE)
    mq.moqae_quantize_kv(cfg, K.cuda(), V.cuda(), T, 0, cache, forced_map=torch.from_numpy(bmap).cuda())
    assert mq.moqae_poll_status(cache) == 0
    H.compare_pools(cache, ocache, 0)
    q = synth.normal((B, Hq, 128), dtype, 700 + chunk, "cpu")
    ws = torch.zeros(mq.moqae_decode_attn_workspace(cfg), dtype=torch.uint8, device="cuda")
    out = torch.full((B, Hq, 128), float("nan"), dtype=torch.float32, device="cuda")
    mq.moqae_decode_attn(cfg, q.cuda(), 0, cache, out, ws)
    torch.cuda.synchronize()
    ok, e_abs, e_rel = H.attn_tolerance_ok(out.cpu().numpy(), O.decode_attn(synth.to_u16(q), dtype, ocache, chunk))
    assert ok, (e_abs, e_rel)


@pytest.mark.parametrize("chunk", [8, 16])
def test_uniform_two_bit_many_chunks_and_wide_query_group(chunk):
    # enough 2-bit tiles for the paired path of the decode kernel, 8 query heads per kv head
    B, T, Hq, Hkv, dtype = 1, chunk * 150 + 3, 8, 1, 1
    K, V = H.make_kv(B, T, Hkv, dtype, 620 + chunk)
    bmap = np.zeros((B, T // chunk), np.uint8)
    ocache = O.quantize_kv(synth.to_u16(K), synth.to_u16(V), dtype, chunk, bmap)
    cfg = mq.make_config(n_layers=1, n_q_heads=Hq, n_kv_heads=Hkv, chunk=chunk, dtype=dtype, d_in=64,
                         max_tokens=T, batch=B)
    cache = mq.moqae_cache_bind(cfg, [T // chunk, 1, 1, 1], zero_pools=True)
    mq.moqae_quantize_kv(cfg, K.cuda(), V.cuda(), T, 0, cache, forced_map=torch.from_numpy(bmap).cuda())
    H.compare_pools(cache, ocache, 0)
    q = synth.normal((B, Hq, 128), dtype, 720 + chunk, "cpu")
    ws = torch.zeros(mq.moqae_decode_attn_workspace(cfg), dtype=torch.uint8, device="cuda")
    out = torch.full((B, Hq, 128), float("nan"), dtype=torch.float32, device="cuda")
    mq.moqae_decode_attn(cfg, q.cuda(), 0, cache, out, ws)
    torch.cuda.synchronize()
    ok, e_abs, e_rel = H.attn_tolerance_ok(out.cpu().numpy(), O.decode_attn(synth.to_u16(q), dtype, ocache, chunk))
    assert ok, (e_abs, e_rel)


@pytest.mark.parametrize("chunk", [8, 16])
def test_append_and_flush(chunk):
    # generation across a chunk boundary: the tail fills up, is routed and packed as one more short chunk
    B, Hq, Hkv, D, dtype = 2, 2, 2, 64, 1
    T1 = chunk * 5
    T0 = T1 - 3
    cfg = mq.make_config(n_layers=1, n_q_heads=Hq, n_kv_heads=Hkv, chunk=chunk, dtype=dtype, d_in=D,
                         max_tokens=T1 + chunk, batch=B, rf_first_chunk=1, tail_capacity=chunk)
    cache = mq.moqae_cache_bind(cfg, [6, 6, 6, 6], zero_pools=True)
    hid = synth.hidden_states(B, T1, D, chunk, dtype, 800 + chunk, "cpu")
    W1, W2, W3, bias = synth.router_weights(D, 4, dtype, 801, "cpu", std=0.2)
    K, V = H.make_kv(B, T1, Hkv, dtype, 802 + chunk)
    mq.moqae_route(cfg, hid[:, :T0].contiguous().cuda(), T0, W1.cuda(), W2.cuda(), W3.cuda(), bias.cuda(), 0, cache)
    mq.moqae_quantize_kv(cfg, K[:, :T0].contiguous().cuda(), V[:, :T0].contiguous().cuda(), T0, 0, cache)
    for s in range(T0, T1):
        mq.moqae_append_kv(cfg, K[:, s].contiguous().cuda(), V[:, s].contiguous().cuda(), 0, cache)
    mq.moqae_flush_tail(cfg, hid[:, T1 - chunk:T1].contiguous().cuda(), W1.cuda(), W2.cuda(), W3.cuda(), bias.cuda(), 0, cache)
    torch.cuda.synchronize()
    assert mq.moqae_poll_status(cache) == 0
    assert (cache.tail_len.cpu().numpy() == 0).all()
    C = T1 // chunk
    gmap = cache.map[0, :, :C].cpu().numpy()
    assert (gmap < 4).all() and (gmap[:, 0] == 3).all()
    w1, w2 = synth.to_u16(W1), synth.to_u16(W2)
    for b in range(B):
        H.check_routed_chunk(synth.to_u16(hid[b, T1 - chunk:T1]), dtype, w1, w2, W3.numpy(), bias.numpy(),
                             cache.votes[0, b, C - 1].cpu().numpy(), gmap[b, C - 1])
    ocache = O.quantize_kv(synth.to_u16(K), synth.to_u16(V), dtype, chunk, gmap)
    H.compare_pools(cache, ocache, 0)
    q = synth.normal((B, Hq, 128), dtype, 803, "cpu")
    ws = torch.zeros(mq.moqae_decode_attn_workspace(cfg), dtype=torch.uint8, device="cuda")
    out = torch.full((B, Hq, 128), float("nan"), dtype=torch.float32, device="cuda")
    mq.moqae_decode_attn(cfg, q.cuda(), 0, cache, out, ws)
    torch.cuda.synchronize()
    ok, e_abs, e_rel = H.attn_tolerance_ok(out.cpu().numpy(), O.decode_attn(synth.to_u16(q), dtype, ocache, chunk))
    assert ok, (e_abs, e_rel)


def test_kernels_that_need_whole_tiles_refuse_short_chunks():
    cfg = mq.make_config(n_layers=1, n_q_heads=2, n_kv_heads=2, chunk=8, dtype=1, d_in=64, max_tokens=64, batch=1)
    cache = mq.moqae_cache_bind(cfg, [1, 1, 1, 1])
    q = torch.zeros((1, 64, 2, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((1, 64, 2, 128), dtype=torch.float32, device="cuda")
    with pytest.raises(mq.MoqaeError) as e:
        mq.moqae_prefill_attn(cfg, q, 64, 0, cache, out)
    assert e.value.code == mq.ERR_UNSUPPORTED
    hid = torch.zeros((1, 64, 64), dtype=torch.bfloat16, device="cuda")
    W = torch.zeros((256, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(mq.MoqaeError) as e:
        mq.moqae_project_quantize_kv(cfg, hid, W, W, 64, 0, cache)
    assert e.value.code == mq.ERR_UNSUPPORTED
