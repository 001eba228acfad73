"""GPU parity at the full size of the two multi-head-attention workloads, in the launch
configurations the benchmark uses for them (query group of one, 32 / 40 kv heads, chunk 128,
router inputs of width 4096 / 5120, bf16):

  * Llama-2-7B shape: one layer, one sequence of 32768 (+ tail) tokens, 32 heads;
  * Llama-2-13B shape: one routing-sharing group of 4 layers, 40 heads, a context that starts 8
    tokens short of 65536: 8 decode steps fill the 16-bit tail (Section 3.2: tokens that do not
    fill a chunk stay 16-bit), moqae_flush_tail turns it into one more routed, quantised chunk, and
    8 more steps follow; attention is checked after every step.

Inputs are drawn on the device; sampled pieces are copied to the host and recomputed by the
oracle: router chunks (near-tie chunks through the reachable-winner rule), packed slots byte for
byte, and the attention of sampled heads over the whole context from the GPU's own packed cache.
"""
import numpy as np
import pytest
import torch

from oracle import moqae_oracle as O
from paper_2506_07533_b200 import binding as mq
from paper_2506_07533_b200 import synth
from paper_2506_07533_b200 import workloads as W
from tests import helpers as H

pytestmark = pytest.mark.gpu


def check_slots(cache, layer, K, V, wl, picks):
    """Packed bytes of sampled (sequence, chunk, head) slots against the oracle's quantiser + packer."""
    g = layer // cache.cfg.rs_group
    for b, c, h in picks:
        w = int(cache.map[g, b, c].item())
        s = int(cache.slot[g, b, c].item())
        Kc = K[b, c * wl.chunk:(c + 1) * wl.chunk, h].unsqueeze(0).unsqueeze(2)
        Vc = V[b, c * wl.chunk:(c + 1) * wl.chunk, h].unsqueeze(0).unsqueeze(2)
        ref = O.quantize_kv(synth.to_u16(Kc), synth.to_u16(Vc), wl.dtype, wl.chunk, np.array([[w]], np.uint8))
        got = cache.pool(w)[layer, b, h, s].cpu().numpy()
        assert (got == ref["pools"][w][0, 0, 0]).all(), (layer, b, c, h, w)


def check_decode_head(cache, layer, b, h, q_row, out_row, wl, C):
    oc = H.oracle_cache_of_head(cache, layer, b, h, C)
    ref = O.decode_attn(synth.to_u16(q_row).reshape(1, 1, 128), wl.dtype, oc, wl.chunk)
    ok, e_abs, e_rel = H.attn_tolerance_ok(out_row.cpu().numpy().reshape(1, 1, 128), ref)
    assert ok, (layer, b, h, e_abs, e_rel)


def test_llama2_7b_shape_one_layer():
    wl = W.WORKLOADS["cfg2"]
    B, Hkv, Hq, chunk, D, dtype = wl.batch, wl.n_kv_heads, wl.n_q_heads, wl.chunk, wl.d_in, wl.dtype
    assert Hq == Hkv == 32 and chunk == 128 and D == 4096
    T = wl.context + 29
    C = T // chunk
    dev = "cuda"
    cfg = mq.make_config(n_layers=1, n_q_heads=Hq, n_kv_heads=Hkv, chunk=chunk, dtype=dtype, d_in=D,
                         max_tokens=T, batch=B, rs_group=1, rf_first_chunk=1, tail_capacity=chunk)
    hidden = synth.hidden_states(B, T, D, chunk, dtype, 6161, dev)
    W1, W2, W3, bias = synth.router_weights(D, 4, dtype, 6162, dev)
    K, V = synth.keys_values(B, T, Hkv, 128, dtype, 6163, dev, outlier_frac=wl.outlier_frac)
    q = synth.normal((B, Hq, 128), dtype, 6164, dev)
    cache = mq.moqae_cache_bind(cfg, [C, C, C, C])
    mq.moqae_route(cfg, hidden, T, W1, W2, W3, bias, 0, cache)
    torch.cuda.synchronize()
    gmap, gvotes = cache.map[0, :, :C].cpu().numpy().copy(), cache.votes[0, :, :C].cpu().numpy().copy()
    assert (gmap[:, 0] == 3).all()
    w1, w2 = synth.to_u16(W1), synth.to_u16(W2)
    rs = np.random.RandomState(15)
    chunks = [1, C - 1] + list(rs.choice(np.arange(2, C - 1), 14, replace=False))
    n_fragile = 0
    for c in chunks:
        rows = synth.to_u16(hidden[0, c * chunk:(c + 1) * chunk])
        n_fragile += H.check_routed_chunk(rows, dtype, w1, w2, W3.cpu().numpy(), bias.cpu().numpy(), gvotes[0, c], gmap[0, c])
    assert n_fragile <= len(chunks) // 2
    slot, count = O.assign_slots(gmap)
    assert (cache.slot[0, :, :C].cpu().numpy() == slot).all() and (cache.count[0].cpu().numpy() == count).all()
    # the cache is built from a seeded map with the workload's 10/40/40/10 mix
    forced = synth.multinomial_map(B, C, wl.mix, 79)
    mq.moqae_quantize_kv(cfg, K, V, T, 0, cache, forced_map=torch.from_numpy(forced).to(dev))
    torch.cuda.synchronize()
    assert mq.moqae_poll_status(cache) == 0
    picks = []
    for w in range(4):
        where = np.argwhere(forced[0] == w)[:, 0]
        picks += [(0, int(c), int(rs.randint(Hkv))) for c in rs.choice(where, 6, replace=False)]
    check_slots(cache, 0, K, V, wl, picks)
    ws = torch.zeros(mq.moqae_decode_attn_workspace(cfg), dtype=torch.uint8, device=dev)
    out = torch.full((B, Hq, 128), float("nan"), dtype=torch.float32, device=dev)
    mq.moqae_decode_attn(cfg, q, 0, cache, out, ws)
    torch.cuda.synchronize()
    assert mq.moqae_poll_status(cache) == 0 and torch.isfinite(out).all()
    for h in (0, 17, Hkv - 1):
        check_decode_head(cache, 0, 0, h, q[0, h], out[0, h], wl, C)


def test_llama2_13b_shape_generation_across_a_chunk_boundary():
    wl = W.WORKLOADS["cfg3"]
    Hkv, Hq, chunk, D, dtype, L = wl.n_kv_heads, wl.n_q_heads, wl.chunk, wl.d_in, wl.dtype, wl.rs_group
    assert Hq == Hkv == 40 and chunk == 128 and D == 5120 and L == 4
    B, n_new = 1, 8
    T1 = wl.context                      # 65536 = 512 whole chunks once the tail has been flushed
    T0 = T1 - n_new
    T2 = T1 + n_new
    dev = "cuda"
    cfg = mq.make_config(n_layers=L, n_q_heads=Hq, n_kv_heads=Hkv, chunk=chunk, dtype=dtype, d_in=D,
                         max_tokens=T1 + chunk, batch=B, rs_group=L, rf_first_chunk=1, tail_capacity=chunk)
    hidden = synth.hidden_states(B, T1, D, chunk, dtype, 7171, dev)
    W1, W2, W3, bias = synth.router_weights(D, 4, dtype, 7172, dev)
    KV = [synth.keys_values(B, T2, Hkv, 128, dtype, 7180 + l, dev, outlier_frac=wl.outlier_frac) for l in range(L)]
    C0, C1 = T0 // chunk, T1 // chunk
    cache = mq.moqae_cache_bind(cfg, [C1, C1, C1, C1])
    mq.moqae_route(cfg, hidden[:, :T0].contiguous(), T0, W1, W2, W3, bias, 0, cache)
    for l in range(L):
        mq.moqae_quantize_kv(cfg, KV[l][0][:, :T0].contiguous(), KV[l][1][:, :T0].contiguous(), T0, l, cache)
    torch.cuda.synchronize()
    assert mq.moqae_poll_status(cache) == 0
    assert (cache.tail_len.cpu().numpy() == chunk - n_new).all()
    gmap = cache.map[0, :, :C0].cpu().numpy().copy()
    w1, w2 = synth.to_u16(W1), synth.to_u16(W2)
    rs = np.random.RandomState(16)
    for c in [1, C0 - 1] + list(rs.choice(np.arange(2, C0 - 1), 8, replace=False)):
        H.check_routed_chunk(synth.to_u16(hidden[0, c * chunk:(c + 1) * chunk]), dtype, w1, w2, W3.cpu().numpy(),
                             bias.cpu().numpy(), cache.votes[0, 0, c].cpu().numpy(), gmap[0, c])
    for l in range(L):
        picks = [(0, int(c), int(rs.randint(Hkv))) for c in rs.choice(C0, 5, replace=False)]
        check_slots(cache, l, KV[l][0], KV[l][1], wl, picks)

    ws = torch.zeros(mq.moqae_decode_attn_workspace(cfg), dtype=torch.uint8, device=dev)
    out = torch.full((L, B, Hq, 128), float("nan"), dtype=torch.float32, device=dev)

    def step(s, n_chunks):
        # one generated token: its K/V rows join every layer's tail, then every layer attends
        for l in range(L):
            K, V = KV[l]
            mq.moqae_append_kv(cfg, K[:, T0 + s].contiguous(), V[:, T0 + s].contiguous(), l, cache)
        q = synth.normal((L, B, Hq, 128), dtype, 7300 + s, dev)
        for l in range(L):
            mq.moqae_decode_attn(cfg, q[l], l, cache, out[l], ws)
        torch.cuda.synchronize()
        assert mq.moqae_poll_status(cache) == 0 and torch.isfinite(out).all()
        l, h = s % L, int(rs.randint(Hkv))                # one sampled (layer, head) per step
        check_decode_head(cache, l, 0, h, q[l, 0, h], out[l, 0, h], wl, n_chunks)

    for s in range(n_new):
        step(s, C0)
        assert (cache.tail_len.cpu().numpy() == chunk - n_new + s + 1).all()
    # the tail is a complete chunk now: route it on the buffered hidden rows, quantise it in all layers
    mq.moqae_flush_tail(cfg, hidden[:, T1 - chunk:T1].contiguous(), W1, W2, W3, bias, 0, cache)
    torch.cuda.synchronize()
    assert mq.moqae_poll_status(cache) == 0
    assert (cache.tail_len.cpu().numpy() == 0).all()
    new_w = int(cache.map[0, 0, C1 - 1].item())
    assert new_w < 4 and (cache.map[0, :, :C0].cpu().numpy() == gmap).all()       # older chunks keep their widths
    H.check_routed_chunk(synth.to_u16(hidden[0, T1 - chunk:T1]), dtype, w1, w2, W3.cpu().numpy(), bias.cpu().numpy(),
                         cache.votes[0, 0, C1 - 1].cpu().numpy(), new_w)
    slot, count = O.assign_slots(cache.map[0, :, :C1].cpu().numpy())
    assert (cache.slot[0, :, :C1].cpu().numpy() == slot).all() and (cache.count[0].cpu().numpy() == count).all()
    for l in range(L):
        check_slots(cache, l, KV[l][0], KV[l][1], wl, [(0, C1 - 1, int(rs.randint(Hkv))), (0, C1 - 1, 0)])
    for s in range(n_new, 2 * n_new):
        step(s, C1)
        assert (cache.tail_len.cpu().numpy() == s - n_new + 1).all()
