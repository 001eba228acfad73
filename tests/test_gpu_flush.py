"""GPU parity: moqae_flush_tail.  Prefill a context that ends 8 tokens short of a chunk boundary,
append the 8 tokens to every layer, flush, and compare with the oracle run on the full context
(one more routed chunk, empty tail): map / slot / count, packed bytes of every layer, attention."""
import numpy as np
import pytest
import torch

from oracle import moqae_oracle as O
from paper_2506_07533_b200 import binding as mq
from paper_2506_07533_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu

TAU = 1e-4


def _votes_ok(got_votes, got_w, ref, c, chunk):
    """Vote histogram of chunk c against the oracle's, allowing flips of near-tied tokens."""
    sl = slice(c * chunk, (c + 1) * chunk)
    frag = np.where(ref["margin"][sl] < TAU * np.maximum(ref["pmax"][sl], 1e-30))[0]
    diff = got_votes.astype(np.int64) - ref["votes"][c]
    assert diff.sum() == 0 and np.abs(diff).sum() // 2 <= len(frag), (diff, len(frag))
    if len(frag) == 0:
        assert got_w == ref["map"][c]


@pytest.mark.parametrize("dtype,gated", [(1, True), (0, False)])
def test_flush_adds_one_routed_chunk(dtype, gated):
    B, Hq, Hkv, chunk, D, L, rs = 2, 4, 2, 64, 128, 3, 2
    n_new = 8
    T1 = chunk * 4                      # context after the flush: 4 whole chunks
    T0 = T1 - n_new                     # prefill: 3 chunks + 56 tail tokens
    n_groups = 2
    cfg = mq.make_config(n_layers=L, n_q_heads=Hq, n_kv_heads=Hkv, chunk=chunk, dtype=dtype, d_in=D,
                         max_tokens=T1 + chunk, batch=B, rs_group=rs, rf_first_chunk=1, tail_capacity=chunk)
    cache = mq.moqae_cache_bind(cfg, [5, 5, 5, 5], zero_pools=True)
    hid = [synth.hidden_states(B, T1, D, chunk, dtype, 300 + g, "cpu") for g in range(n_groups)]
    Wg = [synth.router_weights(D, 4, dtype, 310 + g, "cpu", std=0.2, gated=gated) for g in range(n_groups)]
    KV = [H.make_kv(B, T1, Hkv, dtype, 320 + l) for l in range(L)]
    cu = lambda t: None if t is None else t.cuda()
    # prefill
    for g in range(n_groups):
        W1, W2, W3, bias = Wg[g]
        mq.moqae_route(cfg, hid[g][:, :T0].contiguous().cuda(), T0, cu(W1), cu(W2), cu(W3), cu(bias), g, cache)
    for l in range(L):
        K, V = KV[l]
        mq.moqae_quantize_kv(cfg, K[:, :T0].contiguous().cuda(), V[:, :T0].contiguous().cuda(), T0, l, cache)
    assert (cache.tail_len.cpu().numpy() == chunk - n_new).all()
    # a flush with tails that are not full changes nothing
    before = [b.clone() for b in cache.buffers[4:8]]
    for g in range(n_groups):
        W1, W2, W3, bias = Wg[g]
        mq.moqae_flush_tail(cfg, hid[g][:, T1 - chunk:T1].contiguous().cuda(), cu(W1), cu(W2), cu(W3), cu(bias), g, cache)
    torch.cuda.synchronize()
    assert (cache.tail_len.cpu().numpy() == chunk - n_new).all()
    assert torch.equal(before[0], cache.buffers[4]) and torch.equal(before[1], cache.buffers[5])
    assert torch.equal(before[2], cache.buffers[6])
    # generation: 8 tokens appended to every layer, then the flush
    for s in range(n_new):
        for l in range(L):
            K, V = KV[l]
            mq.moqae_append_kv(cfg, K[:, T0 + s].contiguous().cuda(), V[:, T0 + s].contiguous().cuda(), l, cache)
    assert (cache.tail_len.cpu().numpy() == chunk).all()
    for g in range(n_groups):
        W1, W2, W3, bias = Wg[g]
        mq.moqae_flush_tail(cfg, hid[g][:, T1 - chunk:T1].contiguous().cuda(), cu(W1), cu(W2), cu(W3), cu(bias), g, cache)
    torch.cuda.synchronize()
    assert mq.moqae_poll_status(cache) == 0
    assert (cache.tail_len.cpu().numpy() == 0).all()
    C = T1 // chunk
    for g in range(n_groups):
        W1, W2, W3, bias = Wg[g]
        gmap = cache.map[g, :, :C].cpu().numpy()
        assert (gmap < 4).all()                                      # no marker bit left behind
        gvotes = cache.votes[g, :, :C].cpu().numpy()
        ref = O.route(synth.to_u16(hid[g]), dtype, chunk, synth.to_u16(W1),
                      None if W2 is None else synth.to_u16(W2), None if W3 is None else W3.numpy(), bias.numpy())
        for b in range(B):
            one = {k: (v[b] if hasattr(v, "shape") and v.shape[0] == B else v) for k, v in ref.items()}
            for c in range(1, C):
                _votes_ok(gvotes[b, c], gmap[b, c], one, c, chunk)
        slot, count = O.assign_slots(gmap)
        assert (cache.slot[g, :, :C].cpu().numpy() == slot).all()
        assert (cache.count[g].cpu().numpy() == count).all()
    # packed bytes of every layer equal the oracle's on the full context with the GPU's map
    ws = torch.zeros(mq.moqae_decode_attn_workspace(cfg), dtype=torch.uint8, device="cuda")
    for l in range(L):
        K, V = KV[l]
        gmap = cache.map[l // rs, :, :C].cpu().numpy()
        ocache = O.quantize_kv(synth.to_u16(K), synth.to_u16(V), dtype, chunk, gmap)
        assert ocache["tail_len"] == 0
        H.compare_pools(cache, ocache, l)
        q = synth.normal((B, Hq, 128), dtype, 400 + l, "cpu")
        out = torch.empty((B, Hq, 128), dtype=torch.float32, device="cuda")
        mq.moqae_decode_attn(cfg, q.cuda(), l, cache, out, ws)
        torch.cuda.synchronize()
        ok, e_abs, e_rel = H.attn_tolerance_ok(out.cpu().numpy(), O.decode_attn(synth.to_u16(q), dtype, ocache, chunk))
        assert ok, (l, e_abs, e_rel)


def test_flush_of_a_first_chunk_is_frozen_to_16_bit():
    # a sequence shorter than one chunk at prefill: its first chunk appears at flush time and is 16-bit
    B, Hkv, chunk, D, dtype = 1, 1, 32, 64, 1
    cfg = mq.make_config(n_layers=1, n_q_heads=1, n_kv_heads=Hkv, chunk=chunk, dtype=dtype, d_in=D,
                         max_tokens=4 * chunk, batch=B, rf_first_chunk=1, tail_capacity=chunk)
    cache = mq.moqae_cache_bind(cfg, [2, 2, 2, 2], zero_pools=True)
    K, V = H.make_kv(B, chunk, Hkv, dtype, 500)
    hid = synth.hidden_states(B, chunk, D, chunk, dtype, 501, "cpu")
    W1, W2, W3, bias = synth.router_weights(D, 4, dtype, 502, "cpu", std=0.2)
    bias = torch.tensor([9.0, 0.0, 0.0, 0.0])                       # the router itself would say 2-bit
    mq.moqae_quantize_kv(cfg, K[:, :20].contiguous().cuda(), V[:, :20].contiguous().cuda(), 20, 0, cache)
    for s in range(20, chunk):
        mq.moqae_append_kv(cfg, K[:, s].contiguous().cuda(), V[:, s].contiguous().cuda(), 0, cache)
    mq.moqae_flush_tail(cfg, hid.cuda(), W1.cuda(), W2.cuda(), W3.cuda(), bias.cuda(), 0, cache)
    torch.cuda.synchronize()
    assert mq.moqae_poll_status(cache) == 0
    assert cache.map[0, 0, 0].item() == 3 and cache.count[0, 0].cpu().tolist() == [0, 0, 0, 1]
    assert cache.tail_len[0, 0].item() == 0
    ocache = O.quantize_kv(synth.to_u16(K), synth.to_u16(V), dtype, chunk, np.array([[3]], np.uint8))
    H.compare_pools(cache, ocache, 0)
