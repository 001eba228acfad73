"""GPU parity: per-head routing with a 128-wide router input (the variant of Section 4.1 in which
every head routes its own chunks).  The library keeps one bit-width map per sequence, so a caller
gets per-head maps by handing over head-major tensors: sequence b, head h becomes "sequence"
b * H + h of a configuration with one kv head.  The whole path (route -> quantise+pack ->
decode attention) is checked against the oracle run the same way."""
import numpy as np
import pytest
import torch

from oracle import moqae_oracle as O
from paper_2506_07533_b200 import binding as mq
from paper_2506_07533_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu

TAU = 1e-4


def test_per_head_routing_as_head_major_batch():
    B, Hkv, G, chunk, dtype = 2, 3, 2, 64, 1
    T = chunk * 7 + 9
    K, V = H.make_kv(B, T, Hkv, dtype, 810, outlier_channels=(5, 64))
    head_major = lambda x: x.permute(0, 2, 1, 3).reshape(B * Hkv, T, 1, 128).contiguous()
    Kh, Vh = head_major(K), head_major(V)
    # each head's own 128 router features per token (seeded like the hidden states of the other tests)
    hidden = synth.hidden_states(B * Hkv, T, 128, chunk, dtype, 813, "cpu")
    W1, W2, W3, bias = synth.router_weights(128, 4, dtype, 811, "cpu", std=0.1)
    q = synth.normal((B * Hkv, G, 128), dtype, 812, "cpu")

    cfg = mq.make_config(n_layers=1, n_q_heads=G, n_kv_heads=1, chunk=chunk, dtype=dtype, d_in=128,
                         max_tokens=T, batch=B * Hkv)
    C = T // chunk
    cache = mq.moqae_cache_bind(cfg, [C, C, C, C], zero_pools=True)
    mq.moqae_route(cfg, hidden.cuda(), T, W1.cuda(), W2.cuda(), W3.cuda(), bias.cuda(), 0, cache)
    mq.moqae_quantize_kv(cfg, Kh.cuda(), Vh.cuda(), T, 0, cache)
    ws = torch.zeros(mq.moqae_decode_attn_workspace(cfg), dtype=torch.uint8, device="cuda")
    out = torch.full((B * Hkv, G, 128), float("nan"), dtype=torch.float32, device="cuda")
    mq.moqae_decode_attn(cfg, q.cuda(), 0, cache, out, ws)
    torch.cuda.synchronize()
    assert mq.moqae_poll_status(cache) == 0

    # the maps: equal to the oracle's wherever no token of the chunk sits on a near-tie
    ref = O.route(synth.to_u16(hidden), dtype, chunk, synth.to_u16(W1), synth.to_u16(W2), W3.numpy(), bias.numpy())
    gmap = cache.map[0, :, :C].cpu().numpy()
    firm = 0
    for s in range(B * Hkv):
        for c in range(C):
            sl = slice(c * chunk, (c + 1) * chunk)
            if (ref["margin"][s, sl] >= TAU * np.maximum(ref["pmax"][s, sl], 1e-30)).all():
                assert gmap[s, c] == ref["map"][s, c], (s, c)
                firm += 1
    assert firm > (B * Hkv * C) // 2
    assert (gmap[:, 0] == 3).all()                                         # routing freezing, per head
    assert any((gmap[b * Hkv] != gmap[b * Hkv + h]).any() for b in range(B) for h in range(1, Hkv))   # heads differ

    # packed bytes and attention against the oracle on the GPU's own maps
    ocache = O.quantize_kv(synth.to_u16(Kh), synth.to_u16(Vh), dtype, chunk, gmap)
    H.compare_pools(cache, ocache, 0)
    want = O.decode_attn(synth.to_u16(q), dtype, ocache, chunk)
    ok, e_abs, e_rel = H.attn_tolerance_ok(out.cpu().numpy(), want)
    assert ok, (e_abs, e_rel)


@pytest.mark.parametrize("chunk", [64, 16])
def test_per_head_routing_token_major(chunk):
    """cfg.per_head_routing: the tensors stay token-major ([batch][T][heads][128] for the router
    input, K and V alike) and the library keeps one map per (sequence, kv head).  The oracle sees
    the same data head by head (one single-head sequence per (b, h)): maps with the near-tie rule,
    packed bytes exactly, attention within tolerance."""
    B, Hkv, G, dtype = 2, 3, 2, 1
    T = chunk * 9 + 5
    C = T // chunk
    K, V = H.make_kv(B, T, Hkv, dtype, 820, outlier_channels=(5, 64))
    # every head's own 128 router features per token, chunk-structured per (sequence, head)
    hid_hm = synth.hidden_states(B * Hkv, T, 128, chunk, dtype, 823, "cpu")            # [(b, h), T, 128]
    hidden = hid_hm.view(B, Hkv, T, 128).permute(0, 2, 1, 3).contiguous()             # [B, T, H, 128]
    W1, W2, W3, bias = synth.router_weights(128, 4, dtype, 821, "cpu", std=0.1)
    q = synth.normal((B, Hkv * G, 128), dtype, 822, "cpu")
    cfg = mq.make_config(n_layers=1, n_q_heads=Hkv * G, n_kv_heads=Hkv, chunk=chunk, dtype=dtype, d_in=128,
                         max_tokens=T, batch=B, per_head_routing=True)
    cache = mq.moqae_cache_bind(cfg, [C, C, C, C], zero_pools=True)
    assert cache.map.shape == (1, B * Hkv, C)
    votes_out = torch.full((B * Hkv, C, 4), -1, dtype=torch.int32, device="cuda")
    mq.moqae_route(cfg, hidden.cuda(), T, W1.cuda(), W2.cuda(), W3.cuda(), bias.cuda(), 0, cache, votes_out)
    mq.moqae_quantize_kv(cfg, K.cuda(), V.cuda(), T, 0, cache)
    ws = torch.zeros(mq.moqae_decode_attn_workspace(cfg), dtype=torch.uint8, device="cuda")
    out = torch.full((B, Hkv * G, 128), float("nan"), dtype=torch.float32, device="cuda")
    mq.moqae_decode_attn(cfg, q.cuda(), 0, cache, out, ws)
    torch.cuda.synchronize()
    assert mq.moqae_poll_status(cache) == 0
    gmap = cache.map[0].cpu().numpy()
    gvotes = cache.votes[0].cpu().numpy()
    assert (votes_out.cpu().numpy() == gvotes[:, :C]).all()
    assert (gmap[:, 0] == 3).all()
    assert any((gmap[b * Hkv] != gmap[b * Hkv + h]).any() for b in range(B) for h in range(1, Hkv))   # heads differ
    w1, w2 = synth.to_u16(W1), synth.to_u16(W2)
    n_fragile = 0
    for b in range(B):
        for h in range(Hkv):
            s = b * Hkv + h
            for c in range(1, C):
                n_fragile += H.check_routed_chunk(synth.to_u16(hidden[b, c * chunk:(c + 1) * chunk, h]), dtype, w1, w2,
                                                  W3.numpy(), bias.numpy(), gvotes[s, c], gmap[s, c])
            # this head's slots against the oracle run on it as a one-head sequence with its own map
            oc = O.quantize_kv(synth.to_u16(K[b:b + 1, :, h:h + 1]), synth.to_u16(V[b:b + 1, :, h:h + 1]), dtype, chunk,
                               gmap[s:s + 1])
            assert (cache.count[0, s].cpu().numpy() == oc["count"][0]).all()
            assert (cache.slot[0, s, :C].cpu().numpy() == oc["slot"][0]).all()
            for w in range(4):
                n = int(oc["count"][0, w])
                if n:
                    assert (cache.pool(w)[0, b, h, :n].cpu().numpy() == oc["pools"][w][0, 0, :n]).all(), (b, h, w)
            want = O.decode_attn(synth.to_u16(q[b:b + 1, h * G:(h + 1) * G]), dtype, oc, chunk)
            ok, e_abs, e_rel = H.attn_tolerance_ok(out[b:b + 1, h * G:(h + 1) * G].cpu().numpy(), want)
            assert ok, (b, h, e_abs, e_rel)
    assert n_fragile < B * Hkv * C // 2


def test_per_head_routing_argument_rules():
    # the per-head router input is the head's own 128 channels
    bad = mq.make_config(n_layers=1, n_q_heads=2, n_kv_heads=2, chunk=32, dtype=1, d_in=256, max_tokens=64, batch=1,
                         per_head_routing=True)
    with pytest.raises(mq.MoqaeError) as e:
        mq.moqae_cache_bytes(bad, [1, 1, 1, 1])
    assert e.value.code == mq.ERR_UNSUPPORTED
    cfg = mq.make_config(n_layers=1, n_q_heads=2, n_kv_heads=2, chunk=32, dtype=1, d_in=128, max_tokens=64, batch=3,
                         per_head_routing=True)
    sizes = mq.moqae_cache_bytes(cfg, [1, 1, 1, 1])
    assert sizes[4] == 3 * 2 * 2 and sizes[6] == 3 * 2 * 16            # map and count rows per (sequence, head)
