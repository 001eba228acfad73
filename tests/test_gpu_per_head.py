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
