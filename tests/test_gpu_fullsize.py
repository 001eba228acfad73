"""GPU parity at the full size of the 128k-context workload (batch 4, 131072 (+ tail) tokens,
8 kv heads / 32 query heads, chunk 256, bf16, d_in 4096), one layer, in the launch
configuration the benchmark times.  Inputs are drawn on the device; sampled pieces are copied
to the host and recomputed by the oracle one by one:
  * router: sampled chunks (vote histograms away from near-ties, winner),
  * quantise+pack: every tile of sampled (sequence, kv head, chunk) slots, byte for byte,
  * decode attention: sampled (sequence, kv head) pairs over the whole context, all four
    query heads of the group, against the oracle run on the GPU's own packed cache and map,
  * prefill attention (32k prompt) and the fused projection + quantise (one layer of the 128k
    workload): sampled rows / slots, each in its own test below.
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

TAU = 1e-4


@pytest.fixture(scope="module")
def job():
    wl = W.WORKLOADS["cfg4"]
    B, Hkv, Hq, chunk, D, dtype = wl.batch, wl.n_kv_heads, wl.n_q_heads, wl.chunk, wl.d_in, wl.dtype
    T = wl.context + 37                                   # a ragged tail on top of 512 chunks
    dev = "cuda"
    cfg = mq.make_config(n_layers=1, n_q_heads=Hq, n_kv_heads=Hkv, chunk=chunk, dtype=dtype, d_in=D,
                         max_tokens=T, batch=B, rs_group=1, rf_first_chunk=1, tail_capacity=chunk)
    hidden = synth.hidden_states(B, T, D, chunk, dtype, 4242, dev)
    W1, W2, W3, bias = synth.router_weights(D, 4, dtype, 4243, dev)
    K, V = synth.keys_values(B, T, Hkv, 128, dtype, 4244, dev, outlier_frac=wl.outlier_frac)
    q = synth.normal((B, Hq, 128), dtype, 4245, dev)
    C = T // chunk
    cache = mq.moqae_cache_bind(cfg, [C, C, C, C])
    mq.moqae_route(cfg, hidden, T, W1, W2, W3, bias, 0, cache)
    torch.cuda.synchronize()
    routed = dict(map=cache.map[0, :, :C].cpu().numpy().copy(), votes=cache.votes[0, :, :C].cpu().numpy().copy(),
                  slot=cache.slot[0, :, :C].cpu().numpy().copy(), count=cache.count[0].cpu().numpy().copy())
    # the cache itself is built from a seeded map with the workload's 60/30/5/5 mix, so that every
    # width is present whatever the untrained synthetic router prefers
    forced = torch.from_numpy(synth.multinomial_map(B, C, wl.mix, 77)).to(dev)
    mq.moqae_quantize_kv(cfg, K, V, T, 0, cache, forced_map=forced)
    ws = torch.zeros(mq.moqae_decode_attn_workspace(cfg), dtype=torch.uint8, device=dev)
    out = torch.full((B, Hq, 128), float("nan"), dtype=torch.float32, device=dev)
    mq.moqae_decode_attn(cfg, q, 0, cache, out, ws)
    torch.cuda.synchronize()
    assert mq.moqae_poll_status(cache) == 0
    return dict(wl=wl, cfg=cfg, T=T, C=C, hidden=hidden, routed=routed, W=(W1, W2, W3, bias), K=K, V=V, q=q, cache=cache, out=out)


def test_router_sampled_chunks(job):
    wl, T, C, cache = job["wl"], job["T"], job["C"], job["cache"]
    W1, W2, W3, bias = job["W"]
    gmap, gvotes = job["routed"]["map"], job["routed"]["votes"]
    assert (gmap[:, 0] == 3).all()                        # routing freezing
    w1, w2 = synth.to_u16(W1), synth.to_u16(W2)
    rs = np.random.RandomState(5)
    picks = [(b, c) for b in range(wl.batch) for c in rs.choice(np.arange(1, C), 6, replace=False)]
    picks += [(0, 1), (wl.batch - 1, C - 1)]
    n_fragile = 0
    for b, c in picks:
        rows = job["hidden"][b, c * wl.chunk:(c + 1) * wl.chunk]
        n_fragile += H.check_routed_chunk(synth.to_u16(rows), wl.dtype, w1, w2, W3.cpu().numpy(), bias.cpu().numpy(),
                                          gvotes[b, c], gmap[b, c])
    assert n_fragile <= len(picks) // 2
    slot, count = O.assign_slots(gmap)
    assert (job["routed"]["slot"] == slot).all() and (job["routed"]["count"] == count).all()


def test_quantize_sampled_slots_byte_exact(job):
    wl, C, cache = job["wl"], job["C"], job["cache"]
    gmap = cache.map[0, :, :C].cpu().numpy()
    slot, _ = O.assign_slots(gmap)
    rs = np.random.RandomState(6)
    for w in range(4):                                    # ten slots of every width
        where = np.argwhere(gmap == w)
        assert len(where) >= 10
        for b, c in where[rs.choice(len(where), 10, replace=False)]:
            h = rs.randint(wl.n_kv_heads)
            Kc = job["K"][b, c * wl.chunk:(c + 1) * wl.chunk, h].unsqueeze(0).unsqueeze(2)
            Vc = job["V"][b, c * wl.chunk:(c + 1) * wl.chunk, h].unsqueeze(0).unsqueeze(2)
            ref = O.quantize_kv(synth.to_u16(Kc), synth.to_u16(Vc), wl.dtype, wl.chunk, gmap[b:b + 1, c:c + 1])
            got = cache.pool(w)[0, b, h, int(slot[b, c])].cpu().numpy()
            assert (got == ref["pools"][w][0, 0, 0]).all(), (b, h, c, w)
    r = job["T"] % wl.chunk
    assert (cache.tail_len[0].cpu().numpy() == r).all()
    tk = cache.tail("k")[0, 1, 3, :r].cpu().numpy().view(np.uint16)
    assert (tk == synth.to_u16(job["K"][1, C * wl.chunk:, 3])).all()


def test_decode_sampled_heads_whole_context(job):
    wl, C, T, cache = job["wl"], job["C"], job["T"], job["cache"]
    G = wl.n_q_heads // wl.n_kv_heads
    gmap = cache.map[0, :, :C].cpu().numpy()
    slot, count = O.assign_slots(gmap)
    out = job["out"].cpu().numpy()
    r = T % wl.chunk
    for b, h in [(0, 0), (3, 7), (2, 5)]:
        # the oracle reads the GPU's own packed bytes of this (sequence, head)
        pools = []
        for w in range(4):
            n = int(count[b, w])
            pools.append(cache.pool(w)[0, b, h, :max(n, 1)].cpu().numpy()[None, None])
        oc = dict(pools=pools, slot=slot[b:b + 1], count=count[b:b + 1], tail_len=r,
                  tail_k=cache.tail("k")[0, b, h, :r].cpu().numpy().view(np.uint16)[None, None],
                  tail_v=cache.tail("v")[0, b, h, :r].cpu().numpy().view(np.uint16)[None, None])
        qh = synth.to_u16(job["q"][b, h * G:(h + 1) * G]).reshape(1, G, 128)
        ref = O.decode_attn(qh, wl.dtype, oc, wl.chunk)
        ok, e_abs, e_rel = H.attn_tolerance_ok(out[b, h * G:(h + 1) * G][None], ref)
        assert ok, (b, h, e_abs, e_rel)


def test_prefill_attention_sampled_rows_at_the_32k_prompt():
    """Prefill attention at the size the benchmark times it (32 heads, 32768 (+ tail) tokens, chunk
    128, bf16, seeded mixed map), both with and without the fp16 workspace: sampled (head, position)
    rows are recomputed by the oracle from the GPU's own packed cache of that head."""
    wl = W.WORKLOADS["cfg2"]
    B, Hq, Hkv, chunk, dtype = 1, wl.n_q_heads, wl.n_kv_heads, wl.chunk, wl.dtype
    T = wl.context + 37
    C = T // chunk
    dev = "cuda"
    cfg = mq.make_config(n_layers=1, n_q_heads=Hq, n_kv_heads=Hkv, chunk=chunk, dtype=dtype, d_in=64,
                         max_tokens=T, batch=B, tail_capacity=chunk)
    K, V = synth.keys_values(B, T, Hkv, 128, dtype, 5151, dev, outlier_frac=wl.outlier_frac)
    q = synth.normal((B, T, Hq, 128), dtype, 5152, dev)
    cache = mq.moqae_cache_bind(cfg, [C, C, C, C])
    forced = torch.from_numpy(synth.multinomial_map(B, C, wl.mix, 78)).to(dev)
    mq.moqae_quantize_kv(cfg, K, V, T, 0, cache, forced_map=forced)
    outs = []
    ws = torch.empty(mq.moqae_prefill_attn_workspace(cfg, T), dtype=torch.uint8, device=dev)
    for workspace in (None, ws):
        out = torch.full((B, T, Hq, 128), float("nan"), dtype=torch.float32, device=dev)
        mq.moqae_prefill_attn(cfg, q, T, 0, cache, out, workspace=workspace)
        torch.cuda.synchronize()
        assert mq.moqae_poll_status(cache) == 0
        outs.append(out)
    gmap = cache.map[0, :, :C].cpu().numpy()
    slot, count = O.assign_slots(gmap)
    r = T % chunk
    abs_tol = 3 * 2.0 ** -11 * float(V.float().abs().max())
    G = Hq // Hkv
    rows = [0, 1, 31, 127, 128, 255, 256, 257, 4095, 4096, 17011, wl.context - 1, wl.context, T - 1]
    for h in (0, 13, Hkv - 1):
        pools = []
        for w in range(4):
            n = int(count[0, w])
            pools.append(cache.pool(w)[0, 0, h, :max(n, 1)].cpu().numpy()[None, None])
        oc = dict(pools=pools, map=gmap, slot=slot, count=count, tail_len=r,
                  tail_k=cache.tail("k")[0, 0, h, :r].cpu().numpy().view(np.uint16)[None, None],
                  tail_v=cache.tail("v")[0, 0, h, :r].cpu().numpy().view(np.uint16)[None, None])
        K64, V64 = O.cache_kv_rows_in_order(oc, dtype, chunk, 0, 0)
        assert K64.shape[0] == T
        for g in range(G):
            hq = h * G + g
            qh = O.to_f64(synth.to_u16(q[0, rows, hq]), dtype)                 # [rows, 128]
            for n, t in enumerate(rows):
                s = (K64[:t + 1] @ qh[n]) / np.sqrt(128.0)
                p = np.exp(s - s.max())
                want = (p @ V64[:t + 1]) / p.sum()
                for out in outs:
                    got = out[0, t, hq].cpu().numpy().astype(np.float64)
                    err = np.abs(got - want)
                    assert err.max() <= abs_tol and err.max() <= 1e-2 * max(np.abs(want).max(), 1e-30), (h, g, t, err.max())


def test_fused_producer_sampled_slots_at_the_layer_size():
    """moqae_project_quantize_kv at the size the benchmark times it (one layer of the 128k workload:
    4 x 131072 (+ tail) tokens, d_in 4096, 8 kv heads, seeded mixed map).  Sampled (sequence, chunk, kv
    head) slots: the rows the kernel rounded are within one unit in the last place (plus the float32
    accumulation bound) of the oracle's float64 projection of the same hidden rows, and the slot's
    packed bytes are what the oracle's quantiser makes of the kernel's own rows."""
    wl = W.WORKLOADS["cfg4"]
    B, Hkv, chunk, D, dtype = wl.batch, wl.n_kv_heads, wl.chunk, wl.d_in, wl.dtype
    T = wl.context + 37
    C = T // chunk
    dev = "cuda"
    cfg = mq.make_config(n_layers=1, n_q_heads=wl.n_q_heads, n_kv_heads=Hkv, chunk=chunk, dtype=dtype, d_in=D,
                         max_tokens=T, batch=B, rs_group=1, rf_first_chunk=1, tail_capacity=chunk)
    hidden = synth.hidden_states(B, T, D, chunk, dtype, 6161, dev)
    Wk = synth.normal((Hkv * 128, D), dtype, 6162, dev, std=1.0 / np.sqrt(D))
    Wv = synth.normal((Hkv * 128, D), dtype, 6163, dev, std=1.0 / np.sqrt(D))
    Wk[5] *= 10.0                                          # an outlier key channel
    cache = mq.moqae_cache_bind(cfg, [C, C, C, C])
    gmap = synth.multinomial_map(B, C, wl.mix, 79)
    tdt = synth.torch_dtype(dtype)
    k_r = torch.zeros((B, T, Hkv, 128), dtype=tdt, device=dev)
    v_r = torch.zeros((B, T, Hkv, 128), dtype=tdt, device=dev)
    mq.moqae_project_quantize_kv(cfg, hidden, Wk, Wv, T, 0, cache, forced_map=torch.from_numpy(gmap).to(dev),
                                 k_rounded=k_r, v_rounded=v_r)
    torch.cuda.synchronize()
    assert mq.moqae_poll_status(cache) == 0
    assert (cache.map[0, :, :C].cpu().numpy() == gmap).all()
    slot, count = O.assign_slots(gmap)
    assert (cache.slot[0, :, :C].cpu().numpy() == slot).all() and (cache.count[0].cpu().numpy() == count).all()
    wk, wv = synth.to_u16(Wk), synth.to_u16(Wv)

    def ulp_of(x64):
        sig, emin = (11, -14) if dtype == 0 else (8, -126)
        _, e = np.frexp(x64)
        return np.ldexp(1.0, np.maximum(e, emin + 1) - sig)

    def check_rows(b, t0, t1, h):
        rows = synth.to_u16(hidden[b, t0:t1])[None]                       # [1, n, D]
        _, _, K64, V64 = O.project_kv(rows, wk[h * 128:(h + 1) * 128], wv[h * 128:(h + 1) * 128], dtype, 1)
        absh = np.abs(O.to_f64(rows[0], dtype))
        for got_t, x64, wm in ((k_r, K64, wk), (v_r, V64, wv)):
            g = O.to_f64(synth.to_u16(got_t[b, t0:t1, h]), dtype)
            acc = D * 2.0 ** -24 * (absh @ np.abs(O.to_f64(wm[h * 128:(h + 1) * 128], dtype)).T)
            assert (np.abs(g - x64[0, :, 0]) <= ulp_of(x64[0, :, 0]) * 1.001 + acc).all(), (b, t0, h)

    rs = np.random.RandomState(8)
    for w in range(4):                                     # four slots of every width
        where = np.argwhere(gmap == w)
        for b, c in where[rs.choice(len(where), 4, replace=False)]:
            h = rs.randint(Hkv)
            check_rows(b, c * chunk, (c + 1) * chunk, h)
            Kc = synth.to_u16(k_r[b, c * chunk:(c + 1) * chunk, h])[None, :, None]
            Vc = synth.to_u16(v_r[b, c * chunk:(c + 1) * chunk, h])[None, :, None]
            ref = O.quantize_kv(Kc, Vc, dtype, chunk, gmap[b:b + 1, c:c + 1])
            got = cache.pool(w)[0, b, h, int(slot[b, c])].cpu().numpy()
            assert (got == ref["pools"][w][0, 0, 0]).all(), (b, h, c, w)
    # the trailing tokens stay 16-bit: the tail holds the kernel's rounded rows
    r = T % chunk
    assert (cache.tail_len[0].cpu().numpy() == r).all()
    check_rows(2, C * chunk, T, 6)
    assert (cache.tail("k")[0, 2, 6, :r].cpu().numpy().view(np.uint16) == synth.to_u16(k_r[2, C * chunk:, 6])).all()
    assert (cache.tail("v")[0, 2, 6, :r].cpu().numpy().view(np.uint16) == synth.to_u16(v_r[2, C * chunk:, 6])).all()
