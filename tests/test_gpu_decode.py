"""GPU parity: moqae_decode_attn against the oracle on the same packed cache."""
import numpy as np
import pytest
import torch

from oracle import moqae_oracle as O
from paper_2506_07533_b200 import binding as mq
from paper_2506_07533_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def decode_case(B, T, Hq, Hkv, chunk, dtype, bmap, seed, from_oracle_cache, q_scale=1.0):
    K, V = H.make_kv(B, T, Hkv, dtype, seed)
    q = synth.normal((B, Hq, 128), dtype, seed + 1, "cpu", std=q_scale)
    ocache = O.quantize_kv(synth.to_u16(K), synth.to_u16(V), dtype, chunk, bmap)
    ref = O.decode_attn(synth.to_u16(q), dtype, ocache, chunk)
    cfg = mq.make_config(n_layers=2, n_q_heads=Hq, n_kv_heads=Hkv, chunk=chunk, dtype=dtype, d_in=64,
                         max_tokens=max(T, chunk), batch=B)
    cap = [max(1, int(ocache["count"][:, w].max())) if bmap.size else 1 for w in range(4)]
    cache = mq.moqae_cache_bind(cfg, cap, zero_pools=True)
    layer = 1
    if from_oracle_cache:
        H.upload_oracle_cache(cache, ocache, layer)
    else:
        fm = torch.from_numpy(bmap).cuda() if bmap.size else None
        mq.moqae_quantize_kv(cfg, K.cuda(), V.cuda(), T, layer, cache, forced_map=fm)
    ws = torch.zeros(mq.moqae_decode_attn_workspace(cfg), dtype=torch.uint8, device="cuda")
    out = torch.full((B, Hq, 128), float("nan"), dtype=torch.float32, device="cuda")
    mq.moqae_decode_attn(cfg, q.cuda(), layer, cache, out, ws)
    torch.cuda.synchronize()
    ok, e_abs, e_rel = H.attn_tolerance_ok(out.cpu().numpy(), ref)
    assert ok, (e_abs, e_rel)
    return e_abs, e_rel


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("from_oracle_cache", [True, False])
def test_mixed_cache_mha(dtype, from_oracle_cache):
    B, T, chunk = 2, 32 * 9 + 11, 32
    rs = np.random.RandomState(3 + dtype)
    bmap = rs.randint(0, 4, size=(B, T // chunk)).astype(np.uint8)
    decode_case(B, T, 4, 4, chunk, dtype, bmap, 40 + dtype, from_oracle_cache)


@pytest.mark.parametrize("G", [1, 2, 3, 4, 5, 6, 7, 8])
def test_query_groups(G):
    B, T, chunk, Hkv = 2, 128 * 6 + 5, 128, 2
    rs = np.random.RandomState(G)
    bmap = rs.randint(0, 4, size=(B, T // chunk)).astype(np.uint8)
    decode_case(B, T, Hkv * G, Hkv, chunk, 1, bmap, 50 + G, True)


@pytest.mark.parametrize("w", [0, 1, 2, 3])
def test_uniform_width_config1_shape(w):
    # config 1: batch 1, 8 heads, context 4096, chunk 128, fp16
    bmap = np.full((1, 32), w, np.uint8)
    decode_case(1, 4096, 8, 8, 128, 0, bmap, 60 + w, False)


def test_config1_mixed_with_frozen_first_chunk():
    bmap = synth.multinomial_map(1, 32, [0.25, 0.25, 0.25, 0.25], seed=9)
    assert bmap[0, 0] == 3
    decode_case(1, 4096, 8, 8, 128, 0, bmap, 70, False)


def test_edge_cases():
    decode_case(1, 7, 2, 2, 32, 0, np.zeros((1, 0), np.uint8), 80, False)         # tail only
    decode_case(2, 32, 2, 1, 32, 1, np.array([[0], [3]], np.uint8), 81, False)    # one chunk, no tail
    decode_case(1, 33, 1, 1, 32, 0, np.array([[1]], np.uint8), 82, True)          # one chunk + 1 tail token
    decode_case(1, 512 * 2 + 500, 4, 1, 512, 1, np.array([[2, 0]], np.uint8), 83, False)   # long tail, big chunk
    decode_case(1, 256, 2, 2, 64, 0, np.array([[0, 0, 0, 0]], np.uint8), 84, False, q_scale=4.0)  # peaky softmax


def test_overlapped_chain_of_layers_matches_oracle():
    # decode calls over consecutive layers, each allowed to start while the previous one finishes
    # (MOQAE_DECODE_OVERLAP_PREVIOUS): the shared workspace and the outputs must come out as in
    # separate, serialised calls, several times over
    B, T, Hq, Hkv, chunk, dtype, L = 2, 64 * 7 + 13, 8, 2, 64, 1, 4
    cfg = mq.make_config(n_layers=L, n_q_heads=Hq, n_kv_heads=Hkv, chunk=chunk, dtype=dtype, d_in=64,
                         max_tokens=T, batch=B)
    cache = mq.moqae_cache_bind(cfg, [7, 7, 7, 7], zero_pools=True)
    refs, qs = [], []
    for l in range(L):
        K, V = H.make_kv(B, T, Hkv, dtype, 300 + l)
        bmap = np.random.RandomState(300 + l).randint(0, 4, size=(B, T // chunk)).astype(np.uint8)
        mq.moqae_quantize_kv(cfg, K.cuda(), V.cuda(), T, l, cache, forced_map=torch.from_numpy(bmap).cuda())
        q = synth.normal((B, Hq, 128), dtype, 400 + l, "cpu")
        ocache = O.quantize_kv(synth.to_u16(K), synth.to_u16(V), dtype, chunk, bmap)
        refs.append(O.decode_attn(synth.to_u16(q), dtype, ocache, chunk))
        qs.append(q.cuda())
    torch.cuda.synchronize()
    ws = torch.zeros(mq.moqae_decode_attn_workspace(cfg), dtype=torch.uint8, device="cuda")
    out = torch.full((L, B, Hq, 128), float("nan"), dtype=torch.float32, device="cuda")
    for rep in range(3):
        for l in range(L):
            flags = mq.DECODE_OVERLAP_PREVIOUS if (l > 0 or rep > 0) else 0
            mq.moqae_decode_attn_ex(cfg, qs[l], l, cache, out[l], ws, flags=flags)
    torch.cuda.synchronize()
    for l in range(L):
        ok, e_abs, e_rel = H.attn_tolerance_ok(out[l].cpu().numpy(), refs[l])
        assert ok, (l, e_abs, e_rel)
    assert mq.moqae_poll_status(cache) == 0
    with pytest.raises(mq.MoqaeError) as e:
        mq.moqae_decode_attn_ex(cfg, qs[0], 0, cache, out[0], ws, flags=2)
    assert e.value.code == mq.ERR_INVALID_ARG


def scaled_case(bits_index, kv_range, q_abs, dtype, seed):
    """Uniform-width cache whose K/V groups span about `kv_range` and queries of magnitude about
    `q_abs`: the products q * s_k and p * s_v reach far beyond what N(0,1) inputs produce."""
    B, T, Hq, Hkv, chunk = 1, 128 * 3 + 5, 4, 2, 128
    rs = np.random.RandomState(seed)
    tdt = synth.torch_dtype(dtype)
    K = torch.from_numpy(rs.uniform(-0.5, 0.5, size=(B, T, Hkv, 128)).astype(np.float32) * kv_range).to(tdt)
    V = torch.from_numpy(rs.uniform(-0.5, 0.5, size=(B, T, Hkv, 128)).astype(np.float32) * kv_range).to(tdt)
    q = torch.from_numpy(rs.choice([-1.0, 1.0], size=(B, Hq, 128)).astype(np.float32) * q_abs *
                         rs.uniform(0.5, 1.0, size=(B, Hq, 128)).astype(np.float32)).to(tdt)
    bmap = np.full((B, T // chunk), bits_index, np.uint8)
    ocache = O.quantize_kv(synth.to_u16(K), synth.to_u16(V), dtype, chunk, bmap)
    # a softmax scale that keeps the logits of such inputs in a range where several tokens matter
    scale = 4.0 / (q_abs * kv_range * np.sqrt(128.0))
    ref = O.decode_attn(synth.to_u16(q), dtype, ocache, chunk, scale=scale)
    cfg = mq.make_config(n_layers=1, n_q_heads=Hq, n_kv_heads=Hkv, chunk=chunk, dtype=dtype, d_in=64,
                         max_tokens=T, batch=B)
    cache = mq.moqae_cache_bind(cfg, [3, 3, 3, 3], zero_pools=True)
    H.upload_oracle_cache(cache, ocache, 0)
    ws = torch.zeros(mq.moqae_decode_attn_workspace(cfg), dtype=torch.uint8, device="cuda")
    out = torch.full((B, Hq, 128), float("nan"), dtype=torch.float32, device="cuda")
    mq.moqae_decode_attn(cfg, q.cuda(), 0, cache, out, ws, scale=scale)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    assert np.isfinite(got).all()
    # outputs are of the order of kv_range: the tolerances scale with it
    err = np.abs(got - ref)
    assert err.max() <= 2e-3 * max(1.0, kv_range), (err.max(), kv_range)
    assert (err.max(-1) / np.abs(ref).max(-1)).max() <= 1e-2


@pytest.mark.parametrize("w", [0, 1, 2])
@pytest.mark.parametrize("kv_range", [1e3, 8e3, 3e4])
def test_large_group_ranges_and_queries_stay_finite_and_accurate(w, kv_range):
    # group ranges of thousands at 2 bits give key / value scales of thousands: the folded query
    # q * s_k and the scaled weight p * s_v must not leave the fp16 range
    scaled_case(w, kv_range, 8.0, 0, 500 + w)
    scaled_case(w, kv_range, 8.0, 1, 510 + w)


def test_tiny_and_huge_queries():
    scaled_case(0, 4.0, 1e-3, 0, 520)
    scaled_case(1, 4.0, 3e4, 0, 521)
    scaled_case(0, 2e4, 6e4, 0, 522)
    scaled_case(2, 4.0, 1e6, 1, 523)


def test_empty_cache_gives_zeros():
    cfg = mq.make_config(n_layers=1, n_q_heads=2, n_kv_heads=2, chunk=32, dtype=0, d_in=64,
                         max_tokens=32, batch=1)
    cache = mq.moqae_cache_bind(cfg, [1, 1, 1, 1])
    ws = torch.zeros(mq.moqae_decode_attn_workspace(cfg), dtype=torch.uint8, device="cuda")
    out = torch.full((1, 2, 128), float("nan"), dtype=torch.float32, device="cuda")
    q = synth.normal((1, 2, 128), 0, 1, "cuda")
    mq.moqae_decode_attn(cfg, q, 0, cache, out, ws)
    torch.cuda.synchronize()
    assert (out == 0).all()


def test_append_then_decode_matches_oracle_with_longer_tail():
    # decode loop: new tokens are appended to the 16-bit tail, routing is not re-run
    B, T, Hq, Hkv, chunk, dtype = 2, 64 * 3, 4, 2, 64, 1
    bmap = np.array([[3, 0, 1], [3, 2, 0]], np.uint8)
    K, V = H.make_kv(B, T + 5, Hkv, dtype, 90)
    cfg = mq.make_config(n_layers=1, n_q_heads=Hq, n_kv_heads=Hkv, chunk=chunk, dtype=dtype, d_in=64,
                         max_tokens=T + chunk, batch=B)
    cache = mq.moqae_cache_bind(cfg, [2, 2, 2, 2], zero_pools=True)
    Kc, Vc = K.cuda(), V.cuda()
    mq.moqae_quantize_kv(cfg, Kc[:, :T].contiguous(), Vc[:, :T].contiguous(), T, 0, cache,
                         forced_map=torch.from_numpy(bmap).cuda())
    ws = torch.zeros(mq.moqae_decode_attn_workspace(cfg), dtype=torch.uint8, device="cuda")
    out = torch.empty((B, Hq, 128), dtype=torch.float32, device="cuda")
    for step in range(5):
        mq.moqae_append_kv(cfg, Kc[:, T + step].contiguous(), Vc[:, T + step].contiguous(), 0, cache)
        q = synth.normal((B, Hq, 128), dtype, 200 + step, "cpu")
        mq.moqae_decode_attn(cfg, q.cuda(), 0, cache, out, ws)
        torch.cuda.synchronize()
        n = T + step + 1
        ocache = O.quantize_kv(synth.to_u16(K[:, :n]), synth.to_u16(V[:, :n]), dtype, chunk, bmap)
        assert ocache["tail_len"] == step + 1
        ref = O.decode_attn(synth.to_u16(q), dtype, ocache, chunk)
        ok, e_abs, e_rel = H.attn_tolerance_ok(out.cpu().numpy(), ref)
        assert ok, (step, e_abs, e_rel)
    assert mq.moqae_poll_status(cache) == 0


def test_generation_steps_attend_to_the_new_token_before_it_is_appended():
    # moqae_decode_attn_step: the current token's K/V rows take part in the attention without being in the
    # cache; the layers of a step are chained (each launch may overlap the previous one), the appends follow
    # the step.  After every step the outputs equal the oracle on "cache + tail + the new token".
    B, Hq, Hkv, chunk, dtype, L = 2, 4, 2, 64, 1, 3
    T = 64 * 3 + 7
    cfg = mq.make_config(n_layers=L, n_q_heads=Hq, n_kv_heads=Hkv, chunk=chunk, dtype=dtype, d_in=64,
                         max_tokens=T + chunk, batch=B)
    cache = mq.moqae_cache_bind(cfg, [3, 3, 3, 3], zero_pools=True)
    KV, maps = [], []
    for l in range(L):
        K, V = H.make_kv(B, T + 6, Hkv, dtype, 950 + l)
        bmap = np.random.RandomState(950 + l).randint(0, 4, size=(B, T // chunk)).astype(np.uint8)
        mq.moqae_quantize_kv(cfg, K[:, :T].contiguous().cuda(), V[:, :T].contiguous().cuda(), T, l, cache,
                             forced_map=torch.from_numpy(bmap).cuda())
        KV.append((K, V))
        maps.append(bmap)
    torch.cuda.synchronize()
    ws = torch.zeros(mq.moqae_decode_attn_workspace(cfg), dtype=torch.uint8, device="cuda")
    out = torch.full((L, B, Hq, 128), float("nan"), dtype=torch.float32, device="cuda")
    for step in range(6):
        qs = [synth.normal((B, Hq, 128), dtype, 970 + 10 * step + l, "cpu") for l in range(L)]
        new = [(KV[l][0][:, T + step].contiguous().cuda(), KV[l][1][:, T + step].contiguous().cuda()) for l in range(L)]
        qd = [x.cuda() for x in qs]
        torch.cuda.synchronize()
        for l in range(L):
            mq.moqae_decode_attn_step(cfg, qd[l], new[l][0], new[l][1], l, cache, out[l], ws,
                                      flags=mq.DECODE_OVERLAP_PREVIOUS if l > 0 else 0)
        for l in range(L):
            mq.moqae_append_kv(cfg, new[l][0], new[l][1], l, cache)
        torch.cuda.synchronize()
        n = T + step + 1
        for l in range(L):
            K, V = KV[l]
            ocache = O.quantize_kv(synth.to_u16(K[:, :n]), synth.to_u16(V[:, :n]), dtype, chunk, maps[l])
            assert ocache["tail_len"] == 7 + step + 1
            ok, e_abs, e_rel = H.attn_tolerance_ok(out[l].cpu().numpy(), O.decode_attn(synth.to_u16(qs[l]), dtype, ocache, chunk))
            assert ok, (step, l, e_abs, e_rel)
        assert (cache.tail_len.cpu().numpy() == 7 + step + 1).all()
    assert mq.moqae_poll_status(cache) == 0
    # an empty cache plus the new token: the output is that token's value row
    cfg1 = mq.make_config(n_layers=1, n_q_heads=2, n_kv_heads=1, chunk=32, dtype=0, d_in=64, max_tokens=32, batch=1)
    c1 = mq.moqae_cache_bind(cfg1, [1, 1, 1, 1])
    k1, v1 = synth.normal((1, 1, 128), 0, 1, "cuda"), synth.normal((1, 1, 128), 0, 2, "cuda")
    o1 = torch.full((1, 2, 128), float("nan"), dtype=torch.float32, device="cuda")
    w1 = torch.zeros(mq.moqae_decode_attn_workspace(cfg1), dtype=torch.uint8, device="cuda")
    mq.moqae_decode_attn_step(cfg1, synth.normal((1, 2, 128), 0, 3, "cuda"), k1, v1, 0, c1, o1, w1)
    torch.cuda.synchronize()
    assert torch.allclose(o1[0, 0], v1[0, 0].float(), atol=2e-3) and torch.allclose(o1[0, 1], v1[0, 0].float(), atol=2e-3)


def test_decode_is_deterministic_and_leaves_neighbours_alone():
    # same call twice -> identical bits; bytes around `out` are never touched
    B, T, Hq, Hkv, chunk, dtype = 2, 64 * 5 + 9, 8, 2, 64, 1
    K, V = H.make_kv(B, T, Hkv, dtype, 95)
    bmap = np.random.RandomState(95).randint(0, 4, size=(B, T // chunk)).astype(np.uint8)
    cfg = mq.make_config(n_layers=1, n_q_heads=Hq, n_kv_heads=Hkv, chunk=chunk, dtype=dtype, d_in=64,
                         max_tokens=T, batch=B)
    cache = mq.moqae_cache_bind(cfg, [5, 5, 5, 5], zero_pools=True)
    mq.moqae_quantize_kv(cfg, K.cuda(), V.cuda(), T, 0, cache, forced_map=torch.from_numpy(bmap).cuda())
    ws = torch.zeros(mq.moqae_decode_attn_workspace(cfg), dtype=torch.uint8, device="cuda")
    q = synth.normal((B, Hq, 128), dtype, 96, "cuda")
    n = B * Hq * 128
    buf = torch.full((n + 64,), -7.25, dtype=torch.float32, device="cuda")      # 32 canary floats on either side
    out = buf[32:32 + n].view(B, Hq, 128)
    mq.moqae_decode_attn(cfg, q, 0, cache, out, ws)
    first = out.clone()
    # stale partials must not matter; the arrival counters behind them (one int32 per sequence and
    # kv head) are the only part a call relies on, and every call leaves them zero again
    n_partial_bytes = ws.numel() - (B * Hkv * 4 + 15) // 16 * 16
    ws[:n_partial_bytes].fill_(0xAB)
    assert (ws[n_partial_bytes:] == 0).all()
    mq.moqae_decode_attn(cfg, q, 0, cache, out, ws)
    torch.cuda.synchronize()
    assert torch.equal(first, out)
    assert (buf[:32] == -7.25).all() and (buf[32 + n:] == -7.25).all()
