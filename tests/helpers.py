"""Shared helpers of the parity tests: build seeded inputs once, hand the same bits to the
CPU oracle and to the CUDA library (through its C ABI binding)."""
from __future__ import annotations

import numpy as np
import torch

from oracle import moqae_oracle as O
from paper_2506_07533_b200 import synth


def gpu_available() -> bool:
    return torch.cuda.is_available()


def make_kv(B, T, H, dtype, seed, outlier_channels=(5, 37, 64, 101)):
    K, V = synth.keys_values(B, T, H, 128, dtype, seed, "cpu", outlier_channels=outlier_channels)
    return K, V


def upload_oracle_cache(cache, ocache, layer):
    """Copy a cache built by the oracle into the device buffers of `cache` for one layer."""
    dev = cache.buffers[0].device
    g = layer // cache.cfg.rs_group
    for w in range(4):
        n = int(ocache["count"][:, w].max()) if ocache["count"].size else 0
        if n:
            cache.pool(w)[layer, :, :, :n] = torch.from_numpy(ocache["pools"][w][:, :, :n]).to(dev)
    C = ocache["slot"].shape[1]
    cache.count[g] = torch.from_numpy(ocache["count"]).to(dev)
    cache.slot[g, :, :C] = torch.from_numpy(ocache["slot"]).to(dev)
    r = ocache["tail_len"]
    if r:
        cache.tail("k")[layer, :, :, :r] = torch.from_numpy(ocache["tail_k"].view(np.int16)).to(dev)
        cache.tail("v")[layer, :, :, :r] = torch.from_numpy(ocache["tail_v"].view(np.int16)).to(dev)
    cache.tail_len[layer] = r


def compare_pools(cache, ocache, layer):
    """Byte-exact comparison of every used slot, the tables and the tail."""
    g = layer // cache.cfg.rs_group
    C = ocache["slot"].shape[1]
    assert (cache.count[g].cpu().numpy() == ocache["count"]).all()
    assert (cache.slot[g, :, :C].cpu().numpy() == ocache["slot"]).all()
    for w in range(4):
        got = cache.pool(w)[layer].cpu().numpy()
        for b in range(ocache["count"].shape[0]):
            n = int(ocache["count"][b, w])
            if n:
                exp = ocache["pools"][w][b, :, :n]
                if not (got[b, :, :n] == exp).all():
                    bad = np.argwhere(got[b, :, :n] != exp)
                    raise AssertionError(f"pool {w} seq {b}: {len(bad)} bytes differ, first at {bad[0]}")
    r = ocache["tail_len"]
    assert (cache.tail_len[layer].cpu().numpy() == r).all()
    if r:
        assert (cache.tail("k")[layer, :, :, :r].cpu().numpy().view(np.uint16) == ocache["tail_k"]).all()
        assert (cache.tail("v")[layer, :, :, :r].cpu().numpy().view(np.uint16) == ocache["tail_v"]).all()


TAU = 1e-4      # a token whose top-2 logits differ by less than TAU * max|P| may flip in float32


def check_routed_chunk(rows_u16, dtype, W1_u16, W2_u16, W3, bias, got_votes, got_winner, abs_margin=None):
    """One chunk's vote histogram and winner from the GPU against the oracle router run on the
    chunk's hidden rows [chunk, d_in]: exact unless near-tie tokens exist; then the histograms may
    differ by at most those tokens and the winner must be reachable by flipping them between
    their two best experts.  Returns True if the chunk was fragile."""
    chunk = rows_u16.shape[0]
    ref = O.route(rows_u16[None], dtype, chunk, W1_u16, W2_u16, W3, bias, rf_first_chunk=False)
    thr = abs_margin if abs_margin is not None else TAU * np.maximum(ref["pmax"][0], 1e-30)
    frag = np.where(ref["margin"][0] < thr)[0]
    diff = np.asarray(got_votes).astype(np.int64) - ref["votes"][0, 0]
    assert diff.sum() == 0 and np.abs(diff).sum() // 2 <= len(frag), (diff, len(frag))
    if len(frag) == 0:
        assert (diff == 0).all() and int(got_winner) == int(ref["map"][0, 0])
        return False
    x = O.to_f64(rows_u16[frag], dtype)
    P = O.router_logits(x, O.to_f64(W1_u16, dtype), None if W2_u16 is None else O.to_f64(W2_u16, dtype),
                        None if W3 is None else np.asarray(W3, np.float32).astype(np.float64),
                        None if bias is None else np.asarray(bias, np.float32).astype(np.float64))
    order = np.argsort(-P, axis=1, kind="stable")
    assert int(got_winner) in O.reachable_winners(ref["votes"][0, 0], list(order[:, 0]), list(order[:, 1]))
    return True


def oracle_cache_of_head(cache, layer, b, h, C):
    """The GPU's own packed cache of one (layer, sequence, kv head), in the form the oracle's
    decode functions take (one sequence, one head): its bytes, its map-derived tables, its tail."""
    g = layer // cache.cfg.rs_group
    gmap = cache.map[g, b:b + 1, :C].cpu().numpy()
    slot, count = O.assign_slots(gmap)
    assert (cache.slot[g, b:b + 1, :C].cpu().numpy() == slot).all()
    assert (cache.count[g, b:b + 1].cpu().numpy() == count).all()
    pools = []
    for w in range(4):
        n = int(count[0, w])
        pools.append(cache.pool(w)[layer, b, h, :max(n, 1)].cpu().numpy()[None, None])
    r = int(cache.tail_len[layer, b].item())
    return dict(pools=pools, map=gmap, slot=slot, count=count, tail_len=r,
                tail_k=cache.tail("k")[layer, b, h, :r].cpu().numpy().view(np.uint16)[None, None],
                tail_v=cache.tail("v")[layer, b, h, :r].cpu().numpy().view(np.uint16)[None, None])


def attn_tolerance_ok(got, ref, abs_tol=2e-3, rel_tol=1e-2):
    """max-abs error <= abs_tol and, per (batch, head) row, max|err| / max|ref| <= rel_tol."""
    err = np.abs(got.astype(np.float64) - ref)
    row_rel = err.max(-1) / np.maximum(np.abs(ref).max(-1), 1e-30)
    return err.max() <= abs_tol and row_rel.max() <= rel_tol, float(err.max()), float(row_rel.max())
