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


def attn_tolerance_ok(got, ref, abs_tol=2e-3, rel_tol=1e-2):
    """max-abs error <= abs_tol and, per (batch, head) row, max|err| / max|ref| <= rel_tol."""
    err = np.abs(got.astype(np.float64) - ref)
    row_rel = err.max(-1) / np.maximum(np.abs(ref).max(-1), 1e-30)
    return err.max() <= abs_tol and row_rel.max() <= rel_tol, float(err.max()), float(row_rel.max())
