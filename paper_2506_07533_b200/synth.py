"""Seeded synthetic inputs with the shapes and value structure of the workloads.

This module only draws random tensors; it contains none of the method's
arithmetic (no routing, no quantisation, no attention).  Both the CPU checker
used by the tests and the CUDA library are fed from here, so they see the same
bits.  Everything is a function of (seed, shape); `device` may be "cpu" or a
CUDA device (large workloads are drawn directly in device memory).
"""
from __future__ import annotations

import numpy as np
import torch

DT_FP16 = 0
DT_BF16 = 1
_TORCH_DT = {DT_FP16: torch.float16, DT_BF16: torch.bfloat16}


def torch_dtype(dtype: int) -> torch.dtype:
    return _TORCH_DT[dtype]


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def normal(shape, dtype: int, seed: int, device="cpu", std: float = 1.0) -> torch.Tensor:
    """N(0, std^2) drawn in float32, rounded once to the 16-bit dtype."""
    x = torch.randn(*shape, generator=_gen(seed, device), device=device, dtype=torch.float32)
    if std != 1.0:
        x = x * std
    return x.to(_TORCH_DT[dtype])


def hidden_states(B: int, T: int, D: int, chunk: int, dtype: int, seed: int, device="cpu",
                  rho: float = 0.5) -> torch.Tensor:
    """[B, T, D] router input with chunk-level structure: every token is
    sqrt(1-rho) * eps + sqrt(rho) * u_chunk with eps, u ~ N(0, I), so marginals
    stay N(0, 1) while tokens of one chunk share a direction (without it every
    chunk of an i.i.d. sequence would vote alike)."""
    g = _gen(seed, device)
    n_chunks = (T + chunk - 1) // chunk
    u = torch.randn(B, n_chunks, D, generator=g, device=device, dtype=torch.float32)
    out = torch.empty(B, T, D, device=device, dtype=_TORCH_DT[dtype])
    a, c = float(np.sqrt(1.0 - rho)), float(np.sqrt(rho))
    step = max(1, (1 << 24) // D)                 # bound the float32 scratch
    for b in range(B):
        for t0 in range(0, T, step):
            t1 = min(T, t0 + step)
            eps = torch.randn(t1 - t0, D, generator=g, device=device, dtype=torch.float32)
            idx = torch.arange(t0, t1, device=device) // chunk
            out[b, t0:t1] = (a * eps + c * u[b, idx]).to(_TORCH_DT[dtype])
    return out


def keys_values(B: int, T: int, H: int, d: int, dtype: int, seed: int, device="cpu",
                outlier_channels=None, outlier_frac: float = 0.0, outlier_scale: float = 10.0):
    """K, V [B, T, H, d] ~ N(0,1).  Key outlier channels (fixed over tokens) are
    multiplied by `outlier_scale`: either `outlier_channels` (list of channel
    indices applied in every head) or a seeded `outlier_frac` of the H*d channels."""
    g = _gen(seed, device)
    K = torch.empty(B, T, H, d, device=device, dtype=_TORCH_DT[dtype])
    V = torch.empty(B, T, H, d, device=device, dtype=_TORCH_DT[dtype])
    mult = torch.ones(H, d, device=device, dtype=torch.float32)
    if outlier_channels is not None:
        mult[:, list(outlier_channels)] = outlier_scale
    elif outlier_frac > 0:
        n_out = max(1, int(round(outlier_frac * H * d)))
        rs = np.random.RandomState(seed ^ 0x5EED)
        pick = rs.choice(H * d, size=n_out, replace=False)
        flat = mult.view(-1)
        flat[torch.as_tensor(pick, device=device)] = outlier_scale
    step = max(1, (1 << 24) // (H * d))
    for b in range(B):
        for t0 in range(0, T, step):
            t1 = min(T, t0 + step)
            k = torch.randn(t1 - t0, H, d, generator=g, device=device, dtype=torch.float32)
            K[b, t0:t1] = (k * mult).to(_TORCH_DT[dtype])
            v = torch.randn(t1 - t0, H, d, generator=g, device=device, dtype=torch.float32)
            V[b, t0:t1] = v.to(_TORCH_DT[dtype])
    return K, V


def router_weights(D: int, M: int, dtype: int, seed: int, device="cpu", std: float = 0.02,
                   gated: bool = True):
    """W1, W2 [D, M] in the 16-bit dtype, W3 [M, M] and bias [M] float32."""
    g = _gen(seed, device)
    W1 = (torch.randn(D, M, generator=g, device=device) * std).to(_TORCH_DT[dtype])
    if not gated:
        return W1, None, None, torch.zeros(M, device=device, dtype=torch.float32)
    W2 = (torch.randn(D, M, generator=g, device=device) * std).to(_TORCH_DT[dtype])
    W3 = torch.randn(M, M, generator=g, device=device, dtype=torch.float32)
    return W1, W2, W3, torch.zeros(M, device=device, dtype=torch.float32)


def multinomial_map(B: int, C: int, mix, seed: int, rf_first_chunk: bool = True) -> np.ndarray:
    """Seeded per-chunk expert indices with the given probabilities (a stand-in
    for a trained router's choices); chunk 0 is the 16-bit expert when frozen."""
    rs = np.random.RandomState(seed)
    p = np.asarray(mix, dtype=np.float64)
    m = rs.choice(len(p), size=(B, C), p=p / p.sum()).astype(np.uint8)
    if rf_first_chunk and C > 0:
        m[:, 0] = len(p) - 1
    return m


def to_u16(t: torch.Tensor) -> np.ndarray:
    """Bit patterns of a 16-bit tensor as numpy uint16 (host copy)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
