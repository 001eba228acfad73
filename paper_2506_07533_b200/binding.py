"""ctypes binding of libmoqae.so: argument marshalling only.

Function names follow the C ABI (`include/moqae.h`); tensors are torch CUDA tensors whose
`data_ptr()` is handed to the library, work runs on torch's current stream.  There is no
CPU path: loading fails loudly if the CUDA library has not been built.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass, field

import torch

from . import build as _build

EXPERT_BITS = (2, 4, 8, 16)
N_CACHE_BUFFERS = 12
DT_FP16, DT_BF16 = 0, 1

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_MISALIGNED, ERR_POOL_FULL = -1, -2, -3, -4
ERR_WORKSPACE_TOO_SMALL, ERR_CUDA, ERR_TIMEOUT = -5, -6, -7
ERR_CORRUPT_TABLE = -8

EXPORTS = ["moqae_version", "moqae_last_cuda_error", "moqae_error_string", "moqae_cache_bytes",
           "moqae_cache_bind", "moqae_route", "moqae_quantize_kv", "moqae_append_kv",
           "moqae_decode_attn_workspace", "moqae_decode_attn", "moqae_poll_status",
           "moqae_decode_attn_static", "moqae_decode_attn_static_max_bytes", "moqae_flush_tail", "moqae_prefill_attn",
           "moqae_prefill_attn_workspace", "moqae_decode_attn_ex", "moqae_project_quantize_kv",
           "moqae_validate_tables", "moqae_validate_tables_host", "moqae_decode_attn_step"]


class MoqaeConfig(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("chunk", C.c_int32), ("group", C.c_int32),
                ("dtype", C.c_int32), ("n_experts", C.c_int32), ("expert_bits", C.c_int32 * 4),
                ("rs_group", C.c_int32), ("rf_first_chunk", C.c_int32), ("d_in", C.c_int32),
                ("max_tokens", C.c_int32), ("tail_capacity", C.c_int32), ("batch", C.c_int32),
                ("per_head_routing", C.c_int32)]


class MoqaeCache(C.Structure):
    _fields_ = [("pool", C.c_void_p * 4), ("capacity", C.c_int64 * 4), ("map", C.c_void_p),
                ("slot", C.c_void_p), ("count", C.c_void_p), ("votes", C.c_void_p),
                ("tail_k", C.c_void_p), ("tail_v", C.c_void_p), ("tail_len", C.c_void_p),
                ("status", C.c_void_p)]


class MoqaeError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().moqae_error_string(code).decode()
        if code == ERR_CUDA:
            msg += f" [cuda error {lib().moqae_last_cuda_error()}]"
        super().__init__(f"{where}: {msg} ({code})")


_LIB = None


def lib_path() -> str:
    return _build.LIB


def lib() -> C.CDLL:
    """The loaded C-ABI library.  Raises if it has not been built (no fallback exists)."""
    global _LIB
    if _LIB is None:
        path = lib_path()
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: run `python -m paper_2506_07533_b200.build` "
                               "(the CUDA library is the only implementation)")
        L = C.CDLL(path)
        L.moqae_version.restype = C.c_int
        L.moqae_last_cuda_error.restype = C.c_int
        L.moqae_error_string.restype = C.c_char_p
        L.moqae_error_string.argtypes = [C.c_int]
        L.moqae_cache_bytes.argtypes = [C.POINTER(MoqaeConfig), C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
        L.moqae_cache_bind.argtypes = [C.POINTER(MoqaeConfig), C.POINTER(C.c_int64), C.POINTER(C.c_void_p),
                                       C.POINTER(MoqaeCache)]
        L.moqae_route.argtypes = [C.POINTER(MoqaeConfig), C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p,
                                  C.c_void_p, C.c_void_p, C.c_int32, C.POINTER(MoqaeCache), C.c_void_p,
                                  C.c_void_p]
        L.moqae_quantize_kv.argtypes = [C.POINTER(MoqaeConfig), C.c_void_p, C.c_void_p, C.c_int32, C.c_int32,
                                        C.c_void_p, C.POINTER(MoqaeCache), C.c_void_p]
        L.moqae_project_quantize_kv.argtypes = [C.POINTER(MoqaeConfig), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                                C.c_int32, C.c_void_p, C.POINTER(MoqaeCache), C.c_void_p, C.c_void_p,
                                                C.c_void_p]
        L.moqae_append_kv.argtypes = [C.POINTER(MoqaeConfig), C.c_void_p, C.c_void_p, C.c_int32,
                                      C.POINTER(MoqaeCache), C.c_void_p]
        L.moqae_flush_tail.argtypes = [C.POINTER(MoqaeConfig), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                       C.c_void_p, C.c_int32, C.POINTER(MoqaeCache), C.c_void_p]
        L.moqae_prefill_attn.argtypes = [C.POINTER(MoqaeConfig), C.c_void_p, C.c_int32, C.c_int32,
                                         C.POINTER(MoqaeCache), C.c_void_p, C.c_float, C.c_void_p, C.c_int64, C.c_void_p]
        L.moqae_prefill_attn_workspace.argtypes = [C.POINTER(MoqaeConfig), C.c_int32, C.POINTER(C.c_int64)]
        L.moqae_decode_attn_workspace.argtypes = [C.POINTER(MoqaeConfig), C.POINTER(C.c_int64)]
        L.moqae_decode_attn.argtypes = [C.POINTER(MoqaeConfig), C.c_void_p, C.c_int32, C.POINTER(MoqaeCache),
                                        C.c_void_p, C.c_float, C.c_void_p, C.c_int64, C.c_void_p]
        L.moqae_decode_attn_ex.argtypes = [C.POINTER(MoqaeConfig), C.c_void_p, C.c_int32, C.POINTER(MoqaeCache),
                                           C.c_void_p, C.c_float, C.c_void_p, C.c_int64, C.c_int32, C.c_void_p]
        L.moqae_decode_attn_step.argtypes = [C.POINTER(MoqaeConfig), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                             C.POINTER(MoqaeCache), C.c_void_p, C.c_float, C.c_void_p, C.c_int64,
                                             C.c_int32, C.c_void_p]
        L.moqae_poll_status.argtypes = [C.POINTER(MoqaeCache), C.c_void_p, C.POINTER(C.c_int32)]
        L.moqae_validate_tables.argtypes = [C.POINTER(MoqaeConfig), C.POINTER(MoqaeCache), C.c_int32, C.c_int32,
                                            C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        L.moqae_validate_tables_host.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32,
                                                 C.POINTER(C.c_int64), C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        L.moqae_decode_attn_static.argtypes = [C.POINTER(MoqaeConfig), C.c_void_p, C.c_int32,
                                               C.POINTER(MoqaeCache), C.c_void_p, C.c_float, C.c_void_p]
        L.moqae_decode_attn_static_max_bytes.argtypes = []
        for name in EXPORTS:
            if name not in ("moqae_error_string",):
                getattr(L, name).restype = C.c_int
        L.moqae_decode_attn_static_max_bytes.restype = C.c_int64
        _LIB = L
    return _LIB


def _check(rc: int, where: str):
    if rc != OK:
        raise MoqaeError(rc, where)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def make_config(*, n_layers, n_q_heads, n_kv_heads, chunk, dtype, d_in, max_tokens, batch, rs_group=1,
                rf_first_chunk=1, tail_capacity=None, per_head_routing=False) -> MoqaeConfig:
    cfg = MoqaeConfig()
    cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads = n_layers, n_q_heads, n_kv_heads
    cfg.head_dim, cfg.chunk, cfg.group, cfg.dtype, cfg.n_experts = 128, chunk, 32, dtype, 4
    cfg.expert_bits = (C.c_int32 * 4)(*EXPERT_BITS)
    cfg.rs_group, cfg.rf_first_chunk, cfg.d_in = rs_group, int(rf_first_chunk), d_in
    cfg.max_tokens, cfg.batch = max_tokens, batch
    cfg.tail_capacity = chunk if tail_capacity is None else tail_capacity
    cfg.per_head_routing = int(bool(per_head_routing))
    return cfg


def moqae_version() -> int:
    return lib().moqae_version()


def moqae_cache_bytes(cfg: MoqaeConfig, capacity) -> list:
    cap = (C.c_int64 * 4)(*[int(c) for c in capacity])
    out = (C.c_int64 * N_CACHE_BUFFERS)()
    _check(lib().moqae_cache_bytes(C.byref(cfg), cap, out), "moqae_cache_bytes")
    return list(out)


@dataclass
class Cache:
    """Device buffers of one cache plus the C view handed to the library."""
    cfg: MoqaeConfig
    capacity: list
    buffers: list = field(default_factory=list)      # 12 torch uint8 tensors
    view: MoqaeCache = None

    @property
    def n_groups(self):
        return (self.cfg.n_layers + self.cfg.rs_group - 1) // self.cfg.rs_group

    @property
    def max_chunks(self):
        return self.cfg.max_tokens // self.cfg.chunk

    @property
    def table_rows(self):
        """Rows of the map / slot / count / votes tables per group: one per sequence, or one per
        (sequence, kv head) with per-head routing."""
        return self.cfg.batch * (self.cfg.n_kv_heads if self.cfg.per_head_routing else 1)

    def table(self, idx, dtype, shape):
        n = 1
        for d in shape:
            n *= d
        nbytes = n * torch.empty(0, dtype=dtype).element_size()
        return self.buffers[idx][:nbytes].view(dtype).view(*shape)

    @property
    def map(self):
        return self.table(4, torch.uint8, (self.n_groups, self.table_rows, self.max_chunks))

    @property
    def slot(self):
        return self.table(5, torch.int32, (self.n_groups, self.table_rows, self.max_chunks))

    @property
    def count(self):
        return self.table(6, torch.int32, (self.n_groups, self.table_rows, 4))

    @property
    def votes(self):
        return self.table(7, torch.int32, (self.n_groups, self.table_rows, self.max_chunks, 4))

    @property
    def tail_len(self):
        return self.table(10, torch.int32, (self.cfg.n_layers, self.cfg.batch))

    def pool(self, w):
        """uint8 view [n_layers, batch, n_kv_heads, capacity_w, slot_bytes_w]."""
        tb = 16384 if w == 3 else 1024 + 1024 * EXPERT_BITS[w]
        sb = max(1, self.cfg.chunk // 32) * tb      # a chunk of 8 or 16 tokens is one (padded) tile
        n = self.cfg.n_layers * self.cfg.batch * self.cfg.n_kv_heads * self.capacity[w] * sb
        return self.buffers[w][:n].view(self.cfg.n_layers, self.cfg.batch, self.cfg.n_kv_heads,
                                        self.capacity[w], sb)

    def tail(self, which):
        n = self.cfg.n_layers * self.cfg.batch * self.cfg.n_kv_heads * self.cfg.tail_capacity * 256
        t = self.buffers[8 if which == "k" else 9][:n].view(torch.int16)
        return t.view(self.cfg.n_layers, self.cfg.batch, self.cfg.n_kv_heads, self.cfg.tail_capacity, 128)


def moqae_cache_bind(cfg: MoqaeConfig, capacity, device="cuda", zero_pools=False) -> Cache:
    """Allocate the twelve buffers with torch and bind them (the library allocates nothing)."""
    sizes = moqae_cache_bytes(cfg, capacity)
    bufs = []
    for i, n in enumerate(sizes):
        n_alloc = max(16, (n + 15) // 16 * 16)
        if i < 4 and not zero_pools:
            bufs.append(torch.empty(n_alloc, dtype=torch.uint8, device=device))
        else:
            bufs.append(torch.zeros(n_alloc, dtype=torch.uint8, device=device))
    cap = (C.c_int64 * 4)(*[int(c) for c in capacity])
    ptrs = (C.c_void_p * N_CACHE_BUFFERS)(*[b.data_ptr() for b in bufs])
    view = MoqaeCache()
    _check(lib().moqae_cache_bind(C.byref(cfg), cap, ptrs, C.byref(view)), "moqae_cache_bind")
    return Cache(cfg=cfg, capacity=[int(c) for c in capacity], buffers=bufs, view=view)


def moqae_route(cfg, hidden, T, W1, W2, W3, bias, layer_group, cache: Cache, votes_out=None):
    _check(lib().moqae_route(C.byref(cfg), _ptr(hidden), int(T), _ptr(W1), _ptr(W2), _ptr(W3), _ptr(bias),
                             int(layer_group), C.byref(cache.view), _ptr(votes_out), _stream()), "moqae_route")


def moqae_quantize_kv(cfg, K, V, T, layer, cache: Cache, forced_map=None):
    _check(lib().moqae_quantize_kv(C.byref(cfg), _ptr(K), _ptr(V), int(T), int(layer), _ptr(forced_map),
                                   C.byref(cache.view), _stream()), "moqae_quantize_kv")


def moqae_project_quantize_kv(cfg, hidden, Wk, Wv, T, layer, cache: Cache, forced_map=None, k_rounded=None, v_rounded=None):
    _check(lib().moqae_project_quantize_kv(C.byref(cfg), _ptr(hidden), _ptr(Wk), _ptr(Wv), int(T), int(layer),
                                           _ptr(forced_map), C.byref(cache.view), _ptr(k_rounded), _ptr(v_rounded),
                                           _stream()), "moqae_project_quantize_kv")


def moqae_append_kv(cfg, k_new, v_new, layer, cache: Cache):
    _check(lib().moqae_append_kv(C.byref(cfg), _ptr(k_new), _ptr(v_new), int(layer), C.byref(cache.view),
                                 _stream()), "moqae_append_kv")


def moqae_flush_tail(cfg, hidden_tail, W1, W2, W3, bias, layer_group, cache: Cache):
    _check(lib().moqae_flush_tail(C.byref(cfg), _ptr(hidden_tail), _ptr(W1), _ptr(W2), _ptr(W3), _ptr(bias),
                                  int(layer_group), C.byref(cache.view), _stream()), "moqae_flush_tail")


def moqae_prefill_attn_workspace(cfg, T) -> int:
    out = C.c_int64(0)
    _check(lib().moqae_prefill_attn_workspace(C.byref(cfg), int(T), C.byref(out)), "moqae_prefill_attn_workspace")
    return int(out.value)


def moqae_prefill_attn(cfg, q, T, layer, cache: Cache, out, scale=0.0, workspace=None):
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().moqae_prefill_attn(C.byref(cfg), _ptr(q), int(T), int(layer), C.byref(cache.view), _ptr(out),
                                    C.c_float(scale), _ptr(workspace), C.c_int64(nbytes), _stream()), "moqae_prefill_attn")


def moqae_decode_attn_workspace(cfg) -> int:
    out = C.c_int64(0)
    _check(lib().moqae_decode_attn_workspace(C.byref(cfg), C.byref(out)), "moqae_decode_attn_workspace")
    return int(out.value)


DECODE_OVERLAP_PREVIOUS = 1


def moqae_decode_attn(cfg, q, layer, cache: Cache, out, workspace, scale=0.0):
    _check(lib().moqae_decode_attn(C.byref(cfg), _ptr(q), int(layer), C.byref(cache.view), _ptr(out),
                                   C.c_float(scale), _ptr(workspace), int(workspace.numel() * workspace.element_size()),
                                   _stream()), "moqae_decode_attn")


def moqae_decode_attn_ex(cfg, q, layer, cache: Cache, out, workspace, flags=0, scale=0.0):
    """moqae_decode_attn with flags; DECODE_OVERLAP_PREVIOUS lets the launch start while the
    previous kernel on the stream is finishing (see include/moqae.h for the caller's promise)."""
    _check(lib().moqae_decode_attn_ex(C.byref(cfg), _ptr(q), int(layer), C.byref(cache.view), _ptr(out),
                                      C.c_float(scale), _ptr(workspace), int(workspace.numel() * workspace.element_size()),
                                      int(flags), _stream()), "moqae_decode_attn_ex")


def moqae_decode_attn_step(cfg, q, k_new, v_new, layer, cache: Cache, out, workspace, flags=0, scale=0.0):
    """Decode attention that also attends to the current token's own rows k_new / v_new (not yet in the
    cache); append them afterwards with moqae_append_kv."""
    _check(lib().moqae_decode_attn_step(C.byref(cfg), _ptr(q), _ptr(k_new), _ptr(v_new), int(layer), C.byref(cache.view),
                                        _ptr(out), C.c_float(scale), _ptr(workspace),
                                        int(workspace.numel() * workspace.element_size()), int(flags), _stream()),
           "moqae_decode_attn_step")


def moqae_decode_attn_static_max_bytes() -> int:
    return int(lib().moqae_decode_attn_static_max_bytes())


def moqae_decode_attn_static(cfg, q, layer, cache: Cache, out, scale=0.0):
    """moqae_decode_attn without a caller-provided workspace: for callers that cannot allocate
    device memory, the split partials live in a fixed array inside the library."""
    _check(lib().moqae_decode_attn_static(C.byref(cfg), _ptr(q), int(layer), C.byref(cache.view), _ptr(out),
                                          C.c_float(scale), _stream()), "moqae_decode_attn_static")


def moqae_validate_tables(cfg, cache: Cache, T, layer_group=0):
    """(code, bad_row, bad_chunk): OK, or ERR_CORRUPT_TABLE with the first offending position."""
    r, c = C.c_int32(-1), C.c_int32(-1)
    rc = lib().moqae_validate_tables(C.byref(cfg), C.byref(cache.view), int(T), int(layer_group), _stream(),
                                     C.byref(r), C.byref(c))
    if rc not in (OK, ERR_CORRUPT_TABLE):
        raise MoqaeError(rc, "moqae_validate_tables")
    return rc, int(r.value), int(c.value)


def moqae_validate_tables_host(map_u8, slot_i32, count_i32, n_chunks, capacity):
    """The same check on host numpy arrays map / slot [rows, max_chunks] and count [rows, 4]."""
    import numpy as np
    m = np.ascontiguousarray(map_u8, dtype=np.uint8)
    s = np.ascontiguousarray(slot_i32, dtype=np.int32)
    k = np.ascontiguousarray(count_i32, dtype=np.int32)
    cap = (C.c_int64 * 4)(*[int(x) for x in capacity])
    r, c = C.c_int32(-1), C.c_int32(-1)
    rc = lib().moqae_validate_tables_host(m.ctypes.data_as(C.c_void_p), s.ctypes.data_as(C.c_void_p),
                                          k.ctypes.data_as(C.c_void_p), m.shape[0], m.shape[1], int(n_chunks), cap,
                                          C.byref(r), C.byref(c))
    return rc, int(r.value), int(c.value)


def moqae_poll_status(cache: Cache) -> int:
    out = C.c_int32(0)
    _check(lib().moqae_poll_status(C.byref(cache.view), _stream(), C.byref(out)), "moqae_poll_status")
    return int(out.value)
