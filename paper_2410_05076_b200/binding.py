"""Thin ctypes binding of libtidal.so (same names as include/tidal.h).

Argument marshalling only: every step of the attention path runs in the CUDA
kernels behind the C-ABI. PyTorch supplies device memory and the current
stream. If the shared library is missing and cannot be built the import of
this module's `load()` raises; there is no fallback of any kind.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

from . import build as _build

OK = 0
ERR_INVALID, ERR_UNSUPPORTED, ERR_NOMEM, ERR_CUDA, ERR_TIMEOUT, ERR_INDEX = -1, -2, -3, -4, -5, -6
ERR_TOO_LARGE, ERR_INTERNAL = -7, -8
KV_CONTIG, KV_PAGED = 0, 1
KV_BF16, KV_FP8_E4M3 = 0, 1
SEL_PER_QHEAD, SEL_PER_KVHEAD, SEL_SHARED = 0, 1, 2
LAYER_FULL, LAYER_SELECT, LAYER_SPARSE = 0, 1, 2

EXPORTS = [
    "tidal_create", "tidal_destroy", "tidal_workspace_bytes", "tidal_full_attn", "tidal_select_attn",
    "tidal_sparse_attn", "tidal_decode_step", "tidal_decode_step_host", "tidal_device_status",
    "tidal_launch_count", "tidal_strerror", "tidal_sparse_attn_noalloc", "tidal_kv_append",
    "tidal_decode_step_append", "tidal_set_graphs", "tidal_set_output_dtype", "tidal_set_attend_newest",
    "tidal_set_layer_overlap", "tidal_reserve", "tidal_set_select_margin",
]


class tidal_kv_t(C.Structure):
    _fields_ = [
        ("batch", C.c_int32), ("num_q_heads", C.c_int32), ("num_kv_heads", C.c_int32),
        ("head_dim", C.c_int32), ("kv_layout", C.c_int32),
        ("k", C.c_void_p), ("v", C.c_void_p),
        ("stride_b", C.c_int64), ("stride_pos", C.c_int64), ("stride_head", C.c_int64),
        ("stride_page", C.c_int64),
        ("page_table", C.c_void_p), ("page_size", C.c_int32), ("max_pages_per_seq", C.c_int32),
        ("num_pages", C.c_int32),
        ("ctx_lens", C.c_void_p), ("max_ctx_len", C.c_int32), ("sm_scale", C.c_float),
        ("kv_dtype", C.c_int32), ("k_scale", C.c_void_p), ("v_scale", C.c_void_p),
    ]


class TidalError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {strerror(status)} ({status})")


_lib = None


def load() -> C.CDLL:
    """Load libtidal.so, building it with nvcc first if it is missing or stale."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB
    if not os.path.exists(path) or _build.is_stale():
        try:
            _build.build()
        except Exception as exc:  # no silent fallback: neither to another implementation nor to an outdated library
            what = "is older than its sources" if os.path.exists(path) else "is missing"
            raise ImportError(f"libtidal.so {what} and could not be rebuilt: {exc}") from exc
    L = C.CDLL(path)
    P, I32, I64 = C.c_void_p, C.c_int32, C.c_int64
    KVP = C.POINTER(tidal_kv_t)
    L.tidal_create.argtypes = [C.POINTER(P), C.c_int, C.c_size_t]
    L.tidal_create.restype = I32
    L.tidal_destroy.argtypes = [P]
    L.tidal_destroy.restype = I32
    L.tidal_workspace_bytes.argtypes = [KVP, I32]
    L.tidal_workspace_bytes.restype = C.c_size_t
    L.tidal_decode_step_append.argtypes = [P, I32, P, KVP, P, P, P, P, I32, I32, P, P, P]
    L.tidal_decode_step_append.restype = I32
    L.tidal_set_attend_newest.argtypes = [P, I32]
    L.tidal_set_attend_newest.restype = I32
    L.tidal_set_output_dtype.argtypes = [P, I32]
    L.tidal_set_output_dtype.restype = I32
    L.tidal_set_layer_overlap.argtypes = [P, I32]
    L.tidal_set_layer_overlap.restype = I32
    L.tidal_set_select_margin.argtypes = [P, C.c_float]
    L.tidal_set_select_margin.restype = I32
    L.tidal_reserve.argtypes = [P, KVP, I32, I32]
    L.tidal_reserve.restype = I32
    L.tidal_set_graphs.argtypes = [P, I32]
    L.tidal_set_graphs.restype = I32
    L.tidal_kv_append.argtypes = [P, KVP, P, P, P]
    L.tidal_kv_append.restype = I32
    L.tidal_full_attn.argtypes = [P, KVP, P, P, P]
    L.tidal_full_attn.restype = I32
    L.tidal_select_attn.argtypes = [P, KVP, P, I32, I32, P, P, P, P, P]
    L.tidal_select_attn.restype = I32
    L.tidal_sparse_attn.argtypes = [P, KVP, P, P, P, I32, I32, P, P]
    L.tidal_sparse_attn.restype = I32
    L.tidal_sparse_attn_noalloc.argtypes = [KVP, P, P, P, I32, I32, P, P]
    L.tidal_sparse_attn_noalloc.restype = I32
    L.tidal_decode_step.argtypes = [P, I32, P, KVP, C.POINTER(P), C.POINTER(P), I32, I32, P, P, P]
    L.tidal_decode_step.restype = I32
    L.tidal_decode_step_host.argtypes = [P, I32, P, KVP, P, P, I32, I32, P]
    L.tidal_decode_step_host.restype = I32
    L.tidal_device_status.argtypes = [P, P]
    L.tidal_device_status.restype = I32
    L.tidal_launch_count.argtypes = [P]
    L.tidal_launch_count.restype = I64
    L.tidal_strerror.argtypes = [I32]
    L.tidal_strerror.restype = C.c_char_p
    _lib = L
    return L


def strerror(status: int) -> str:
    return load().tidal_strerror(status).decode()


def kv_struct(layer) -> tidal_kv_t:
    """Descriptor of one layer's cache from any object with LayerKV's fields."""
    s = tidal_kv_t()
    s.batch, s.num_q_heads, s.num_kv_heads, s.head_dim = (
        layer.batch, layer.num_q_heads, layer.num_kv_heads, layer.head_dim)
    paged = layer.page_table is not None
    s.kv_layout = KV_PAGED if paged else KV_CONTIG
    s.k, s.v = layer.k.data_ptr(), layer.v.data_ptr()
    s.stride_b, s.stride_pos, s.stride_head, s.stride_page = (
        layer.stride_b, layer.stride_pos, layer.stride_head, layer.stride_page)
    if paged:
        s.page_table = layer.page_table.data_ptr()
        s.page_size = layer.page_size
        s.max_pages_per_seq = layer.max_pages_per_seq
        s.num_pages = getattr(layer, "num_pages", 0) or layer.keep[0].shape[0]
    s.ctx_lens = layer.ctx_lens.data_ptr()
    s.max_ctx_len = layer.max_ctx_len
    s.sm_scale = layer.sm_scale
    s.kv_dtype = getattr(layer, "kv_dtype", 0)
    if s.kv_dtype:
        s.k_scale = layer.k_scale.data_ptr() if layer.k_scale is not None else None
        s.v_scale = layer.v_scale.data_ptr() if layer.v_scale is not None else None
    return s


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(status: int, what: str) -> None:
    if status != OK:
        raise TidalError(status, what)


def sparse_attn_noalloc(layer, q: torch.Tensor, idx: torch.Tensor, idx_count: Optional[torch.Tensor] = None,
                        out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """tidal_sparse_attn_noalloc on the current device and stream: sparse attention for callers that
    may not allocate device memory. No context is involved; the library's fixed static scratch is
    used, so batch * num_q_heads is limited to 4096 and overlapping calls on one GPU race. `out`
    should be passed by such callers (this wrapper allocates it with torch only as a convenience)."""
    if out is None:
        out = torch.empty(layer.batch, layer.num_q_heads, layer.head_dim, dtype=torch.float32, device=q.device)
    s = kv_struct(layer)
    _, hi, k = idx.shape
    _check(load().tidal_sparse_attn_noalloc(C.byref(s), q.data_ptr(), idx.data_ptr(),
                                            idx_count.data_ptr() if idx_count is not None else None, k, hi,
                                            out.data_ptr(), _stream()), "tidal_sparse_attn_noalloc")
    return out


class Tidal:
    """A libtidal context on one CUDA device (use one context per stream)."""

    def __init__(self, device: int = 0, workspace_bytes: int = 0):
        self.lib = load()
        self.ctx = C.c_void_p()
        _check(self.lib.tidal_create(C.byref(self.ctx), device, workspace_bytes), "tidal_create")
        self.device = device
        self.out_dtype = torch.float32

    def close(self) -> None:
        if getattr(self, "ctx", None) and self.ctx.value:
            self.lib.tidal_destroy(self.ctx)
            self.ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @staticmethod
    def workspace_bytes(layer, k: int) -> int:
        s = kv_struct(layer)
        return load().tidal_workspace_bytes(C.byref(s), k)

    def reserve(self, layer, k: int, num_layers_host: int = 0) -> None:
        """Allocate everything later calls with this cache shape and budget need (then they can be captured)."""
        s = kv_struct(layer)
        _check(self.lib.tidal_reserve(self.ctx, C.byref(s), k, num_layers_host), "tidal_reserve")

    def kv_append(self, layer, k_new: torch.Tensor, v_new: torch.Tensor) -> None:
        """Write the new token's rows (bf16 [B, Hkv, d]) at position ctx_lens[b] - 1 of the layer's cache."""
        s = kv_struct(layer)
        _check(self.lib.tidal_kv_append(self.ctx, C.byref(s), k_new.data_ptr(), v_new.data_ptr(), _stream()),
               "tidal_kv_append")

    def full_attn(self, layer, q: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        if out is None:
            out = torch.empty(layer.batch, layer.num_q_heads, layer.head_dim, dtype=self.out_dtype, device=q.device)
        s = kv_struct(layer)
        _check(self.lib.tidal_full_attn(self.ctx, C.byref(s), q.data_ptr(), out.data_ptr(), _stream()),
               "tidal_full_attn")
        return out

    def select_attn(self, layer, q: torch.Tensor, k: int, granularity: int = SEL_PER_QHEAD,
                    out: Optional[torch.Tensor] = None, idx: Optional[torch.Tensor] = None,
                    idx_count: Optional[torch.Tensor] = None, scores: Optional[torch.Tensor] = None):
        hi = {SEL_PER_QHEAD: layer.num_q_heads, SEL_PER_KVHEAD: layer.num_kv_heads, SEL_SHARED: 1}.get(granularity, 1)
        if out is None:
            out = torch.empty(layer.batch, layer.num_q_heads, layer.head_dim, dtype=self.out_dtype, device=q.device)
        if idx is None:
            idx = torch.empty(layer.batch, hi, max(k, 1), dtype=torch.int32, device=q.device)
        if idx_count is None:
            idx_count = torch.empty(layer.batch, dtype=torch.int32, device=q.device)
        s = kv_struct(layer)
        _check(self.lib.tidal_select_attn(self.ctx, C.byref(s), q.data_ptr(), k, granularity, out.data_ptr(),
                                          idx.data_ptr(), idx_count.data_ptr(),
                                          scores.data_ptr() if scores is not None else None, _stream()),
               "tidal_select_attn")
        return out, idx, idx_count

    def sparse_attn(self, layer, q: torch.Tensor, idx: torch.Tensor, idx_count: Optional[torch.Tensor] = None,
                    out: Optional[torch.Tensor] = None) -> torch.Tensor:
        if out is None:
            out = torch.empty(layer.batch, layer.num_q_heads, layer.head_dim, dtype=self.out_dtype, device=q.device)
        s = kv_struct(layer)
        _, hi, k = idx.shape
        _check(self.lib.tidal_sparse_attn(self.ctx, C.byref(s), q.data_ptr(), idx.data_ptr(),
                                          idx_count.data_ptr() if idx_count is not None else None, k, hi,
                                          out.data_ptr(), _stream()), "tidal_sparse_attn")
        return out

    def make_step(self, sched: Sequence[int], layers: Sequence, qs: Sequence[torch.Tensor],
                  outs: Sequence[torch.Tensor], k: int, granularity: int = SEL_PER_QHEAD):
        """Marshal the per-layer arrays once; the returned callable enqueues one decode step."""
        L = len(sched)
        sched_arr = (C.c_uint8 * L)(*sched)
        kvs = (tidal_kv_t * L)(*[kv_struct(l) for l in layers])
        qp = (C.c_void_p * L)(*[q.data_ptr() for q in qs])
        op = (C.c_void_p * L)(*[o.data_ptr() for o in outs])
        hi = {SEL_PER_QHEAD: layers[0].num_q_heads, SEL_PER_KVHEAD: layers[0].num_kv_heads, SEL_SHARED: 1}[granularity]
        dev = qs[0].device
        idx = torch.full((layers[0].batch, hi, k), -1, dtype=torch.int32, device=dev)
        cnt = torch.zeros(layers[0].batch, dtype=torch.int32, device=dev)
        keep = (sched_arr, kvs, qp, op, list(layers), list(qs), list(outs))

        def step():
            _check(self.lib.tidal_decode_step(self.ctx, L, sched_arr, kvs, qp, op, k, granularity,
                                              idx.data_ptr(), cnt.data_ptr(), _stream()), "tidal_decode_step")

        step.idx, step.idx_count, step.keep = idx, cnt, keep
        return step

    def decode_step_append(self, sched, layers, qs, k_new, v_new, k: int, granularity: int = SEL_PER_QHEAD):
        """One step including the cache update: k_new[i], v_new[i] (bf16 [B, Hkv, d]) go to position
        ctx_lens[b] - 1 of layer i's cache before the layers run. Returns (outs, idx, idx_count)."""
        L = len(sched)
        outs = [torch.empty(l.batch, l.num_q_heads, l.head_dim, dtype=self.out_dtype, device=qs[0].device)
                for l in layers]
        hi = {SEL_PER_QHEAD: layers[0].num_q_heads, SEL_PER_KVHEAD: layers[0].num_kv_heads, SEL_SHARED: 1}[granularity]
        idx = torch.full((layers[0].batch, hi, k), -1, dtype=torch.int32, device=qs[0].device)
        cnt = torch.zeros(layers[0].batch, dtype=torch.int32, device=qs[0].device)
        ptrs = lambda ts: (C.c_void_p * L)(*[t.data_ptr() for t in ts])
        _check(self.lib.tidal_decode_step_append(
            self.ctx, L, (C.c_uint8 * L)(*sched), (tidal_kv_t * L)(*[kv_struct(l) for l in layers]), ptrs(qs),
            ptrs(k_new), ptrs(v_new), ptrs(outs), k, granularity, idx.data_ptr(), cnt.data_ptr(), _stream()),
            "tidal_decode_step_append")
        return outs, idx, cnt

    def decode_step(self, sched, layers, qs, k: int, granularity: int = SEL_PER_QHEAD):
        outs = [torch.empty(l.batch, l.num_q_heads, l.head_dim, dtype=self.out_dtype, device=qs[0].device)
                for l in layers]
        step = self.make_step(sched, layers, qs, outs, k, granularity)
        step()
        return outs, step.idx, step.idx_count

    def make_step_host(self, sched, layers, q_host: torch.Tensor, out_host: torch.Tensor, k: int,
                       granularity: int = SEL_PER_QHEAD):
        """q_host bf16 [L,B,Hq,d] and out_host fp32 [L,B,Hq,d] in (pinned) host memory."""
        L = len(sched)
        sched_arr = (C.c_uint8 * L)(*sched)
        kvs = (tidal_kv_t * L)(*[kv_struct(l) for l in layers])
        assert q_host.device.type == "cpu" and out_host.device.type == "cpu"
        assert q_host.is_contiguous() and out_host.is_contiguous()

        def step():
            _check(self.lib.tidal_decode_step_host(self.ctx, L, sched_arr, kvs, q_host.data_ptr(),
                                                   out_host.data_ptr(), k, granularity, _stream()),
                   "tidal_decode_step_host")

        step.keep = (sched_arr, kvs, list(layers), q_host, out_host)
        return step

    def set_attend_newest(self, enabled: bool) -> None:
        """Sparse layers also attend the newest token (an optional deviation from the paper's algorithm)."""
        _check(self.lib.tidal_set_attend_newest(self.ctx, 1 if enabled else 0), "tidal_set_attend_newest")

    def set_output_bf16(self, enabled: bool) -> None:
        """Later calls write bf16 outputs (pass bf16 `out` tensors) instead of fp32."""
        _check(self.lib.tidal_set_output_dtype(self.ctx, 1 if enabled else 0), "tidal_set_output_dtype")
        self.out_dtype = torch.bfloat16 if enabled else torch.float32

    def set_graphs(self, enabled: bool) -> None:
        """Record whole steps as CUDA graphs and replay them (on by default; needs a non-default stream)."""
        _check(self.lib.tidal_set_graphs(self.ctx, 1 if enabled else 0), "tidal_set_graphs")

    def set_select_margin(self, margin: float) -> None:
        """Safety factor of the selection layers' provisional thresholds (default 3; 0: rank all scores)."""
        _check(self.lib.tidal_set_select_margin(self.ctx, margin), "tidal_set_select_margin")

    def set_layer_overlap(self, enabled: bool) -> None:
        """Layers of a step may stream their inputs while the layer before them finishes (on by default)."""
        _check(self.lib.tidal_set_layer_overlap(self.ctx, 1 if enabled else 0), "tidal_set_layer_overlap")

    def device_status(self) -> int:
        return self.lib.tidal_device_status(self.ctx, _stream())

    def launch_count(self) -> int:
        return self.lib.tidal_launch_count(self.ctx)
