"""ctypes front end of the CPU oracle (test infrastructure, not the product).

The oracle itself is `tidal_oracle.c`: a plain C restatement of Eq. 1 and
Algorithm 1 of the TidalDecode paper (full attention, argTopK by full sort,
sparse attention over the selected positions, the layer schedule). This module
only compiles it with gcc and marshals numpy arrays; it holds no arithmetic.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
it. It never imports the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tidal_oracle.c")
_HDR = os.path.join(_HERE, "tidal_oracle.h")
_LIB = os.path.join(_HERE, "libtidal_oracle.so")

LAYER_FULL, LAYER_SELECT, LAYER_SPARSE = 0, 1, 2
KV_BF16, KV_FP8_E4M3 = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP) if the shared object is stale."""
    stale = force or not os.path.exists(_LIB) or any(
        os.path.getmtime(p) > os.path.getmtime(_LIB) for p in (_SRC, _HDR))
    if stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _KV(C.Structure):
    _fields_ = [
        ("batch", C.c_int32), ("num_q_heads", C.c_int32), ("num_kv_heads", C.c_int32),
        ("head_dim", C.c_int32), ("paged", C.c_int32),
        ("k", C.c_void_p), ("v", C.c_void_p),
        ("stride_b", C.c_int64), ("stride_pos", C.c_int64), ("stride_head", C.c_int64),
        ("stride_page", C.c_int64),
        ("page_table", C.c_void_p), ("page_size", C.c_int32), ("max_pages_per_seq", C.c_int32),
        ("ctx_lens", C.c_void_p), ("sm_scale", C.c_float),
        ("kv_dtype", C.c_int32), ("k_scale", C.c_void_p), ("v_scale", C.c_void_p),
    ]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        P, I, I64 = C.c_void_p, C.c_int, C.c_int64
        L.oracle_logits.argtypes = [C.POINTER(_KV), P, I, I, P]
        L.oracle_logits.restype = None
        L.oracle_softmax_weights.argtypes = [P, I, P]
        L.oracle_softmax_weights.restype = None
        L.oracle_full_attn.argtypes = [C.POINTER(_KV), P, P, P, I64]
        L.oracle_full_attn.restype = I
        L.oracle_topk.argtypes = [P, I, I, P]
        L.oracle_topk.restype = I
        L.oracle_select_attn.argtypes = [C.POINTER(_KV), P, I, I, P, P, P, P, I64]
        L.oracle_select_attn.restype = I
        L.oracle_sparse_attn.argtypes = [C.POINTER(_KV), P, P, P, I, I, P]
        L.oracle_sparse_attn.restype = I
        L.oracle_decode_step.argtypes = [I, P, C.POINTER(_KV), C.POINTER(P), C.POINTER(P), I, I, P, P]
        L.oracle_decode_step.restype = I
        L.oracle_kv_append.argtypes = [C.POINTER(_KV), P, P]
        L.oracle_kv_append.restype = None
        L.oracle_schedule.argtypes = [I, I, P]
        L.oracle_schedule.restype = None
        L.oracle_num_threads.restype = I
        L.oracle_e4m3_decode.argtypes = [C.c_uint8]
        L.oracle_e4m3_decode.restype = C.c_float
        _lib = L
    return _lib


@dataclass
class KV:
    """One layer's KV cache on the host: uint16 (bf16 bits) arrays plus element
    strides, contiguous or paged (see oracle_kv_t in tidal_oracle.h)."""
    k: np.ndarray
    v: np.ndarray
    batch: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    ctx_lens: np.ndarray
    stride_b: int = 0
    stride_pos: int = 0
    stride_head: int = 0
    stride_page: int = 0
    page_table: Optional[np.ndarray] = None
    page_size: int = 16
    max_pages_per_seq: int = 0
    sm_scale: float = 0.0
    k_offset: int = 0   # element offsets of K and V inside their arrays
    v_offset: int = 0
    kv_dtype: int = 0   # 0: bf16 bits in uint16 arrays; 1: OCP FP8 E4M3 codes in uint8 arrays
    k_scale: Optional[np.ndarray] = None   # fp8: float32 [num_kv_heads], None = 1
    v_scale: Optional[np.ndarray] = None

    def c_struct(self) -> _KV:
        want = np.uint8 if self.kv_dtype == KV_FP8_E4M3 else np.uint16
        assert self.k.dtype == want and self.v.dtype == want
        esz = 1 if self.kv_dtype == KV_FP8_E4M3 else 2
        self.ctx_lens = np.ascontiguousarray(self.ctx_lens, dtype=np.int32)
        s = _KV()
        s.batch, s.num_q_heads, s.num_kv_heads, s.head_dim = (
            self.batch, self.num_q_heads, self.num_kv_heads, self.head_dim)
        s.paged = 1 if self.page_table is not None else 0
        s.k = self.k.ctypes.data + esz * self.k_offset
        s.v = self.v.ctypes.data + esz * self.v_offset
        s.kv_dtype = self.kv_dtype
        if self.k_scale is not None:
            self.k_scale = np.ascontiguousarray(self.k_scale, dtype=np.float32)
            s.k_scale = self.k_scale.ctypes.data
        if self.v_scale is not None:
            self.v_scale = np.ascontiguousarray(self.v_scale, dtype=np.float32)
            s.v_scale = self.v_scale.ctypes.data
        s.stride_b, s.stride_pos, s.stride_head, s.stride_page = (
            self.stride_b, self.stride_pos, self.stride_head, self.stride_page)
        if self.page_table is not None:
            self.page_table = np.ascontiguousarray(self.page_table, dtype=np.int32)
            s.page_table = self.page_table.ctypes.data
            s.max_pages_per_seq = self.max_pages_per_seq or self.page_table.shape[-1]
        s.page_size = self.page_size
        s.ctx_lens = self.ctx_lens.ctypes.data
        s.sm_scale = self.sm_scale
        return s


def _q(q: np.ndarray) -> np.ndarray:
    assert q.dtype == np.uint16
    return np.ascontiguousarray(q)


def logits(kv: KV, q: np.ndarray, b: int, h: int) -> np.ndarray:
    q = _q(q)
    s = np.empty(int(kv.ctx_lens[b]), dtype=np.float32)
    st = kv.c_struct()
    lib().oracle_logits(C.byref(st), q.ctypes.data, b, h, s.ctypes.data)
    return s


def softmax_weights(s: np.ndarray) -> np.ndarray:
    s = np.ascontiguousarray(s, dtype=np.float32)
    w = np.empty(s.shape[0], dtype=np.float64)
    lib().oracle_softmax_weights(s.ctypes.data, s.shape[0], w.ctypes.data)
    return w


def full_attn(kv: KV, q: np.ndarray, want_scores: bool = False):
    q = _q(q)
    out = np.zeros((kv.batch, kv.num_q_heads, kv.head_dim), dtype=np.float32)
    st = kv.c_struct()
    if want_scores:
        nmax = int(max(1, kv.ctx_lens.max()))
        sc = np.full((kv.batch, kv.num_q_heads, nmax), -np.inf, dtype=np.float32)
        lib().oracle_full_attn(C.byref(st), q.ctypes.data, out.ctypes.data, sc.ctypes.data, nmax)
        return out, sc
    lib().oracle_full_attn(C.byref(st), q.ctypes.data, out.ctypes.data, None, 0)
    return out


def topk(s: np.ndarray, k: int) -> np.ndarray:
    s = np.ascontiguousarray(s, dtype=np.float32)
    idx = np.empty(k, dtype=np.int32)
    lib().oracle_topk(s.ctypes.data, s.shape[0], k, idx.ctypes.data)
    return idx


def select_attn(kv: KV, q: np.ndarray, k: int, num_index_heads: Optional[int] = None,
                want_scores: bool = False):
    q = _q(q)
    hi = num_index_heads or kv.num_q_heads
    out = np.zeros((kv.batch, kv.num_q_heads, kv.head_dim), dtype=np.float32)
    idx = np.empty((kv.batch, hi, k), dtype=np.int32)
    cnt = np.empty(kv.batch, dtype=np.int32)
    st = kv.c_struct()
    sc, stride, scp = None, 0, None
    if want_scores:
        stride = int(max(1, kv.ctx_lens.max()))
        sc = np.full((kv.batch, kv.num_q_heads, stride), -np.inf, dtype=np.float32)
        scp = sc.ctypes.data
    rc = lib().oracle_select_attn(C.byref(st), q.ctypes.data, k, hi, out.ctypes.data,
                                  idx.ctypes.data, cnt.ctypes.data, scp, stride)
    if rc:
        raise ValueError("oracle_select_attn: bad arguments")
    return (out, idx, cnt, sc) if want_scores else (out, idx, cnt)


def sparse_attn(kv: KV, q: np.ndarray, idx: np.ndarray, idx_count: Optional[np.ndarray] = None):
    q = _q(q)
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    _, hi, k = idx.shape
    out = np.zeros((kv.batch, kv.num_q_heads, kv.head_dim), dtype=np.float32)
    st = kv.c_struct()
    cp = None
    if idx_count is not None:
        idx_count = np.ascontiguousarray(idx_count, dtype=np.int32)
        cp = idx_count.ctypes.data
    rc = lib().oracle_sparse_attn(C.byref(st), q.ctypes.data, idx.ctypes.data, cp, k, hi,
                                  out.ctypes.data)
    if rc:
        raise ValueError("oracle_sparse_attn: bad arguments")
    return out


def with_newest(kv: KV, idx: np.ndarray, idx_count: np.ndarray):
    """Index lists for the optional 'always attend the newest token' variant (not in the paper): every
    list gets one more slot holding position ctx_len - 1, or -1 if the list already ends with it. Data
    preparation only; the attention itself is sparse_attn on the returned lists."""
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    B, hi, k = idx.shape
    out = np.full((B, hi, k + 1), -1, dtype=np.int32)
    cnt = np.asarray(idx_count, dtype=np.int32)
    for b in range(B):
        c, n = int(min(cnt[b], k)), int(kv.ctx_lens[b])
        out[b, :, :c] = idx[b, :, :c]
        for h in range(hi):
            last = idx[b, h, c - 1] if c > 0 else -1
            out[b, h, c] = n - 1 if (n > 0 and last != n - 1) else -1
    return out, cnt + 1


def kv_append(kv: KV, k_new: np.ndarray, v_new: np.ndarray) -> None:
    """C.append(k, v): writes the rows [B, Hkv, d] at position ctx_lens[b] - 1 of kv's arrays, in place."""
    want = np.uint8 if kv.kv_dtype == KV_FP8_E4M3 else np.uint16
    assert k_new.dtype == want and v_new.dtype == want
    k_new, v_new = np.ascontiguousarray(k_new), np.ascontiguousarray(v_new)
    st = kv.c_struct()
    lib().oracle_kv_append(C.byref(st), k_new.ctypes.data, v_new.ctypes.data)


def e4m3_decode(codes) -> np.ndarray:
    """Values of OCP FP8 E4M3 codes (any array of uint8), one call of the C decoder per element."""
    codes = np.asarray(codes, dtype=np.uint8)
    f = lib().oracle_e4m3_decode
    return np.array([f(int(c)) for c in codes.reshape(-1)], dtype=np.float32).reshape(codes.shape)


def schedule(num_layers: int, reselect_layer: int) -> np.ndarray:
    s = np.empty(num_layers, dtype=np.uint8)
    lib().oracle_schedule(num_layers, reselect_layer, s.ctypes.data)
    return s


def decode_step(sched: Sequence[int], kvs: Sequence[KV], qs: Sequence[np.ndarray], k: int,
                num_index_heads: Optional[int] = None):
    """Algorithm 1's attention branch over all layers. Returns (outs, idx, idx_count)."""
    L = len(sched)
    sched = np.ascontiguousarray(sched, dtype=np.uint8)
    hi = num_index_heads or kvs[0].num_q_heads
    B = kvs[0].batch
    structs = (_KV * L)(*[kv.c_struct() for kv in kvs])
    qs = [_q(q) for q in qs]
    outs = [np.zeros((kv.batch, kv.num_q_heads, kv.head_dim), dtype=np.float32) for kv in kvs]
    qp = (C.c_void_p * L)(*[q.ctypes.data for q in qs])
    op = (C.c_void_p * L)(*[o.ctypes.data for o in outs])
    idx = np.full((B, hi, k), -1, dtype=np.int32)
    cnt = np.zeros(B, dtype=np.int32)
    rc = lib().oracle_decode_step(L, sched.ctypes.data, structs, qp, op, k, hi,
                                  idx.ctypes.data, cnt.ctypes.data)
    if rc:
        raise ValueError("oracle_decode_step: sparse layer before any selection layer")
    return outs, idx, cnt


def num_threads() -> int:
    return lib().oracle_num_threads()
