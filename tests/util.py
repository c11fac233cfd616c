"""Test helpers: turn a synthetic LayerKV into the oracle's host descriptor and
compare CUDA results with oracle results under the acceptance rules."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2410_05076_b200 import synth

MAX_ABS_TOL = 2e-2      # attention output, max |gpu - oracle|
MEAN_ABS_TOL = 2e-3     # attention output, mean |gpu - oracle|
TIE_BAND = 1e-3         # index sets must agree outside this band around the k-th score


def _host_bits(t: torch.Tensor, keep):
    """(uint16 array of the whole owning buffer, element offset of t in it)."""
    for buf in keep:
        if buf.untyped_storage().data_ptr() == t.untyped_storage().data_ptr():
            flat = buf.detach().reshape(-1)
            return synth.bits(flat), t.storage_offset() - buf.storage_offset()
    flat = t.detach().contiguous().reshape(-1)
    return synth.bits(flat), 0


def oracle_kv(layer: synth.LayerKV) -> oracle.KV:
    kb, koff = _host_bits(layer.k, layer.keep)
    if layer.v.untyped_storage().data_ptr() == layer.k.untyped_storage().data_ptr():
        vb, voff = kb, layer.v.storage_offset() - layer.keep[0].storage_offset()
    else:
        vb, voff = _host_bits(layer.v, layer.keep)
    return oracle.KV(
        k=kb, v=vb, k_offset=koff, v_offset=voff, batch=layer.batch,
        num_q_heads=layer.num_q_heads, num_kv_heads=layer.num_kv_heads, head_dim=layer.head_dim,
        ctx_lens=layer.ctx_lens.cpu().numpy().astype(np.int32),
        stride_b=layer.stride_b, stride_pos=layer.stride_pos, stride_head=layer.stride_head,
        stride_page=layer.stride_page,
        page_table=None if layer.page_table is None else layer.page_table.cpu().numpy(),
        page_size=layer.page_size, max_pages_per_seq=layer.max_pages_per_seq,
        sm_scale=layer.sm_scale)


def check_out(got, ref, what=""):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    err = np.abs(got - ref)
    assert err.max() <= MAX_ABS_TOL, f"{what}: max abs err {err.max():.3e}"
    assert err.mean() <= MEAN_ABS_TOL, f"{what}: mean abs err {err.mean():.3e}"


def check_idx_row(got_row, ref_scores, k, n, what=""):
    """One (sequence, index head): `got_row` int32 [k] from the CUDA path,
    `ref_scores` float32 [n] from the oracle. The set must have k' = min(k, n)
    distinct in-range members followed by -1 padding; every position scoring
    more than TIE_BAND above the oracle's k'-th largest score must be present
    and none scoring more than TIE_BAND below it may be."""
    kk = min(k, n)
    got = np.asarray(got_row)
    sel = got[:kk]
    assert (got[kk:] == -1).all(), f"{what}: padding is not -1"
    assert ((sel >= 0) & (sel < n)).all(), f"{what}: index out of range"
    assert len(np.unique(sel)) == kk, f"{what}: duplicate or missing entries"
    assert (np.diff(sel) > 0).all(), f"{what}: not ascending"
    if kk == n:
        return 0
    s = np.asarray(ref_scores[:n], dtype=np.float32)
    kth = np.partition(s, n - kk)[n - kk]
    must = np.nonzero(s > kth + TIE_BAND)[0]
    chosen = np.zeros(n, dtype=bool)
    chosen[sel] = True
    assert chosen[must].all(), f"{what}: {int((~chosen[must]).sum())} clear winners missing"
    assert (s[sel] >= kth - TIE_BAND).all(), f"{what}: member below the tie band"
    ref_sel = oracle.topk(s, k)[:kk]
    return int(kk - np.intersect1d(sel, ref_sel).size)   # differences inside the band
