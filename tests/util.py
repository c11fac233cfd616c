"""Test helpers: turn a synthetic LayerKV into the oracle's host descriptor and
compare CUDA results with oracle results under the acceptance rules."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from oracle import adapter
from paper_2410_05076_b200 import synth

MAX_ABS_TOL = 2e-2      # attention output, max |gpu - oracle|
MEAN_ABS_TOL = 2e-3     # attention output, mean |gpu - oracle|
TIE_BAND = 1e-3         # index sets must agree outside this band around the k-th score


def oracle_kv(layer: synth.LayerKV) -> oracle.KV:
    return adapter.kv_from_layer(layer)


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


CANARY_BYTES = 512      # guard zone on each side of a guarded buffer


class Guarded:
    """A device tensor with CANARY_BYTES of a fixed pattern directly before and after it in memory.
    compute-sanitizer is not available where these tests run; the guard zones catch stores that
    stray past either end of an output buffer. `t` is the tensor to hand to the library."""

    def __init__(self, shape, dtype, device, fill=None):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        body = (n + 255) // 256 * 256                      # keeps the alignment of whatever follows
        self.raw = torch.empty(CANARY_BYTES + body + CANARY_BYTES, dtype=torch.uint8, device=device)
        self.pattern = (torch.arange(CANARY_BYTES, device=device) * 37 + 11).to(torch.uint8)
        self.raw[:CANARY_BYTES] = self.pattern
        self.raw[CANARY_BYTES + n:] = 0xA5
        self.raw[CANARY_BYTES + body:] = self.pattern
        self.n, self.body = n, body
        self.t = self.raw[CANARY_BYTES:CANARY_BYTES + n].view(dtype).view(*shape)
        if fill is not None:
            self.t.fill_(fill)

    def check(self, what=""):
        torch.cuda.synchronize()
        assert torch.equal(self.raw[:CANARY_BYTES], self.pattern), f"{what}: store before the buffer"
        assert (self.raw[CANARY_BYTES + self.n:CANARY_BYTES + self.body] == 0xA5).all(), f"{what}: store just past the buffer"
        assert torch.equal(self.raw[CANARY_BYTES + self.body:], self.pattern), f"{what}: store after the buffer"
