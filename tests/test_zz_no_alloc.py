"""The allocation-free sparse-attention entry point, through the C-ABI.

Some users of this library cannot allocate device memory when they call it (a server that gave all
memory to its own pool, a latency-critical loop that cannot afford cudaMalloc's synchronisation).
For them tidal_sparse_attn_noalloc keeps its scratch in a fixed static device array. This file
checks that it returns what the CPU oracle and tidal_sparse_attn return, twice in a row (the array keeps the previous
call's contents), that it refuses problems larger than its scratch, and that it works in a fresh
process as well as after every other test (pytest collects this file last)."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle

from paper_2410_05076_b200 import binding, synth
from tests import util

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _case(batch, hq, hkv, ctx, k, layout, seed):
    w = synth.Workload(f"na{seed}", batch, hq, hkv, 2, ctx, k, min(8, ctx),
                       [synth.LAYER_SELECT, synth.LAYER_SPARSE], synth.BASE_SEED + 900 + seed,
                       ragged=batch > 1, ctx_min=max(1, ctx // 2))
    q = synth.make_q(w, 0, DEV)
    if layout == "paged":
        pt, total = synth.make_page_table(w, extra_pages=2)
        lay = synth.make_layer(w, 0, DEV, layout="paged", q=q, page_table=pt, num_pages=total)
    else:
        lay = synth.make_layer(w, 0, DEV, layout=layout, q=q)
    return w, q, lay


@pytest.mark.parametrize("batch,hq,hkv,ctx,k,layout,hi,with_count", [
    (1, 8, 2, 3000, 200, "hnd_interleaved", 8, True),
    (2, 8, 2, 1500, 96, "paged", 8, True),
    (1, 32, 8, 20000, 2048, "hnd_interleaved", 32, True),
    (128, 32, 8, 300, 48, "hnd_interleaved", 32, True),      # 4096 rows: the most the scratch holds, one CTA per item
    (3, 8, 2, 2000, 512, "nhd_separate", 2, True),           # one token set per KV head
    (2, 8, 2, 2000, 512, "paged", 1, True),                  # one set shared by all heads
    (1, 8, 2, 3000, 200, "hnd_interleaved", 8, False),       # no idx_count: the -1 padding ends the lists
    (40, 16, 2, 900, 512, "hnd_interleaved", 16, True),      # 640 items: more CTAs than are resident at once
])
def test_noalloc_matches_the_oracle_and_the_context_entry_point_twice(batch, hq, hkv, ctx, k, layout, hi, with_count):
    w, q, lay = _case(batch, hq, hkv, ctx, k, layout, seed=ctx % 97)
    td = binding.Tidal(0)
    try:
        gran = {hq: binding.SEL_PER_QHEAD, hkv: binding.SEL_PER_KVHEAD, 1: binding.SEL_SHARED}[hi]
        _, idx, cnt = td.select_attn(lay, q, k, granularity=gran)
        cnt_arg = cnt if with_count else None
        ref = td.sparse_attn(lay, q, idx, cnt_arg)
        torch.cuda.synchronize()
        # the independent check: the CPU oracle on the same token sets
        want = oracle.sparse_attn(util.oracle_kv(lay), synth.bits(q), idx.cpu().numpy(),
                                  cnt.cpu().numpy() if with_count else None)
        out = torch.full_like(ref, float("nan"))
        for call in range(2):                       # second call sees the first call's leftovers
            out.fill_(float("nan"))
            binding.sparse_attn_noalloc(lay, q, idx, cnt_arg, out=out)
            torch.cuda.synchronize()
            util.check_out(out.cpu().numpy(), want, f"noalloc call {call} vs oracle")
            # the two entry points split the index list differently, so the bf16 rounding of the
            # softmax weights differs term by term; both stay far inside the oracle tolerance
            util.check_out(out.cpu().numpy(), ref.cpu().numpy(), f"noalloc call {call} vs tidal_sparse_attn")
            assert torch.allclose(out, ref, rtol=0, atol=1e-3)
        assert td.device_status() == binding.OK
    finally:
        td.close()


def test_noalloc_refuses_more_rows_than_its_scratch_holds():
    w, q, lay = _case(1, 8, 2, 64, 8, "hnd_interleaved", seed=3)
    lib = binding.load()
    s = binding.kv_struct(lay)
    s.batch = 1025                                   # 1025 * 8 rows > 4096; rejected on the host
    out = torch.empty(1, 8, 128, dtype=torch.float32, device=DEV)
    idx = torch.zeros(1, 8, 8, dtype=torch.int32, device=DEV)
    rc = lib.tidal_sparse_attn_noalloc(C.byref(s), q.data_ptr(), idx.data_ptr(), None, 8, 8,
                                       out.data_ptr(), None)
    assert rc == binding.ERR_TOO_LARGE
    assert "scratch" in binding.strerror(rc)
    s = binding.kv_struct(lay)
    assert lib.tidal_sparse_attn_noalloc(C.byref(s), q.data_ptr(), idx.data_ptr(), None, 0, 8,
                                         out.data_ptr(), None) == binding.ERR_INVALID
