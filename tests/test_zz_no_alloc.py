"""The allocation-free sparse-attention entry point, through the C-ABI.

Some users of this library cannot allocate device memory when they call it (a server that gave all
memory to its own pool, a latency-critical loop that cannot afford cudaMalloc's synchronisation).
For them tidal_sparse_attn_noalloc keeps its scratch in a fixed static device array. This file
checks that it returns what tidal_sparse_attn returns, twice in a row (the array keeps the previous
call's contents), that it refuses problems larger than its scratch, and that it works in a fresh
process as well as after every other test (pytest collects this file last)."""
import ctypes as C

import numpy as np
import pytest
import torch

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


@pytest.mark.parametrize("batch,hq,hkv,ctx,k,layout", [
    (1, 8, 2, 3000, 200, "hnd_interleaved"),
    (2, 8, 2, 1500, 96, "paged"),
    (1, 32, 8, 20000, 2048, "hnd_interleaved"),
])
def test_noalloc_matches_the_context_entry_point_twice(batch, hq, hkv, ctx, k, layout):
    w, q, lay = _case(batch, hq, hkv, ctx, k, layout, seed=ctx % 97)
    td = binding.Tidal(0)
    try:
        _, idx, cnt = td.select_attn(lay, q, k)
        ref = td.sparse_attn(lay, q, idx, cnt)
        torch.cuda.synchronize()
        out = torch.full_like(ref, float("nan"))
        for call in range(2):                       # second call sees the first call's leftovers
            out.fill_(float("nan"))
            binding.sparse_attn_noalloc(lay, q, idx, cnt, out=out)
            torch.cuda.synchronize()
            util.check_out(out.cpu().numpy(), ref.cpu().numpy(), f"noalloc call {call}")
            # the two entry points split the index list differently, so the bf16 rounding of the
            # softmax weights differs term by term; both stay far inside the oracle tolerance
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
