"""The C-ABI library loads without a GPU, exports every symbol the header
declares, validates arguments on the host, and refuses to run without a GPU."""
import ctypes as C
import os
import re

import pytest
import torch

from paper_2410_05076_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "tidal.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tidal_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = binding.load()
    names = declared_functions()
    assert len(names) >= 11
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == [n for n in names if n in binding.EXPORTS]
    assert set(names) == set(binding.EXPORTS)


def test_strerror_covers_all_codes():
    for code in range(0, -7, -1):
        assert binding.strerror(code) != "unknown status"
    assert binding.strerror(-99) == "unknown status"


def _kv(**over):
    s = binding.tidal_kv_t()
    s.batch, s.num_q_heads, s.num_kv_heads, s.head_dim = 1, 32, 8, 128
    s.kv_layout = binding.KV_CONTIG
    s.k, s.v = 4096, 8192                 # never dereferenced by the size query
    s.stride_b, s.stride_pos, s.stride_head = 8 * 1024 * 256, 256, 1024 * 256
    s.ctx_lens = 4096
    s.max_ctx_len = 1024
    for k, v in over.items():
        setattr(s, k, v)
    return s


def test_host_validation_through_workspace_query():
    lib = binding.load()
    ok = _kv()
    assert lib.tidal_workspace_bytes(C.byref(ok), 64) > 0
    assert lib.tidal_workspace_bytes(C.byref(ok), 0) == 0
    for bad in (dict(head_dim=64), dict(num_kv_heads=5), dict(num_kv_heads=2), dict(k=4097),
                dict(stride_pos=100), dict(max_ctx_len=0), dict(max_ctx_len=262145),
                dict(kv_layout=7), dict(kv_layout=binding.KV_PAGED), dict(ctx_lens=None),
                dict(sm_scale=-1.0)):
        assert lib.tidal_workspace_bytes(C.byref(_kv(**bad)), 64) == 0, bad
    paged = _kv(kv_layout=binding.KV_PAGED, page_table=4096, page_size=16, max_pages_per_seq=64,
                num_pages=64, stride_page=8 * 16 * 256)
    assert lib.tidal_workspace_bytes(C.byref(paged), 64) > 0
    paged.max_pages_per_seq = 63          # 63 * 16 < max_ctx_len
    assert lib.tidal_workspace_bytes(C.byref(paged), 64) == 0


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU failure mode")
def test_no_gpu_means_no_context():
    with pytest.raises(binding.TidalError) as e:
        binding.Tidal(0)
    assert e.value.status == binding.ERR_CUDA
