"""Parity at the benchmark's full sizes, in the launch configuration bench.py times (same entry
points, same persistent grids): one selection layer and one sparse layer of every configuration,
every head compared with the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2410_05076_b200 import binding, synth
from tests import util

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def td():
    t = binding.Tidal(0)
    yield t
    assert t.device_status() == binding.OK
    t.close()


def select_then_sparse(td, w, sel_layer, sp_layer, max_band_members_per_head=64):
    qs = {i: synth.make_q(w, i, DEV) for i in (sel_layer, sp_layer)}
    if w.paged:
        pt, total = synth.make_page_table(w)
        mk = lambda i: synth.make_layer(w, i, DEV, layout="paged", q=qs[i], page_table=pt, num_pages=total)
    else:
        mk = lambda i: synth.make_layer(w, i, DEV, q=qs[i])
    lay = mk(sel_layer)
    lens = lay.ctx_lens.cpu().numpy()
    out, idx, cnt = td.select_attn(lay, qs[sel_layer], w.k)
    full = td.full_attn(lay, qs[sel_layer])
    torch.cuda.synchronize()
    okv, qb = util.oracle_kv(lay), synth.bits(qs[sel_layer])
    ref, sc = oracle.full_attn(okv, qb, want_scores=True)
    util.check_out(out.cpu().numpy(), ref, f"{w.name}.select")
    util.check_out(full.cpu().numpy(), ref, f"{w.name}.full")
    idx_h, cnt_h = idx.cpu().numpy(), cnt.cpu().numpy()
    assert cnt_h.tolist() == [min(w.k, int(n)) for n in lens]
    for b in range(w.batch):
        for h in range(w.num_q_heads):
            inside = util.check_idx_row(idx_h[b, h], sc[b, h], w.k, int(lens[b]), f"{w.name}.idx[{b},{h}]")
            assert inside <= max_band_members_per_head
    # Heavy hitters are selected: always when the oracle scores them clear of the k'-th score, and nearly
    # all of them anyway (their logits are about 5.7 +- 1; only at the smallest k / N of the sweep does
    # the k'-th score, about 2.9 there, reach into that distribution's tail).
    planted = synth.planted_positions(w, sel_layer, [int(n) for n in lens])
    found = planted_total = 0
    for b in range(w.batch):
        if w.k >= lens[b]:
            continue
        n = int(lens[b])
        for g in range(w.num_kv_heads):
            for i, pos in enumerate(planted[b, g].tolist()):
                h = g * w.group + i % w.group
                kth = np.partition(sc[b, h, :n], n - w.k)[n - w.k]
                hit = pos in idx_h[b, h]
                assert hit or sc[b, h, pos] <= kth + util.TIE_BAND
                found += hit
                planted_total += 1
    assert found >= 0.97 * planted_total
    del okv, lay
    torch.cuda.empty_cache()
    lay2 = mk(sp_layer)
    sp = td.sparse_attn(lay2, qs[sp_layer], idx, cnt)
    torch.cuda.synchronize()
    ref2 = oracle.sparse_attn(util.oracle_kv(lay2), synth.bits(qs[sp_layer]), idx_h, cnt_h)
    util.check_out(sp.cpu().numpy(), ref2, f"{w.name}.sparse")
    assert td.device_status() == binding.OK


def test_config2_llama2_7b_shapes(td):
    select_then_sparse(td, synth.workload("cfg2"), 2, 3)


def test_config3_llama3_8b_128k(td):
    select_then_sparse(td, synth.workload("cfg3"), 13, 14)


def test_config4_paged_ragged_batch(td):
    w = synth.workload("cfg4")
    lens = w.ctx_lens()
    assert len(lens) == 8 and min(lens) >= 8192 and max(lens) <= 65536 and len(set(lens)) > 1
    select_then_sparse(td, w, 2, 3)


@pytest.mark.parametrize("gran,hi", [(binding.SEL_PER_KVHEAD, 8), (binding.SEL_SHARED, 1)])
def test_config3_with_one_set_per_kv_head_or_one_shared_set(td, gran, hi):
    """128K selection layer ranking by the summed logits of a KV head's group (or of all heads), then a sparse
    layer over those sets, against the oracle."""
    w = synth.workload("cfg3")
    q = synth.make_q(w, 2, DEV)
    lay = synth.make_layer(w, 2, DEV, q=q)
    out, idx, cnt = td.select_attn(lay, q, w.k, granularity=gran)
    sp = td.sparse_attn(lay, q, idx, cnt)
    torch.cuda.synchronize()
    okv, qb = util.oracle_kv(lay), synth.bits(q)
    ref, sc = oracle.full_attn(okv, qb, want_scores=True)
    util.check_out(out.cpu().numpy(), ref, "select")
    idx_h, cnt_h = idx.cpu().numpy(), cnt.cpu().numpy()
    assert idx_h.shape == (1, hi, w.k) and cnt_h.tolist() == [w.k]
    members = w.num_q_heads // hi
    for h in range(hi):
        agg = sc[0, h * members:(h + 1) * members].astype(np.float64).sum(0).astype(np.float32)
        assert util.check_idx_row(idx_h[0, h], agg, w.k, w.ctx, f"idx[{h}]") <= 64
    util.check_out(sp.cpu().numpy(), oracle.sparse_attn(okv, qb, idx_h, cnt_h), "sparse")
    assert td.device_status() == binding.OK


def test_sixty_four_layer_variant_group_of_eight(td):
    """The 64-layer variant of Section 4.3 at Llama-3-70B attention shapes: its re-selection layer and the
    sparse layer after it."""
    w = synth.workload("cfg64")
    assert w.sched.count(0) == 2 and w.sched.count(1) == 2 and w.sched.count(2) == 60 and w.sched[31] == 1
    select_then_sparse(td, w, 31, 32)


@pytest.mark.parametrize("ctx", synth.SWEEP_CTX)
@pytest.mark.parametrize("k", synth.SWEEP_K)
def test_config5_sweep_points(td, ctx, k):
    """All 25 points of the context x budget sweep that bench.py times."""
    w = synth.sweep_point(ctx, min(k, ctx))      # the API takes k <= max_ctx_len; k' = min(k, N)
    select_then_sparse(td, w, 0, 1)


def test_whole_step_of_config3_runs_and_matches_on_sampled_layers(td):
    """All 32 layers at 128K through tidal_decode_step (16 GiB of KV); layers 0, 2, 3, 13 and 31
    are compared with the oracle, the sparse ones on the token sets the GPU selected."""
    w = synth.workload("cfg3")
    qs = [synth.make_q(w, i, DEV) for i in range(w.num_layers)]
    layers = [synth.make_layer(w, i, DEV, q=qs[i]) for i in range(w.num_layers)]
    rho = {}
    for i in (2, 13):
        _, idx, cnt = td.select_attn(layers[i], qs[i], w.k)
        rho[i] = (idx.cpu().numpy().copy(), cnt.cpu().numpy().copy())
    outs, idx, cnt = td.decode_step(w.sched, layers, qs, w.k)
    torch.cuda.synchronize()
    assert np.array_equal(idx.cpu().numpy(), rho[13][0])
    for i in (0, 2, 3, 13, 31):
        okv, qb = util.oracle_kv(layers[i]), synth.bits(qs[i])
        if w.sched[i] == synth.LAYER_SPARSE:
            r = rho[2] if i < 13 else rho[13]
            ref = oracle.sparse_attn(okv, qb, r[0], r[1])
        else:
            ref = oracle.full_attn(okv, qb)
        util.check_out(outs[i].cpu().numpy(), ref, f"cfg3.step.layer{i}")
    assert td.device_status() == binding.OK
