"""CUDA path vs CPU oracle, element by element, through the C-ABI (GPU only)."""
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


def wl(batch, hq, hkv, ctx, k, planted=8, seed=1, ragged=False, ctx_min=0, layers=2):
    return synth.Workload(f"t{batch}_{hq}_{hkv}_{ctx}_{k}", batch, hq, hkv, layers, ctx, k, planted,
                          [synth.LAYER_SELECT, synth.LAYER_SPARSE], synth.BASE_SEED + 100 + seed,
                          ragged=ragged, ctx_min=ctx_min)


def paged_layer(w, layer, q):
    pt, total = synth.make_page_table(w, extra_pages=3)
    return synth.make_layer(w, layer, DEV, layout="paged", q=q, page_table=pt, num_pages=total)


def build(w, layout, layer=0):
    q = synth.make_q(w, layer, DEV)
    if layout == "paged":
        lay = paged_layer(w, layer, q)
    else:
        lay = synth.make_layer(w, layer, DEV, layout=layout, q=q)
    return q, lay


CASES = [
    # batch, Hq, Hkv, ctx, k, ragged
    (1, 8, 2, 300, 40, False),
    (2, 8, 2, 1000, 64, True),
    (1, 4, 4, 4097, 256, False),       # MHA, ragged tail of one position
    (3, 16, 2, 777, 100, True),        # group 8
    (1, 2, 1, 2500, 17, False),        # group 2
    (1, 8, 2, 16, 5, False),           # exactly one tile
    (1, 8, 2, 17, 17, False),          # one tile + 1, k = N
    (1, 8, 2, 15, 3, False),
    (1, 4, 2, 1, 1, False),            # single cached token
]


@pytest.mark.parametrize("layout", ["hnd_interleaved", "nhd_separate", "paged"])
@pytest.mark.parametrize("B,Hq,Hkv,N,k,ragged", CASES)
def test_layers_match_oracle(td, layout, B, Hq, Hkv, N, k, ragged):
    w = wl(B, Hq, Hkv, N, k, planted=min(8, N), ragged=ragged, ctx_min=max(1, N // 3))
    q, lay = build(w, layout)
    okv = util.oracle_kv(lay)
    qb = synth.bits(q)
    lens = lay.ctx_lens.cpu().numpy()

    # full attention layer
    out = td.full_attn(lay, q)
    ref_out, ref_sc = oracle.full_attn(okv, qb, want_scores=True)
    util.check_out(out.cpu().numpy(), ref_out, "full")

    # token selection layer: output, emitted scores, index sets
    scores = torch.full((B, Hq, N), float("nan"), dtype=torch.float32, device=DEV)
    out2, idx, cnt = td.select_attn(lay, q, k, scores=scores)
    util.check_out(out2.cpu().numpy(), ref_out, "select.out")
    sc = scores.cpu().numpy()
    idx_h = idx.cpu().numpy()
    assert cnt.cpu().numpy().tolist() == [min(k, int(n)) for n in lens]
    for b in range(B):
        n = int(lens[b])
        assert np.abs(sc[b, :, :n] - ref_sc[b, :, :n]).max() <= 1e-4
        for h in range(Hq):
            util.check_idx_row(idx_h[b, h], ref_sc[b, h], k, n, f"idx[{b},{h}]")

    # same call with the scores kept in the workspace
    _, idx_ws, _ = td.select_attn(lay, q, k)
    assert torch.equal(idx_ws, idx)

    # sparse layer on the oracle's own index sets
    _, ref_idx, ref_cnt = oracle.select_attn(okv, qb, k)
    sp = td.sparse_attn(lay, q, torch.from_numpy(ref_idx).to(DEV), torch.from_numpy(ref_cnt).to(DEV))
    util.check_out(sp.cpu().numpy(), oracle.sparse_attn(okv, qb, ref_idx, ref_cnt), "sparse")
    # and without idx_count: the -1 padding alone delimits the list
    sp2 = td.sparse_attn(lay, q, torch.from_numpy(ref_idx).to(DEV))
    util.check_out(sp2.cpu().numpy(), oracle.sparse_attn(okv, qb, ref_idx), "sparse.nocount")
    assert td.device_status() == binding.OK


def test_config1_select_then_sparse(td):
    """Configuration 1 at full size: 8q/2kv, context 4096, k 256, 32 planted per KV head."""
    w = synth.workload("cfg1")
    q0 = synth.make_q(w, 0, DEV)
    q1 = synth.make_q(w, 1, DEV)
    l0 = synth.make_layer(w, 0, DEV, q=q0)
    l1 = synth.make_layer(w, 1, DEV, q=q1)
    outs, idx, cnt = td.decode_step(w.sched, [l0, l1], [q0, q1], w.k)
    o0, s0 = oracle.full_attn(util.oracle_kv(l0), synth.bits(q0), want_scores=True)
    util.check_out(outs[0].cpu().numpy(), o0, "cfg1.select")
    idx_h = idx.cpu().numpy()
    inside = 0
    for h in range(w.num_q_heads):
        inside += util.check_idx_row(idx_h[0, h], s0[0, h], w.k, w.ctx, f"cfg1.idx[{h}]")
    # planted heavy hitters of a head's own group are selected by that head
    planted = synth.planted_positions(w, 0, [w.ctx])
    for g in range(w.num_kv_heads):
        for i, pos in enumerate(planted[0, g].tolist()):
            h = g * w.group + i % w.group
            assert pos in idx_h[0, h]
    # sparse layer: oracle evaluated on the GPU's (validated) token sets
    ref1 = oracle.sparse_attn(util.oracle_kv(l1), synth.bits(q1), idx_h, cnt.cpu().numpy())
    util.check_out(outs[1].cpu().numpy(), ref1, "cfg1.sparse")
    assert inside <= 8


@pytest.mark.parametrize("gran,hi_of", [(binding.SEL_PER_KVHEAD, lambda w: w.num_kv_heads),
                                        (binding.SEL_SHARED, lambda w: 1)])
def test_aggregated_granularities(td, gran, hi_of):
    w = wl(2, 8, 2, 900, 50, ragged=True, ctx_min=300, seed=7)
    q, lay = build(w, "hnd_interleaved")
    okv, qb = util.oracle_kv(lay), synth.bits(q)
    Hi = hi_of(w)
    ref_out, ref_idx, ref_cnt, ref_sc = oracle.select_attn(okv, qb, w.k, Hi, want_scores=True)
    lens = lay.ctx_lens.cpu().numpy()
    members = w.num_q_heads // Hi
    # without a score buffer the attention kernel stores the group sums itself; with one it stores the
    # per-head scores and the top-k sums them: both must give the oracle's sets
    for scores in (None, torch.full((w.batch, w.num_q_heads, w.ctx), float("nan"), dtype=torch.float32, device=DEV)):
        out, idx, cnt = td.select_attn(lay, q, w.k, granularity=gran, scores=scores)
        util.check_out(out.cpu().numpy(), ref_out, "agg.out")
        idx_h = idx.cpu().numpy()
        assert cnt.cpu().numpy().tolist() == ref_cnt.tolist()
        for b in range(w.batch):
            n = int(lens[b])
            for hi in range(Hi):
                agg = ref_sc[b, hi * members:(hi + 1) * members, :n].astype(np.float64).sum(0).astype(np.float32)
                util.check_idx_row(idx_h[b, hi], agg, w.k, n, f"agg.idx[{b},{hi}]")
        if scores is not None:
            for b in range(w.batch):
                n = int(lens[b])
                assert np.abs(scores[b, :, :n].cpu().numpy() - ref_sc[b, :, :n]).max() <= 1e-4
    sp = td.sparse_attn(lay, q, torch.from_numpy(ref_idx).to(DEV), torch.from_numpy(ref_cnt).to(DEV))
    util.check_out(sp.cpu().numpy(), oracle.sparse_attn(okv, qb, ref_idx, ref_cnt), "agg.sparse")


def test_decode_step_schedule_and_rho_persistence(td):
    """Seven layers F,F,S,sp,S,sp,sp on a paged ragged batch; sparse layers are
    checked against the oracle run on the token sets the GPU selected."""
    sched = [0, 0, 1, 2, 1, 2, 2]
    w = wl(2, 8, 2, 1200, 96, ragged=True, ctx_min=500, seed=9, layers=len(sched))
    pt, total = synth.make_page_table(w, extra_pages=5)
    qs = [synth.make_q(w, i, DEV) for i in range(len(sched))]
    layers = [synth.make_layer(w, i, DEV, layout="paged", q=qs[i], page_table=pt, num_pages=total)
              for i in range(len(sched))]
    lens = layers[0].ctx_lens.cpu().numpy()

    # run layer by layer to capture rho after each selection layer
    rho = {}
    for i, t in enumerate(sched):
        if t == 1:
            _, idx, cnt = td.select_attn(layers[i], qs[i], w.k)
            rho[i] = (idx.cpu().numpy().copy(), cnt.cpu().numpy().copy())
    outs, idx, cnt = td.decode_step(sched, layers, qs, w.k)
    assert np.array_equal(idx.cpu().numpy(), rho[4][0])          # rho was replaced wholesale at layer 4
    cur = None
    for i, t in enumerate(sched):
        okv, qb = util.oracle_kv(layers[i]), synth.bits(qs[i])
        got = outs[i].cpu().numpy()
        if t in (0, 1):
            ref, sc = oracle.full_attn(okv, qb, want_scores=True)
            util.check_out(got, ref, f"step.layer{i}")
            if t == 1:
                cur = rho[i]
                for b in range(w.batch):
                    for h in range(w.num_q_heads):
                        util.check_idx_row(cur[0][b, h], sc[b, h], w.k, int(lens[b]), f"step.idx{i}")
        else:
            util.check_out(got, oracle.sparse_attn(okv, qb, cur[0], cur[1]), f"step.layer{i}")
    assert td.device_status() == binding.OK


def test_decode_step_host_buffers(td):
    sched = [0, 1, 2, 2]
    w = wl(1, 8, 2, 640, 48, seed=11, layers=len(sched))
    qs = [synth.make_q(w, i, DEV) for i in range(len(sched))]
    layers = [synth.make_layer(w, i, DEV, q=qs[i]) for i in range(len(sched))]
    q_host = torch.stack([q.cpu() for q in qs]).contiguous().pin_memory()
    out_host = torch.zeros(len(sched), 1, 8, 128, dtype=torch.float32).pin_memory()
    td.make_step_host(sched, layers, q_host, out_host, w.k)()
    outs, _, _ = td.decode_step(sched, layers, qs, w.k)
    # tiles are handed to warps dynamically, so the fp32 summation order (not the result
    # beyond rounding) may differ between two runs
    for i in range(len(sched)):
        assert torch.allclose(out_host[i], outs[i].cpu(), rtol=0, atol=5e-4)
    # pageable host buffers take the staging path (copies) instead of being accessed by the kernels
    q_page = torch.stack([q.cpu() for q in qs]).contiguous()
    out_page = torch.zeros(len(sched), 1, 8, 128, dtype=torch.float32)
    assert not q_page.is_pinned() and not out_page.is_pinned()
    td.make_step_host(sched, layers, q_page, out_page, w.k)()
    for i in range(len(sched)):
        assert torch.allclose(out_page[i], outs[i].cpu(), rtol=0, atol=5e-4)
    # and every layer against the oracle, through the pinned path
    cur = None
    for i, t in enumerate(sched):
        okv, qb = util.oracle_kv(layers[i]), synth.bits(qs[i])
        if t != 2:
            util.check_out(out_host[i].numpy(), oracle.full_attn(okv, qb), f"host.layer{i}")
            if t == 1:
                _, gi, gc = td.select_attn(layers[i], qs[i], w.k)
                cur = (gi.cpu().numpy(), gc.cpu().numpy())
        else:
            util.check_out(out_host[i].numpy(), oracle.sparse_attn(okv, qb, cur[0], cur[1]), f"host.layer{i}")


@pytest.mark.parametrize("N,k", [(333, 20), (9000, 700), (40000, 5000)])
def test_ties_and_constant_scores(td, N, k):
    """q = 0: every score is equal, so the lowest positions win and the output is the mean of V. The sizes
    cover a threshold bin that fits shared memory, one that overflows it in a single CTA, and one that
    overflows it across several CTAs."""
    w = wl(1, 4, 2, N, k, seed=13)
    q, lay = build(w, "hnd_interleaved")
    q.zero_()
    out, idx, _ = td.select_attn(lay, q, w.k)
    assert idx.cpu().numpy()[0].tolist() == [list(range(k))] * 4
    ref = oracle.full_attn(util.oracle_kv(lay), synth.bits(q))
    util.check_out(out.cpu().numpy(), ref, "ties.out")


def test_sparse_skips_padding_duplicates_and_flags_bad_indices(td):
    w = wl(1, 4, 2, 200, 12, seed=15)
    q, lay = build(w, "nhd_separate")
    okv, qb = util.oracle_kv(lay), synth.bits(q)
    idx = np.full((1, 4, 12), -1, np.int32)
    idx[0, 0, :5] = [199, 3, 3, 50, 0]           # unsorted with a duplicate
    idx[0, 1, :1] = [7]
    idx[0, 3, :12] = np.arange(100, 112)         # head 2 has no entries at all
    sp = td.sparse_attn(lay, q, torch.from_numpy(idx).to(DEV))
    ref = oracle.sparse_attn(okv, qb, idx)
    util.check_out(sp.cpu().numpy(), ref, "sparse.dups")
    assert (sp.cpu().numpy()[0, 2] == 0).all()
    assert td.device_status() == binding.OK
    idx[0, 1, 1] = 200                            # one past the end of the cache
    sp = td.sparse_attn(lay, q, torch.from_numpy(idx).to(DEV))
    assert td.device_status() == binding.ERR_INDEX
    assert td.device_status() == binding.OK       # sticky word was cleared
    util.check_out(sp.cpu().numpy(), ref, "sparse.badidx")   # the bad entry was skipped
    idx[0, 1, 1] = -5                             # negative but not the padding value
    sp = td.sparse_attn(lay, q, torch.from_numpy(idx).to(DEV))
    assert td.device_status() == binding.ERR_INDEX
    util.check_out(sp.cpu().numpy(), ref, "sparse.negidx")   # skipped as well


def test_host_side_argument_errors(td):
    w = wl(1, 8, 2, 64, 8, seed=17)
    q, lay = build(w, "hnd_interleaved")
    lib, ctx = td.lib, td.ctx
    import ctypes as C
    out = torch.empty(1, 8, 128, dtype=torch.float32, device=DEV)
    idx = torch.empty(1, 8, 8, dtype=torch.int32, device=DEV)

    def sel(s, k=8, gran=0, q_=q, idx_=idx):
        return lib.tidal_select_attn(ctx, C.byref(s), q_.data_ptr(), k, gran, out.data_ptr(),
                                     idx_.data_ptr(), None, None, None)

    s = binding.kv_struct(lay)
    assert sel(s) == binding.OK
    assert sel(s, k=0) == binding.ERR_INVALID
    assert sel(s, k=65) == binding.ERR_INVALID
    assert sel(s, gran=9) == binding.ERR_INVALID
    s = binding.kv_struct(lay); s.head_dim = 64
    assert sel(s) == binding.ERR_UNSUPPORTED
    s = binding.kv_struct(lay); s.num_kv_heads = 3
    assert sel(s) == binding.ERR_INVALID
    s = binding.kv_struct(lay); s.k = None
    assert sel(s) == binding.ERR_INVALID
    s = binding.kv_struct(lay); s.stride_pos = 260
    assert sel(s) == binding.ERR_INVALID
    s = binding.kv_struct(lay); s.kv_layout = binding.KV_PAGED
    assert sel(s) == binding.ERR_INVALID          # paged without a page table
    s = binding.kv_struct(lay)
    assert lib.tidal_sparse_attn(ctx, C.byref(s), q.data_ptr(), idx.data_ptr(), None, 8, 3,
                                 out.data_ptr(), None) == binding.ERR_INVALID
    # a sparse layer before any selection layer
    with pytest.raises(binding.TidalError) as e:
        td.decode_step([0, 2], [lay, lay], [q, q], 8)
    assert e.value.status == binding.ERR_INVALID
    assert binding.Tidal.workspace_bytes(lay, 8) > 0
    torch.cuda.synchronize()


def test_results_are_reproducible(td):
    w = wl(1, 8, 2, 5000, 300, seed=19)
    q, lay = build(w, "hnd_interleaved")
    a = td.select_attn(lay, q, w.k)
    b = td.select_attn(lay, q, w.k)
    assert torch.equal(a[1], b[1])                       # the selected sets are reproducible bit for bit
    assert torch.allclose(a[0], b[0], rtol=0, atol=5e-4)  # outputs up to fp32 summation order


def test_many_short_sequences_use_the_flat_split(td):
    """A batch of 37 ragged short sequences: every CTA walks several (sequence, head) segments."""
    w = wl(37, 4, 2, 700, 33, ragged=True, ctx_min=20, seed=21)
    q, lay = build(w, "paged")
    okv, qb = util.oracle_kv(lay), synth.bits(q)
    lens = lay.ctx_lens.cpu().numpy()
    out, idx, cnt = td.select_attn(lay, q, w.k)
    ref, sc = oracle.full_attn(okv, qb, want_scores=True)
    util.check_out(out.cpu().numpy(), ref, "batch.select")
    idx_h = idx.cpu().numpy()
    for b in range(w.batch):
        for h in range(w.num_q_heads):
            util.check_idx_row(idx_h[b, h], sc[b, h], w.k, int(lens[b]), f"batch.idx[{b},{h}]")
    sp = td.sparse_attn(lay, q, idx, cnt)
    util.check_out(sp.cpu().numpy(), oracle.sparse_attn(okv, qb, idx_h, cnt.cpu().numpy()), "batch.sparse")
    assert td.device_status() == binding.OK


def test_explicit_softmax_scale(td):
    w = wl(1, 8, 2, 600, 30, seed=23)
    q, lay = build(w, "hnd_interleaved")
    lay.sm_scale = 0.05
    okv, qb = util.oracle_kv(lay), synth.bits(q)
    scores = torch.empty(1, 8, 600, dtype=torch.float32, device=DEV)
    out, idx, cnt = td.select_attn(lay, q, w.k, scores=scores)
    ref, sc = oracle.full_attn(okv, qb, want_scores=True)
    util.check_out(out.cpu().numpy(), ref, "scale.out")
    assert np.abs(scores.cpu().numpy() - sc).max() <= 1e-4
    # the stored logits scale with sm_scale: compare with the default scale 1/sqrt(128)
    lay.sm_scale = 0.0
    _, sc_default = oracle.full_attn(util.oracle_kv(lay), qb, want_scores=True)
    assert np.allclose(sc, sc_default * (0.05 * np.sqrt(128.0)), atol=1e-5)


def test_group_of_eight_with_shared_sets_at_32k(td):
    """64 query heads over 8 KV heads (Llama-3-70B-like), context 32768, one token set per KV head:
    the sparse layer then runs all eight heads of a group as MMA columns over the same gathered rows."""
    w = synth.Workload("g8", 1, 64, 8, 2, 32768, 1024, 64, [1, 2], synth.BASE_SEED + 777)
    q, lay = build(w, "hnd_interleaved")
    okv, qb = util.oracle_kv(lay), synth.bits(q)
    out, idx, cnt = td.select_attn(lay, q, w.k, granularity=binding.SEL_PER_KVHEAD)
    ref, ref_idx, ref_cnt, sc = oracle.select_attn(okv, qb, w.k, 8, want_scores=True)
    util.check_out(out.cpu().numpy(), ref, "g8.select")
    idx_h = idx.cpu().numpy()
    for g in range(8):
        agg = sc[0, 8 * g: 8 * g + 8].astype(np.float64).sum(0).astype(np.float32)
        util.check_idx_row(idx_h[0, g], agg, w.k, w.ctx, f"g8.idx[{g}]")
    sp = td.sparse_attn(lay, q, idx, cnt)
    util.check_out(sp.cpu().numpy(), oracle.sparse_attn(okv, qb, idx_h, cnt.cpu().numpy()), "g8.sparse")
    # the paper's per-head sets on the same cache (histogram with 1024 bins for a group of 8)
    out2, idx2, cnt2 = td.select_attn(lay, q, w.k)
    idx2_h = idx2.cpu().numpy()
    for h in range(0, 64, 7):
        util.check_idx_row(idx2_h[0, h], sc[0, h], w.k, w.ctx, f"g8.idx_q[{h}]")
    sp2 = td.sparse_attn(lay, q, idx2, cnt2)
    util.check_out(sp2.cpu().numpy(), oracle.sparse_attn(okv, qb, idx2_h, cnt2.cpu().numpy()), "g8.sparse_q")


def test_budget_equal_to_a_long_context_keeps_everything(td):
    w = synth.sweep_point(65536, 65536)
    q, lay = build(w, "hnd_interleaved")
    out, idx, cnt = td.select_attn(lay, q, w.k)
    assert cnt.item() == 65536
    assert torch.equal(idx[0, 5], torch.arange(65536, dtype=torch.int32, device=DEV))
    sp = td.sparse_attn(lay, q, idx, cnt)
    torch.cuda.synchronize()
    # sparse over everything is full attention; the two kernels round the softmax weights to bf16 at
    # different running maxima and sum in different orders (each is within about 1.5e-4 of the exact
    # result at this size), so they agree to a few 1e-4, not bit for bit
    assert torch.allclose(sp, out, rtol=0, atol=1e-3)


def test_sixty_four_layer_schedule_matches_the_oracle_step(td):
    """The 64-layer composition of Section 4.3 (2 full + 2 selection + 60 sparse layers, selection at
    layers 2 and 13) as one tidal_decode_step call against the oracle's own step driver."""
    L = 64
    sched = synth.schedule(L, 13)
    assert (sched.count(0), sched.count(1), sched.count(2)) == (2, 2, 60)
    w = synth.Workload("l64", 1, 8, 2, L, 320, 40, 8, sched, synth.BASE_SEED + 64)
    qs = [synth.make_q(w, i, DEV) for i in range(L)]
    layers = [synth.make_layer(w, i, DEV, q=qs[i]) for i in range(L)]
    outs, idx, cnt = td.decode_step(sched, layers, qs, w.k)
    ref_outs, ref_idx, ref_cnt = oracle.decode_step(sched, [util.oracle_kv(l) for l in layers],
                                                    [synth.bits(q) for q in qs], w.k)
    # with well separated scores the selected sets agree exactly and every layer can be compared directly
    assert np.array_equal(cnt.cpu().numpy(), ref_cnt)
    if np.array_equal(idx.cpu().numpy(), ref_idx):
        for i in range(L):
            util.check_out(outs[i].cpu().numpy(), ref_outs[i], f"l64.layer{i}")
    else:       # a legal swap inside the tie band at the last selection layer: compare on the GPU's sets
        for i in (0, 1, 2, 13):
            util.check_out(outs[i].cpu().numpy(), ref_outs[i], f"l64.layer{i}")
        for i in range(14, L):
            ref = oracle.sparse_attn(util.oracle_kv(layers[i]), synth.bits(qs[i]), idx.cpu().numpy(), cnt.cpu().numpy())
            util.check_out(outs[i].cpu().numpy(), ref, f"l64.layer{i}")
    assert td.launch_count() > 0 and td.device_status() == binding.OK


@pytest.mark.parametrize("layout", ["hnd_interleaved", "nhd_separate", "paged"])
def test_kv_append_writes_the_same_rows_as_the_oracle(td, layout):
    """C.append of Algorithm 1: the whole cache is bit-identical to the oracle's after the append, and
    full attention over it matches."""
    w = wl(3, 8, 2, 333, 32, ragged=True, ctx_min=1)
    q, lay = build(w, layout)
    okv = util.oracle_kv(lay)                     # host copy taken BEFORE the append
    g = torch.Generator(device="cpu").manual_seed(99)
    kn = torch.randn(w.batch, w.num_kv_heads, w.head_dim, generator=g).to(torch.bfloat16)
    vn = torch.randn(w.batch, w.num_kv_heads, w.head_dim, generator=g).to(torch.bfloat16)
    oracle.kv_append(okv, synth.bits(kn), synth.bits(vn))
    td.kv_append(lay, kn.to(DEV), vn.to(DEV))
    torch.cuda.synchronize()
    after = util.oracle_kv(lay)                   # host copy of what the kernel wrote
    assert np.array_equal(after.k, okv.k) and np.array_equal(after.v, okv.v)
    util.check_out(td.full_attn(lay, q).cpu().numpy(), oracle.full_attn(okv, synth.bits(q)), "full after append")
    assert td.device_status() == binding.OK


@pytest.mark.parametrize("layout", ["hnd_interleaved", "paged"])
def test_batch_with_an_empty_and_a_one_token_sequence(td, layout):
    """Degenerate lengths inside a batch: an empty cache gives a zero output row, no indices and a count
    of 0; a one-token cache returns v_0; the other sequences are unaffected."""
    w = wl(4, 8, 2, 200, 24, ragged=False, seed=11)
    q, lay = build(w, layout)
    lay.ctx_lens = torch.tensor([200, 0, 1, 77], dtype=torch.int32, device=DEV)
    okv, qb = util.oracle_kv(lay), synth.bits(q)
    ref_out, ref_idx, ref_cnt, ref_sc = oracle.select_attn(okv, qb, w.k, want_scores=True)
    assert ref_cnt.tolist() == [24, 0, 1, 24] and (ref_out[1] == 0).all()
    util.check_out(td.full_attn(lay, q).cpu().numpy(), ref_out, "full")
    out, idx, cnt = td.select_attn(lay, q, w.k)
    util.check_out(out.cpu().numpy(), ref_out, "select")
    assert (out.cpu().numpy()[1] == 0).all()
    assert cnt.cpu().numpy().tolist() == ref_cnt.tolist()
    idx_h = idx.cpu().numpy()
    assert (idx_h[1] == -1).all() and (idx_h[2, :, 0] == 0).all() and (idx_h[2, :, 1:] == -1).all()
    for b in (0, 3):
        for h in range(w.num_q_heads):
            util.check_idx_row(idx_h[b, h], ref_sc[b, h], w.k, int(lay.ctx_lens[b]), f"idx[{b},{h}]")
    sp = td.sparse_attn(lay, q, idx, cnt)
    util.check_out(sp.cpu().numpy(), oracle.sparse_attn(okv, qb, idx_h, cnt.cpu().numpy()), "sparse")
    assert (sp.cpu().numpy()[1] == 0).all()
    assert td.device_status() == binding.OK


def test_decode_step_with_the_cache_update(td):
    """Algorithm 1's loop with C.append: every layer's new rows are written, then F,S,sp,S,sp run; compared
    with the oracle appending to host copies of the caches and stepping over them."""
    sched = [0, 1, 2, 1, 2]
    w = wl(2, 8, 2, 500, 48, ragged=True, ctx_min=100, seed=21, layers=len(sched))
    qs = [synth.make_q(w, i, DEV) for i in range(len(sched))]
    layers = [synth.make_layer(w, i, DEV, layout="nhd_separate" if i % 2 else "hnd_interleaved", q=qs[i])
              for i in range(len(sched))]
    g = torch.Generator(device="cpu").manual_seed(5)
    k_new = [(3.0 * torch.randn(w.batch, w.num_kv_heads, w.head_dim, generator=g)).to(torch.bfloat16) for _ in sched]
    v_new = [torch.randn(w.batch, w.num_kv_heads, w.head_dim, generator=g).to(torch.bfloat16) for _ in sched]
    okvs = [util.oracle_kv(l) for l in layers]                     # host copies taken before the update
    for okv, kn, vn in zip(okvs, k_new, v_new):
        oracle.kv_append(okv, synth.bits(kn), synth.bits(vn))
    outs, idx, cnt = td.decode_step_append(sched, layers, qs, [t.to(DEV) for t in k_new], [t.to(DEV) for t in v_new], w.k)
    torch.cuda.synchronize()
    for l, okv in zip(layers, okvs):                               # the caches themselves
        after = util.oracle_kv(l)
        assert np.array_equal(after.k, okv.k) and np.array_equal(after.v, okv.v)
    lens = layers[0].ctx_lens.cpu().numpy()
    cur = None
    for i, t in enumerate(sched):
        qb = synth.bits(qs[i])
        got = outs[i].cpu().numpy()
        if t in (0, 1):
            ref, sc = oracle.full_attn(okvs[i], qb, want_scores=True)
            util.check_out(got, ref, f"layer{i}")
            if t == 1:
                _, gi, gc = td.select_attn(layers[i], qs[i], w.k)      # the cache now holds the new rows
                cur = (gi.cpu().numpy(), gc.cpu().numpy())
                for b in range(w.batch):
                    for h in range(w.num_q_heads):
                        util.check_idx_row(cur[0][b, h], sc[b, h], w.k, int(lens[b]), f"idx{i}")
        else:
            util.check_out(got, oracle.sparse_attn(okvs[i], qb, cur[0], cur[1]), f"layer{i}")
    assert np.array_equal(idx.cpu().numpy(), cur[0])
    assert td.device_status() == binding.OK


def _fuzz_cases(n, seed):
    r = np.random.default_rng(seed)
    out = []
    for _ in range(n):
        hkv = int(r.choice([1, 2, 3, 4, 8]))
        g = int(r.choice([1, 2, 4, 8]))
        batch = int(r.integers(1, 5))
        ctx = int(r.choice([int(r.integers(1, 40)), int(r.integers(40, 700)), int(r.integers(700, 5000))]))
        k = int(r.integers(1, ctx + 1)) if r.random() < 0.7 else ctx
        out.append((batch, hkv * g, hkv, ctx, k, bool(r.random() < 0.6), str(r.choice(["hnd_interleaved", "nhd_separate", "paged"])),
                    int(r.choice([binding.SEL_PER_QHEAD, binding.SEL_PER_KVHEAD, binding.SEL_SHARED]))))
    return out


@pytest.mark.parametrize("B,Hq,Hkv,N,k,ragged,layout,gran", _fuzz_cases(36, 20241005))
def test_random_shapes_match_the_oracle(td, B, Hq, Hkv, N, k, ragged, layout, gran):
    """Seeded random shapes: head counts, groups 1-8, batch, context from one token to a few thousand, budget,
    layout and index granularity all vary; selection and sparse layers against the oracle."""
    w = wl(B, Hq, Hkv, N, k, planted=min(8, N), ragged=ragged, ctx_min=max(1, N // 4), seed=N + k)
    q, lay = build(w, layout)
    okv, qb = util.oracle_kv(lay), synth.bits(q)
    Hi = {binding.SEL_PER_QHEAD: Hq, binding.SEL_PER_KVHEAD: Hkv, binding.SEL_SHARED: 1}[gran]
    ref_out, ref_idx, ref_cnt, ref_sc = oracle.select_attn(okv, qb, k, Hi, want_scores=True)
    out, idx, cnt = td.select_attn(lay, q, k, granularity=gran)
    util.check_out(out.cpu().numpy(), ref_out, "select")
    assert cnt.cpu().numpy().tolist() == ref_cnt.tolist()
    lens = lay.ctx_lens.cpu().numpy()
    idx_h = idx.cpu().numpy()
    members = Hq // Hi
    for b in range(B):
        n = int(lens[b])
        for hi in range(Hi):
            agg = ref_sc[b, hi * members:(hi + 1) * members, :n].astype(np.float64).sum(0).astype(np.float32)
            util.check_idx_row(idx_h[b, hi], agg, k, n, f"idx[{b},{hi}]")
    sp = td.sparse_attn(lay, q, idx, cnt)
    util.check_out(sp.cpu().numpy(), oracle.sparse_attn(okv, qb, idx_h, cnt.cpu().numpy()), "sparse")
    assert td.device_status() == binding.OK


def test_decode_step_replays_from_a_cuda_graph(td):
    """The step allocates nothing once its workspace exists, so it can be captured into a CUDA graph
    (programmatic dependent launches included) and replayed: same token sets, same outputs."""
    sched = [0, 1, 2, 2, 1, 2]
    w = wl(1, 8, 2, 3000, 128, seed=23, layers=len(sched))
    qs = [synth.make_q(w, i, DEV) for i in range(len(sched))]
    layers = [synth.make_layer(w, i, DEV, q=qs[i]) for i in range(len(sched))]
    outs = [torch.zeros(1, 8, 128, dtype=torch.float32, device=DEV) for _ in sched]
    step = td.make_step(sched, layers, qs, outs, w.k)
    step()                                                    # sizes the workspace outside the capture
    torch.cuda.synchronize()
    eager = [o.clone() for o in outs]
    eager_idx = step.idx.clone()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())      # the inputs were built on the current stream
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            step()
    for o in outs:
        o.zero_()
    step.idx.fill_(-7)
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(step.idx, eager_idx)
    for o, e in zip(outs, eager):
        assert torch.allclose(o, e, rtol=0, atol=5e-4)
    assert td.device_status() == binding.OK


def test_library_records_and_replays_step_graphs(td):
    """On an ordinary stream the step is recorded once and replayed; lengths live in device memory, so a
    replay follows them when they change. Compared with the same step enqueued kernel by kernel."""
    sched = [0, 1, 2, 2]
    w = wl(2, 8, 2, 2000, 64, ragged=True, ctx_min=500, seed=29, layers=len(sched))
    qs = [synth.make_q(w, i, DEV) for i in range(len(sched))]
    layers = [synth.make_layer(w, i, DEV, q=qs[i]) for i in range(len(sched))]
    lens0 = layers[0].ctx_lens.clone()
    for l in layers:
        l.ctx_lens = layers[0].ctx_lens                   # one length vector for all layers, changed in place below
    outs = [torch.zeros(2, 8, 128, dtype=torch.float32, device=DEV) for _ in sched]
    step = td.make_step(sched, layers, qs, outs, w.k)
    q_host = torch.stack([q.cpu() for q in qs]).contiguous().pin_memory()
    out_host = torch.zeros(len(sched), 2, 8, 128, dtype=torch.float32).pin_memory()
    step_host = td.make_step_host(sched, layers, q_host, out_host, w.k)

    def run_direct():
        step()                                            # default stream: kernel by kernel
        torch.cuda.synchronize()
        return [o.clone() for o in outs], step.idx.clone()

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())      # the inputs were built on the current stream
    for new_lens in (lens0, (lens0 // 2).clamp(min=70), lens0):
        layers[0].ctx_lens.copy_(new_lens)
        ref_outs, ref_idx = run_direct()
        for o in outs:
            o.zero_()
        with torch.cuda.stream(side):
            n0 = td.launch_count()
            step()
            n1 = td.launch_count()
            step()                                        # a replay at the latest
            n2 = td.launch_count()
            side.synchronize()
            assert n1 - n0 == n2 - n1 == 6                # full, key pass, value pass, top-k, two sparse layers
            assert torch.equal(step.idx, ref_idx)
            for o, r in zip(outs, ref_outs):
                assert torch.allclose(o, r, rtol=0, atol=5e-4)
            step_host()
            step_host()
            for i, r in enumerate(ref_outs):
                assert torch.allclose(out_host[i].to(DEV), r, rtol=0, atol=5e-4)
    td.set_graphs(False)
    with torch.cuda.stream(side):
        step()
        side.synchronize()
    td.set_graphs(True)
    for o, r in zip(outs, ref_outs):
        assert torch.allclose(o, r, rtol=0, atol=5e-4)
    assert td.device_status() == binding.OK


def test_a_repeated_call_is_replayed_only_while_nothing_changes(td):
    """A step call that repeats the previous one byte for byte skips validation and launches the same graph
    again; any change (another budget, other output buffers, other queries, a setting) must take the long
    way. Two steps over the same caches are interleaved and every result is compared with the same step
    enqueued kernel by kernel."""
    sched = [0, 1, 2, 2]
    w = wl(1, 8, 2, 3000, 64, seed=37, layers=len(sched))
    qs = [synth.make_q(w, i, DEV) for i in range(len(sched))]
    qs_b = [synth.make_q(w, i + 10, DEV) for i in range(len(sched))]
    layers = [synth.make_layer(w, i, DEV, q=qs[i]) for i in range(len(sched))]
    outs_a = [torch.zeros(1, 8, 128, device=DEV) for _ in sched]
    outs_b = [torch.zeros(1, 8, 128, device=DEV) for _ in sched]
    step_a = td.make_step(sched, layers, qs, outs_a, 64)
    step_b = td.make_step(sched, layers, qs_b, outs_b, 32)

    def reference(step, outs):
        step()                                            # default stream: kernel by kernel
        torch.cuda.synchronize()
        ref = ([o.clone() for o in outs], step.idx.clone())
        for o in outs:
            o.zero_()
        step.idx.fill_(-7)
        torch.cuda.synchronize()
        return ref

    ref_a, ref_b = reference(step_a, outs_a), reference(step_b, outs_b)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())      # the inputs were built on the current stream
    with torch.cuda.stream(side):
        for which in "aabaabbbab":
            step, outs, ref = (step_a, outs_a, ref_a) if which == "a" else (step_b, outs_b, ref_b)
            for o in outs:
                o.zero_()
            step.idx.fill_(-7)
            step()
            side.synchronize()
            assert torch.equal(step.idx, ref[1]), which
            for o, r in zip(outs, ref[0]):
                assert torch.allclose(o, r, rtol=0, atol=5e-4), which
        # a setting changes between two otherwise identical calls
        step_a()
        td.set_layer_overlap(False)
        try:
            for o in outs_a:
                o.zero_()
            step_a()
            side.synchronize()
        finally:
            td.set_layer_overlap(True)
        for o, r in zip(outs_a, ref_a[0]):
            assert torch.allclose(o, r, rtol=0, atol=5e-4)
    assert td.device_status() == binding.OK


def test_bf16_outputs_are_the_fp32_results_rounded(td):
    """With the bf16 output type every call writes the rounded fp32 result; everything else is unchanged."""
    sched = [0, 1, 2]
    w = wl(2, 8, 2, 700, 64, ragged=True, ctx_min=300, seed=31, layers=len(sched))
    qs = [synth.make_q(w, i, DEV) for i in range(len(sched))]
    layers = [synth.make_layer(w, i, DEV, q=qs[i]) for i in range(len(sched))]
    # (bf16 outputs always come from the fused selection kernel; without the overlap so do the fp32 ones)
    td.set_layer_overlap(False)
    try:
        ref_outs, ref_idx, _ = td.decode_step(sched, layers, qs, w.k)
    finally:
        td.set_layer_overlap(True)
    ref_full = td.full_attn(layers[0], qs[0])
    torch.cuda.synchronize()
    td.set_output_bf16(True)
    try:
        outs, idx, cnt = td.decode_step(sched, layers, qs, w.k)
        full = td.full_attn(layers[0], qs[0])
        _, idx2, cnt2 = td.select_attn(layers[1], qs[1], w.k)
        sp = td.sparse_attn(layers[2], qs[2], idx2, cnt2)
        q_host = torch.stack([q.cpu() for q in qs]).contiguous().pin_memory()
        out_host = torch.zeros(len(sched), 2, 8, 128, dtype=torch.bfloat16).pin_memory()
        td.make_step_host(sched, layers, q_host, out_host, w.k)()
        torch.cuda.synchronize()
    finally:
        td.set_output_bf16(False)
    assert torch.equal(idx, ref_idx) and torch.equal(idx2, ref_idx)
    for o, r, h in zip(outs, ref_outs, out_host):
        assert o.dtype == torch.bfloat16
        # equal to the rounded fp32 result up to the run-to-run variation of the fp32 value (one bf16 step)
        assert torch.allclose(o.float(), r.to(torch.bfloat16).float(), rtol=2 ** -7, atol=5e-4)
        assert torch.allclose(h.to(DEV).float(), r, rtol=2 ** -7, atol=5e-4)
    assert torch.allclose(full.float(), ref_full, rtol=2 ** -7, atol=5e-4)
    assert torch.allclose(sp.float(), ref_outs[2], rtol=2 ** -7, atol=5e-4)
    okv, qb = util.oracle_kv(layers[0]), synth.bits(qs[0])
    util.check_out(full.float().cpu().numpy(), oracle.full_attn(okv, qb), "bf16 full vs oracle")
    again = td.full_attn(layers[0], qs[0])
    assert again.dtype == torch.float32
    assert td.device_status() == binding.OK


def test_two_contexts_on_two_streams_do_not_interfere(td):
    """Each context owns its workspace, counters and step graphs: two of them driven alternately on two
    streams give the results of one."""
    sched = [0, 1, 2, 2]
    w = wl(1, 8, 2, 2500, 96, seed=37, layers=len(sched))
    qs = [synth.make_q(w, i, DEV) for i in range(len(sched))]
    layers = [synth.make_layer(w, i, DEV, q=qs[i]) for i in range(len(sched))]
    ref_outs, ref_idx, _ = td.decode_step(sched, layers, qs, w.k)
    torch.cuda.synchronize()
    other = binding.Tidal(0)
    try:
        sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
        sa.wait_stream(torch.cuda.current_stream())        # the inputs were built on the current stream
        sb.wait_stream(torch.cuda.current_stream())
        outs_a = [torch.zeros_like(o) for o in ref_outs]
        outs_b = [torch.zeros_like(o) for o in ref_outs]
        step_a = td.make_step(sched, layers, qs, outs_a, w.k)
        step_b = other.make_step(sched, layers, qs, outs_b, w.k)
        for _ in range(4):
            with torch.cuda.stream(sa):
                step_a()
            with torch.cuda.stream(sb):
                step_b()
        torch.cuda.synchronize()
        for oa, ob, r in zip(outs_a, outs_b, ref_outs):
            assert torch.allclose(oa, r, rtol=0, atol=5e-4) and torch.allclose(ob, r, rtol=0, atol=5e-4)
        assert torch.equal(step_a.idx, ref_idx) and torch.equal(step_b.idx, ref_idx)
        assert other.device_status() == binding.OK
    finally:
        other.close()


@pytest.mark.parametrize("layout", ["hnd_interleaved", "paged"])
def test_sparse_layers_can_always_attend_the_newest_token(td, layout):
    """The optional variant (not in the paper): every list is extended by the newest position unless it
    already ends with it; compared with the oracle on lists extended the same way, alone and in a step."""
    sched = [1, 2, 2]
    w = wl(3, 8, 2, 900, 48, ragged=True, ctx_min=100, seed=41, layers=len(sched))
    qs = [synth.make_q(w, i, DEV) for i in range(len(sched))]
    if layout == "paged":
        pt, total = synth.make_page_table(w, extra_pages=2)
        layers = [synth.make_layer(w, i, DEV, layout="paged", q=qs[i], page_table=pt, num_pages=total) for i in range(len(sched))]
    else:
        layers = [synth.make_layer(w, i, DEV, q=qs[i]) for i in range(len(sched))]
    lens = layers[0].ctx_lens.cpu().numpy()
    _, idx, cnt = td.select_attn(layers[0], qs[0], w.k)
    idx_h, cnt_h = idx.cpu().numpy().copy(), cnt.cpu().numpy().copy()
    idx_h[0, 0, w.k - 1] = lens[0] - 1                    # one list that already ends with the newest token
    idx_h[0, 0, : w.k - 1] = np.arange(w.k - 1)
    idx_d = torch.from_numpy(idx_h).to(DEV)
    td.set_attend_newest(True)
    try:
        sp = td.sparse_attn(layers[1], qs[1], idx_d, cnt)
        outs, idx2, cnt2 = td.decode_step(sched, layers, qs, w.k)
        with pytest.raises(binding.TidalError):
            td.sparse_attn(layers[1], qs[1], idx_d)       # the end of the lists must be known
        torch.cuda.synchronize()
    finally:
        td.set_attend_newest(False)
    okv1, okv2 = util.oracle_kv(layers[1]), util.oracle_kv(layers[2])
    aug, cnt_aug = oracle.with_newest(okv1, idx_h, cnt_h)
    util.check_out(sp.cpu().numpy(), oracle.sparse_attn(okv1, synth.bits(qs[1]), aug, cnt_aug), "newest.sparse")
    plain = td.sparse_attn(layers[1], qs[1], idx_d, cnt)
    assert not torch.allclose(plain, sp, atol=1e-6)      # the extra token changes the result ...
    assert torch.allclose(plain[0, 0], sp[0, 0], atol=5e-4)   # ... except where the list had it already
    aug2, cnt_aug2 = oracle.with_newest(okv1, idx2.cpu().numpy(), cnt2.cpu().numpy())
    util.check_out(outs[1].cpu().numpy(), oracle.sparse_attn(okv1, synth.bits(qs[1]), aug2, cnt_aug2), "newest.step1")
    util.check_out(outs[2].cpu().numpy(), oracle.sparse_attn(okv2, synth.bits(qs[2]), aug2, cnt_aug2), "newest.step2")
    assert td.device_status() == binding.OK


@pytest.mark.parametrize("layout", ["hnd_interleaved", "paged"])
@pytest.mark.parametrize("B,Hq,Hkv,N,k,ragged", [(1, 8, 2, 300, 40, False), (3, 16, 2, 777, 100, True), (1, 4, 4, 4097, 256, False)])
def test_no_call_writes_outside_its_output_buffers(td, layout, B, Hq, Hkv, N, k, ragged):
    """Every caller-owned output (out, idx, idx_count, scores) sits between guard zones of a fixed pattern,
    which must be intact after each call: full, selection (scores in the caller's buffer and in the
    workspace), sparse, a whole step, and the step with bf16 outputs (half the bytes in the same buffer)."""
    w = wl(B, Hq, Hkv, N, k, planted=min(8, N), ragged=ragged, ctx_min=max(1, N // 3), seed=43, layers=3)
    qs = [synth.make_q(w, i, DEV) for i in range(3)]
    if layout == "paged":
        pt, total = synth.make_page_table(w, extra_pages=3)
        lays = [synth.make_layer(w, i, DEV, layout="paged", q=qs[i], page_table=pt, num_pages=total) for i in range(3)]
    else:
        lays = [synth.make_layer(w, i, DEV, q=qs[i]) for i in range(3)]
    okv, qb = util.oracle_kv(lays[0]), synth.bits(qs[0])
    out = util.Guarded((B, Hq, 128), torch.float32, DEV, fill=float("nan"))
    idx = util.Guarded((B, Hq, k), torch.int32, DEV, fill=-7)
    cnt = util.Guarded((B,), torch.int32, DEV, fill=-7)
    sc = util.Guarded((B, Hq, N), torch.float32, DEV, fill=float("nan"))
    guards = {"out": out, "idx": idx, "idx_count": cnt, "scores": sc}

    def check_all(what):
        for name, g in guards.items():
            g.check(f"{what}: {name}")

    td.full_attn(lays[0], qs[0], out=out.t)
    check_all("full")
    ref_out, ref_sc = oracle.full_attn(okv, qb, want_scores=True)
    util.check_out(out.t.cpu().numpy(), ref_out, "full")
    out.t.fill_(float("nan"))
    td.select_attn(lays[0], qs[0], k, out=out.t, idx=idx.t, idx_count=cnt.t, scores=sc.t)
    check_all("select with caller scores")
    util.check_out(out.t.cpu().numpy(), ref_out, "select")
    lens = lays[0].ctx_lens.cpu().numpy()
    for b in range(B):
        for h in range(Hq):
            util.check_idx_row(idx.t[b, h].cpu().numpy(), ref_sc[b, h], k, int(lens[b]), "select.idx")
    idx.t.fill_(-7)
    td.select_attn(lays[0], qs[0], k, out=out.t, idx=idx.t, idx_count=cnt.t)
    check_all("select with workspace scores")
    out.t.fill_(float("nan"))
    td.sparse_attn(lays[1], qs[1], idx.t, cnt.t, out=out.t)
    check_all("sparse")
    util.check_out(out.t.cpu().numpy(), oracle.sparse_attn(util.oracle_kv(lays[1]), synth.bits(qs[1]),
                                                           idx.t.cpu().numpy(), cnt.t.cpu().numpy()), "sparse")
    # a whole step writing three guarded outputs and the guarded index list
    outs = [util.Guarded((B, Hq, 128), torch.float32, DEV, fill=float("nan")) for _ in range(3)]
    for i, g in enumerate(outs):
        guards[f"out{i}"] = g
    step = td.make_step([0, 1, 2], lays, qs, [g.t for g in outs], k)
    # make_step owns its idx / idx_count; run it, then the same schedule by hand into the guarded ones
    step()
    check_all("step")
    td.set_output_bf16(True)
    try:
        bouts = [util.Guarded((B, Hq, 128), torch.bfloat16, DEV) for _ in range(3)]
        for i, g in enumerate(bouts):
            guards[f"bf16 out{i}"] = g
        td.make_step([0, 1, 2], lays, qs, [g.t for g in bouts], k)()
        check_all("bf16 step")
    finally:
        td.set_output_bf16(False)
    assert td.device_status() == binding.OK


def test_bf16_outputs_match_the_oracle(td):
    """Outputs rounded to bf16 against the oracle: the usual bounds widened by one bf16 step of the value
    (2^-8 relative: the rounding of a correctly computed fp32 result moves it by at most half a step, the
    fp32 result itself may sit on the other side of a rounding boundary)."""
    sched = [0, 1, 2]
    w = wl(2, 8, 2, 700, 64, ragged=True, ctx_min=300, seed=31, layers=len(sched))
    qs = [synth.make_q(w, i, DEV) for i in range(len(sched))]
    layers = [synth.make_layer(w, i, DEV, q=qs[i]) for i in range(len(sched))]
    td.set_output_bf16(True)
    try:
        outs, idx, cnt = td.decode_step(sched, layers, qs, w.k)
        sel, idx2, cnt2 = td.select_attn(layers[1], qs[1], w.k)
        sp = td.sparse_attn(layers[2], qs[2], idx2, cnt2)
        torch.cuda.synchronize()
    finally:
        td.set_output_bf16(False)
    idx_h, cnt_h = idx.cpu().numpy(), cnt.cpu().numpy()
    refs = [oracle.full_attn(util.oracle_kv(layers[0]), synth.bits(qs[0])),
            oracle.full_attn(util.oracle_kv(layers[1]), synth.bits(qs[1])),
            oracle.sparse_attn(util.oracle_kv(layers[2]), synth.bits(qs[2]), idx_h, cnt_h)]

    def check_bf16(got, ref, what):
        got = got.float().cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all()
        err = np.abs(got - ref)
        assert (err <= util.MAX_ABS_TOL + np.abs(ref) * 2.0 ** -8).all(), f"{what}: max abs err {err.max():.3e}"
        assert err.mean() <= util.MEAN_ABS_TOL + np.abs(ref).mean() * 2.0 ** -8, f"{what}: mean abs err {err.mean():.3e}"
        # and in fact the error is the rounding alone
        assert (err <= 1e-3 + np.abs(ref) * 2.0 ** -8).all(), what

    for i in range(3):
        assert outs[i].dtype == torch.bfloat16
        check_bf16(outs[i], refs[i], f"bf16 step layer {i}")
    check_bf16(sel, refs[1], "bf16 select")
    assert torch.equal(idx2, idx)
    check_bf16(sp, refs[2], "bf16 sparse")
    assert td.device_status() == binding.OK


def test_an_invalid_step_leaves_the_caches_untouched(td):
    """tidal_decode_step_append validates the whole step before it writes a single row: a schedule with a
    sparse layer ahead of any selection layer is refused and every cache byte is as before."""
    sched = [0, 2, 1]
    w = wl(2, 8, 2, 300, 16, ragged=True, ctx_min=50, seed=47, layers=3)
    qs = [synth.make_q(w, i, DEV) for i in range(3)]
    layers = [synth.make_layer(w, i, DEV, q=qs[i]) for i in range(3)]
    before = [l.keep[0].clone() for l in layers]
    kn = [torch.ones(w.batch, w.num_kv_heads, 128, dtype=torch.bfloat16, device=DEV) for _ in sched]
    with pytest.raises(binding.TidalError) as e:
        td.decode_step_append(sched, layers, qs, kn, kn, w.k)
    assert e.value.status == binding.ERR_INVALID
    torch.cuda.synchronize()
    for l, b in zip(layers, before):
        assert torch.equal(l.keep[0], b)
    # k larger than a selection layer's max_ctx_len is refused the same way
    with pytest.raises(binding.TidalError):
        td.decode_step_append([0, 1, 2], layers, qs, kn, kn, 301)
    torch.cuda.synchronize()
    for l, b in zip(layers, before):
        assert torch.equal(l.keep[0], b)


def test_reserve_then_capture_the_first_call(td):
    """tidal_reserve sizes workspace and counters, so that the very first call of a fresh context can be
    recorded into a CUDA graph (nothing allocates, nothing touches the legacy stream)."""
    sched = [0, 1, 2, 2]
    w = wl(2, 8, 2, 1500, 64, ragged=True, ctx_min=400, seed=53, layers=len(sched))
    qs = [synth.make_q(w, i, DEV) for i in range(len(sched))]
    layers = [synth.make_layer(w, i, DEV, q=qs[i]) for i in range(len(sched))]
    ref_outs, ref_idx, _ = td.decode_step(sched, layers, qs, w.k)
    torch.cuda.synchronize()
    fresh = binding.Tidal(0)
    try:
        fresh.reserve(layers[0], w.k)
        outs = [torch.zeros_like(o) for o in ref_outs]
        step = fresh.make_step(sched, layers, qs, outs, w.k)
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())      # the inputs were built on the current stream
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                step()                                    # the context's first call ever
        graph.replay()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(step.idx, ref_idx)
        for o, r in zip(outs, ref_outs):
            assert torch.allclose(o, r, rtol=0, atol=5e-4)
        assert fresh.device_status() == binding.OK
    finally:
        fresh.close()


def test_extreme_ragged_batches_stay_within_the_split_bound(td):
    """One long sequence among many one-token ones, and the reverse: the number of CTAs that share a row
    is bounded on the host; a kernel that found the bound too small would set the status word."""
    for lens in ([4000] + [1] * 60, [1] * 60 + [4000], [4000, 3999] + [17] * 30, [16] * 64):
        B = len(lens)
        w = wl(B, 4, 2, max(lens), min(32, max(lens)), planted=1, seed=59)
        q, lay = build(w, "paged")
        lay.ctx_lens = torch.tensor(lens, dtype=torch.int32, device=DEV)
        okv, qb = util.oracle_kv(lay), synth.bits(q)
        out, idx, cnt = td.select_attn(lay, q, w.k)
        ref, sc = oracle.full_attn(okv, qb, want_scores=True)
        util.check_out(out.cpu().numpy(), ref, "ragged.select")
        for b in (0, B - 1):
            for h in range(4):
                util.check_idx_row(idx.cpu().numpy()[b, h], sc[b, h], w.k, lens[b], "ragged.idx")
        sp = td.sparse_attn(lay, q, idx, cnt)
        util.check_out(sp.cpu().numpy(), oracle.sparse_attn(okv, qb, idx.cpu().numpy(), cnt.cpu().numpy()), "ragged.sparse")
        assert td.device_status() == binding.OK


@pytest.mark.parametrize("N,k,Hq,Hkv", [(8200, 300, 8, 2), (40000, 2000, 4, 4), (131072, 4096, 8, 2)])
def test_candidate_compaction_is_exact_with_and_without_its_fallback(td, N, k, Hq, Hkv):
    """The optional compaction of top-k candidates inside the selection kernel: with a generous margin the
    list decides, with a margin below 1 the provisional thresholds are too high and the kernel must notice
    and rank all scores instead; either way the sets are the ones the oracle's full sort gives, twice in a
    row (the lists' cursors and thresholds must be left clean)."""
    w = wl(1, Hq, Hkv, N, k, planted=16, seed=61)
    q, lay = build(w, "hnd_interleaved")
    ref, sc = oracle.full_attn(util.oracle_kv(lay), synth.bits(q), want_scores=True)
    _, base_idx, _ = td.select_attn(lay, q, k)                 # compaction off
    try:
        for margin in (3.0, 1.0, 0.3):
            td.set_select_margin(margin)
            for _ in range(2):
                out, idx, cnt = td.select_attn(lay, q, k)
                util.check_out(out.cpu().numpy(), ref, f"margin {margin}")
                assert cnt.item() == k
                for h in range(Hq):
                    util.check_idx_row(idx.cpu().numpy()[0, h], sc[0, h], k, N, f"margin {margin} head {h}")
                assert torch.equal(idx, base_idx)               # the tie rule is the same on every path
    finally:
        td.set_select_margin(0.0)
    assert td.device_status() == binding.OK


def test_candidate_compaction_on_scores_that_drift_along_the_context(td):
    """Provisional thresholds come from the first tiles each CTA sees. Here the keys of the second half
    of the context are scaled up, so CTAs disagree widely about the threshold: the result must still be
    exact (through the list where it is complete, through the fallback where it is not), also inside a
    decode step followed by a sparse layer."""
    N, k = 65536, 1024
    w = wl(1, 8, 2, N, k, planted=16, seed=67, layers=2)
    qs = [synth.make_q(w, i, DEV) for i in range(2)]
    lays = [synth.make_layer(w, i, DEV, q=qs[i]) for i in range(2)]
    buf = lays[0].keep[0]                                         # [B][Hkv][N][K|V][d]
    buf[:, :, N // 2:, 0, :] *= 3.0
    buf[:, :, : N // 8, 0, :] *= 0.25
    ref, sc = oracle.full_attn(util.oracle_kv(lays[0]), synth.bits(qs[0]), want_scores=True)
    try:
        for margin in (3.0, 1.5):
            td.set_select_margin(margin)
            outs, idx, cnt = td.decode_step([1, 2], lays, qs, k)
            util.check_out(outs[0].cpu().numpy(), ref, "drift.select")
            idx_h = idx.cpu().numpy()
            for h in range(8):
                util.check_idx_row(idx_h[0, h], sc[0, h], k, N, f"drift head {h}")
            util.check_out(outs[1].cpu().numpy(), oracle.sparse_attn(util.oracle_kv(lays[1]), synth.bits(qs[1]), idx_h,
                                                                     cnt.cpu().numpy()), "drift.sparse")
    finally:
        td.set_select_margin(0.0)
    assert td.device_status() == binding.OK


def test_scores_that_are_not_numbers_never_leave_stale_indices(td):
    """Keys holding NaN (and infinities) make some scores NaN: what is selected among them is unspecified,
    but every entry of the list must be a valid position or -1, in every top-k path."""
    N, k = 20000, 1500
    w = wl(1, 4, 2, N, k, planted=4, seed=71)
    q, lay = build(w, "hnd_interleaved")
    buf = lay.keep[0]
    buf[0, :, 100:19000:7, 0, 5] = float("nan")
    buf[0, :, 3, 0, 0] = float("inf")
    idx = torch.full((1, 4, k), 123456789, dtype=torch.int32, device=DEV)
    try:
        for margin in (0.0, 3.0, 0.3):
            td.set_select_margin(margin)
            idx.fill_(123456789)
            td.select_attn(lay, q, k, idx=idx)
            got = idx.cpu().numpy()
            assert ((got >= -1) & (got < N)).all(), margin
            for h in range(4):
                sel = got[0, h][got[0, h] >= 0]
                assert len(np.unique(sel)) == len(sel) and (np.diff(sel) > 0).all()
    finally:
        td.set_select_margin(0.0)
    td.device_status()


# ---- 8-bit (FP8 E4M3) caches ------------------------------------------------------------------------
FP8_CASES = [
    # batch, Hq, Hkv, ctx, k, ragged
    (1, 8, 2, 300, 40, False),
    (2, 8, 2, 1000, 64, True),
    (1, 4, 4, 4097, 256, False),       # MHA, ragged tail of one position
    (3, 16, 2, 777, 100, True),        # group 8
    (1, 2, 1, 2500, 17, False),
    (1, 8, 2, 17, 17, False),
    (1, 4, 2, 1, 1, False),
    (1, 32, 8, 20000, 1024, False),    # pooled grid, several CTAs per head
]


@pytest.mark.parametrize("layout", ["hnd_interleaved", "paged"])
@pytest.mark.parametrize("B,Hq,Hkv,N,k,ragged", FP8_CASES)
def test_fp8_cache_layers_match_the_oracle(td, layout, B, Hq, Hkv, N, k, ragged):
    """Full, selection and sparse layers over a cache of E4M3 codes with per-KV-head scales, against the
    oracle's dequantise-then-Eq. 1 on the same codes and scales."""
    w = wl(B, Hq, Hkv, N, k, planted=min(8, N), ragged=ragged, ctx_min=max(1, N // 3), seed=73)
    q, lay16 = build(w, layout)
    lay = synth.to_fp8(lay16)
    assert lay.kv_dtype == synth.KV_FP8_E4M3 and lay.k.element_size() == 1
    okv, qb = util.oracle_kv(lay), synth.bits(q)
    lens = lay.ctx_lens.cpu().numpy()
    ref_out, ref_sc = oracle.full_attn(okv, qb, want_scores=True)
    util.check_out(td.full_attn(lay, q).cpu().numpy(), ref_out, "fp8.full")
    scores = torch.full((B, Hq, N), float("nan"), dtype=torch.float32, device=DEV)
    out, idx, cnt = td.select_attn(lay, q, k, scores=scores)
    util.check_out(out.cpu().numpy(), ref_out, "fp8.select")
    assert cnt.cpu().numpy().tolist() == [min(k, int(n)) for n in lens]
    sc, idx_h = scores.cpu().numpy(), idx.cpu().numpy()
    for b in range(B):
        n = int(lens[b])
        assert np.abs(sc[b, :, :n] - ref_sc[b, :, :n]).max() <= 1e-4
        for h in range(Hq):
            util.check_idx_row(idx_h[b, h], ref_sc[b, h], k, n, f"fp8.idx[{b},{h}]")
    _, ref_idx, ref_cnt = oracle.select_attn(okv, qb, k)
    sp = td.sparse_attn(lay, q, torch.from_numpy(ref_idx).to(DEV), torch.from_numpy(ref_cnt).to(DEV))
    util.check_out(sp.cpu().numpy(), oracle.sparse_attn(okv, qb, ref_idx, ref_cnt), "fp8.sparse")
    # quantisation is visible: the 8-bit result is close to, but not the same as, the 16-bit one
    if N > 16:
        assert not torch.equal(td.full_attn(lay16, q), td.full_attn(lay, q))
    assert td.device_status() == binding.OK


def test_fp8_decode_step_with_aggregated_sets_and_append(td):
    """A whole step (F, S, sp, S, sp) over E4M3 caches with the cache update (codes are copied), one token
    set per KV head, against the oracle stepping over host copies."""
    sched = [0, 1, 2, 1, 2]
    w = wl(2, 8, 2, 900, 64, ragged=True, ctx_min=200, seed=79, layers=len(sched))
    qs = [synth.make_q(w, i, DEV) for i in range(len(sched))]
    layers = [synth.to_fp8(synth.make_layer(w, i, DEV, q=qs[i])) for i in range(len(sched))]
    g = torch.Generator(device="cpu").manual_seed(3)
    k_new = [torch.randn(w.batch, w.num_kv_heads, 128, generator=g).to(torch.float8_e4m3fn) for _ in sched]
    v_new = [torch.randn(w.batch, w.num_kv_heads, 128, generator=g).to(torch.float8_e4m3fn) for _ in sched]
    okvs = [util.oracle_kv(l) for l in layers]
    for okv, kn, vn in zip(okvs, k_new, v_new):
        oracle.kv_append(okv, synth.bits(kn), synth.bits(vn))
    outs, idx, cnt = td.decode_step_append(sched, layers, qs, [t.to(DEV) for t in k_new], [t.to(DEV) for t in v_new],
                                           w.k, granularity=binding.SEL_PER_KVHEAD)
    torch.cuda.synchronize()
    for l, okv in zip(layers, okvs):
        after = util.oracle_kv(l)
        assert np.array_equal(after.k, okv.k) and np.array_equal(after.v, okv.v)
    lens = layers[0].ctx_lens.cpu().numpy()
    cur = None
    for i, t in enumerate(sched):
        qb, got = synth.bits(qs[i]), outs[i].cpu().numpy()
        if t in (0, 1):
            ref, sc = oracle.full_attn(okvs[i], qb, want_scores=True)
            util.check_out(got, ref, f"fp8.step.layer{i}")
            if t == 1:
                _, gi, gc = td.select_attn(layers[i], qs[i], w.k, granularity=binding.SEL_PER_KVHEAD)
                cur = (gi.cpu().numpy(), gc.cpu().numpy())
                for b in range(w.batch):
                    for g_ in range(w.num_kv_heads):
                        agg = sc[b, 4 * g_: 4 * g_ + 4, : lens[b]].astype(np.float64).sum(0).astype(np.float32)
                        util.check_idx_row(cur[0][b, g_], agg, w.k, int(lens[b]), f"fp8.step.idx{i}")
        else:
            util.check_out(got, oracle.sparse_attn(okvs[i], qb, cur[0], cur[1]), f"fp8.step.layer{i}")
    assert np.array_equal(idx.cpu().numpy(), cur[0])
    assert td.device_status() == binding.OK


def test_fp8_argument_rules(td):
    w = wl(1, 8, 2, 64, 8, seed=83)
    q, lay16 = build(w, "hnd_interleaved")
    lay = synth.to_fp8(lay16)
    import ctypes as C
    out = torch.empty(1, 8, 128, dtype=torch.float32, device=DEV)
    s = binding.kv_struct(lay)
    assert td.lib.tidal_full_attn(td.ctx, C.byref(s), q.data_ptr(), out.data_ptr(), None) == binding.OK
    s.stride_pos = 264                                    # not a multiple of 16 bytes
    assert td.lib.tidal_full_attn(td.ctx, C.byref(s), q.data_ptr(), out.data_ptr(), None) == binding.ERR_INVALID
    s = binding.kv_struct(lay); s.kv_dtype = 7
    assert td.lib.tidal_full_attn(td.ctx, C.byref(s), q.data_ptr(), out.data_ptr(), None) == binding.ERR_INVALID
    idx = torch.zeros(1, 8, 8, dtype=torch.int32, device=DEV)
    s = binding.kv_struct(lay)
    assert td.lib.tidal_sparse_attn_noalloc(C.byref(s), q.data_ptr(), idx.data_ptr(), None, 8, 8, out.data_ptr(), None) == binding.ERR_UNSUPPORTED
    torch.cuda.synchronize()


@pytest.mark.parametrize("shape", ["one sequence, chains of sparse layers", "paged ragged batch", "small grids",
                                   "full and sparse layers interleaved"])
def test_overlapping_layers_repeatably_equal_the_non_overlapped_step(td, shape):
    """Layers of a step overlap (late wait, early trigger, several sparse layers in flight, pool cursors
    used ahead of the wait). Run the step hundreds of times back to back, so that consecutive steps overlap
    too, against the same step with the overlap switched off: identical token sets every time, outputs
    equal up to the rounding of a different split; the non-overlapped step is itself checked against the
    oracle on its sparse layers."""
    if shape == "one sequence, chains of sparse layers":
        w = synth.Workload("ov1", 1, 32, 8, 16, 20000, 1024, 8, [0, 0, 1] + [2] * 6 + [1] + [2] * 6, 6)
    elif shape == "paged ragged batch":
        w = synth.Workload("ov2", 4, 16, 4, 12, 9000, 512, 8, [0, 1] + [2] * 5 + [0, 1] + [2] * 3, 7,
                           ragged=True, ctx_min=2000, paged=True)
    elif shape == "small grids":
        w = synth.Workload("ov3", 1, 8, 2, 12, 3000, 256, 8, [0, 1] + [2] * 10, 5)
    else:
        w = synth.Workload("ov4", 1, 32, 8, 11, 24000, 2048, 8, [1, 2, 0, 2, 0, 0, 2, 1, 1, 2, 0], 8)
    L = len(w.sched)
    qs = [synth.make_q(w, i, DEV) for i in range(L)]
    if w.paged:
        pt, total = synth.make_page_table(w)
        lays = [synth.make_layer(w, i, DEV, layout="paged", q=qs[i], page_table=pt, num_pages=total) for i in range(L)]
    else:
        lays = [synth.make_layer(w, i, DEV, q=qs[i]) for i in range(L)]
    outs = [torch.zeros(w.batch, w.num_q_heads, 128, device=DEV) for _ in range(L)]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())      # the inputs were built on the current stream
    with torch.cuda.stream(side):
        td.set_layer_overlap(False)
        try:
            plain = td.make_step(w.sched, lays, qs, outs, w.k)
            plain()
            side.synchronize()
        finally:
            td.set_layer_overlap(True)
        ref, ref_idx, ref_cnt = [o.clone() for o in outs], plain.idx.clone(), plain.idx_count.clone()
        last = max(i for i, kind in enumerate(w.sched) if kind == 2)      # a sparse layer, fed by the last selection layer
        want = oracle.sparse_attn(util.oracle_kv(lays[last]), synth.bits(qs[last]), ref_idx.cpu().numpy(), ref_cnt.cpu().numpy())
        util.check_out(ref[last].cpu().numpy(), want, "non-overlapped reference")
        step = td.make_step(w.sched, lays, qs, outs, w.k)
        for it in range(120):
            for o in outs:
                o.fill_(float("nan"))
            step.idx.fill_(-9)
            for _ in range(3):
                step()
            side.synchronize()
            assert torch.equal(step.idx, ref_idx), it
            for o, r in zip(outs, ref):
                assert torch.allclose(o, r, rtol=0, atol=2e-3), it
    assert td.device_status() == binding.OK


def _two_pass_cases():
    shapes = [(32, 8, 20011, 1024), (16, 16, 24000, 900), (16, 2, 40001, 3000), (8, 4, 70000, 2048)]
    cases = [(layout, *shape, False) for layout in ("hnd_interleaved", "nhd_separate", "paged") for shape in shapes]
    # the same over caches of E4M3 codes (units of 32 positions: lengths that end in the first and in the second
    # tile of a unit, a single tile, three tiles)
    cases += [(layout, *shape, True) for layout in ("hnd_interleaved", "paged") for shape in shapes]
    cases += [("paged", 32, 8, 20011 + 16, 1024, True), ("hnd_interleaved", 8, 1, 15, 8, True),
              ("paged", 8, 2, 16 * 2 + 3, 16, True), ("hnd_interleaved", 16, 4, 16 * 64, 100, True)]
    return cases


@pytest.mark.parametrize("layout,Hq,Hkv,N,k,fp8", _two_pass_cases())
def test_two_pass_selection_layers_match_the_oracle(td, layout, Hq, Hkv, N, k, fp8):
    """Inside a step (one sequence, per-head sets) a selection layer runs as a key pass and a value pass on
    two streams. Its output, its token sets and the sparse layers after it against the oracle, for groups of
    1, 2, 4 and 8, context lengths with a ragged last tile, all layouts, bf16 and FP8 caches; and against the
    fused kernel that the single-layer call uses. Two selection layers in a row share the score buffer: the
    second key pass must wait for the first value pass."""
    sched = [0, 1, 1, 2, 2]
    w = wl(1, Hq, Hkv, N, k, planted=8, seed=97, layers=len(sched))
    qs = [synth.make_q(w, i, DEV) for i in range(len(sched))]
    if layout == "paged":
        pt, total = synth.make_page_table(w, extra_pages=3)
        lays = [synth.make_layer(w, i, DEV, layout="paged", q=qs[i], page_table=pt, num_pages=total) for i in range(len(sched))]
    else:
        lays = [synth.make_layer(w, i, DEV, layout=layout, q=qs[i]) for i in range(len(sched))]
    if fp8:
        lays = [synth.to_fp8(lay) for lay in lays]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())      # the inputs were built on the current stream
    with torch.cuda.stream(side):
        outs, idx, cnt = td.decode_step(sched, lays, qs, w.k)
        side.synchronize()
    for i in (1, 2):
        okv, qb = util.oracle_kv(lays[i]), synth.bits(qs[i])
        ref, sc = oracle.full_attn(okv, qb, want_scores=True)
        util.check_out(outs[i].cpu().numpy(), ref, f"two-pass layer {i}")
        fused, fidx, _ = td.select_attn(lays[i], qs[i], w.k)
        assert torch.allclose(outs[i], fused, rtol=0, atol=1e-3)
        if i == 2:
            assert torch.equal(idx, fidx)                  # same scores, same sets as the fused kernel
            for h in range(0, Hq, max(1, Hq // 4)):
                util.check_idx_row(idx.cpu().numpy()[0, h], sc[0, h], w.k, N, f"two-pass idx[{h}]")
    for i in (3, 4):
        ref = oracle.sparse_attn(util.oracle_kv(lays[i]), synth.bits(qs[i]), idx.cpu().numpy(), cnt.cpu().numpy())
        util.check_out(outs[i].cpu().numpy(), ref, f"sparse layer {i} after a two-pass selection")
    assert td.device_status() == binding.OK


@pytest.mark.parametrize("B,Hq,Hkv,N,k,ragged,layout", [
    (3, 16, 4, 9000, 500, True, "hnd_interleaved"), (8, 8, 2, 5000, 256, True, "paged"),
    (2, 32, 8, 20000, 1024, False, "nhd_separate"), (5, 8, 8, 700, 64, True, "paged"),
    (4, 8, 1, 90, 16, True, "hnd_interleaved"), (6, 16, 2, 33000, 2048, True, "paged")])
def test_two_pass_selection_layers_of_a_batch_match_the_oracle(td, B, Hq, Hkv, N, k, ragged, layout):
    """Batches run the two passes over a flat split of the (sequence, KV head, tile) space: CTAs cross item
    and sequence boundaries. Outputs, token sets and the sparse layers after two consecutive selection
    layers against the oracle, ragged lengths, all layouts."""
    sched = [0, 1, 1, 2, 2]
    w = wl(B, Hq, Hkv, N, k, planted=min(8, N), seed=131, ragged=ragged, ctx_min=max(1, N // 5), layers=len(sched))
    qs = [synth.make_q(w, i, DEV) for i in range(len(sched))]
    if layout == "paged":
        pt, total = synth.make_page_table(w, extra_pages=3)
        lays = [synth.make_layer(w, i, DEV, layout="paged", q=qs[i], page_table=pt, num_pages=total) for i in range(len(sched))]
    else:
        lays = [synth.make_layer(w, i, DEV, layout=layout, q=qs[i]) for i in range(len(sched))]
    lens = lays[0].ctx_lens.cpu().numpy()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())      # the inputs were built on the current stream
    with torch.cuda.stream(side):
        outs, idx, cnt = td.decode_step(sched, lays, qs, w.k)
        side.synchronize()
    assert cnt.cpu().numpy().tolist() == [min(k, int(n)) for n in lens]
    for i in (1, 2):
        okv, qb = util.oracle_kv(lays[i]), synth.bits(qs[i])
        ref, sc = oracle.full_attn(okv, qb, want_scores=True)
        util.check_out(outs[i].cpu().numpy(), ref, f"batch two-pass layer {i}")
        if i == 2:
            idx_h = idx.cpu().numpy()
            for b in range(B):
                for h in range(0, Hq, max(1, Hq // 4)):
                    util.check_idx_row(idx_h[b, h], sc[b, h], w.k, int(lens[b]), f"batch two-pass idx[{b},{h}]")
    for i in (3, 4):
        ref = oracle.sparse_attn(util.oracle_kv(lays[i]), synth.bits(qs[i]), idx.cpu().numpy(), cnt.cpu().numpy())
        util.check_out(outs[i].cpu().numpy(), ref, f"sparse layer {i} after a batch's two-pass selection")
    assert td.device_status() == binding.OK


def _step_fuzz_cases(n, seed):
    import random
    rng = random.Random(seed)
    cases = []
    for _ in range(n):
        B = rng.choice([1, 1, 1, 2, 3, 5])
        Hkv = rng.choice([1, 2, 4, 8])
        G = min(rng.choice([1, 2, 4, 8]), 32 // Hkv)
        N = rng.choice([17, 100, 1000, 4096, 9001, 20000, 33333])
        k = min(rng.choice([8, 64, 300, 1024]), N)
        ragged = B > 1 and rng.random() < 0.7
        layout = rng.choice(["hnd_interleaved", "paged", "nhd_separate"])
        fp8 = layout != "nhd_separate" and rng.random() < 0.35
        sched = rng.choice(["12", "0112", "12122", "00122212"])
        cases.append((B, Hkv * G, Hkv, N, k, ragged, layout, fp8, sched))
    return cases


@pytest.mark.parametrize("B,Hq,Hkv,N,k,ragged,layout,fp8,sched", _step_fuzz_cases(24, 20241006))
def test_random_decode_steps_match_the_oracle(td, B, Hq, Hkv, N, k, ragged, layout, fp8, sched):
    """Whole steps over random shapes, layouts, cache types and schedules (two calls in a row, the second a
    replay): every full and selection layer, the last token sets and the sparse layers that use them against
    the oracle. Covers the pooled, the flat-split and the FP8 variants of the two selection passes."""
    sched = [int(c) for c in sched]
    w = wl(B, Hq, Hkv, N, k, planted=min(8, N), seed=500 + N % 97 + B, ragged=ragged, ctx_min=max(1, N // 4), layers=len(sched))
    qs = [synth.make_q(w, i, DEV) for i in range(len(sched))]
    if layout == "paged":
        pt, total = synth.make_page_table(w, extra_pages=3)
        lays = [synth.make_layer(w, i, DEV, layout="paged", q=qs[i], page_table=pt, num_pages=total) for i in range(len(sched))]
    else:
        lays = [synth.make_layer(w, i, DEV, layout=layout, q=qs[i]) for i in range(len(sched))]
    if fp8:
        lays = [synth.to_fp8(lay) for lay in lays]
    lens = lays[0].ctx_lens.cpu().numpy()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())      # the inputs were built on the current stream
    with torch.cuda.stream(side):
        outs, idx, cnt = td.decode_step(sched, lays, qs, w.k)
        outs2, idx2, _ = td.decode_step(sched, lays, qs, w.k)
        side.synchronize()
    assert torch.equal(idx, idx2)
    last_sel = max(i for i, t in enumerate(sched) if t == 1)
    for i, t in enumerate(sched):
        okv, qb = util.oracle_kv(lays[i]), synth.bits(qs[i])
        if t != 2:
            ref = oracle.full_attn(okv, qb)
            util.check_out(outs[i].cpu().numpy(), ref, f"layer {i}")
            util.check_out(outs2[i].cpu().numpy(), ref, f"layer {i}, second call")
        elif i > last_sel:
            ref = oracle.sparse_attn(okv, qb, idx.cpu().numpy(), cnt.cpu().numpy())
            util.check_out(outs[i].cpu().numpy(), ref, f"sparse layer {i}")
    _, sc = oracle.full_attn(util.oracle_kv(lays[last_sel]), synth.bits(qs[last_sel]), want_scores=True)
    idx_h = idx.cpu().numpy()
    for b in range(B):
        for h in range(0, Hq, max(1, Hq // 3)):
            util.check_idx_row(idx_h[b, h], sc[b, h], w.k, int(lens[b]), f"idx[{b},{h}]")
    assert td.device_status() == binding.OK
