"""Pins of the CPU oracle against things other than itself: an independent
evaluation of Eq. 1, closed forms, invariances, brute force, and the facts the
paper prints (layer mix, KV-cache size). CPU only."""
import os

import numpy as np
import pytest
import torch

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")
D = 128


def bf16_bits(x: np.ndarray) -> np.ndarray:
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def bf16_val(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def make(B, Hq, Hkv, N, seed, lens=None, scale=0.0):
    """NHD contiguous cache K,V [B,N,Hkv,D] as bf16 bits + oracle descriptor."""
    r = np.random.default_rng(seed)
    q = bf16_bits(r.standard_normal((B, Hq, D)))
    k = bf16_bits(r.standard_normal((B, N, Hkv, D)))
    v = bf16_bits(r.standard_normal((B, N, Hkv, D)))
    lens = np.full(B, N, np.int32) if lens is None else np.asarray(lens, np.int32)
    kv = oracle.KV(k=k.reshape(-1), v=v.reshape(-1), batch=B, num_q_heads=Hq, num_kv_heads=Hkv,
                   head_dim=D, ctx_lens=lens, stride_b=N * Hkv * D, stride_pos=Hkv * D,
                   stride_head=D, sm_scale=scale)
    return q, k, v, kv


def eq1_numpy(q, k, v, lens, idx=None):
    """Eq. 1 evaluated independently in float64 with numpy matmul/softmax."""
    B, Hq, _ = q.shape
    Hkv = k.shape[2]
    G = Hq // Hkv
    qf, kf, vf = bf16_val(q), bf16_val(k), bf16_val(v)
    out = np.zeros((B, Hq, D))
    for b in range(B):
        for h in range(Hq):
            rows = np.arange(lens[b]) if idx is None else idx[b][h]
            K = kf[b, rows, h // G]
            V = vf[b, rows, h // G]
            a = (K @ qf[b, h]) / np.sqrt(D)
            p = np.exp(a - a.max())
            out[b, h] = (p / p.sum()) @ V
    return out


# ---- P1: softmax weights -------------------------------------------------
def test_softmax_weights_sum_to_one():
    q, k, v, kv = make(1, 2, 2, 777, 1)
    for h in range(2):
        s = oracle.logits(kv, q, 0, h)
        w = oracle.softmax_weights(s)
        assert abs(w.sum() - 1.0) < 1e-6
        assert (w >= 0).all()
        # textbook softmax of the same logits
        e = np.exp(s.astype(np.float64) - s.max())
        np.testing.assert_allclose(w, e / e.sum(), rtol=1e-12)


# ---- P2: full attention vs an independent formulation ---------------------
@pytest.mark.parametrize("B,Hq,Hkv,N", [(1, 1, 1, 1), (2, 4, 4, 33), (1, 8, 2, 300), (3, 6, 2, 65)])
def test_full_attention_matches_eq1(B, Hq, Hkv, N):
    lens = [max(1, N - 7 * b) for b in range(B)]
    q, k, v, kv = make(B, Hq, Hkv, N, 10 + N, lens)
    out, sc = oracle.full_attn(kv, q, want_scores=True)
    ref = eq1_numpy(q, k, v, lens)
    np.testing.assert_allclose(out, ref, rtol=0, atol=2e-7)
    # the emitted scores are A = q K^T / sqrt(d), not the raw inner product and not transposed
    G = Hq // Hkv
    for b in range(B):
        for h in range(Hq):
            a = bf16_val(k)[b, : lens[b], h // G] @ bf16_val(q)[b, h] / np.sqrt(D)
            np.testing.assert_allclose(sc[b, h, : lens[b]], a, rtol=0, atol=1e-6)


def test_full_attention_matches_torch_sdpa():
    q, k, v, kv = make(2, 4, 4, 97, 5)
    out = oracle.full_attn(kv, q)
    qt = torch.from_numpy(bf16_val(q))[:, :, None, :]
    kt = torch.from_numpy(bf16_val(k)).permute(0, 2, 1, 3)
    vt = torch.from_numpy(bf16_val(v)).permute(0, 2, 1, 3)
    ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt)[:, :, 0, :].numpy()
    np.testing.assert_allclose(out, ref, rtol=0, atol=2e-7)


def test_explicit_scale_is_used():
    q, k, v, kv = make(1, 2, 2, 50, 6, scale=0.25)
    _, sc = oracle.full_attn(kv, q, want_scores=True)
    a = bf16_val(k)[0, :, 0] @ bf16_val(q)[0, 0] * 0.25
    np.testing.assert_allclose(sc[0, 0], a, atol=1e-5)


# ---- P3: k >= N makes sparse attention equal to full attention ------------
@pytest.mark.parametrize("k", [40, 41, 64])
def test_sparse_with_full_budget_equals_full(k):
    q, k_, v, kv = make(2, 4, 2, 40, 3, lens=[40, 29])
    full = oracle.full_attn(kv, q)
    out, idx, cnt = oracle.select_attn(kv, q, k)
    assert cnt.tolist() == [min(k, 40), min(k, 29)]
    for b, n in enumerate([40, 29]):
        assert (idx[b, :, : min(k, n)] == np.arange(min(k, n))).all()
        assert (idx[b, :, min(k, n):] == -1).all()
    sp = oracle.sparse_attn(kv, q, idx, cnt)
    assert np.array_equal(out, full)
    if k >= 40:
        assert np.array_equal(sp, full)          # bit for bit
    else:
        assert np.array_equal(sp[1], full[1])    # the shorter sequence is fully covered


# ---- P4: top-k vs brute force and vs ranking by probability ---------------
def brute_topk(s, k):
    s = s.astype(np.float64).copy()
    picked = []
    for _ in range(min(k, len(s))):
        j = int(np.argmax(s))           # numpy argmax returns the lowest index among equals
        picked.append(j)
        s[j] = -np.inf
    return sorted(picked)


@pytest.mark.parametrize("n,k", [(1, 1), (17, 5), (256, 64), (512, 511), (100, 100), (100, 130)])
def test_topk_matches_brute_force(n, k):
    r = np.random.default_rng(n * 1000 + k)
    s = r.standard_normal(n).astype(np.float32)
    s[r.integers(0, n, n // 4)] = np.float32(0.5)      # many exact ties
    idx = oracle.topk(s, k)
    kk = min(n, k)
    assert idx[:kk].tolist() == brute_topk(s, k)
    assert (idx[kk:] == -1).all()


def test_topk_by_logit_equals_topk_by_probability():
    q, k, v, kv = make(1, 4, 4, 400, 8)
    _, idx, _ = oracle.select_attn(kv, q, 37)
    for h in range(4):
        w = oracle.softmax_weights(oracle.logits(kv, q, 0, h))
        by_prob = np.sort(np.argsort(-w, kind="stable")[:37])
        assert idx[0, h].tolist() == by_prob.tolist()


def test_topk_all_equal_takes_lowest_positions():
    s = np.zeros(50, np.float32)
    assert oracle.topk(s, 7).tolist() == list(range(7))


# ---- P5: the selected set retains the most softmax mass --------------------
def test_selected_set_maximises_retained_mass():
    q, k, v, kv = make(1, 2, 2, 300, 9)
    _, idx, _ = oracle.select_attn(kv, q, 30)
    r = np.random.default_rng(0)
    for h in range(2):
        w = oracle.softmax_weights(oracle.logits(kv, q, 0, h))
        mass = w[idx[0, h]].sum()
        for _ in range(1000):
            assert w[r.choice(300, 30, replace=False)].sum() <= mass + 1e-15
        inside = set(idx[0, h].tolist())
        worst_in = min(w[j] for j in inside)
        best_out = max(w[j] for j in range(300) if j not in inside)
        assert best_out <= worst_in                 # no single swap improves it


# ---- P6: closed-form bound on sparse-vs-full error ------------------------
def test_sparse_error_is_bounded_by_dropped_mass():
    q, k, v, kv = make(1, 4, 2, 500, 11)
    full = oracle.full_attn(kv, q)
    _, idx, cnt = oracle.select_attn(kv, q, 100)
    sp = oracle.sparse_attn(kv, q, idx, cnt)
    vmax = np.abs(bf16_val(v)).max()
    for h in range(4):
        w = oracle.softmax_weights(oracle.logits(kv, q, 0, h))
        dropped = 1.0 - w[idx[0, h]].sum()
        assert np.abs(full[0, h] - sp[0, h]).max() <= 2 * dropped * vmax + 1e-6


# ---- P7: closed-form special cases ----------------------------------------
def test_zero_query_gives_mean_of_values_and_first_positions():
    q, k, v, kv = make(1, 2, 1, 64, 12)
    q[:] = 0
    out, idx, _ = oracle.select_attn(kv, q, 9)
    mean_v = bf16_val(v)[0, :, 0].mean(axis=0)
    np.testing.assert_allclose(out[0, 0], mean_v, atol=1e-6)
    np.testing.assert_allclose(out[0, 1], mean_v, atol=1e-6)
    assert idx[0, 0].tolist() == list(range(9))


def test_single_token_returns_its_value():
    q, k, v, kv = make(1, 2, 2, 1, 13)
    out = oracle.full_attn(kv, q)
    np.testing.assert_array_equal(out[0], bf16_val(v)[0, 0].astype(np.float32))


def test_dominant_key_returns_its_value_row():
    q, k, v, kv = make(1, 1, 1, 128, 14)
    kf = bf16_val(k)
    kf[0, 77, 0] = 8.0 * bf16_val(q)[0, 0]
    kv.k = bf16_bits(kf).reshape(-1)
    out, idx, _ = oracle.select_attn(kv, q, 4)
    assert 77 in idx[0, 0].tolist()
    np.testing.assert_allclose(out[0, 0], bf16_val(v)[0, 77, 0], atol=1e-6)


def test_sparse_uses_only_listed_rows_and_renormalises():
    q, k, v, kv = make(1, 2, 2, 90, 15)
    idx = np.full((1, 2, 6), -1, np.int32)
    idx[0, 0, :4] = [3, 17, 18, 80]
    idx[0, 1, :5] = [0, 1, 2, 88, 89]
    sp = oracle.sparse_attn(kv, q, idx)
    ref = eq1_numpy(q, k, v, [90], idx=[[np.array([3, 17, 18, 80]), np.array([0, 1, 2, 88, 89])]])
    np.testing.assert_allclose(sp, ref, atol=2e-7)
    # a repeated entry counts twice; order does not matter
    idx2 = np.full((1, 2, 6), -1, np.int32)
    idx2[0, 0, :5] = [80, 3, 3, 18, 17]
    idx2[0, 1, :5] = [89, 88, 2, 1, 0]
    sp2 = oracle.sparse_attn(kv, q, idx2)
    ref2 = eq1_numpy(q, k, v, [90], idx=[[np.array([80, 3, 3, 18, 17]), np.array([0, 1, 2, 88, 89])]])
    np.testing.assert_allclose(sp2, ref2, atol=2e-7)
    # idx_count limits how many entries are read
    sp3 = oracle.sparse_attn(kv, q, idx, np.array([2], np.int32))
    ref3 = eq1_numpy(q, k, v, [90], idx=[[np.array([3, 17]), np.array([0, 1])]])
    np.testing.assert_allclose(sp3, ref3, atol=2e-7)


# ---- P8: invariances --------------------------------------------------------
def test_permuting_positions_permutes_indices_only():
    q, k, v, kv = make(1, 2, 2, 120, 16)
    out, idx, _ = oracle.select_attn(kv, q, 20)
    perm = np.random.default_rng(1).permutation(120)          # new position of old j is perm[j]
    k2, v2 = np.empty_like(k), np.empty_like(v)
    k2[0, perm] = k[0]
    v2[0, perm] = v[0]
    kv2 = oracle.KV(k=k2.reshape(-1), v=v2.reshape(-1), batch=1, num_q_heads=2, num_kv_heads=2,
                    head_dim=D, ctx_lens=kv.ctx_lens, stride_b=kv.stride_b,
                    stride_pos=kv.stride_pos, stride_head=kv.stride_head)
    out2, idx2, _ = oracle.select_attn(kv2, q, 20)
    np.testing.assert_allclose(out2, out, atol=1e-6)
    for h in range(2):
        assert sorted(perm[idx[0, h]].tolist()) == idx2[0, h].tolist()


def test_constant_logit_shift_changes_nothing():
    # adding to every key a vector u orthogonal to nothing in particular but with
    # the same q.u for all positions shifts every logit equally
    r = np.random.default_rng(17)
    q, k, v, kv = make(1, 1, 1, 80, 17)
    qf = bf16_val(q)[0, 0]
    u = np.zeros(D)
    u[0] = 4.0 if qf[0] != 0 else 0.0          # exactly representable shift along one axis
    kf = bf16_val(k)
    kf[..., 0] = np.round(kf[..., 0] * 4) / 4   # keep k + u exactly representable in bf16
    k1 = bf16_bits(kf)
    k2 = bf16_bits(kf + u)
    assert np.array_equal(bf16_val(k2), kf + u)
    outs = []
    for kk in (k1, k2):
        kvx = oracle.KV(k=kk.reshape(-1), v=v.reshape(-1), batch=1, num_q_heads=1, num_kv_heads=1,
                        head_dim=D, ctx_lens=kv.ctx_lens, stride_b=kv.stride_b,
                        stride_pos=kv.stride_pos, stride_head=kv.stride_head)
        outs.append(oracle.select_attn(kvx, q, 10))
    np.testing.assert_allclose(outs[0][0], outs[1][0], atol=1e-5)
    assert outs[0][1].tolist() == outs[1][1].tolist()


# ---- P9: GQA equals MHA on a head-repeated cache ----------------------------
def test_gqa_equals_mha_with_repeated_kv_heads():
    B, Hq, Hkv, N = 2, 8, 2, 70
    q, k, v, kv = make(B, Hq, Hkv, N, 18, lens=[70, 33])
    G = Hq // Hkv
    k_rep = np.repeat(k, G, axis=2)
    v_rep = np.repeat(v, G, axis=2)
    kv_mha = oracle.KV(k=k_rep.reshape(-1), v=v_rep.reshape(-1), batch=B, num_q_heads=Hq,
                       num_kv_heads=Hq, head_dim=D, ctx_lens=kv.ctx_lens, stride_b=N * Hq * D,
                       stride_pos=Hq * D, stride_head=D)
    a = oracle.select_attn(kv, q, 12)
    b = oracle.select_attn(kv_mha, q, 12)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    assert np.array_equal(oracle.sparse_attn(kv, q, a[1], a[2]),
                          oracle.sparse_attn(kv_mha, q, b[1], b[2]))


# ---- P10: paged equals contiguous -------------------------------------------
def test_paged_equals_contiguous():
    B, Hq, Hkv, N, PS = 2, 4, 2, 75, 16
    lens = [75, 40]
    q, k, v, kv = make(B, Hq, Hkv, N, 19, lens=lens)
    pages_per = [(n + PS - 1) // PS for n in lens]
    total = sum(pages_per) + 3
    perm = np.random.default_rng(2).permutation(total)
    pt = np.zeros((B, max(pages_per)), np.int32)
    pool_k = np.zeros((total, PS, Hkv, D), np.uint16)
    pool_v = np.zeros((total, PS, Hkv, D), np.uint16)
    at = 0
    for b in range(B):
        for lp in range(pages_per[b]):
            phys = perm[at]; at += 1
            pt[b, lp] = phys
            lo, hi = lp * PS, min(lens[b], lp * PS + PS)
            pool_k[phys, : hi - lo] = k[b, lo:hi]
            pool_v[phys, : hi - lo] = v[b, lo:hi]
    kvp = oracle.KV(k=pool_k.reshape(-1), v=pool_v.reshape(-1), batch=B, num_q_heads=Hq,
                    num_kv_heads=Hkv, head_dim=D, ctx_lens=np.asarray(lens, np.int32),
                    stride_pos=Hkv * D, stride_head=D, stride_page=PS * Hkv * D,
                    page_table=pt, page_size=PS)
    a = oracle.select_attn(kv, q, 21)
    b = oracle.select_attn(kvp, q, 21)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    assert np.array_equal(oracle.sparse_attn(kv, q, a[1], a[2]),
                          oracle.sparse_attn(kvp, q, b[1], b[2]))


# ---- index-head granularities (aggregated ranking) ---------------------------
def test_aggregated_granularity_ranks_by_summed_logits():
    q, k, v, kv = make(1, 8, 2, 200, 20)
    _, _, _, sc = oracle.select_attn(kv, q, 16, want_scores=True)
    _, idx_kv, _ = oracle.select_attn(kv, q, 16, num_index_heads=2)
    _, idx_sh, _ = oracle.select_attn(kv, q, 16, num_index_heads=1)
    for g in range(2):
        agg = sc[0, 4 * g: 4 * g + 4].astype(np.float64).sum(axis=0)
        assert idx_kv[0, g].tolist() == brute_topk(agg.astype(np.float32), 16)
    agg = sc[0].astype(np.float64).sum(axis=0)
    assert idx_sh[0, 0].tolist() == brute_topk(agg.astype(np.float32), 16)
    # sparse attention maps query head h to index head h*Hi/Hq
    sp = oracle.sparse_attn(kv, q, idx_kv)
    ref = eq1_numpy(q, k, v, [200], idx=[[idx_kv[0, h // 4] for h in range(8)]])
    np.testing.assert_allclose(sp, ref, atol=2e-7)


# ---- P11: schedule and rho persistence ---------------------------------------
def _golden(name):
    rows = {}
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                key, val = line.split("=")
                rows[key.strip()] = val.strip()
    return rows


def test_layer_mix_matches_the_paper():
    g = _golden("layer_mix.txt")
    for L in (32, 64):
        s = oracle.schedule(L, 13).tolist()
        full, sel, sparse = (int(x) for x in g[f"layers_{L}"].split("+"))
        assert (s.count(0), s.count(1), s.count(2)) == (full, sel, sparse)
        assert s[0] == s[1] == oracle.LAYER_FULL
        assert s[2] == oracle.LAYER_SELECT and s[13] == oracle.LAYER_SELECT


def test_kv_cache_size_formula_matches_the_paper():
    g = _golden("kv_cache_size.txt")
    layers, heads, dim, seq = (int(g[x]) for x in ("layers", "kv_heads", "head_dim", "seq_len"))
    total = layers * heads * dim * seq * 2 * 2            # K and V, 2 bytes each
    assert total == int(g["gib"]) * 2 ** 30


def test_decode_step_keeps_rho_until_the_next_selection_layer():
    L, B, Hq, Hkv, N, k = 7, 1, 4, 2, 60, 9
    sched = [0, 0, 1, 2, 1, 2, 2]
    caches = [make(B, Hq, Hkv, N, 100 + i) for i in range(L)]
    qs = [c[0] for c in caches]
    kvs = [c[3] for c in caches]
    outs, idx, cnt = oracle.decode_step(sched, kvs, qs, k)
    _, rho2, c2 = oracle.select_attn(kvs[2], qs[2], k)
    _, rho4, c4 = oracle.select_attn(kvs[4], qs[4], k)
    assert not np.array_equal(rho2, rho4)
    assert np.array_equal(idx, rho4)
    assert np.array_equal(outs[0], oracle.full_attn(kvs[0], qs[0]))
    assert np.array_equal(outs[2], oracle.full_attn(kvs[2], qs[2]))     # selection layer output is full attention
    assert np.array_equal(outs[3], oracle.sparse_attn(kvs[3], qs[3], rho2, c2))
    assert np.array_equal(outs[5], oracle.sparse_attn(kvs[5], qs[5], rho4, c4))
    assert np.array_equal(outs[6], oracle.sparse_attn(kvs[6], qs[6], rho4, c4))
    with pytest.raises(ValueError):
        oracle.decode_step([0, 2], kvs[:2], qs[:2], k)


# ---- KV append (Algorithm 1, C.append) ------------------------------------
def test_append_writes_exactly_the_last_counted_row():
    """Independent numpy slice assignment on the [B, N, Hkv, D] arrays gives the same cache."""
    B, Hq, Hkv, N = 3, 4, 2, 37
    lens = [37, 1, 20]
    q, k, v, kv = make(B, Hq, Hkv, N, 41, lens=lens)
    r = np.random.default_rng(5)
    kn, vn = bf16_bits(r.standard_normal((B, Hkv, D))), bf16_bits(r.standard_normal((B, Hkv, D)))
    k_ref, v_ref = k.copy(), v.copy()
    for b in range(B):
        k_ref[b, lens[b] - 1] = kn[b]
        v_ref[b, lens[b] - 1] = vn[b]
    oracle.kv_append(kv, kn, vn)
    assert np.array_equal(kv.k.reshape(k.shape), k_ref)
    assert np.array_equal(kv.v.reshape(v.shape), v_ref)


def test_appended_dominant_key_returns_the_appended_value():
    """Closed form: a new key that dominates every logit makes Eq. 1 return the new value row."""
    B, Hq, Hkv, N = 2, 4, 2, 50
    lens = [50, 13]
    q, k, v, kv = make(B, Hq, Hkv, N, 43, lens=lens)
    qv = bf16_val(q)
    kn = np.zeros((B, Hkv, D))
    for b in range(B):
        for g in range(Hkv):
            kn[b, g] = 40.0 * (qv[b, 2 * g] + qv[b, 2 * g + 1])   # aligned with both heads of the group
    r = np.random.default_rng(6)
    kn, vn = bf16_bits(kn), bf16_bits(r.standard_normal((B, Hkv, D)))
    oracle.kv_append(kv, kn, vn)
    out = oracle.full_attn(kv, q)
    for b in range(B):
        for h in range(Hq):
            assert np.allclose(out[b, h], bf16_val(vn)[b, h // 2], atol=1e-6)


def test_append_through_a_page_table_equals_contiguous_append():
    B, Hq, Hkv, N, PS = 2, 2, 2, 40, 16
    lens = [40, 17]
    q, k, v, kv = make(B, Hq, Hkv, N, 47, lens=lens)
    r = np.random.default_rng(7)
    pages_per_seq = (N + PS - 1) // PS
    perm = r.permutation(B * pages_per_seq + 3)[: B * pages_per_seq].reshape(B, pages_per_seq)
    pool_k = np.zeros((B * pages_per_seq + 3, PS, Hkv, D), np.uint16)
    pool_v = np.zeros_like(pool_k)
    for b in range(B):
        for p in range(pages_per_seq):
            n = min(PS, N - p * PS)
            pool_k[perm[b, p], :n] = k[b, p * PS: p * PS + n]
            pool_v[perm[b, p], :n] = v[b, p * PS: p * PS + n]
    pkv = oracle.KV(k=pool_k.reshape(-1), v=pool_v.reshape(-1), batch=B, num_q_heads=Hq, num_kv_heads=Hkv,
                    head_dim=D, ctx_lens=np.asarray(lens, np.int32), stride_pos=Hkv * D, stride_head=D,
                    stride_page=PS * Hkv * D, page_table=perm.astype(np.int32), page_size=PS,
                    max_pages_per_seq=pages_per_seq)
    kn, vn = bf16_bits(r.standard_normal((B, Hkv, D))), bf16_bits(r.standard_normal((B, Hkv, D)))
    oracle.kv_append(kv, kn, vn)
    oracle.kv_append(pkv, kn, vn)
    assert np.array_equal(oracle.full_attn(kv, q), oracle.full_attn(pkv, q))
    for b in range(B):
        pos = lens[b] - 1
        assert np.array_equal(pkv.k.reshape(pool_k.shape)[perm[b, pos // PS], pos % PS], kn[b])


# ---- optional variant: sparse layers always attend the newest token ----------------------------
def test_newest_token_variant_closed_forms():
    """A dominant newest key returns the newest value row although rho excludes it; a list that already
    ends with the newest position is left alone (no double count)."""
    B, Hq, Hkv, N = 1, 2, 1, 60
    q, k, v, kv = make(B, Hq, Hkv, N, 53)
    qv = bf16_val(q)
    k[0, N - 1, 0] = bf16_bits(40.0 * (qv[0, 0] + qv[0, 1]))
    idx = np.array([[[3, 10, 20], [5, 6, N - 1]]], np.int32)
    cnt = np.array([3], np.int32)
    plain = oracle.sparse_attn(kv, q, idx, cnt)
    aug, cnt2 = oracle.with_newest(kv, idx, cnt)
    assert aug[0, 0].tolist() == [3, 10, 20, N - 1] and aug[0, 1].tolist() == [5, 6, N - 1, -1] and cnt2.tolist() == [4]
    out = oracle.sparse_attn(kv, q, aug, cnt2)
    assert np.allclose(out[0, 0], bf16_val(v)[0, N - 1, 0], atol=1e-6)      # head 0 now sees the dominant key
    assert np.array_equal(out[0, 1], plain[0, 1])                            # head 1 had it already


# ---- 8-bit (FP8 E4M3) caches: dequantise, then Eq. 1 ------------------------------------------------
def make_fp8(B, Hq, Hkv, N, seed, k_scale=None, v_scale=None, lens=None):
    """NHD cache of E4M3 codes drawn from torch's cast of N(0,1) draws, plus the values they stand for."""
    r = np.random.default_rng(seed)
    q = bf16_bits(r.standard_normal((B, Hq, D)))
    kt = torch.from_numpy(r.standard_normal((B, N, Hkv, D)).astype(np.float32)).to(torch.float8_e4m3fn)
    vt = torch.from_numpy(r.standard_normal((B, N, Hkv, D)).astype(np.float32)).to(torch.float8_e4m3fn)
    kc, vc = kt.view(torch.uint8).numpy().copy(), vt.view(torch.uint8).numpy().copy()
    lens = np.full(B, N, np.int32) if lens is None else np.asarray(lens, np.int32)
    kv = oracle.KV(k=kc.reshape(-1), v=vc.reshape(-1), batch=B, num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D,
                   ctx_lens=lens, stride_b=N * Hkv * D, stride_pos=Hkv * D, stride_head=D,
                   kv_dtype=oracle.KV_FP8_E4M3, k_scale=k_scale, v_scale=v_scale)
    return q, kt.float().numpy(), vt.float().numpy(), kv      # torch's own decoding of the codes


def test_e4m3_decoder_matches_torch_and_the_format_definition():
    """All 256 codes against torch.float8_e4m3fn (an independent implementation), plus the landmarks of
    the format: largest finite value 448, smallest subnormal 2^-9, no infinities, two NaN codes."""
    codes = np.arange(256, dtype=np.uint8)
    mine = oracle.e4m3_decode(codes)
    ref = torch.from_numpy(codes).view(torch.float8_e4m3fn).float().numpy()
    assert np.array_equal(np.isnan(mine), np.isnan(ref)) and np.isnan(mine).sum() == 2
    assert np.array_equal(mine[~np.isnan(mine)], ref[~np.isnan(ref)])
    assert mine[0x7e] == 448.0 and mine[0xfe] == -448.0 and mine[0x01] == 2.0 ** -9 and mine[0x08] == 2.0 ** -6
    assert mine[0x38] == 1.0 and mine[0x00] == 0.0 and np.isfinite(mine[~np.isnan(mine)]).all()


def test_fp8_cache_with_unit_scales_equals_the_bf16_path_on_the_same_values():
    """Every E4M3 value is also a bf16 value, so a cache of codes with scale 1 and a bf16 cache holding the
    decoded values must give identical logits, outputs, token sets and sparse outputs, bit for bit."""
    B, Hq, Hkv, N, k = 2, 4, 2, 150, 20
    q, kf, vf, kv8 = make_fp8(B, Hq, Hkv, N, seed=5, lens=[150, 97])
    kv16 = oracle.KV(k=bf16_bits(kf).reshape(-1), v=bf16_bits(vf).reshape(-1), batch=B, num_q_heads=Hq,
                     num_kv_heads=Hkv, head_dim=D, ctx_lens=kv8.ctx_lens, stride_b=N * Hkv * D,
                     stride_pos=Hkv * D, stride_head=D)
    assert np.array_equal(bf16_val(bf16_bits(kf)), kf.astype(np.float64))          # representable indeed
    o8, i8, c8, s8 = oracle.select_attn(kv8, q, k, want_scores=True)
    o16, i16, c16, s16 = oracle.select_attn(kv16, q, k, want_scores=True)
    assert np.array_equal(s8, s16) and np.array_equal(o8, o16) and np.array_equal(i8, i16) and np.array_equal(c8, c16)
    assert np.array_equal(oracle.sparse_attn(kv8, q, i8, c8), oracle.sparse_attn(kv16, q, i16, c16))


def test_fp8_scales_are_per_kv_head_and_match_a_bf16_cache_of_the_scaled_values():
    """Power-of-two scales keep the dequantised values representable in bf16: the result must equal the
    bf16 path on those values bit for bit (each head with its own scale), and equal Eq. 1 in numpy."""
    B, Hq, Hkv, N = 1, 4, 2, 120
    ks, vs = np.array([0.5, 4.0], np.float32), np.array([2.0, 0.25], np.float32)
    q, kf, vf, kv8 = make_fp8(B, Hq, Hkv, N, seed=7, k_scale=ks, v_scale=vs)
    kd, vd = kf * ks[None, None, :, None], vf * vs[None, None, :, None]
    kv16 = oracle.KV(k=bf16_bits(kd).reshape(-1), v=bf16_bits(vd).reshape(-1), batch=B, num_q_heads=Hq,
                     num_kv_heads=Hkv, head_dim=D, ctx_lens=kv8.ctx_lens, stride_b=N * Hkv * D,
                     stride_pos=Hkv * D, stride_head=D)
    o8, s8 = oracle.full_attn(kv8, q, want_scores=True)
    o16, s16 = oracle.full_attn(kv16, q, want_scores=True)
    assert np.array_equal(s8, s16) and np.array_equal(o8, o16)
    ref = eq1_numpy(q, bf16_bits(kd), bf16_bits(vd), kv8.ctx_lens)
    assert np.abs(o8 - ref).max() < 1e-6
    # scales that are not powers of two: against numpy in float64 on decode * scale
    ks2, vs2 = np.array([0.3, 1.7], np.float32), np.array([0.9, 1.1], np.float32)
    kv8.k_scale, kv8.v_scale = ks2, vs2
    qf = bf16_val(q)
    o = oracle.full_attn(kv8, q)
    for h in range(Hq):
        g = h // 2
        a = (kf[0, :, g].astype(np.float64) * float(ks2[g])) @ qf[0, h] / np.sqrt(D)
        p = np.exp(a - a.max())
        want = (p / p.sum()) @ (vf[0, :, g].astype(np.float64) * float(vs2[g]))
        assert np.abs(o[0, h] - want).max() < 1e-6


def test_fp8_value_scale_is_linear_and_key_scale_acts_like_the_softmax_scale():
    B, Hq, Hkv, N = 1, 2, 1, 90
    q, kf, vf, kv = make_fp8(B, Hq, Hkv, N, seed=9)
    base, sc = oracle.full_attn(kv, q, want_scores=True)
    kv.v_scale = np.array([8.0], np.float32)
    assert np.array_equal(oracle.full_attn(kv, q), base * 8.0)
    kv.v_scale = None
    kv.k_scale = np.array([0.5], np.float32)
    half, sc_half = oracle.full_attn(kv, q, want_scores=True)
    assert np.array_equal(sc_half, sc * 0.5)
    kv.k_scale = None
    kv.sm_scale = 0.5 / np.sqrt(D)
    assert np.abs(oracle.full_attn(kv, q) - half).max() < 1e-6


def test_fp8_append_copies_codes_to_the_last_counted_row():
    B, Hq, Hkv, N = 2, 2, 2, 40
    q, kf, vf, kv = make_fp8(B, Hq, Hkv, N, seed=11, lens=[40, 13])
    before_k, before_v = kv.k.copy(), kv.v.copy()
    kn = np.arange(B * Hkv * D, dtype=np.uint8).reshape(B, Hkv, D) % 120
    vn = (kn + 3).astype(np.uint8)
    oracle.kv_append(kv, kn, vn)
    want_k, want_v = before_k.reshape(B, N, Hkv, D).copy(), before_v.reshape(B, N, Hkv, D).copy()
    want_k[0, 39], want_v[0, 39], want_k[1, 12], want_v[1, 12] = kn[0], vn[0], kn[1], vn[1]
    assert np.array_equal(kv.k.reshape(B, N, Hkv, D), want_k) and np.array_equal(kv.v.reshape(B, N, Hkv, D), want_v)
