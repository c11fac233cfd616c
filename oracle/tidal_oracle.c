/*
 * CPU oracle (test infrastructure) for TidalDecode's decode-step attention
 * path. See tidal_oracle.h for what it follows and how it is pinned.
 * Plain C; the only parallelism is an OpenMP loop over (sequence, head).
 */
#include "tidal_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* bf16 is the upper half of an IEEE float: widening is exact. */
static float bf16_to_float(uint16_t bits) {
    uint32_t u = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

float oracle_e4m3_decode(uint8_t code) {
    int sign = code >> 7, e = (code >> 3) & 15, m = code & 7;
    double v;
    if (e == 15 && m == 7) return NAN;                        /* the only non-number; no infinities */
    if (e == 0) v = ldexp((double)m / 8.0, -6);               /* subnormal */
    else v = ldexp(1.0 + (double)m / 8.0, e - 7);
    return (float)(sign ? -v : v);
}

/* Element offset of row (b, pos, g) of K or V: C[pos] of Algorithm 1 for one KV head. */
static int64_t kv_row(const oracle_kv_t *kv, int b, int pos, int g) {
    if (kv->paged) {
        int64_t page = kv->page_table[(int64_t)b * kv->max_pages_per_seq + pos / kv->page_size];
        int64_t slot = pos % kv->page_size;
        return page * kv->stride_page + slot * kv->stride_pos + (int64_t)g * kv->stride_head;
    }
    return (int64_t)b * kv->stride_b + (int64_t)pos * kv->stride_pos + (int64_t)g * kv->stride_head;
}

/* The number stored at element `at` of K (which = 0) or V (which = 1) for KV head g: a bf16 widened
 * exactly, or an fp8 code decoded and multiplied by the head's scale. */
static double kv_value(const oracle_kv_t *kv, int which, int64_t at, int g) {
    const uint16_t *base = which ? kv->v : kv->k;
    if (kv->kv_dtype == ORACLE_KV_FP8_E4M3) {
        const float *scale = which ? kv->v_scale : kv->k_scale;
        double s = scale ? (double)scale[g] : 1.0;
        return (double)oracle_e4m3_decode(((const uint8_t *)base)[at]) * s;
    }
    return (double)bf16_to_float(base[at]);
}

static double scale_of(const oracle_kv_t *kv) {
    if (kv->sm_scale != 0.0f) return (double)kv->sm_scale;
    return 1.0 / sqrt((double)kv->head_dim);   /* the 1/sqrt(d) of Eq. 1 */
}

/* One entry of A = q K^T / sqrt(d) (Eq. 1) for query head h and position pos. */
static float logit_at(const oracle_kv_t *kv, const uint16_t *q, int b, int h, int pos) {
    int d = kv->head_dim;
    int g = h / (kv->num_q_heads / kv->num_kv_heads);
    const uint16_t *qh = q + ((int64_t)b * kv->num_q_heads + h) * d;
    int64_t kr = kv_row(kv, b, pos, g);
    double dot = 0.0;
    for (int c = 0; c < d; ++c) dot += (double)bf16_to_float(qh[c]) * kv_value(kv, 0, kr + c, g);
    return (float)(dot * scale_of(kv));
}

void oracle_logits(const oracle_kv_t *kv, const uint16_t *q, int b, int h, float *s) {
    int n = kv->ctx_lens[b];
    for (int j = 0; j < n; ++j) s[j] = logit_at(kv, q, b, h, j);
}

void oracle_softmax_weights(const float *s, int n, double *w) {
    float m = -INFINITY;
    for (int j = 0; j < n; ++j) if (s[j] > m) m = s[j];
    double l = 0.0;
    for (int j = 0; j < n; ++j) { w[j] = exp((double)s[j] - (double)m); l += w[j]; }
    for (int j = 0; j < n; ++j) w[j] /= l;
}

/* H = softmax(A) V (Eq. 1) over the positions pos[0..n), logits s[0..n). */
static void weighted_values(const oracle_kv_t *kv, int b, int g, const int32_t *pos, const float *s,
                            int n, float *o) {
    int d = kv->head_dim;
    double *acc = (double *)calloc((size_t)d, sizeof(double));
    float m = -INFINITY;
    for (int j = 0; j < n; ++j) if (s[j] > m) m = s[j];
    double l = 0.0;
    for (int j = 0; j < n; ++j) {
        double p = exp((double)s[j] - (double)m);
        l += p;
        int64_t vr = kv_row(kv, b, pos ? pos[j] : j, g);
        for (int c = 0; c < d; ++c) acc[c] += p * kv_value(kv, 1, vr + c, g);
    }
    for (int c = 0; c < d; ++c) o[c] = (n > 0) ? (float)(acc[c] / l) : 0.0f;
    free(acc);
}

int oracle_full_attn(const oracle_kv_t *kv, const uint16_t *q, float *out,
                     float *scores_opt, int64_t score_stride) {
    int B = kv->batch, Hq = kv->num_q_heads, d = kv->head_dim;
    int G = Hq / kv->num_kv_heads;
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < B * Hq; ++bh) {
        int b = bh / Hq, h = bh % Hq, n = kv->ctx_lens[b];
        float *s = (float *)malloc(sizeof(float) * (size_t)(n > 0 ? n : 1));
        oracle_logits(kv, q, b, h, s);
        weighted_values(kv, b, h / G, NULL, s, n, out + (int64_t)bh * d);
        if (scores_opt) memcpy(scores_opt + (int64_t)bh * score_stride, s, sizeof(float) * (size_t)n);
        free(s);
    }
    return 0;
}

typedef struct { float s; int32_t pos; } scored_t;

/* Total order: larger score first, then smaller position. */
static int by_score_desc_pos_asc(const void *a, const void *b) {
    const scored_t *x = (const scored_t *)a, *y = (const scored_t *)b;
    if (x->s > y->s) return -1;
    if (x->s < y->s) return 1;
    return (x->pos > y->pos) - (x->pos < y->pos);
}

static int by_int_asc(const void *a, const void *b) {
    int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

int oracle_topk(const float *s, int n, int k, int32_t *idx) {
    int kk = k < n ? k : n;
    if (kk < 0) kk = 0;
    scored_t *all = (scored_t *)malloc(sizeof(scored_t) * (size_t)(n > 0 ? n : 1));
    for (int j = 0; j < n; ++j) { all[j].s = s[j]; all[j].pos = j; }
    qsort(all, (size_t)n, sizeof(scored_t), by_score_desc_pos_asc);   /* full sort */
    for (int i = 0; i < kk; ++i) idx[i] = all[i].pos;
    qsort(idx, (size_t)kk, sizeof(int32_t), by_int_asc);
    for (int i = kk; i < k; ++i) idx[i] = -1;
    free(all);
    return kk;
}

int oracle_select_attn(const oracle_kv_t *kv, const uint16_t *q, int k, int num_index_heads,
                       float *out, int32_t *idx, int32_t *idx_count,
                       float *scores_opt, int64_t score_stride) {
    int B = kv->batch, Hq = kv->num_q_heads, Hi = num_index_heads;
    if (Hi <= 0 || Hq % Hi != 0 || k <= 0) return -1;
    int members = Hq / Hi;
    int nmax = 1;
    for (int b = 0; b < B; ++b) if (kv->ctx_lens[b] > nmax) nmax = kv->ctx_lens[b];
    float *sc = scores_opt;
    int64_t stride = score_stride;
    if (!sc) { stride = nmax; sc = (float *)malloc(sizeof(float) * (size_t)B * Hq * (size_t)stride); }
    oracle_full_attn(kv, q, out, sc, stride);            /* o = FullAttention(q, C[:]) */
#pragma omp parallel for schedule(dynamic, 1)
    for (int bi = 0; bi < B * Hi; ++bi) {                /* rho := argTopK(<q, K>, m) */
        int b = bi / Hi, hi = bi % Hi, n = kv->ctx_lens[b];
        int32_t *dst = idx + (int64_t)bi * k;
        if (members == 1) {
            oracle_topk(sc + ((int64_t)b * Hq + hi) * stride, n, k, dst);
        } else {
            float *agg = (float *)malloc(sizeof(float) * (size_t)(n > 0 ? n : 1));
            for (int j = 0; j < n; ++j) {
                double t = 0.0;
                for (int m = 0; m < members; ++m)
                    t += (double)sc[((int64_t)b * Hq + hi * members + m) * stride + j];
                agg[j] = (float)t;
            }
            oracle_topk(agg, n, k, dst);
            free(agg);
        }
    }
    if (idx_count)
        for (int b = 0; b < B; ++b) idx_count[b] = k < kv->ctx_lens[b] ? k : kv->ctx_lens[b];
    if (!scores_opt) free(sc);
    return 0;
}

int oracle_sparse_attn(const oracle_kv_t *kv, const uint16_t *q, const int32_t *idx,
                       const int32_t *idx_count, int k, int num_index_heads, float *out) {
    int B = kv->batch, Hq = kv->num_q_heads, d = kv->head_dim, Hi = num_index_heads;
    if (Hi <= 0 || Hq % Hi != 0 || k <= 0) return -1;
    int G = Hq / kv->num_kv_heads;
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < B * Hq; ++bh) {
        int b = bh / Hq, h = bh % Hq;
        int hi = (int)(((int64_t)h * Hi) / Hq);
        const int32_t *row = idx + ((int64_t)b * Hi + hi) * k;
        int cnt = idx_count ? idx_count[b] : k;
        if (cnt > k) cnt = k;
        int32_t *pos = (int32_t *)malloc(sizeof(int32_t) * (size_t)(k > 0 ? k : 1));
        float *s = (float *)malloc(sizeof(float) * (size_t)(k > 0 ? k : 1));
        int n = 0;
        for (int i = 0; i < cnt; ++i) {
            if (row[i] < 0 || row[i] >= kv->ctx_lens[b]) continue;   /* padding / not a cached token */
            pos[n] = row[i];
            s[n] = logit_at(kv, q, b, h, row[i]);
            ++n;
        }
        weighted_values(kv, b, h / G, pos, s, n, out + (int64_t)bh * d);
        free(pos);
        free(s);
    }
    return 0;
}

int oracle_decode_step(int num_layers, const uint8_t *schedule, const oracle_kv_t *kv_per_layer,
                       const uint16_t *const *q_per_layer, float *const *out_per_layer,
                       int k, int num_index_heads, int32_t *idx, int32_t *idx_count) {
    int have_rho = 0;                                    /* rho = [] */
    for (int i = 0; i < num_layers; ++i) {
        const oracle_kv_t *kv = &kv_per_layer[i];
        int rc = 0;
        if (schedule[i] == ORACLE_LAYER_FULL) {
            rc = oracle_full_attn(kv, q_per_layer[i], out_per_layer[i], NULL, 0);
        } else if (schedule[i] == ORACLE_LAYER_SELECT) {
            rc = oracle_select_attn(kv, q_per_layer[i], k, num_index_heads, out_per_layer[i],
                                    idx, idx_count, NULL, 0);
            have_rho = 1;
        } else {
            if (!have_rho) return -1;
            rc = oracle_sparse_attn(kv, q_per_layer[i], idx, idx_count, k, num_index_heads,
                                    out_per_layer[i]);
        }
        if (rc) return rc;
    }
    return 0;
}

void oracle_kv_append(const oracle_kv_t *kv, const uint16_t *k_new, const uint16_t *v_new) {
    int d = kv->head_dim;
    for (int b = 0; b < kv->batch; ++b) {
        int pos = kv->ctx_lens[b] - 1;
        if (pos < 0) continue;
        for (int g = 0; g < kv->num_kv_heads; ++g) {
            int64_t at = kv_row(kv, b, pos, g);
            int64_t from = ((int64_t)b * kv->num_kv_heads + g) * d;
            if (kv->kv_dtype == ORACLE_KV_FP8_E4M3) {
                uint8_t *kr = (uint8_t *)kv->k + at, *vr = (uint8_t *)kv->v + at;
                for (int c = 0; c < d; ++c) { kr[c] = ((const uint8_t *)k_new)[from + c]; vr[c] = ((const uint8_t *)v_new)[from + c]; }
            } else {
                uint16_t *kr = (uint16_t *)kv->k + at, *vr = (uint16_t *)kv->v + at;
                for (int c = 0; c < d; ++c) { kr[c] = k_new[from + c]; vr[c] = v_new[from + c]; }
            }
        }
    }
}

void oracle_schedule(int num_layers, int reselect_layer, uint8_t *schedule) {
    for (int i = 0; i < num_layers; ++i) {
        if (i < 2) schedule[i] = ORACLE_LAYER_FULL;
        else if (i == 2 || i == reselect_layer) schedule[i] = ORACLE_LAYER_SELECT;
        else schedule[i] = ORACLE_LAYER_SPARSE;
    }
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
