/*
 * CPU oracle for the decode-step attention path of TidalDecode's Position
 * Persistent Sparse Attention (arxiv 2410.05076).
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT. It is a plain, slow,
 * deliberately unoptimised restatement of what the paper defines, used only
 * to check the CUDA library and to be timed beside it as a reported CPU
 * baseline. It shares no code, header, table or helper with the CUDA path and
 * must never be called from it.
 *
 * What it follows:
 *   - Eq. 1 (Section 3.1): per head  A = q K^T / sqrt(d),  H = softmax(A) V.
 *   - Algorithm 1: FullAttention over the whole cache C[:]; at a token
 *     selection layer additionally rho := argTopK(<q, K>, m); at every other
 *     layer SparseAttention over C[rho].
 *   - Section 3 / 3.1 prose: the inner product of the query with every cached
 *     key is what is ranked (softmax preserves the order), and a sparse layer
 *     attends only to the selected tokens.
 *
 * Arithmetic: bf16 inputs are widened exactly; every dot product, softmax sum
 * and weighted sum is accumulated in double in plain index order and rounded
 * to float once. There is no blocking, no online softmax, no split context and
 * no radix select: top-k is a full sort by (score descending, position
 * ascending).
 *
 * Parity pins (tests, CPU only): softmax weights sum to 1; full attention
 * equals an independent numpy/torch evaluation of Eq. 1; k >= N makes sparse
 * equal full bit for bit; top-k equals brute-force repeated arg-max and the
 * ranking by post-softmax probability; closed forms (q = 0 gives the mean of
 * V, N = 1 gives v_0, a dominant key returns its value row); permutation and
 * logit-shift invariances; GQA equals MHA on a head-repeated cache; paged
 * equals contiguous; the 2+2+28 / 2+2+60 layer mix of Section 4.3.
 * Parity unpinned: absolute attention outputs of the paper's trained models
 * on its datasets (the paper prints no numeric attention output).
 *
 * 8-bit caches (not in the paper, which assumes half precision; a reading of this
 * build): K and V may be stored as OCP FP8 E4M3 bytes with one float scale per KV
 * head for K and one for V. The oracle's definition is "dequantise, then Eq. 1":
 * every element is decode(byte) * scale[g], taken in double, and everything else
 * is unchanged. Pins: the decoder against torch.float8_e4m3fn for all 256 codes;
 * with power-of-two scales and values that bf16 also represents, every result
 * equals the bf16 path's on the dequantised cache bit for bit; scale linearity.
 */
#ifndef TIDAL_ORACLE_H
#define TIDAL_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* KV cache of ONE layer, host memory, bf16 bit patterns.
 * contiguous (paged == 0): element (b, pos, g, c) of K lives at
 *     k[b*stride_b + pos*stride_pos + g*stride_head + c]
 * paged (paged == 1): pos -> page = page_table[b*max_pages_per_seq + pos/page_size],
 *     slot = pos % page_size, element at
 *     k[page*stride_page + slot*stride_pos + g*stride_head + c]
 * V uses the same strides from its own base pointer. Strides count elements. */
typedef struct {
    int32_t batch, num_q_heads, num_kv_heads, head_dim;
    int32_t paged;
    const uint16_t *k, *v;
    int64_t stride_b, stride_pos, stride_head, stride_page;
    const int32_t *page_table;
    int32_t page_size, max_pages_per_seq;
    const int32_t *ctx_lens;   /* [batch]; the cache already holds the new token (Algorithm 1) */
    float sm_scale;            /* 0 => 1/sqrt(head_dim) */
    int32_t kv_dtype;          /* ORACLE_KV_BF16: k, v point to uint16 bf16 bits (as declared);
                                  ORACLE_KV_FP8_E4M3: they point to bytes, strides still count elements */
    const float *k_scale, *v_scale;   /* fp8 only: [num_kv_heads] each, NULL = 1 */
} oracle_kv_t;

enum { ORACLE_KV_BF16 = 0, ORACLE_KV_FP8_E4M3 = 1 };

/* Value of one OCP FP8 E4M3 code: sign, 4 exponent bits (bias 7), 3 mantissa bits; exponent 0 is
 * subnormal (m/8 * 2^-6); there are no infinities and S.1111.111 is NaN, so the largest finite
 * value is 448. */
float oracle_e4m3_decode(uint8_t code);

enum { ORACLE_LAYER_FULL = 0, ORACLE_LAYER_SELECT = 1, ORACLE_LAYER_SPARSE = 2 };

/* Scaled logits s[j] = (q_h . k_j) * sm_scale for j in [0, ctx_len) of one
 * (sequence, query head); Eq. 1's A for a single query row. */
void oracle_logits(const oracle_kv_t *kv, const uint16_t *q, int b, int h, float *s);

/* Softmax weights p[j]/l over s[0..n) (Eq. 1); exposed so a test can check
 * that they sum to one. */
void oracle_softmax_weights(const float *s, int n, double *w);

/* FullAttention(q, C[:]) of Algorithm 1 for all (b, h).
 * q: bf16 [B, Hq, d]; out: float [B, Hq, d];
 * scores_opt: NULL or float [B, Hq, score_stride], receives s. */
int oracle_full_attn(const oracle_kv_t *kv, const uint16_t *q, float *out,
                     float *scores_opt, int64_t score_stride);

/* argTopK of Algorithm 1 on one score row: the k' = min(k, n) positions with
 * the largest score, lower position first among equals; written ascending by
 * position into idx[0..k'), the rest of idx[0..k) set to -1. Returns k'. */
int oracle_topk(const float *s, int n, int k, int32_t *idx);

/* Token selection layer: full attention, then one token set per index head.
 * num_index_heads in {Hq, Hkv, 1}: with fewer index heads than query heads the
 * ranking score of an index head is the sum of its member heads' scaled
 * logits (a reading of this build; the paper defines the per-head case).
 * idx: int32 [B, Hi, k]; idx_count: NULL or int32 [B]. */
int oracle_select_attn(const oracle_kv_t *kv, const uint16_t *q, int k, int num_index_heads,
                       float *out, int32_t *idx, int32_t *idx_count,
                       float *scores_opt, int64_t score_stride);

/* SparseAttention(q, C[rho]) of Algorithm 1: Eq. 1 restricted to the listed
 * positions, softmax renormalised over them; negative entries are skipped,
 * repeated entries count once per occurrence. count = idx_count[b] if given,
 * else k. */
int oracle_sparse_attn(const oracle_kv_t *kv, const uint16_t *q, const int32_t *idx,
                       const int32_t *idx_count, int k, int num_index_heads, float *out);

/* One decode step of Algorithm 1 without projections and FFN: walk the layer
 * schedule, keep rho across layers, replace it at every selection layer.
 * Returns 0, or -1 if a sparse layer comes before any selection layer. */
int oracle_decode_step(int num_layers, const uint8_t *schedule, const oracle_kv_t *kv_per_layer,
                       const uint16_t *const *q_per_layer, float *const *out_per_layer,
                       int k, int num_index_heads, int32_t *idx, int32_t *idx_count);

/* C.append(k, v) of Algorithm 1 for one layer: the new token's key and value rows (bf16
 * [B, Hkv, d]; for an fp8 cache already-quantised bytes [B, Hkv, d]) are written at position
 * ctx_lens[b] - 1, the slot the lengths already count.
 * The cache arrays are written through the descriptor's (const) base pointers. */
void oracle_kv_append(const oracle_kv_t *kv, const uint16_t *k_new, const uint16_t *v_new);

/* Layer schedule of Sections 3 and 4.3: the first two layers full, layer 2 and
 * one middle layer (0-based `reselect_layer`) select, every other layer sparse. */
void oracle_schedule(int num_layers, int reselect_layer, uint8_t *schedule);

/* Threads the parallel loops over (sequence, head) will use. */
int oracle_num_threads(void);

#ifdef __cplusplus
}
#endif
#endif
