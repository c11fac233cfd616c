/*
 * libtidal — decode-step attention of TidalDecode's Position Persistent Sparse
 * Attention (arxiv 2410.05076) for NVIDIA B200 (sm_100a).
 *
 * The library covers the attention branch of the paper's Algorithm 1 for one
 * decode step: full attention over the whole KV cache (full-attention layers),
 * full attention that also ranks every cached token by its query-key inner
 * product and keeps the top k (token selection layers), and sparse attention
 * over only the positions kept by the last selection layer (all other
 * layers), and the cache update (the new token's key and value rows written
 * into the cache). Projections, position encodings and FFN are the caller's.
 *
 * Conventions shared by every call
 *   - All tensor pointers are DEVICE pointers unless a parameter says "host".
 *     The caller owns every buffer; the library owns only its context and the
 *     workspace inside it and keeps no reference to caller memory after the
 *     work it enqueued has run.
 *   - Calls enqueue work on the CUDA stream passed as `stream` (a cudaStream_t
 *     cast to void*, NULL = the legacy default stream) and return without
 *     waiting for it, except where stated.
 *   - Return value: TIDAL_OK or a negative tidal_status_t. Argument errors are
 *     detected on the host before anything is enqueued. Nothing throws or
 *     aborts across this boundary. Problems only the device can see (a token
 *     index outside the cache, a page id outside the pool) make the kernel skip
 *     that element and set a sticky status word read by tidal_device_status().
 *   - q is bf16 [batch, num_q_heads, head_dim] contiguous; outputs are fp32
 *     [batch, num_q_heads, head_dim] contiguous. Arithmetic: bf16 inputs,
 *     fp32 accumulation.
 *   - A context holds scratch memory and counters that its calls share: use it
 *     from one host thread and on one stream at a time (work of consecutive
 *     calls may overlap on that stream; calls on two streams need two contexts).
 *   - There is no CPU path: on a machine without a usable GPU tidal_create()
 *     fails with TIDAL_ERR_CUDA.
 */
#ifndef TIDAL_H
#define TIDAL_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tidal_ctx tidal_ctx_t;     /* opaque: device, workspace, kernel attributes */
typedef int32_t tidal_status_t;

enum {
    TIDAL_OK = 0,
    TIDAL_ERR_INVALID = -1,       /* bad argument (NULL pointer, k <= 0, misaligned stride, ...) */
    TIDAL_ERR_UNSUPPORTED = -2,   /* valid request outside what is built (head_dim != 128, ...) */
    TIDAL_ERR_NOMEM = -3,         /* workspace allocation failed */
    TIDAL_ERR_CUDA = -4,          /* a CUDA runtime call failed */
    TIDAL_ERR_TIMEOUT = -5,       /* reserved: a bounded device-side wait expired (no kernel waits on another) */
    TIDAL_ERR_INDEX = -6,         /* device saw a token index or page id out of range */
    TIDAL_ERR_TOO_LARGE = -7,     /* tidal_sparse_attn_noalloc only: problem exceeds its fixed scratch */
    TIDAL_ERR_INTERNAL = -8       /* a kernel found the host's launch plan inconsistent: a bug, results invalid */
};

enum { TIDAL_KV_CONTIG = 0, TIDAL_KV_PAGED = 1 };

/* Granularity of the selected token set (number of index heads Hi).
 * PER_QHEAD is the paper's definition (Eq. 1 and Section 3.1 are per attention
 * head): Hi = num_q_heads. The other two rank by the sum of the member heads'
 * scaled logits: PER_KVHEAD has Hi = num_kv_heads, SHARED has Hi = 1. */
enum { TIDAL_SEL_PER_QHEAD = 0, TIDAL_SEL_PER_KVHEAD = 1, TIDAL_SEL_SHARED = 2 };

/* Layer types of Algorithm 1 / Figure 2. */
enum { TIDAL_LAYER_FULL = 0, TIDAL_LAYER_SELECT = 1, TIDAL_LAYER_SPARSE = 2 };

/* KV cache of one layer. Strides count bf16 ELEMENTS and must be multiples of
 * 8 (16 bytes); k and v must be 16-byte aligned; a row (head_dim elements of
 * one position and KV head) is contiguous.
 *   contiguous: K[b, pos, g, c] at k + b*stride_b + pos*stride_pos + g*stride_head + c
 *   paged:      page = page_table[b*max_pages_per_seq + pos/page_size], slot = pos%page_size,
 *               K[b, pos, g, c] at k + page*stride_page + slot*stride_pos + g*stride_head + c
 * V uses the same strides from `v`. The cache already contains the token being
 * decoded (Algorithm 1 appends before attention), so ctx_lens[b] >= 1 counts it. */
typedef struct {
    int32_t batch, num_q_heads, num_kv_heads, head_dim;   /* head_dim == 128; Hq % Hkv == 0; Hq/Hkv <= 8 */
    int32_t kv_layout;                                    /* TIDAL_KV_CONTIG or TIDAL_KV_PAGED */
    const void *k, *v;                                    /* device, bf16 */
    int64_t stride_b, stride_pos, stride_head, stride_page;
    const int32_t *page_table;      /* device int32 [batch, max_pages_per_seq]; paged only */
    int32_t page_size;              /* 16 (paged only) */
    int32_t max_pages_per_seq;
    int32_t num_pages;              /* physical pages in the pool; page ids are checked against it */
    const int32_t *ctx_lens;        /* device int32 [batch] */
    int32_t max_ctx_len;            /* host upper bound of ctx_lens; 1 .. 262144 */
    float sm_scale;                 /* 0 => 1/sqrt(head_dim), the scale of Eq. 1 */
    int32_t kv_dtype;               /* TIDAL_KV_BF16 (0) or TIDAL_KV_FP8_E4M3 */
    const float *k_scale, *v_scale; /* FP8 only: device float [num_kv_heads] each, NULL = 1 */
} tidal_kv_t;

/* Element type of the cache. The paper assumes half precision; TIDAL_KV_FP8_E4M3 is this library's
 * 8-bit variant: k and v hold OCP FP8 E4M3 codes (no infinities, largest value 448) and element
 * (b, pos, g, c) stands for decode(code) * k_scale[g] (v_scale[g] for V); attention is Eq. 1 on those
 * values. Strides still count elements, i.e. bytes, and must be multiples of 16; a row is 128
 * contiguous bytes. The query stays bf16 (it is converted to fp16 inside the kernels, exactly for
 * magnitudes between 6.1e-5 and 65504). Not available: tidal_set_attend_newest,
 * tidal_sparse_attn_noalloc, tidal_set_select_margin (ignored). */
enum { TIDAL_KV_BF16 = 0, TIDAL_KV_FP8_E4M3 = 1 };

/* Create a context on CUDA device `device`. workspace_bytes preallocates that much scratch
 * (0 = none). Whatever a later call needs beyond what the context holds is allocated inside that
 * call (which then also synchronises the device): use tidal_reserve() to do all of it up front. */
tidal_status_t tidal_create(tidal_ctx_t **ctx, int device, size_t workspace_bytes);
tidal_status_t tidal_destroy(tidal_ctx_t *ctx);

/* Allocates, now, everything later calls with this cache shape (batch, heads, max_ctx_len) and a
 * budget up to k will need: the scratch workspace and the small block of counters and histograms
 * that scale with batch * num_q_heads. num_layers_host is the layer count of later
 * tidal_decode_step_host calls (0 if that call is not used). After it, calls with shapes no larger
 * allocate nothing and do not synchronise, so they can be captured into a CUDA graph from the first
 * one on. May allocate and synchronise itself; call it outside any capture. */
tidal_status_t tidal_reserve(tidal_ctx_t *ctx, const tidal_kv_t *kv, int32_t k, int32_t num_layers_host);

/* Workspace a call with this cache shape and budget k needs (split-context
 * partial results, the score buffer of a selection layer, top-k histograms). */
size_t tidal_workspace_bytes(const tidal_kv_t *kv, int32_t k);

/* C.append(k, v) of Algorithm 1 for one layer: writes the new token's key and value rows
 * (k_new, v_new: device bf16 [batch, num_kv_heads, head_dim], contiguous, 16-byte aligned; for an
 * FP8 cache the rows are E4M3 codes already, quantised by the caller with the cache's scales) into
 * the cache at position ctx_lens[b] - 1, the slot that the lengths already count, through the
 * layout described by `kv` (contiguous or paged). The cache memory behind kv->k / kv->v is
 * WRITTEN by this call although the descriptor declares it const. Sequences with
 * ctx_lens[b] < 1 or > max_ctx_len and page ids outside the pool are skipped (the latter is
 * reported by tidal_device_status). q and k are expected position-encoded already: rotary or
 * other position encodings are the caller's. */
tidal_status_t tidal_kv_append(tidal_ctx_t *ctx, const tidal_kv_t *kv, const void *k_new,
                               const void *v_new, void *stream);

/* FullAttention(q, C[:]) of Algorithm 1, Eq. 1 per head:
 *   out[b,h,:] = softmax_j(q[b,h,:] . K[b,j,g,:] * sm_scale) V[b,j,g,:],  j < ctx_lens[b], g = h / (Hq/Hkv).
 * The single decode query sees every cached token (no mask). */
tidal_status_t tidal_full_attn(tidal_ctx_t *ctx, const tidal_kv_t *kv, const void *q,
                               float *out, void *stream);

/* Token selection layer of Algorithm 1 (Section 3: the inner products are
 * stored during full attention, then the k tokens with the highest values are
 * kept): out as tidal_full_attn, and for every (sequence, index head) the
 * k' = min(k, ctx_lens[b]) positions with the largest scaled logit, equal
 * logits resolved toward the lower position.
 *   idx       int32 [batch, Hi, k]: the positions in ascending order, padded with -1.
 *   idx_count int32 [batch] or NULL: receives k'.
 *   scores_opt float [batch, Hq, max_ctx_len] or NULL: receives the scaled
 *             logits q.k*sm_scale (entries at and beyond ctx_lens[b] are unspecified);
 *             with NULL they live in the workspace (with fewer index heads than
 *             query heads the workspace then holds only the per-KV-head sums). */
tidal_status_t tidal_select_attn(tidal_ctx_t *ctx, const tidal_kv_t *kv, const void *q,
                                 int32_t k, int32_t granularity, float *out, int32_t *idx,
                                 int32_t *idx_count, float *scores_opt, void *stream);

/* SparseAttention(q, C[rho]) of Algorithm 1: Eq. 1 restricted to the positions
 * listed for the query head's index head hi = h * Hi / Hq, softmax renormalised
 * over them. -1 is padding and skipped; any other entry outside
 * [0, ctx_lens[b]) is skipped too and reported as TIDAL_ERR_INDEX by
 * tidal_device_status(); a repeated
 * entry counts once per occurrence. Only the first idx_count[b] entries are
 * read when idx_count is given, else k. A head with no valid entry gets zeros.
 * num_index_heads must be Hq, Hkv or 1. */
tidal_status_t tidal_sparse_attn(tidal_ctx_t *ctx, const tidal_kv_t *kv, const void *q,
                                 const int32_t *idx, const int32_t *idx_count, int32_t k,
                                 int32_t num_index_heads, float *out, void *stream);

/* One decode step's attention for all layers (the loop of Algorithm 1):
 * schedule[i] (host, TIDAL_LAYER_*) picks the call for layer i; the token set
 * rho lives in idx/idx_count, is written by every selection layer and read by
 * the sparse layers after it. kv_per_layer (host array of descriptors),
 * q_per_layer and out_per_layer (host arrays of device pointers) have
 * num_layers entries. A sparse layer before the first selection layer is
 * TIDAL_ERR_INVALID. Everything is enqueued without host waits and is complete, in
 * stream order, when the work enqueued on `stream` is: a selection layer may run part
 * of its work (its value pass) on a second stream that the context owns, forked from
 * and joined back into `stream` with events, also inside a stream capture. */
tidal_status_t tidal_decode_step(tidal_ctx_t *ctx, int32_t num_layers, const uint8_t *schedule,
                                 const tidal_kv_t *kv_per_layer, const void *const *q_per_layer,
                                 float *const *out_per_layer, int32_t k, int32_t granularity,
                                 int32_t *idx, int32_t *idx_count, void *stream);

/* Optional deviation from Algorithm 1 (off by default): with enabled != 0 every later sparse layer on
 * this context also attends the newest token, position ctx_lens[b] - 1, whether or not it was
 * selected. A list that already ends with that position (lists from tidal_select_attn are ascending) is
 * left as it is, so the token never counts twice. tidal_sparse_attn then needs idx_count. */
tidal_status_t tidal_set_attend_newest(tidal_ctx_t *ctx, int32_t enabled);

/* Output type of every later call on this context: TIDAL_OUT_F32 (default; `out` arguments are
 * float*) or TIDAL_OUT_BF16 (the same `out` arguments then point to bf16 [batch, Hq, head_dim],
 * each value the fp32 result rounded to nearest even; out_host of tidal_decode_step_host likewise).
 * tidal_sparse_attn_noalloc always writes fp32. */
enum { TIDAL_OUT_F32 = 0, TIDAL_OUT_BF16 = 1 };
tidal_status_t tidal_set_output_dtype(tidal_ctx_t *ctx, int32_t dtype);

/* Step graphs. When `stream` is an ordinary stream (not the legacy or per-thread default, and not
 * being captured by the caller), tidal_decode_step and tidal_decode_step_host record their launches
 * once as a CUDA graph and replay it for as long as every argument (schedule, descriptors, pointers,
 * k, granularity) stays byte-for-byte the same: lengths and page tables live in device memory and
 * may change freely. Up to 16 recordings are kept per context. On by default; enabled = 0 turns it
 * off and frees the recordings. */
tidal_status_t tidal_set_graphs(tidal_ctx_t *ctx, int32_t enabled);

/* Optional candidate compaction inside a selection layer's attention kernel (off by default: on B200
 * it measured slower than ranking all scores from the fused histogram, about 122 against 104
 * microseconds per selection layer at 128K context; it is kept as a tested alternative). Applies to one sequence, one token set per query head, groups of at
 * most four and k <= max_ctx_len / 6; other cases always rank all scores. With margin > 0, every CTA
 * of the attention kernel estimates, from the first few hundred scores it sees, a provisional
 * threshold that about margin * k / N of a head's scores should reach, and lists the scores at or
 * above it; the top-k then runs on that list alone. The result is exact whatever the margin: the list
 * is used only if it provably contains the k best (its k-th best score is not below the largest
 * threshold any CTA used); otherwise all scores are ranked by the same kernel, which is slower.
 * margin: 0 = off (default); 3 is a sensible value; values below 1 make the shortcut fail on purpose
 * (that is how the tests reach the exact fallback). */
tidal_status_t tidal_set_select_margin(tidal_ctx_t *ctx, float margin);

/* Overlap between the layers of a step (on by default). tidal_decode_step receives every layer's
 * query, lengths, page table and cache up front, so all of them are complete, in stream order, before
 * the call. With enabled != 0 a full-attention or sparse layer therefore streams its whole input while
 * the layer before it is still finishing and waits for that layer only before it writes scratch memory
 * and its output (a sparse layer right after a selection layer always waits first: the top-k writes its
 * index list). With enabled = 0 a layer only prefetches cache rows ahead of the previous layer's end and
 * reads its query afterwards, as a caller would need whose queries are produced between the layers.
 * With the overlap on, a selection layer with per-head sets and fp32 outputs (one sequence, or a batch over a
 * 16-bit cache)
 * also runs as two passes: keys first (logits, their histogram, the largest logit per head), then the
 * top-k on `stream` while the values are streamed on the context's second stream beside it and beside
 * the sparse layers that follow.
 * The single-layer calls always wait for all earlier work in the stream before reading anything. */
tidal_status_t tidal_set_layer_overlap(tidal_ctx_t *ctx, int32_t enabled);

/* The step of Algorithm 1 including its cache update: layer i's new key and value rows
 * (k_new_per_layer[i], v_new_per_layer[i]: device bf16 [batch, Hkv, head_dim], as for
 * tidal_kv_append) are written at position ctx_lens[b] - 1 of layer i's cache, then the layers
 * run as in tidal_decode_step. All layers' rows are written by one launch ahead of the first
 * layer, which is equivalent because every layer's inputs are given up front. The caches are
 * WRITTEN although the descriptors declare them const. */
tidal_status_t tidal_decode_step_append(tidal_ctx_t *ctx, int32_t num_layers, const uint8_t *schedule,
                                        const tidal_kv_t *kv_per_layer, const void *const *q_per_layer,
                                        const void *const *k_new_per_layer,
                                        const void *const *v_new_per_layer, float *const *out_per_layer,
                                        int32_t k, int32_t granularity, int32_t *idx,
                                        int32_t *idx_count, void *stream);

/* The same step for a caller whose queries and outputs live in HOST memory
 * (pinned for full speed): q_host is bf16 [num_layers, batch, Hq, head_dim],
 * out_host fp32 of the same shape. Runs tidal_decode_step with idx/idx_count in
 * the workspace and WAITS for the stream. Page-locked buffers are read and written
 * by the kernels directly over the bus (q_host 16-byte aligned); pageable ones are
 * copied to and from a staging area on the device. The KV cache stays resident on
 * the device. */
tidal_status_t tidal_decode_step_host(tidal_ctx_t *ctx, int32_t num_layers, const uint8_t *schedule,
                                      const tidal_kv_t *kv_per_layer, const void *q_host,
                                      float *out_host, int32_t k, int32_t granularity, void *stream);

/* tidal_sparse_attn for callers that are not allowed to allocate device memory. (The paper has
 * no counterpart to this call; it exists for integration, not for the method.) Such callers are,
 * for example, a serving process that handed all device memory to its own pool at start-up, so
 * that a later cudaMalloc fails or is forbidden by policy; code running inside a latency-critical
 * loop where the implicit synchronisation of cudaMalloc/cudaFree is unacceptable; or a plug-in
 * that is called with the device already in a state where allocation is not permitted. The other
 * entry points need a context whose workspace is allocated (and may grow) behind the caller's back.
 *
 * This one takes no context and never calls cudaMalloc, cudaFree or any allocating routine: its
 * scratch (split partial results, arrival counters, pool cursors) is one static device array of
 * about 2.06 MiB (4096 partial rows) that every GPU loading the library holds until the process
 * exits. It runs on the CURRENT device. Arguments and results are those of tidal_sparse_attn,
 * with these differences:
 *   - batch * num_q_heads must not exceed 4096, otherwise TIDAL_ERR_TOO_LARGE (nothing enqueued);
 *   - an index entry >= ctx_lens[b] or a page id outside the pool is skipped but cannot be
 *     reported (there is no context to hold the status word);
 *   - all calls on a device share the one scratch array: two calls whose kernels can overlap on
 *     the GPU (different streams, no dependency) race; keep them on one stream or order them;
 *   - the first call on each device also does the one-time set-up (it resolves the array's device
 *     address and prepares the kernel, still without allocating): that first call should come
 *     before any stream capture. */
tidal_status_t tidal_sparse_attn_noalloc(const tidal_kv_t *kv, const void *q, const int32_t *idx,
                                         const int32_t *idx_count, int32_t k, int32_t num_index_heads,
                                         float *out, void *stream);

/* Waits for `stream`, then returns and clears the sticky device status word: TIDAL_OK,
 * TIDAL_ERR_INDEX, TIDAL_ERR_INTERNAL, or TIDAL_ERR_CUDA if the stream reports an error. */
tidal_status_t tidal_device_status(tidal_ctx_t *ctx, void *stream);

/* Kernels launched through this context since it was created. */
int64_t tidal_launch_count(const tidal_ctx_t *ctx);

const char *tidal_strerror(tidal_status_t status);

#ifdef __cplusplus
}
#endif
#endif
