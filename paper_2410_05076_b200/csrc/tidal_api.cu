// C-ABI of libtidal: argument checking, workspace, launch planning.
// Every step of the attention path runs in the kernels of attn_kernels.cuh and
// topk_kernels.cuh; nothing here computes on the host and there is no CPU path.
#include "../../include/tidal.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <vector>
#include <new>

#include "attn_kernels.cuh"
#include "split_select_kernels.cuh"
#include "topk_kernels.cuh"

using namespace tidal;

namespace {

constexpr int MAX_CTX = 262144;
constexpr int GRID_MAX = 320;            // persistent CTAs per launch never exceed this (2 per SM on 148 SMs)
constexpr int MIN_TILES_PER_CTA = 8;     // do not cut work finer than 128 positions per CTA
constexpr int MAX_GROUP = 8;            // query heads per KV head that fit the 8 MMA columns

// Streaming (full / selection) and gather (sparse) launch shapes.
constexpr int DENSE_NW = 8, DENSE_STAGES = 3;
constexpr int SPARSE_NW = 4, SPARSE_STAGES = 3;
// 8-bit caches: ring slots are half as large, so twice as many keep the same bytes in flight.
constexpr int DENSE_STAGES8 = 4, SPARSE_STAGES8 = 4;
constexpr int SPARSE_NW8 = 6;
constexpr int DENSE_NW8 = 12;
constexpr size_t HIST_SMEM = HIST_SMEM_WORDS * sizeof(uint32_t);

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }


}  // namespace

struct tidal_ctx {
    int device = 0;
    int sm_count = 0;
    int dense_slots = 0, sparse_slots = 0;     // resident CTAs on the whole GPU
    void* ws = nullptr;                         // scratch: contents are garbage between calls
    size_t ws_bytes = 0;
    // Words that must read zero when a kernel starts (split counters, top-k cursors, arrival
    // counters and histograms). The kernels restore the zeros themselves, so this lives apart
    // from the scratch workspace, whose layout changes with the problem shape.
    void* state = nullptr;
    int state_rows = 0;                         // capacity in (sequence, head) rows
    int* status = nullptr;                      // device word, sticky
    int out_bf16 = 0;                           // outputs are written as bf16 instead of fp32
    int attend_newest = 0;                      // sparse layers also attend the newest token (not in the paper)
    int cursor_set = 0;                         // which of the sets of pool cursors the last attention launch used
    float select_margin = 0.f;                  // > 0: selection layers compact candidates above a provisional threshold aimed at this multiple of k'/N
    // Split selection layers run their value pass on a stream of the context's own, beside the top-k and
    // the sparse layers that follow on the caller's stream; two events fork and join the streams.
    cudaStream_t side = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    int split_select = 1;
    int layer_overlap = 1;                      // layers of a step may stream their inputs while the layer before them finishes
    int64_t launches = 0;
    // Whole steps are recorded once as CUDA graphs (programmatic dependent launches included) and
    // replayed while every host-visible argument stays the same: one launch per step instead of one
    // per kernel. Keyed by the bytes of all arguments plus the workspace addresses they bake in.
    struct StepGraph {
        std::vector<unsigned char> key;
        cudaGraphExec_t exec = nullptr;
        int launches = 0;
        uint64_t last_use = 0;
    };
    std::vector<StepGraph> graphs;
    uint64_t graph_clock = 0;
    bool graphs_enabled = true;
    // The call before this one, byte for byte (arguments, the arrays they point to, the settings and the
    // workspace addresses): a step loop repeats it, and then validation, layout and key building are skipped.
    struct LastCall {
        std::vector<unsigned char> raw;
        cudaGraphExec_t exec = nullptr;
        int launches = 0;
    } last;
    std::vector<unsigned char> raw_scratch;
    cudaGraphExec_t ran_exec = nullptr;         // set by run_graphed: the graph it launched, if any
    int ran_launches = 0;
};

namespace {

struct WsLayout {
    size_t part_ml, part_o, scores, cand, bitmap, idx, idx_count, q_stage, out_stage, total;
    long long cand_stride, bitmap_stride;
    long long score_stride;
    int max_splits;
};

// Partial-result slots a (sequence, head) row can need: the CTAs of one launch are at most
// GRID_MAX, and an item of `tiles_max` tiles is cut into at most tiles/per_cta + 2 pieces where
// per_cta >= (one tile per item) * items / GRID_MAX.
int max_splits_for(const tidal_kv_t* kv) {
    const long long items = (long long)kv->batch * kv->num_kv_heads;
    const long long tiles_max = (kv->max_ctx_len + TILE - 1) / TILE;
    const long long bound = tiles_max * GRID_MAX / std::max(items, 1LL) + 2;
    return (int)std::max(1LL, std::min<long long>(GRID_MAX, bound));
}

// Persistent grid: every resident slot gets an equal share of the tiles, but no CTA is
// launched for fewer than MIN_TILES_PER_CTA tiles.
int grid_for(long long tiles_upper_bound, int slots) {
    const long long by_work = std::max(1LL, tiles_upper_bound / MIN_TILES_PER_CTA);
    return (int)std::max(1LL, std::min<long long>(std::min(slots, GRID_MAX), by_work));
}

// 2048 histogram bins per head while the group's columns fit the shared histogram, else 1024.
int hist_shift_for(const tidal_kv_t* kv) { return (kv->num_q_heads / kv->num_kv_heads) <= 4 ? 21 : 22; }

// One sequence: all items have the same length, so whole groups of CTAs can share an item's tiles.
int pooled_splits(const tidal_kv_t* kv, int items, int grid) {
    if (kv->batch != 1) return 0;
    const int S = grid / std::max(items, 1);
    return S >= 2 ? S : 0;
}

int hi_of(const tidal_kv_t* kv, int granularity) {
    switch (granularity) {
        case TIDAL_SEL_PER_QHEAD: return kv->num_q_heads;
        case TIDAL_SEL_PER_KVHEAD: return kv->num_kv_heads;
        case TIDAL_SEL_SHARED: return 1;
        default: return -1;
    }
}

tidal_status_t check_kv(const tidal_kv_t* kv) {
    if (!kv || !kv->k || !kv->v || !kv->ctx_lens) return TIDAL_ERR_INVALID;
    if (kv->batch <= 0 || kv->num_q_heads <= 0 || kv->num_kv_heads <= 0) return TIDAL_ERR_INVALID;
    if (kv->num_q_heads % kv->num_kv_heads != 0) return TIDAL_ERR_INVALID;
    if (kv->head_dim != HEAD_DIM) return TIDAL_ERR_UNSUPPORTED;
    if (kv->num_q_heads / kv->num_kv_heads > MAX_GROUP) return TIDAL_ERR_UNSUPPORTED;
    if (kv->max_ctx_len < 1 || kv->max_ctx_len > MAX_CTX) return TIDAL_ERR_INVALID;
    if (kv->batch > 65535 || kv->num_q_heads > 65535) return TIDAL_ERR_UNSUPPORTED;
    if ((long long)kv->batch * kv->num_q_heads > 262144) return TIDAL_ERR_UNSUPPORTED;   // split counters fit the zeroed head of the workspace
    if (((uintptr_t)kv->k | (uintptr_t)kv->v) & 15) return TIDAL_ERR_INVALID;
    if (kv->kv_dtype != TIDAL_KV_BF16 && kv->kv_dtype != TIDAL_KV_FP8_E4M3) return TIDAL_ERR_INVALID;
    // rows must start on 16-byte boundaries: 8 elements of 16 bits, 16 of 8 bits
    const int64_t align_mask = kv->kv_dtype == TIDAL_KV_FP8_E4M3 ? 15 : 7;
    if ((kv->stride_pos | kv->stride_head | kv->stride_b | kv->stride_page) & align_mask) return TIDAL_ERR_INVALID;
    if (kv->kv_dtype == TIDAL_KV_FP8_E4M3 && ((((uintptr_t)kv->k_scale | (uintptr_t)kv->v_scale) & 3) != 0)) return TIDAL_ERR_INVALID;
    if ((kv->stride_pos | kv->stride_head) & 7) return TIDAL_ERR_INVALID;
    if (kv->stride_pos < 0 || kv->stride_head < 0 || kv->stride_b < 0 || kv->stride_page < 0) return TIDAL_ERR_INVALID;
    if (!(kv->sm_scale >= 0.f) || std::isinf(kv->sm_scale)) return TIDAL_ERR_INVALID;
    if (kv->kv_layout == TIDAL_KV_CONTIG) {
        if (kv->stride_b & 7) return TIDAL_ERR_INVALID;
        if (kv->stride_pos < HEAD_DIM && kv->max_ctx_len > 1) return TIDAL_ERR_INVALID;
    } else if (kv->kv_layout == TIDAL_KV_PAGED) {
        if (!kv->page_table) return TIDAL_ERR_INVALID;
        if (kv->page_size != TILE) return TIDAL_ERR_UNSUPPORTED;
        if (kv->stride_page & 7) return TIDAL_ERR_INVALID;
        if (kv->num_pages <= 0 || kv->max_pages_per_seq <= 0) return TIDAL_ERR_INVALID;
        if ((long long)kv->max_pages_per_seq * kv->page_size < kv->max_ctx_len) return TIDAL_ERR_INVALID;
    } else {
        return TIDAL_ERR_INVALID;
    }
    return TIDAL_OK;
}

// Workspace layout for a cache shape, budget k and (for the host-buffer step) layer count.
WsLayout layout_ws(const tidal_kv_t* kv, int k, int num_layers_host) {
    WsLayout w;
    const size_t rows = (size_t)kv->batch * kv->num_q_heads;
    size_t at = 0;
    w.max_splits = max_splits_for(kv);
    w.part_ml = at;   at += align_up(rows * w.max_splits * sizeof(float2), 256);
    w.part_o = at;    at += align_up(rows * w.max_splits * HEAD_DIM * sizeof(float), 256);
    w.score_stride = (long long)align_up((size_t)kv->max_ctx_len, 16);
    w.scores = at;    at += align_up(rows * (size_t)w.score_stride * sizeof(float), 256);
    w.cand_stride = w.score_stride;
    w.cand = at;      at += align_up(rows * (size_t)w.cand_stride * sizeof(uint2), 256);
    w.bitmap_stride = (long long)align_up((size_t)kv->max_ctx_len, TK_SPAN) / 32;
    w.bitmap = at;    at += align_up(rows * (size_t)w.bitmap_stride * sizeof(unsigned), 256);
    w.idx = at;       at += align_up(rows * (size_t)std::max(k, 1) * sizeof(int), 256);
    w.idx_count = at; at += align_up((size_t)kv->batch * sizeof(int), 256);
    w.q_stage = at;   at += align_up((size_t)num_layers_host * rows * HEAD_DIM * 2, 256);
    w.out_stage = at; at += align_up((size_t)num_layers_host * rows * HEAD_DIM * 4, 256);
    w.total = at;
    return w;
}

size_t ws_bytes_for(const tidal_kv_t* kv, int k, int num_layers_host) {
    return layout_ws(kv, k, num_layers_host).total;
}

void drop_graphs(tidal_ctx* ctx) {
    ctx->last.exec = nullptr;
    if (ctx->graphs.empty()) return;
    cudaDeviceSynchronize();
    for (auto& g : ctx->graphs) if (g.exec) cudaGraphExecDestroy(g.exec);
    ctx->graphs.clear();
}

tidal_status_t ensure_ws(tidal_ctx* ctx, size_t bytes) {
    if (ctx->ws_bytes >= bytes) return TIDAL_OK;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return TIDAL_ERR_CUDA;
    drop_graphs(ctx);                           // they carry addresses inside the old workspace
    if (ctx->ws) { cudaDeviceSynchronize(); cudaFree(ctx->ws); ctx->ws = nullptr; ctx->ws_bytes = 0; }
    void* p = nullptr;
    if (cudaMalloc(&p, bytes) != cudaSuccess) { cudaGetLastError(); return TIDAL_ERR_NOMEM; }
    ctx->ws = p;
    ctx->ws_bytes = bytes;
    return TIDAL_OK;
}

// State layout for a capacity of R rows: counters | cursor | done | thr_max | side counters | side cursors |
// split max | split sum | tile_ctr sets, each
// [R][CTR_STRIDE], then hist[R][TK_BINS]. Consecutive attention launches rotate through the sets of
// pool cursors, so that a launch may use its set before its predecessor has finished with another.
// Every counter has a 128-byte line of its own: hundreds of warps hit them at once, and atomics to one
// line are served one after the other.
constexpr int CTR_STRIDE = 32;
constexpr int CURSOR_SETS = 6;
inline int* state_counters(const tidal_ctx* c) { return (int*)c->state; }
inline int* state_cursor(const tidal_ctx* c) { return (int*)c->state + (size_t)CTR_STRIDE * c->state_rows; }
inline int* state_done(const tidal_ctx* c) { return (int*)c->state + 2 * (size_t)CTR_STRIDE * c->state_rows; }
inline unsigned* state_thr_max(const tidal_ctx* c) { return (unsigned*)c->state + 3 * (size_t)CTR_STRIDE * c->state_rows; }
inline int* state_side_counters(const tidal_ctx* c) { return (int*)c->state + 4 * (size_t)CTR_STRIDE * c->state_rows; }
inline int* state_side_cursors(const tidal_ctx* c) { return (int*)c->state + 5 * (size_t)CTR_STRIDE * c->state_rows; }
inline unsigned* state_split_max(const tidal_ctx* c) { return (unsigned*)c->state + 6 * (size_t)CTR_STRIDE * c->state_rows; }
inline float* state_split_sum(const tidal_ctx* c) { return (float*)c->state + 7 * (size_t)CTR_STRIDE * c->state_rows; }
inline int* state_tile_ctr(const tidal_ctx* c) { return (int*)c->state + 8 * (size_t)CTR_STRIDE * c->state_rows; }
inline unsigned* state_hist(const tidal_ctx* c) { return (unsigned*)c->state + (8 + CURSOR_SETS) * (size_t)CTR_STRIDE * c->state_rows; }

tidal_status_t ensure_state(tidal_ctx* ctx, int rows) {
    if (ctx->state_rows >= rows) return TIDAL_OK;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return TIDAL_ERR_CUDA;
    drop_graphs(ctx);
    if (ctx->state) { cudaDeviceSynchronize(); cudaFree(ctx->state); ctx->state = nullptr; ctx->state_rows = 0; }
    const int cap = (int)align_up((size_t)rows, 64);
    const size_t bytes = (size_t)cap * ((8 + CURSOR_SETS) * CTR_STRIDE + TK_BINS) * sizeof(int);
    void* p = nullptr;
    if (cudaMalloc(&p, bytes) != cudaSuccess) { cudaGetLastError(); return TIDAL_ERR_NOMEM; }
    // on a stream of its own, so that nothing here is the legacy stream's business, and waited for
    cudaStream_t zs = nullptr;
    bool zeroed = cudaStreamCreateWithFlags(&zs, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaMemsetAsync(p, 0, bytes, zs) == cudaSuccess && cudaStreamSynchronize(zs) == cudaSuccess;
    if (zs) cudaStreamDestroy(zs);
    if (!zeroed) { cudaGetLastError(); cudaFree(p); return TIDAL_ERR_CUDA; }
    ctx->state = p;
    ctx->state_rows = cap;
    return TIDAL_OK;
}

tidal_status_t ensure_all(tidal_ctx* ctx, const tidal_kv_t* kv, size_t ws_bytes) {
    const tidal_status_t rc = ensure_state(ctx, kv->batch * kv->num_q_heads);
    return rc != TIDAL_OK ? rc : ensure_ws(ctx, ws_bytes);
}

void fill_common(AttnParams& a, const tidal_ctx* ctx, const tidal_kv_t* kv, const void* q, float* out,
                 const WsLayout& w) {
    std::memset(&a, 0, sizeof a);
    a.q = (const __nv_bfloat16*)q;
    a.k = (const __nv_bfloat16*)kv->k;
    a.v = (const __nv_bfloat16*)kv->v;
    a.out = out;
    a.out_bf16 = ctx->out_bf16;
    a.stride_b = kv->stride_b; a.stride_pos = kv->stride_pos; a.stride_head = kv->stride_head;
    a.stride_page = kv->stride_page;
    a.page_table = kv->page_table; a.max_pages = kv->max_pages_per_seq; a.num_pages = kv->num_pages;
    a.paged = kv->kv_layout == TIDAL_KV_PAGED;
    a.ctx_lens = kv->ctx_lens;
    a.max_ctx = kv->max_ctx_len;
    a.Hq = kv->num_q_heads; a.Hkv = kv->num_kv_heads; a.G = a.Hq / a.Hkv;
    a.scale = kv->sm_scale > 0.f ? kv->sm_scale : 1.0f / std::sqrt((float)kv->head_dim);
    a.scale_log2 = a.scale * 1.4426950408889634f;
    if (kv->kv_dtype == TIDAL_KV_FP8_E4M3) { a.k_scale = kv->k_scale; a.v_scale = kv->v_scale; }
    char* ws = (char*)ctx->ws;
    a.counters = state_counters(ctx);
    a.part_ml = (float2*)(ws + w.part_ml);
    a.part_o = (float*)(ws + w.part_o);
    a.max_splits = w.max_splits;
    a.batch = kv->batch;
    a.tile_ctr = state_tile_ctr(ctx);
    a.ctr_stride = CTR_STRIDE;
    a.hist_shift = hist_shift_for(kv);
    a.status = ctx->status;
}

template <int MODE, int NW, int STAGES, bool KV8 = false>
constexpr size_t attn_smem() {
    return (size_t)NW * STAGES * (KV8 ? STAGE_BYTES8 : STAGE_BYTES) +
           (MODE == MODE_SELECT ? HIST_SMEM : 0) + 1024;   // + alignment slack
}

template <int MODE, int NW, int STAGES, bool NEWEST = false, bool COMPACT = false, bool KV8 = false>
tidal_status_t launch_attn(tidal_ctx* ctx, AttnParams& a, int grid, int full_grid, cudaStream_t st) {
    // Programmatic dependent launch: the kernel may begin while its predecessor in the stream
    // drains; it waits (griddepcontrol.wait) before touching anything that predecessor wrote.
    a.pdl = 1;
    ctx->cursor_set = (ctx->cursor_set + 1) % CURSOR_SETS;
    a.tile_ctr = state_tile_ctr(ctx) + (size_t)ctx->cursor_set * CTR_STRIDE * ctx->state_rows;
    // A kernel that waits late triggers its successor at once, before it has itself waited for its
    // predecessor, so several consecutive launches can be resident together. The one thing a kernel
    // touches before its own wait is its set of pool cursors, last used CURSOR_SETS launches ago by a
    // kernel that must have finished with it. It has: the launches in between either waited before they
    // triggered (then stream order guarantees it), or each of them holds all its CTAs until its own
    // predecessor is complete and (CURSOR_SETS - 1) of them fill every resident slot of the GPU, so this
    // launch cannot have started while a CTA of that old kernel was still resident. Hence the rule:
    // early trigger only for pooled launches (every CTA stays until the wait) whose grid is at least
    // 1 / (CURSOR_SETS - 1) of the resident slots for this kernel's CTA size.
    a.trigger_early = a.wait_late && (long long)(CURSOR_SETS - 1) * grid >= full_grid;
    if (!a.trigger_early) a.wait_late = 0;      // without the early trigger the late wait only delays the successor
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(NW * 32, 1, 1);
    cfg.dynamicSmemBytes = attn_smem<MODE, NW, STAGES, KV8>();
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    ctx->launches++;
    return cudaLaunchKernelEx(&cfg, attn_kernel<MODE, NW, STAGES, NEWEST, COMPACT, KV8>, a) == cudaSuccess ? TIDAL_OK : TIDAL_ERR_CUDA;
}

// How a selection layer produces its ranking scores. Per query head: one row per head, histogram
// fused. Fewer index heads than query heads: the ranking score is the sum of the member heads'
// scaled logits; unless the caller wants the per-head scores, the attention kernel stores the
// group sums directly (one row per KV head; histogram fused when a set belongs to one KV head).
// With one sequence, one set per query head and enough scores per set, the attention kernel compacts
// candidates instead (no histogram) and a single CTA per head finishes the selection on them.
struct SelectPlan { bool agg, fuse, compact, split; int rows; };
constexpr int SCORE_NW = 16, SCORE_STAGES = 3;     // key rows only, 4 KB per tile: sixteen warps keep enough tiles in flight
constexpr int VALUE_NW = 8, VALUE_STAGES = 3;      // value rows + logits, 4.5 KB per tile: two CTAs per SM, also beside a sparse layer's CTA
constexpr size_t SCORE_SMEM = (size_t)SCORE_NW * SCORE_STAGES * TILE_BYTES + HIST_SMEM + 1024;
constexpr size_t VALUE_SMEM = (size_t)VALUE_NW * VALUE_STAGES * (TILE_BYTES + 512) + 1024;
constexpr int VALUE_NW8 = 7;                        // 8-bit caches: 32 positions (4 KB of codes + 1 KB of logits) per slot
constexpr size_t VALUE_SMEM8 = (size_t)VALUE_NW8 * VALUE_STAGES * (UNIT8_BYTES + 1024) + 1024;
constexpr int COMPACT_LIST_SMEM = 12288;      // candidates the compacting top-k keeps in shared memory

int dense_grid(const tidal_ctx* ctx, const tidal_kv_t* kv) {
    const long long tiles = (long long)kv->batch * kv->num_kv_heads * ((kv->max_ctx_len + TILE - 1) / TILE);
    return grid_for(tiles, ctx->dense_slots);
}

SelectPlan select_plan(const tidal_ctx* ctx, const tidal_kv_t* kv, int Hi, int k, bool caller_scores) {
    SelectPlan s;
    s.agg = Hi != kv->num_q_heads && !caller_scores;
    s.rows = s.agg ? kv->num_kv_heads : kv->num_q_heads;
    s.fuse = Hi == s.rows;
    s.compact = ctx->select_margin > 0.f && kv->kv_dtype == TIDAL_KV_BF16 && Hi == kv->num_q_heads && kv->batch == 1 &&
                kv->num_q_heads / kv->num_kv_heads <= CAND_COLS && 6LL * k <= kv->max_ctx_len &&
                pooled_splits(kv, kv->num_kv_heads, dense_grid(ctx, kv)) > 0;
    if (s.compact) s.fuse = false;
    s.split = false;
    return s;
}

// Inside a step a selection layer can run as two passes (split_select_kernels.cuh) when it has one
// sequence (or a batch over a 16-bit cache), per-head scores with the fused histogram and fp32 outputs.
bool can_split(const tidal_ctx* ctx, const tidal_kv_t* kv, const SelectPlan& sp) {
    if (!(ctx->split_select && ctx->layer_overlap && !ctx->out_bf16 && !sp.agg && sp.fuse && !sp.compact)) return false;
    if (kv->batch == 1) return pooled_splits(kv, kv->num_kv_heads, dense_grid(ctx, kv)) > 0;
    return kv->kv_dtype == TIDAL_KV_BF16;       // batches: the flat-split passes (16-bit caches)
}

// hist != nullptr: the kernel also accumulates the per-head histogram the top-k needs.
// How a layer's kernel treats the kernel before it in the stream (see AttnParams::wait_first / wait_late).
enum Dep { DEP_FIRST, DEP_PREFETCH, DEP_LATE };
// Where a sparse layer sits in a run of consecutive sparse layers of a step (see run_sparse).
enum Chain { CHAIN_NONE, CHAIN_FIRST, CHAIN_MIDDLE, CHAIN_LAST };

tidal_status_t run_dense(tidal_ctx* ctx, const tidal_kv_t* kv, const void* q, float* out, float* scores,
                         long long score_stride, bool fuse_hist, Dep dep, const WsLayout& w, cudaStream_t st,
                         bool agg = false, int compact_k = 0, bool private_scores = false) {
    AttnParams a;
    fill_common(a, ctx, kv, q, out, w);
    a.wait_first = dep == DEP_FIRST;
    // A selection layer writes scores while it streams: it may do so ahead of its wait only when no earlier
    // kernel can still be reading the score buffer (the step driver knows), and not with candidate lists.
    a.wait_late = dep == DEP_LATE && (scores == nullptr || (private_scores && compact_k == 0));
    int grid = dense_grid(ctx, kv);
    if (compact_k > 0) {
        a.compact = 1;
        a.cand = (uint2*)((char*)ctx->ws + w.cand);
        a.cand_stride = w.cand_stride;
        a.cand_cursor = state_cursor(ctx);
        a.thr_max = state_thr_max(ctx);
        a.margin = ctx->select_margin;
        a.budget = compact_k;
    }
    if (const int S = pooled_splits(kv, kv->batch * kv->num_kv_heads, grid)) {
        a.splits_per_item = S;        // the grid keeps its size: some items get one CTA more than others
    }
    a.scores = scores;
    a.score_stride = score_stride;
    a.agg = agg ? 1 : 0;
    a.hist = fuse_hist ? state_hist(ctx) : nullptr;
    if (kv->kv_dtype == TIDAL_KV_FP8_E4M3) {
        const int full8 = std::min(ctx->dense_slots, GRID_MAX);
        if (scores) return launch_attn<MODE_SELECT, DENSE_NW8, DENSE_STAGES8, false, false, true>(ctx, a, grid, full8, st);
        return launch_attn<MODE_FULL, DENSE_NW8, DENSE_STAGES8, false, false, true>(ctx, a, grid, full8, st);
    }
    if (scores && a.compact) {
        if (a.splits_per_item <= 0) return TIDAL_ERR_INTERNAL;      // select_plan admits pooled grids only
        return launch_attn<MODE_SELECT, DENSE_NW, DENSE_STAGES, false, true>(ctx, a, grid, std::min(ctx->dense_slots, GRID_MAX), st);
    }
    if (scores) return launch_attn<MODE_SELECT, DENSE_NW, DENSE_STAGES>(ctx, a, grid, std::min(ctx->dense_slots, GRID_MAX), st);
    return launch_attn<MODE_FULL, DENSE_NW, DENSE_STAGES>(ctx, a, grid, std::min(ctx->dense_slots, GRID_MAX), st);
}

// The context's second stream and the two events that fork and join it (created on first use).
tidal_status_t ensure_side_stream(tidal_ctx* ctx) {
    if (ctx->side) return TIDAL_OK;
    if (cudaStreamCreateWithFlags(&ctx->side, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming) != cudaSuccess) {
        cudaGetLastError();
        return TIDAL_ERR_CUDA;
    }
    return TIDAL_OK;
}

// Pass 1 of a split selection layer on the caller's stream: logits, histogram, softmax statistics.
tidal_status_t run_score_pass(tidal_ctx* ctx, const tidal_kv_t* kv, const void* q, float* out, float* scores,
                              long long score_stride, Dep dep, bool scores_free, const WsLayout& w, cudaStream_t st) {
    AttnParams a;
    fill_common(a, ctx, kv, q, out, w);
    const int grid = dense_grid(ctx, kv);
    a.splits_per_item = kv->batch == 1 ? pooled_splits(kv, kv->num_kv_heads, grid) : 0;
    a.scores = scores;
    a.score_stride = score_stride;
    a.hist = state_hist(ctx);
    a.split_max = state_split_max(ctx);
    // the kernel writes scores while it streams: ahead of its wait only if nobody can still be reading them
    a.wait_first = !(dep == DEP_LATE && scores_free);
    a.wait_late = !a.wait_first;
    a.pdl = 1;
    ctx->cursor_set = (ctx->cursor_set + 1) % CURSOR_SETS;
    a.tile_ctr = state_tile_ctr(ctx) + (size_t)ctx->cursor_set * CTR_STRIDE * ctx->state_rows;
    a.trigger_early = a.wait_late && (long long)(CURSOR_SETS - 1) * grid >= std::min(ctx->dense_slots, GRID_MAX);
    if (a.wait_late && !a.trigger_early) { a.wait_late = 0; a.wait_first = 1; }
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(SCORE_NW * 32, 1, 1);
    cfg.dynamicSmemBytes = SCORE_SMEM;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    ctx->launches++;
    const bool rowc = kv->stride_pos == 2 * HEAD_DIM;     // K and V rows interleaved: constant offsets between the rows of a tile
    cudaError_t e;
    if (kv->batch > 1)
        e = rowc ? cudaLaunchKernelEx(&cfg, score_pass_flat_kernel<SCORE_NW, SCORE_STAGES, true>, a)
                 : cudaLaunchKernelEx(&cfg, score_pass_flat_kernel<SCORE_NW, SCORE_STAGES, false>, a);
    else if (kv->kv_dtype == TIDAL_KV_FP8_E4M3)
        e = rowc ? cudaLaunchKernelEx(&cfg, score_pass8_kernel<SCORE_NW, SCORE_STAGES, true>, a)
                 : cudaLaunchKernelEx(&cfg, score_pass8_kernel<SCORE_NW, SCORE_STAGES, false>, a);
    else
        e = rowc ? cudaLaunchKernelEx(&cfg, score_pass_kernel<SCORE_NW, SCORE_STAGES, true>, a)
                 : cudaLaunchKernelEx(&cfg, score_pass_kernel<SCORE_NW, SCORE_STAGES, false>, a);
    return e == cudaSuccess ? TIDAL_OK : TIDAL_ERR_CUDA;
}

// Pass 2 on the context's second stream: it starts when pass 1 is complete and runs beside whatever
// the caller's stream does next. It owns a cursor and a counter array of its own and no other scratch.
tidal_status_t run_value_pass(tidal_ctx* ctx, const tidal_kv_t* kv, float* out, float* out_final, const float* scores,
                              long long score_stride, const WsLayout& w, cudaStream_t st) {
    AttnParams a;
    fill_common(a, ctx, kv, nullptr, out, w);
    a.out_final = out_final;
    a.scores = const_cast<float*>(scores);
    a.score_stride = score_stride;
    a.split_max = state_split_max(ctx);
    a.split_sum = state_split_sum(ctx);
    a.counters = state_side_counters(ctx);
    a.tile_ctr = state_side_cursors(ctx);
    a.pdl = 0;
    // most of the slots (its CTAs are the size of the sparse layers'): it shares the GPU with the top-k and the
    // first sparse layers; between 25 % and 100 % of the slots the step time moved by less than 2 %
    const int per_item = std::max(2, 85 * std::min(ctx->sparse_slots, GRID_MAX) / (100 * kv->num_kv_heads));
    const int grid = kv->batch == 1 ? per_item * kv->num_kv_heads : std::min(ctx->sparse_slots, GRID_MAX);
    a.splits_per_item = kv->batch == 1 ? per_item : 0;
    if (cudaEventRecord(ctx->ev_fork, st) != cudaSuccess || cudaStreamWaitEvent(ctx->side, ctx->ev_fork, 0) != cudaSuccess)
        return TIDAL_ERR_CUDA;
    const bool rowc = kv->stride_pos == 2 * HEAD_DIM;
    if (kv->batch > 1) {
        if (rowc) value_pass_flat_kernel<VALUE_NW, VALUE_STAGES, true><<<grid, VALUE_NW * 32, VALUE_SMEM, ctx->side>>>(a);
        else value_pass_flat_kernel<VALUE_NW, VALUE_STAGES, false><<<grid, VALUE_NW * 32, VALUE_SMEM, ctx->side>>>(a);
    } else if (kv->kv_dtype == TIDAL_KV_FP8_E4M3) {
        if (rowc) value_pass8_kernel<VALUE_NW8, VALUE_STAGES, true><<<grid, VALUE_NW8 * 32, VALUE_SMEM8, ctx->side>>>(a);
        else value_pass8_kernel<VALUE_NW8, VALUE_STAGES, false><<<grid, VALUE_NW8 * 32, VALUE_SMEM8, ctx->side>>>(a);
    } else if (rowc) value_pass_kernel<VALUE_NW, VALUE_STAGES, true><<<grid, VALUE_NW * 32, VALUE_SMEM, ctx->side>>>(a);
    else value_pass_kernel<VALUE_NW, VALUE_STAGES, false><<<grid, VALUE_NW * 32, VALUE_SMEM, ctx->side>>>(a);
    ctx->launches++;
    if (cudaGetLastError() != cudaSuccess) return TIDAL_ERR_CUDA;
    return cudaEventRecord(ctx->ev_join, ctx->side) == cudaSuccess ? TIDAL_OK : TIDAL_ERR_CUDA;
}

// `rows`: score rows per sequence (query heads, or KV heads when the attention kernel stored group sums).
tidal_status_t run_topk(tidal_ctx* ctx, const tidal_kv_t* kv, const float* scores, long long score_stride,
                        int k, int rows, int Hi, bool hist_done, int* idx, int* idx_count, const WsLayout& w,
                        cudaStream_t st, bool compact = false) {
    TopkParams t;
    std::memset(&t, 0, sizeof t);
    t.scores = scores; t.score_stride = score_stride;
    t.ctx_lens = kv->ctx_lens; t.max_ctx = kv->max_ctx_len;
    t.Hq = rows; t.Hi = Hi; t.k = k;
    t.idx = idx; t.idx_count = idx_count;
    char* ws = (char*)ctx->ws;
    t.hist = state_hist(ctx);
    t.cursor = state_cursor(ctx);
    t.ctr_stride = CTR_STRIDE;
    t.done = state_done(ctx);
    t.cand = (uint2*)(ws + w.cand);
    t.cand_stride = w.cand_stride;
    t.bitmap = (unsigned*)(ws + w.bitmap);
    t.bitmap_stride = w.bitmap_stride;
    const int items = kv->batch * Hi;
    if (items > 65535) return TIDAL_ERR_UNSUPPORTED;
    const int parts = (kv->max_ctx_len + TK_SLICE - 1) / TK_SLICE;        // histogram kernel
    const int sel_parts = (kv->max_ctx_len + TK_SPAN - 1) / TK_SPAN;     // select kernel
    t.shift = hist_shift_for(kv);
    t.vec_ok = (((uintptr_t)scores & 15) == 0 && (score_stride & 3) == 0) ? 1 : 0;
    // Candidates the last CTA of a head can hold in shared memory (a threshold bin's population is about
    // 2000 of 131072 scores; larger lists are read from global memory). With more CTAs than fit the GPU at
    // once (batches), the buffer is cut to what fits beside the bitmaps in the 64 KB the score staging needs
    // anyway, so that three CTAs share an SM instead of two.
    const size_t words = (size_t)(kv->max_ctx_len + 31) / 32;
    t.cand_smem = 8192;
    {
        const long long ctas = (long long)((kv->max_ctx_len + TK_SPAN - 1) / TK_SPAN) * kv->batch * Hi;
        const size_t staging = (size_t)TK_SPAN * sizeof(float), bitmaps = 2 * words * sizeof(unsigned);
        if (ctas > 2LL * ctx->sm_count && bitmaps + 2048 * sizeof(uint2) <= staging)
            t.cand_smem = (int)((staging - bitmaps) / sizeof(uint2));
    }
    // the last CTA's bitmaps and candidate buffer, or every CTA's score staging area, whichever is larger
    size_t smem = std::max(2 * words * sizeof(unsigned) + (size_t)t.cand_smem * sizeof(uint2),
                           (size_t)TK_SPAN * sizeof(float));
    if (kv->max_ctx_len <= TK_SPAN) {
        // every row fits one CTA: staged scores, two bitmaps and 4096 candidates in shared memory
        t.solo_cand = 4096;
        smem = (size_t)TK_SPAN * sizeof(float) + 2 * (TK_SPAN / 32) * sizeof(unsigned) + (size_t)t.solo_cand * sizeof(uint2);
    }
    // Both kernels may become resident while the kernel before them drains (they wait for it first).
    t.pdl = 1;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof cfg);
    cfg.blockDim = dim3(TK_THREADS, 1, 1);
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (compact) {
        t.thr_max = state_thr_max(ctx);
        t.list_smem = COMPACT_LIST_SMEM;
        const size_t bm_words = (size_t)(kv->max_ctx_len + 31) / 32;
        cfg.gridDim = dim3(items, 1, 1);
        cfg.dynamicSmemBytes = 2 * (bm_words + 1) * sizeof(unsigned) + (size_t)COMPACT_LIST_SMEM * sizeof(uint2);
        ctx->launches++;
        return cudaLaunchKernelEx(&cfg, topk_compact_kernel, t) == cudaSuccess ? TIDAL_OK : TIDAL_ERR_CUDA;
    }
    if (!hist_done) {
        cfg.gridDim = dim3(parts, items, 1);
        cfg.dynamicSmemBytes = 0;
        ctx->launches++;
        if (cudaLaunchKernelEx(&cfg, topk_hist_kernel, t) != cudaSuccess) return TIDAL_ERR_CUDA;
    }
    cfg.gridDim = dim3(sel_parts, items, 1);
    cfg.dynamicSmemBytes = smem;
    ctx->launches++;
    if (cudaLaunchKernelEx(&cfg, topk_select_kernel, t) != cudaSuccess) return TIDAL_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? TIDAL_OK : TIDAL_ERR_CUDA;
}

tidal_status_t run_sparse(tidal_ctx* ctx, const tidal_kv_t* kv, const void* q, const int* idx,
                          const int* idx_count, int k, int Hi, float* out, Dep dep, Chain chain, const WsLayout& w,
                          cudaStream_t st) {
    AttnParams a;
    fill_common(a, ctx, kv, q, out, w);
    a.wait_first = dep == DEP_FIRST;
    a.wait_late = dep == DEP_LATE;
    const int per_batch = (Hi == kv->num_q_heads) ? kv->num_q_heads : kv->num_kv_heads;
    const long long tiles = (long long)kv->batch * per_batch * ((k + TILE - 1) / TILE);
    const int full = std::min(ctx->sparse_slots, GRID_MAX);
    int grid = grid_for(tiles, ctx->sparse_slots);
    a.idx = idx; a.idx_count = idx_count; a.budget = k; a.Hi = Hi;
    // In a chain of sparse layers that overlap (late wait, early trigger) a launch takes about a third
    // of the resident slots, so that about three layers are in flight at any time, one behind the
    // other: while the CTAs of one layer start up (lengths, index entries, first rows: a chain of
    // dependent loads) or merge their results, the others keep the memory system busy. Every item gets
    // the same number of CTAs.
    // The first layer of a chain runs alone until its successors have joined it and gets about half
    // the slots; the last one, which nothing follows into the slots it frees, gets one CTA per item
    // more than a third (measured at cfg3: step 658 -> 645 us against a third everywhere).
    const int items = kv->batch * per_batch;
    if (chain != CHAIN_NONE) {
        // (a layer that gathers fewer bytes, an 8-bit cache or a small budget, still has the same start-up and
        // merge phases: four layers in flight below 48 MB per layer)
        const long long row_bytes = kv->kv_dtype == TIDAL_KV_FP8_E4M3 ? 2 * ROW_BYTES8 : 4 * HEAD_DIM;
        const int depth = (long long)items * k * row_bytes < (48ll << 20) ? 4 : 3;
        const int third = std::max(1, (full + depth * items / 2) / (depth * items));
        const int S = chain == CHAIN_FIRST ? std::max(third, (full + items) / (2 * items))
                      : chain == CHAIN_LAST ? third + 1 : third;
        grid = std::min(grid, S * items);
    }
    if (const int S = pooled_splits(kv, items, grid)) {
        a.splits_per_item = S;
    }
    if (kv->kv_dtype == TIDAL_KV_FP8_E4M3) {
        if (ctx->attend_newest) return TIDAL_ERR_UNSUPPORTED;
        return launch_attn<MODE_SPARSE, SPARSE_NW8, SPARSE_STAGES8, false, false, true>(ctx, a, grid, std::min(ctx->sparse_slots, GRID_MAX), st);
    }
    if (ctx->attend_newest) return launch_attn<MODE_SPARSE, SPARSE_NW, SPARSE_STAGES, true>(ctx, a, grid, std::min(ctx->sparse_slots, GRID_MAX), st);
    return launch_attn<MODE_SPARSE, SPARSE_NW, SPARSE_STAGES>(ctx, a, grid, std::min(ctx->sparse_slots, GRID_MAX), st);
}

template <typename K>
int resident_ctas(K kernel, int threads, size_t smem, int sm_count) {
    int per_sm = 0;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return -1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, smem) != cudaSuccess) return -1;
    return per_sm * sm_count;
}

// ---- step graphs ------------------------------------------------------------------------------------
struct KeyBuilder {
    std::vector<unsigned char> bytes;
    template <typename T> void add(const T& v) {
        const unsigned char* p = reinterpret_cast<const unsigned char*>(&v);
        bytes.insert(bytes.end(), p, p + sizeof(T));
    }
    void add_raw(const void* p, size_t n) {
        const unsigned char* c = static_cast<const unsigned char*>(p);
        bytes.insert(bytes.end(), c, c + n);
    }
};

void step_key(KeyBuilder& kb, const tidal_ctx* ctx, int tag, int32_t num_layers, const uint8_t* schedule,
                     const tidal_kv_t* kvs, int32_t k, int32_t granularity, int host_layers) {
    kb.add(tag); kb.add(num_layers); kb.add(k); kb.add(granularity); kb.add(host_layers);
    kb.add(ctx->ws); kb.add(ctx->state); kb.add(ctx->out_bf16); kb.add(ctx->attend_newest); kb.add(ctx->layer_overlap); kb.add(ctx->select_margin); kb.add(ctx->split_select);
    kb.add_raw(schedule, (size_t)num_layers);
    for (int i = 0; i < num_layers; ++i) {
        // field by field: the struct has padding whose bytes are not the caller's to define
        const tidal_kv_t& v = kvs[i];
        kb.add(v.batch); kb.add(v.num_q_heads); kb.add(v.num_kv_heads); kb.add(v.head_dim); kb.add(v.kv_layout);
        kb.add(v.k); kb.add(v.v); kb.add(v.stride_b); kb.add(v.stride_pos); kb.add(v.stride_head); kb.add(v.stride_page);
        kb.add(v.page_table); kb.add(v.page_size); kb.add(v.max_pages_per_seq); kb.add(v.num_pages);
        kb.add(v.ctx_lens); kb.add(v.max_ctx_len); kb.add(v.sm_scale); kb.add(v.kv_dtype); kb.add(v.k_scale); kb.add(v.v_scale);
    }
}

// A stream can record a graph if it is a real stream (not the legacy or per-thread default) that is
// not already being captured by the caller.
bool graphable(const tidal_ctx* ctx, cudaStream_t st) {
    if (!ctx->graphs_enabled || st == nullptr || st == cudaStreamLegacy || st == cudaStreamPerThread) return false;
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cs) != cudaSuccess) { cudaGetLastError(); return false; }
    return cs == cudaStreamCaptureStatusNone;
}

// Replays the recorded graph of `key`, or records one from `enqueue` (which must only launch work on
// `st`). Falls back to plain enqueueing when recording is not possible.
template <typename F>
tidal_status_t run_graphed(tidal_ctx* ctx, KeyBuilder& kb, cudaStream_t st, F&& enqueue) {
    constexpr size_t MAX_GRAPHS = 16;
    ctx->ran_exec = nullptr;
    if (!graphable(ctx, st)) return enqueue();
    ++ctx->graph_clock;
    for (auto& g : ctx->graphs) {
        if (g.key == kb.bytes) {
            g.last_use = ctx->graph_clock;
            if (cudaGraphLaunch(g.exec, st) != cudaSuccess) return TIDAL_ERR_CUDA;
            ctx->launches += g.launches;
            ctx->ran_exec = g.exec; ctx->ran_launches = g.launches;
            return TIDAL_OK;
        }
    }
    if (cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) != cudaSuccess) { cudaGetLastError(); return enqueue(); }
    const int64_t before = ctx->launches;
    const tidal_status_t rc = enqueue();
    cudaGraph_t graph = nullptr;
    const cudaError_t end = cudaStreamEndCapture(st, &graph);
    const int recorded = (int)(ctx->launches - before);
    ctx->launches = before;                     // nothing has run yet
    if (rc != TIDAL_OK || end != cudaSuccess || !graph) {
        if (graph) cudaGraphDestroy(graph);
        cudaGetLastError();
        return rc != TIDAL_OK ? rc : enqueue();
    }
    cudaGraphExec_t exec = nullptr;
    const cudaError_t inst = cudaGraphInstantiate(&exec, graph, 0);
    cudaGraphDestroy(graph);
    if (inst != cudaSuccess || !exec) { cudaGetLastError(); return enqueue(); }
    if (ctx->graphs.size() >= MAX_GRAPHS) {     // forget the entry that has gone unused the longest
        size_t victim = 0;
        for (size_t i = 1; i < ctx->graphs.size(); ++i)
            if (ctx->graphs[i].last_use < ctx->graphs[victim].last_use) victim = i;
        if (ctx->last.exec == ctx->graphs[victim].exec) ctx->last.exec = nullptr;
        cudaGraphExecDestroy(ctx->graphs[victim].exec);   // deferred by the runtime while a launch is in flight
        ctx->graphs.erase(ctx->graphs.begin() + victim);
    }
    tidal_ctx::StepGraph g;
    g.key = std::move(kb.bytes);
    g.exec = exec;
    g.launches = recorded;
    g.last_use = ctx->graph_clock;
    ctx->graphs.push_back(std::move(g));
    if (cudaGraphLaunch(exec, st) != cudaSuccess) return TIDAL_ERR_CUDA;
    ctx->launches += recorded;
    ctx->ran_exec = exec; ctx->ran_launches = recorded;
    return TIDAL_OK;
}

// The bytes that decide what a step call does: compared with the previous call's before anything else.
void raw_call_key(std::vector<unsigned char>& r, const tidal_ctx* ctx, int tag, int32_t num_layers, const uint8_t* schedule,
                  const tidal_kv_t* kvs, const void* const* qs, float* const* outs, const void* p0, const void* p1,
                  int32_t k, int32_t granularity, cudaStream_t st) {
    struct Head {
        int tag; int32_t num_layers, k, granularity; cudaStream_t st; const void *p0, *p1, *ws, *state;
        int out_bf16, attend_newest, layer_overlap, split_select; float select_margin;
    } h;
    std::memset(&h, 0, sizeof h);
    h.tag = tag; h.num_layers = num_layers; h.k = k; h.granularity = granularity; h.st = st; h.p0 = p0; h.p1 = p1;
    h.ws = ctx->ws; h.state = ctx->state; h.out_bf16 = ctx->out_bf16; h.attend_newest = ctx->attend_newest;
    h.layer_overlap = ctx->layer_overlap; h.split_select = ctx->split_select; h.select_margin = ctx->select_margin;
    const size_t L = (size_t)num_layers;
    const size_t n_q = qs ? L * sizeof(void*) : 0, n_o = outs ? L * sizeof(void*) : 0;
    r.resize(sizeof h + L + L * sizeof(tidal_kv_t) + n_q + n_o);
    unsigned char* d = r.data();
    std::memcpy(d, &h, sizeof h); d += sizeof h;
    std::memcpy(d, schedule, L); d += L;
    std::memcpy(d, kvs, L * sizeof(tidal_kv_t)); d += L * sizeof(tidal_kv_t);
    if (n_q) { std::memcpy(d, qs, n_q); d += n_q; }
    if (n_o) std::memcpy(d, outs, n_o);
}

// Same call as the last one, which ran as a graph: launch that graph again.
bool replay_last(tidal_ctx* ctx, cudaStream_t st, tidal_status_t& rc) {
    if (!ctx->last.exec || ctx->raw_scratch != ctx->last.raw || !graphable(ctx, st)) return false;
    rc = cudaGraphLaunch(ctx->last.exec, st) == cudaSuccess ? TIDAL_OK : TIDAL_ERR_CUDA;
    if (rc == TIDAL_OK) ctx->launches += ctx->last.launches;
    return true;
}

void remember_last(tidal_ctx* ctx) {
    if (!ctx->ran_exec) { ctx->last.exec = nullptr; return; }
    ctx->last.raw = ctx->raw_scratch;
    ctx->last.exec = ctx->ran_exec;
    ctx->last.launches = ctx->ran_launches;
}

}  // namespace

extern "C" {

tidal_status_t tidal_create(tidal_ctx_t** out, int device, size_t workspace_bytes) {
    if (!out) return TIDAL_ERR_INVALID;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) { cudaGetLastError(); return TIDAL_ERR_CUDA; }
    if (cudaSetDevice(device) != cudaSuccess) return TIDAL_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return TIDAL_ERR_CUDA;
    if (prop.major < 10) return TIDAL_ERR_UNSUPPORTED;
    tidal_ctx* ctx = new (std::nothrow) tidal_ctx();
    if (!ctx) return TIDAL_ERR_NOMEM;
    ctx->device = device;
    ctx->sm_count = prop.multiProcessorCount;
    const int d0 = resident_ctas(attn_kernel<MODE_FULL, DENSE_NW, DENSE_STAGES>, DENSE_NW * 32, attn_smem<MODE_FULL, DENSE_NW, DENSE_STAGES>(), ctx->sm_count);
    const int d1 = resident_ctas(attn_kernel<MODE_SELECT, DENSE_NW, DENSE_STAGES>, DENSE_NW * 32, attn_smem<MODE_SELECT, DENSE_NW, DENSE_STAGES>(), ctx->sm_count);
    const int d2 = resident_ctas(attn_kernel<MODE_SELECT, DENSE_NW, DENSE_STAGES, false, true>, DENSE_NW * 32, attn_smem<MODE_SELECT, DENSE_NW, DENSE_STAGES>(), ctx->sm_count);
    const int s0 = resident_ctas(attn_kernel<MODE_SPARSE, SPARSE_NW, SPARSE_STAGES>, SPARSE_NW * 32, attn_smem<MODE_SPARSE, SPARSE_NW, SPARSE_STAGES>(), ctx->sm_count);
    const int s1 = resident_ctas(attn_kernel<MODE_SPARSE, SPARSE_NW, SPARSE_STAGES, true>, SPARSE_NW * 32, attn_smem<MODE_SPARSE, SPARSE_NW, SPARSE_STAGES>(), ctx->sm_count);
    const int e0 = resident_ctas(attn_kernel<MODE_FULL, DENSE_NW8, DENSE_STAGES8, false, false, true>, DENSE_NW8 * 32, attn_smem<MODE_FULL, DENSE_NW8, DENSE_STAGES8, true>(), ctx->sm_count);
    const int e1 = resident_ctas(attn_kernel<MODE_SELECT, DENSE_NW8, DENSE_STAGES8, false, false, true>, DENSE_NW8 * 32, attn_smem<MODE_SELECT, DENSE_NW8, DENSE_STAGES8, true>(), ctx->sm_count);
    const int e2 = resident_ctas(attn_kernel<MODE_SPARSE, SPARSE_NW8, SPARSE_STAGES8, false, false, true>, SPARSE_NW8 * 32, attn_smem<MODE_SPARSE, SPARSE_NW8, SPARSE_STAGES8, true>(), ctx->sm_count);
    const bool split_ok =
        cudaFuncSetAttribute(score_pass_kernel<SCORE_NW, SCORE_STAGES, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SCORE_SMEM) == cudaSuccess &&
        cudaFuncSetAttribute(score_pass_kernel<SCORE_NW, SCORE_STAGES, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SCORE_SMEM) == cudaSuccess &&
        cudaFuncSetAttribute(score_pass_flat_kernel<SCORE_NW, SCORE_STAGES, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SCORE_SMEM) == cudaSuccess &&
        cudaFuncSetAttribute(score_pass_flat_kernel<SCORE_NW, SCORE_STAGES, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SCORE_SMEM) == cudaSuccess &&
        cudaFuncSetAttribute(value_pass_flat_kernel<VALUE_NW, VALUE_STAGES, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)VALUE_SMEM) == cudaSuccess &&
        cudaFuncSetAttribute(value_pass_flat_kernel<VALUE_NW, VALUE_STAGES, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)VALUE_SMEM) == cudaSuccess &&
        cudaFuncSetAttribute(score_pass8_kernel<SCORE_NW, SCORE_STAGES, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SCORE_SMEM) == cudaSuccess &&
        cudaFuncSetAttribute(score_pass8_kernel<SCORE_NW, SCORE_STAGES, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SCORE_SMEM) == cudaSuccess &&
        cudaFuncSetAttribute(value_pass8_kernel<VALUE_NW8, VALUE_STAGES, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)VALUE_SMEM8) == cudaSuccess &&
        cudaFuncSetAttribute(value_pass8_kernel<VALUE_NW8, VALUE_STAGES, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)VALUE_SMEM8) == cudaSuccess &&
        cudaFuncSetAttribute(value_pass_kernel<VALUE_NW, VALUE_STAGES, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)VALUE_SMEM) == cudaSuccess &&
        cudaFuncSetAttribute(value_pass_kernel<VALUE_NW, VALUE_STAGES, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)VALUE_SMEM) == cudaSuccess;
    const size_t topk_smem = 2 * (size_t)(MAX_CTX / 32) * sizeof(unsigned) + 8192 * sizeof(uint2);
    const bool topk_ok = cudaFuncSetAttribute(topk_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)topk_smem) == cudaSuccess;
    const size_t compact_smem = 2 * ((size_t)(MAX_CTX / 32) + 1) * sizeof(unsigned) + (size_t)COMPACT_LIST_SMEM * sizeof(uint2);
    const bool compact_ok = cudaFuncSetAttribute(topk_compact_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)compact_smem) == cudaSuccess;
    if (d0 <= 0 || d1 <= 0 || d2 < d1 || s0 <= 0 || s1 < s0 || e0 < d0 || e1 < d1 || e2 < s0 || !topk_ok || !compact_ok || !split_ok) { cudaGetLastError(); delete ctx; return TIDAL_ERR_CUDA; }
    ctx->dense_slots = std::min(d0, d1);
    ctx->sparse_slots = s0;
    if (cudaMalloc((void**)&ctx->status, 256) != cudaSuccess || cudaMemset(ctx->status, 0, 256) != cudaSuccess) {
        cudaGetLastError(); delete ctx; return TIDAL_ERR_NOMEM;
    }
    if (workspace_bytes) {
        const tidal_status_t rc = ensure_ws(ctx, workspace_bytes);
        if (rc != TIDAL_OK) { cudaFree(ctx->status); delete ctx; return rc; }
    }
    *out = ctx;
    return TIDAL_OK;
}

tidal_status_t tidal_destroy(tidal_ctx_t* ctx) {
    if (!ctx) return TIDAL_ERR_INVALID;
    cudaSetDevice(ctx->device);
    cudaDeviceSynchronize();
    drop_graphs(ctx);
    if (ctx->side) cudaStreamDestroy(ctx->side);
    if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
    if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
    if (ctx->ws) cudaFree(ctx->ws);
    if (ctx->state) cudaFree(ctx->state);
    if (ctx->status) cudaFree(ctx->status);
    delete ctx;
    return TIDAL_OK;
}

size_t tidal_workspace_bytes(const tidal_kv_t* kv, int32_t k) {
    if (check_kv(kv) != TIDAL_OK || k <= 0) return 0;
    return ws_bytes_for(kv, k, 0);
}

tidal_status_t tidal_reserve(tidal_ctx_t* ctx, const tidal_kv_t* kv, int32_t k, int32_t num_layers_host) {
    if (!ctx || k <= 0 || num_layers_host < 0 || num_layers_host > 1024) return TIDAL_ERR_INVALID;
    const tidal_status_t rc = check_kv(kv);
    if (rc != TIDAL_OK) return rc;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return TIDAL_ERR_CUDA;
    const tidal_status_t rs = ensure_side_stream(ctx);       // a later step's selection layers may use it
    if (rs != TIDAL_OK) return rs;
    return ensure_all(ctx, kv, ws_bytes_for(kv, k, num_layers_host));
}

static void fill_append(AppendParams& a, const tidal_ctx* ctx, const tidal_kv_t* kv, const void* k_new,
                        const void* v_new);

tidal_status_t tidal_kv_append(tidal_ctx_t* ctx, const tidal_kv_t* kv, const void* k_new, const void* v_new,
                               void* stream) {
    if (!ctx || !k_new || !v_new || (((uintptr_t)k_new | (uintptr_t)v_new) & 15)) return TIDAL_ERR_INVALID;
    const tidal_status_t rc = check_kv(kv);
    if (rc != TIDAL_OK) return rc;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return TIDAL_ERR_CUDA;
    AppendParams a;
    fill_append(a, ctx, kv, k_new, v_new);
    const int pairs = kv->batch * kv->num_kv_heads;
    kv_append_kernel<<<(pairs + 3) / 4, 128, 0, (cudaStream_t)stream>>>(a);
    ctx->launches++;
    return cudaGetLastError() == cudaSuccess ? TIDAL_OK : TIDAL_ERR_CUDA;
}

static void fill_append(AppendParams& a, const tidal_ctx* ctx, const tidal_kv_t* kv, const void* k_new,
                        const void* v_new) {
    std::memset(&a, 0, sizeof a);
    a.k = (__nv_bfloat16*)const_cast<void*>(kv->k);
    a.v = (__nv_bfloat16*)const_cast<void*>(kv->v);
    a.k_new = (const __nv_bfloat16*)k_new;
    a.v_new = (const __nv_bfloat16*)v_new;
    a.stride_b = kv->stride_b; a.stride_pos = kv->stride_pos; a.stride_head = kv->stride_head;
    a.stride_page = kv->stride_page;
    a.page_table = kv->page_table; a.max_pages = kv->max_pages_per_seq; a.num_pages = kv->num_pages;
    a.paged = kv->kv_layout == TIDAL_KV_PAGED;
    a.ctx_lens = kv->ctx_lens; a.max_ctx = kv->max_ctx_len;
    a.batch = kv->batch; a.Hkv = kv->num_kv_heads;
    a.elem_bytes = kv->kv_dtype == TIDAL_KV_FP8_E4M3 ? 1 : 2;
    a.status = ctx->status;
}

tidal_status_t tidal_full_attn(tidal_ctx_t* ctx, const tidal_kv_t* kv, const void* q, float* out, void* stream) {
    if (!ctx || !q || !out || ((uintptr_t)q & 15)) return TIDAL_ERR_INVALID;
    tidal_status_t rc = check_kv(kv);
    if (rc != TIDAL_OK) return rc;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return TIDAL_ERR_CUDA;
    const WsLayout w = layout_ws(kv, 1, 0);
    if ((rc = ensure_all(ctx, kv, w.total)) != TIDAL_OK) return rc;
    return run_dense(ctx, kv, q, out, nullptr, 0, false, DEP_FIRST, w, (cudaStream_t)stream);
}

tidal_status_t tidal_select_attn(tidal_ctx_t* ctx, const tidal_kv_t* kv, const void* q, int32_t k,
                                 int32_t granularity, float* out, int32_t* idx, int32_t* idx_count,
                                 float* scores_opt, void* stream) {
    if (!ctx || !q || !out || !idx || ((uintptr_t)q & 15)) return TIDAL_ERR_INVALID;
    tidal_status_t rc = check_kv(kv);
    if (rc != TIDAL_OK) return rc;
    if (k <= 0 || k > kv->max_ctx_len) return TIDAL_ERR_INVALID;
    const int Hi = hi_of(kv, granularity);
    if (Hi <= 0) return TIDAL_ERR_INVALID;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return TIDAL_ERR_CUDA;
    const WsLayout w = layout_ws(kv, k, 0);
    if ((rc = ensure_all(ctx, kv, w.total)) != TIDAL_OK) return rc;
    float* scores = scores_opt ? scores_opt : (float*)((char*)ctx->ws + w.scores);
    const long long stride = scores_opt ? (long long)kv->max_ctx_len : w.score_stride;
    cudaStream_t st = (cudaStream_t)stream;
    const SelectPlan sp = select_plan(ctx, kv, Hi, k, scores_opt != nullptr);
    if ((rc = run_dense(ctx, kv, q, out, scores, stride, sp.fuse, DEP_FIRST, w, st, sp.agg, sp.compact ? k : 0)) != TIDAL_OK) return rc;
    return run_topk(ctx, kv, scores, stride, k, sp.rows, Hi, sp.fuse, idx, idx_count, w, st, sp.compact);
}

tidal_status_t tidal_sparse_attn(tidal_ctx_t* ctx, const tidal_kv_t* kv, const void* q, const int32_t* idx,
                                 const int32_t* idx_count, int32_t k, int32_t num_index_heads, float* out,
                                 void* stream) {
    if (!ctx || !q || !out || !idx || ((uintptr_t)q & 15)) return TIDAL_ERR_INVALID;
    tidal_status_t rc = check_kv(kv);
    if (rc != TIDAL_OK) return rc;
    if (k <= 0) return TIDAL_ERR_INVALID;
    const int Hi = num_index_heads;
    if (Hi != kv->num_q_heads && Hi != kv->num_kv_heads && Hi != 1) return TIDAL_ERR_INVALID;
    if (ctx->attend_newest && !idx_count) return TIDAL_ERR_INVALID;   // the end of each list must be known
    if (cudaSetDevice(ctx->device) != cudaSuccess) return TIDAL_ERR_CUDA;
    const WsLayout w = layout_ws(kv, k, 0);
    if ((rc = ensure_all(ctx, kv, w.total)) != TIDAL_OK) return rc;
    return run_sparse(ctx, kv, q, idx, idx_count, k, Hi, out, DEP_FIRST, CHAIN_NONE, w, (cudaStream_t)stream);
}

// Validates a step and sizes the workspace for it (may allocate and synchronise).
static tidal_status_t decode_step_prepare(tidal_ctx_t* ctx, int32_t num_layers, const uint8_t* schedule,
                                          const tidal_kv_t* kvs, const void* const* qs, float* const* outs,
                                          int32_t k, int32_t granularity, int host_layers) {
    // Validate everything before enqueuing anything.
    bool have_rho = false;
    size_t need = 0;
    for (int i = 0; i < num_layers; ++i) {
        tidal_status_t rc = check_kv(&kvs[i]);
        if (rc != TIDAL_OK) return rc;
        if (!qs[i] || !outs[i] || ((uintptr_t)qs[i] & 15)) return TIDAL_ERR_INVALID;
        if (kvs[i].batch != kvs[0].batch || kvs[i].num_q_heads != kvs[0].num_q_heads ||
            kvs[i].num_kv_heads != kvs[0].num_kv_heads) return TIDAL_ERR_INVALID;
        if (schedule[i] == TIDAL_LAYER_SELECT) {
            if (k > kvs[i].max_ctx_len) return TIDAL_ERR_INVALID;
            have_rho = true;
        } else if (schedule[i] == TIDAL_LAYER_SPARSE) {
            if (!have_rho) return TIDAL_ERR_INVALID;
        } else if (schedule[i] != TIDAL_LAYER_FULL) {
            return TIDAL_ERR_INVALID;
        }
        need = std::max(need, ws_bytes_for(&kvs[i], k, host_layers));
    }
    if (hi_of(&kvs[0], granularity) <= 0) return TIDAL_ERR_INVALID;
    return ensure_all(ctx, &kvs[0], need);
}

// Enqueues the layers of a prepared step: launches only, nothing that a stream capture forbids.
static tidal_status_t decode_step_enqueue(tidal_ctx_t* ctx, int32_t num_layers, const uint8_t* schedule,
                                          const tidal_kv_t* kvs, const void* const* qs, float* const* outs,
                                          int32_t k, int32_t granularity, int32_t* idx, int32_t* idx_count,
                                          int host_layers, cudaStream_t st, float* const* acc = nullptr) {
    const int Hi = hi_of(&kvs[0], granularity);
    tidal_status_t rc = TIDAL_OK;
    bool side_pending = false;                  // a value pass is in flight on the second stream
    for (int i = 0; i < num_layers; ++i) {
        const tidal_kv_t* kv = &kvs[i];
        const WsLayout w = layout_ws(kv, k, host_layers);
        // Every query, length, page table and cache row of the step was complete before the call, so a
        // layer may read all of them while the layer before it is still running and needs that layer to
        // have finished only before it writes scratch memory (DEP_LATE). The exceptions: the first
        // kernel of the step (whatever ran before it in the stream may have produced its inputs), and a
        // sparse layer right after a selection layer, whose index list is written by the top-k.
        const Dep dep = i == 0 ? DEP_FIRST : (ctx->layer_overlap ? DEP_LATE : DEP_PREFETCH);
        if (schedule[i] == TIDAL_LAYER_FULL) {
            rc = run_dense(ctx, kv, qs[i], outs[i], nullptr, 0, false, dep, w, st);
        } else if (schedule[i] == TIDAL_LAYER_SELECT) {
            float* scores = (float*)((char*)ctx->ws + w.scores);
            const SelectPlan sp = select_plan(ctx, kv, Hi, k, false);
            // The score buffer's last reader is the top-k of the selection layer before this one. If a
            // sparse layer ran in between, its first kernel waited for that top-k before it let anything
            // else start, so nobody reads the buffer any more; right after another selection layer, wait.
            const bool scores_free = i > 0 && schedule[i - 1] != TIDAL_LAYER_SELECT;
            // The value pass adds to the output rows, four floats at a time: in place, or in the device rows the
            // caller of this function set aside (outputs in host memory), from where its last CTAs write outs[i].
            float* const sums = (acc && acc[i]) ? acc[i] : outs[i];
            if (can_split(ctx, kv, sp) && ((uintptr_t)sums & 15) == 0 && ensure_side_stream(ctx) == TIDAL_OK) {
                // key pass -> (value pass on the second stream) | top-k -> the layers that follow. A value
                // pass still in flight reads the score buffer and the statistics this key pass overwrites.
                if (side_pending) { if (cudaStreamWaitEvent(st, ctx->ev_join, 0) != cudaSuccess) return TIDAL_ERR_CUDA; side_pending = false; }
                rc = run_score_pass(ctx, kv, qs[i], sums, scores, w.score_stride, dep, scores_free, w, st);
                if (rc == TIDAL_OK) rc = run_value_pass(ctx, kv, sums, sums == outs[i] ? nullptr : outs[i], scores, w.score_stride, w, st);
                side_pending = rc == TIDAL_OK;
            } else {
                rc = run_dense(ctx, kv, qs[i], outs[i], scores, w.score_stride, sp.fuse, dep, w, st, sp.agg, sp.compact ? k : 0, scores_free);
            }
            if (rc == TIDAL_OK) rc = run_topk(ctx, kv, scores, w.score_stride, k, sp.rows, Hi, sp.fuse, idx, idx_count, w, st, sp.compact);
        } else {
            const bool fresh_idx = i == 0 || schedule[i - 1] == TIDAL_LAYER_SELECT;
            const bool has_prev = i > 0 && schedule[i - 1] == TIDAL_LAYER_SPARSE;
            const bool has_next = i + 1 < num_layers && schedule[i + 1] == TIDAL_LAYER_SPARSE;
            const Chain chain = !ctx->layer_overlap || (!has_prev && !has_next) ? CHAIN_NONE
                                : !has_prev ? CHAIN_FIRST : !has_next ? CHAIN_LAST : CHAIN_MIDDLE;
            rc = run_sparse(ctx, kv, qs[i], idx, idx_count, k, Hi, outs[i], fresh_idx ? DEP_FIRST : dep, chain, w, st);
        }
        if (rc != TIDAL_OK) return rc;
    }
    // the step is complete on the caller's stream only when the second stream's work is
    if (side_pending && cudaStreamWaitEvent(st, ctx->ev_join, 0) != cudaSuccess) return TIDAL_ERR_CUDA;
    return TIDAL_OK;
}

tidal_status_t tidal_decode_step_append(tidal_ctx_t* ctx, int32_t num_layers, const uint8_t* schedule,
                                        const tidal_kv_t* kv_per_layer, const void* const* q_per_layer,
                                        const void* const* k_new_per_layer, const void* const* v_new_per_layer,
                                        float* const* out_per_layer, int32_t k, int32_t granularity, int32_t* idx,
                                        int32_t* idx_count, void* stream) {
    if (!ctx || num_layers <= 0 || !schedule || !kv_per_layer || !q_per_layer || !out_per_layer || !idx || !idx_count ||
        !k_new_per_layer || !v_new_per_layer || k <= 0)
        return TIDAL_ERR_INVALID;
    for (int i = 0; i < num_layers; ++i) {
        const tidal_status_t rc = check_kv(&kv_per_layer[i]);
        if (rc != TIDAL_OK) return rc;
        if (!k_new_per_layer[i] || !v_new_per_layer[i] ||
            (((uintptr_t)k_new_per_layer[i] | (uintptr_t)v_new_per_layer[i]) & 15)) return TIDAL_ERR_INVALID;
        if (kv_per_layer[i].batch != kv_per_layer[0].batch || kv_per_layer[i].num_kv_heads != kv_per_layer[0].num_kv_heads)
            return TIDAL_ERR_INVALID;
    }
    if (cudaSetDevice(ctx->device) != cudaSuccess) return TIDAL_ERR_CUDA;
    // The whole step is validated (and its workspace sized) before the first row is written: an
    // argument error must leave the caches as they were.
    const tidal_status_t ok = decode_step_prepare(ctx, num_layers, schedule, kv_per_layer, q_per_layer, out_per_layer,
                                                  k, granularity, 0);
    if (ok != TIDAL_OK) return ok;
    const int pairs = kv_per_layer[0].batch * kv_per_layer[0].num_kv_heads;
    for (int l0 = 0; l0 < num_layers; l0 += APPEND_MAX_LAYERS) {
        const int n = std::min(APPEND_MAX_LAYERS, num_layers - l0);
        AppendBatchParams bp;
        std::memset(&bp, 0, sizeof bp);
        for (int j = 0; j < n; ++j) fill_append(bp.layer[j], ctx, &kv_per_layer[l0 + j], k_new_per_layer[l0 + j], v_new_per_layer[l0 + j]);
        kv_append_layers_kernel<<<dim3((pairs + 3) / 4, n, 1), 128, 0, (cudaStream_t)stream>>>(bp);
        ctx->launches++;
        if (cudaGetLastError() != cudaSuccess) return TIDAL_ERR_CUDA;
    }
    return tidal_decode_step(ctx, num_layers, schedule, kv_per_layer, q_per_layer, out_per_layer, k, granularity, idx,
                             idx_count, stream);
}

tidal_status_t tidal_decode_step(tidal_ctx_t* ctx, int32_t num_layers, const uint8_t* schedule,
                                 const tidal_kv_t* kv_per_layer, const void* const* q_per_layer,
                                 float* const* out_per_layer, int32_t k, int32_t granularity, int32_t* idx,
                                 int32_t* idx_count, void* stream) {
    if (!ctx || num_layers <= 0 || !schedule || !kv_per_layer || !q_per_layer || !out_per_layer || !idx || k <= 0)
        return TIDAL_ERR_INVALID;
    if (num_layers > 1024) return TIDAL_ERR_INVALID;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return TIDAL_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    tidal_status_t rc;
    raw_call_key(ctx->raw_scratch, ctx, 0, num_layers, schedule, kv_per_layer, q_per_layer, out_per_layer, idx, idx_count, k, granularity, st);
    if (replay_last(ctx, st, rc)) return rc;
    rc = decode_step_prepare(ctx, num_layers, schedule, kv_per_layer, q_per_layer, out_per_layer, k, granularity, 0);
    if (rc != TIDAL_OK) return rc;
    // (the workspace may just have moved: the remembered bytes must name the addresses the graph was built with)
    raw_call_key(ctx->raw_scratch, ctx, 0, num_layers, schedule, kv_per_layer, q_per_layer, out_per_layer, idx, idx_count, k, granularity, st);
    KeyBuilder kb;
    step_key(kb, ctx, 0, num_layers, schedule, kv_per_layer, k, granularity, 0);
    kb.add_raw(q_per_layer, sizeof(void*) * (size_t)num_layers);
    kb.add_raw(out_per_layer, sizeof(void*) * (size_t)num_layers);
    kb.add(idx); kb.add(idx_count);
    rc = run_graphed(ctx, kb, st, [&]() {
        return decode_step_enqueue(ctx, num_layers, schedule, kv_per_layer, q_per_layer, out_per_layer, k, granularity,
                                   idx, idx_count, 0, st);
    });
    if (rc == TIDAL_OK) remember_last(ctx); else ctx->last.exec = nullptr;
    return rc;
}

tidal_status_t tidal_set_attend_newest(tidal_ctx_t* ctx, int32_t enabled) {
    if (!ctx) return TIDAL_ERR_INVALID;
    ctx->attend_newest = enabled != 0;
    return TIDAL_OK;
}

tidal_status_t tidal_set_select_margin(tidal_ctx_t* ctx, float margin) {
    if (!ctx || !(margin >= 0.f) || margin > 64.f) return TIDAL_ERR_INVALID;
    ctx->select_margin = margin;
    return TIDAL_OK;
}

tidal_status_t tidal_set_layer_overlap(tidal_ctx_t* ctx, int32_t enabled) {
    if (!ctx) return TIDAL_ERR_INVALID;
    ctx->layer_overlap = enabled != 0;
    return TIDAL_OK;
}

tidal_status_t tidal_set_output_dtype(tidal_ctx_t* ctx, int32_t dtype) {
    if (!ctx || (dtype != TIDAL_OUT_F32 && dtype != TIDAL_OUT_BF16)) return TIDAL_ERR_INVALID;
    ctx->out_bf16 = dtype == TIDAL_OUT_BF16;
    return TIDAL_OK;
}

tidal_status_t tidal_set_graphs(tidal_ctx_t* ctx, int32_t enabled) {
    if (!ctx) return TIDAL_ERR_INVALID;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return TIDAL_ERR_CUDA;
    ctx->graphs_enabled = enabled != 0;
    if (!ctx->graphs_enabled) drop_graphs(ctx);
    return TIDAL_OK;
}

tidal_status_t tidal_decode_step_host(tidal_ctx_t* ctx, int32_t num_layers, const uint8_t* schedule,
                                      const tidal_kv_t* kv_per_layer, const void* q_host, float* out_host,
                                      int32_t k, int32_t granularity, void* stream) {
    if (!ctx || num_layers <= 0 || num_layers > 1024 || !schedule || !kv_per_layer || !q_host || !out_host || k <= 0)
        return TIDAL_ERR_INVALID;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return TIDAL_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    tidal_status_t rc;
    raw_call_key(ctx->raw_scratch, ctx, 1, num_layers, schedule, kv_per_layer, nullptr, nullptr, q_host, out_host, k, granularity, st);
    if (replay_last(ctx, st, rc)) {
        if (rc != TIDAL_OK) return rc;
        return cudaStreamSynchronize(st) == cudaSuccess ? TIDAL_OK : TIDAL_ERR_CUDA;
    }
    rc = check_kv(&kv_per_layer[0]);
    if (rc != TIDAL_OK) return rc;
    // Size the workspace for every layer first so that the staging pointers stay put.
    size_t need = 0;
    for (int i = 0; i < num_layers; ++i) {
        if ((rc = check_kv(&kv_per_layer[i])) != TIDAL_OK) return rc;
        need = std::max(need, ws_bytes_for(&kv_per_layer[i], k, num_layers));
    }
    if ((rc = ensure_all(ctx, &kv_per_layer[0], need)) != TIDAL_OK) return rc;
    // All layers must share batch and head counts (checked again below); the staging
    // offsets depend only on those and on max_ctx_len of the layer used for the layout.
    const tidal_kv_t* kv0 = &kv_per_layer[0];
    for (int i = 1; i < num_layers; ++i)
        if (kv_per_layer[i].max_ctx_len != kv0->max_ctx_len) return TIDAL_ERR_UNSUPPORTED;
    const WsLayout w = layout_ws(kv0, k, num_layers);
    const size_t rows = (size_t)kv0->batch * kv0->num_q_heads;
    char* ws = (char*)ctx->ws;
    char* qd = ws + w.q_stage;
    float* od = (float*)(ws + w.out_stage);
    const size_t out_elem = ctx->out_bf16 ? 2 : 4;            // bytes per output element, device and host side
    // Page-locked host memory is addressable from the device: the kernels then read the queries from the
    // caller's buffer and write their outputs straight into it (each output element once, as posted
    // writes over the bus), and the two copies, which would otherwise run before the first and after
    // the last layer, disappear (cfg3: 699 -> 679 us per step). Pageable buffers go through the staging
    // area and copies.
    auto device_alias = [](const void* p) -> void* {
        cudaPointerAttributes at;
        if (cudaPointerGetAttributes(&at, p) != cudaSuccess) { cudaGetLastError(); return nullptr; }
        if (at.type != cudaMemoryTypeHost || at.devicePointer == nullptr) return nullptr;
        return at.devicePointer;
    };
    char* out_alias = (char*)device_alias(out_host);
    char* q_alias = (char*)device_alias(q_host);
    if (q_alias && ((uintptr_t)q_alias & 15)) q_alias = nullptr;      // query rows are read as 16-byte pieces
    const void* qs[1024];
    float* outs[1024];
    // (a selection layer may run as two passes whose second adds to the output rows with reductions: those
    // sums stay in the staging area and the pass's last CTAs write the finished rows to the caller's buffer)
    float* acc[1024];
    for (int i = 0; i < num_layers; ++i) {
        qs[i] = (q_alias ? q_alias : qd) + (size_t)i * rows * HEAD_DIM * 2;
        outs[i] = (float*)((out_alias ? out_alias : (char*)od) + (size_t)i * rows * HEAD_DIM * out_elem);
        acc[i] = (out_alias && schedule[i] == TIDAL_LAYER_SELECT) ? (float*)((char*)od + (size_t)i * rows * HEAD_DIM * out_elem) : nullptr;
    }
    if ((rc = decode_step_prepare(ctx, num_layers, schedule, kv_per_layer, qs, outs, k, granularity, num_layers)) != TIDAL_OK)
        return rc;
    auto enqueue = [&]() -> tidal_status_t {
        if (!q_alias && cudaMemcpyAsync(qd, q_host, (size_t)num_layers * rows * HEAD_DIM * 2, cudaMemcpyHostToDevice, st) != cudaSuccess)
            return TIDAL_ERR_CUDA;
        const tidal_status_t r = decode_step_enqueue(ctx, num_layers, schedule, kv_per_layer, qs, outs, k, granularity,
                                                     (int*)(ws + w.idx), (int*)(ws + w.idx_count), num_layers, st, acc);
        if (r != TIDAL_OK) return r;
        if (!out_alias && cudaMemcpyAsync(out_host, od, (size_t)num_layers * rows * HEAD_DIM * out_elem, cudaMemcpyDeviceToHost, st) != cudaSuccess)
            return TIDAL_ERR_CUDA;
        return TIDAL_OK;
    };
    // The copies can be recorded with the layers only when both host buffers are page-locked.
    auto pinned = [](const void* p) {
        cudaPointerAttributes at;
        if (cudaPointerGetAttributes(&at, p) != cudaSuccess) { cudaGetLastError(); return false; }
        return at.type == cudaMemoryTypeHost;
    };
    if (pinned(q_host) && pinned(out_host)) {
        KeyBuilder kb;
        step_key(kb, ctx, 1, num_layers, schedule, kv_per_layer, k, granularity, num_layers);
        kb.add(q_host); kb.add(out_host);
        rc = run_graphed(ctx, kb, st, enqueue);
        if (rc == TIDAL_OK) {
            raw_call_key(ctx->raw_scratch, ctx, 1, num_layers, schedule, kv_per_layer, nullptr, nullptr, q_host, out_host, k, granularity, st);
            remember_last(ctx);
        } else {
            ctx->last.exec = nullptr;
        }
    } else {
        ctx->last.exec = nullptr;
        rc = enqueue();
    }
    if (rc != TIDAL_OK) return rc;
    return cudaStreamSynchronize(st) == cudaSuccess ? TIDAL_OK : TIDAL_ERR_CUDA;
}

tidal_status_t tidal_device_status(tidal_ctx_t* ctx, void* stream) {
    if (!ctx) return TIDAL_ERR_INVALID;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return TIDAL_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaStreamSynchronize(st) != cudaSuccess) return TIDAL_ERR_CUDA;
    int word = 0;
    if (cudaMemcpy(&word, ctx->status, sizeof word, cudaMemcpyDeviceToHost) != cudaSuccess) return TIDAL_ERR_CUDA;
    if (word != 0 && cudaMemset(ctx->status, 0, sizeof(int)) != cudaSuccess) return TIDAL_ERR_CUDA;
    if (word & STATUS_SPLIT_OVERFLOW) return TIDAL_ERR_INTERNAL;
    return word ? TIDAL_ERR_INDEX : TIDAL_OK;
}


int64_t tidal_launch_count(const tidal_ctx_t* ctx) { return ctx ? ctx->launches : 0; }

const char* tidal_strerror(tidal_status_t s) {
    switch (s) {
        case TIDAL_OK: return "ok";
        case TIDAL_ERR_INVALID: return "invalid argument";
        case TIDAL_ERR_UNSUPPORTED: return "unsupported configuration";
        case TIDAL_ERR_NOMEM: return "out of device memory";
        case TIDAL_ERR_CUDA: return "CUDA runtime error";
        case TIDAL_ERR_TIMEOUT: return "device-side wait timed out";
        case TIDAL_ERR_INDEX: return "token index or page id out of range";
        case TIDAL_ERR_TOO_LARGE: return "problem exceeds the fixed scratch of the allocation-free entry point";
        case TIDAL_ERR_INTERNAL: return "launch plan inconsistency detected on the device (results are invalid)";
        default: return "unknown status";
    }
}

}  // extern "C"

// =====================================================================================================
// Sparse attention for callers that must not allocate.
//
// Everything the kernel needs beyond the caller's inputs and outputs (the split partial results,
// the arrival counters, the pool cursors and a status word) lives in one file-scope device array
// of fixed size, so this entry point never calls cudaMalloc, cudaFree or anything that allocates.
// =====================================================================================================
namespace {

constexpr int NOALLOC_MAX_ROWS = 4096;      // (sequence, query head) rows; also the number of partial slots
constexpr size_t NOALLOC_PART_O = (size_t)NOALLOC_MAX_ROWS * HEAD_DIM * sizeof(float);   // 2 MiB
constexpr size_t NOALLOC_PART_ML = (size_t)NOALLOC_MAX_ROWS * sizeof(float2);           // 32 KiB
constexpr size_t NOALLOC_WORDS = 2 * (size_t)NOALLOC_MAX_ROWS * sizeof(int) + 256;      // counters, cursors, status
constexpr size_t NOALLOC_BYTES = NOALLOC_PART_O + NOALLOC_PART_ML + NOALLOC_WORDS;      // 2 MiB + 64 KiB + 256 B, about 2.06 MiB

// Held by every GPU that loads the library until the process exits. In host code this name is
// only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_BYTES];

constexpr int NOALLOC_MAX_DEVICES = 64;
struct NoallocDevice {
    bool ready = false;
    unsigned char* scratch = nullptr;       // device address of g_noalloc_scratch on this GPU
    int slots = 0;                          // resident CTAs of the sparse kernel on this GPU
};
NoallocDevice g_noalloc_dev[NOALLOC_MAX_DEVICES];
std::mutex g_noalloc_mutex;

// Once per device, with that device current: resolve the scratch array's device address and
// prepare the kernel (shared-memory opt-in, occupancy). Allocates nothing.
tidal_status_t noalloc_setup(int device, const NoallocDevice** out) {
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    NoallocDevice& d = g_noalloc_dev[device];
    if (!d.ready) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || ptr == nullptr) {
            cudaGetLastError();
            return TIDAL_ERR_CUDA;
        }
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) return TIDAL_ERR_CUDA;
        const int slots = resident_ctas(attn_kernel<MODE_SPARSE, SPARSE_NW, SPARSE_STAGES>, SPARSE_NW * 32,
                                        attn_smem<MODE_SPARSE, SPARSE_NW, SPARSE_STAGES>(), sms);
        if (slots <= 0) { cudaGetLastError(); return TIDAL_ERR_CUDA; }
        d.scratch = static_cast<unsigned char*>(ptr);
        d.slots = slots;
        d.ready = true;
    }
    *out = &d;
    return TIDAL_OK;
}

}  // namespace

extern "C" tidal_status_t tidal_sparse_attn_noalloc(const tidal_kv_t* kv, const void* q, const int32_t* idx,
                                                    const int32_t* idx_count, int32_t k,
                                                    int32_t num_index_heads, float* out, void* stream) {
    if (!q || !out || !idx || ((uintptr_t)q & 15)) return TIDAL_ERR_INVALID;
    tidal_status_t rc = check_kv(kv);
    if (rc != TIDAL_OK) return rc;
    if (k <= 0) return TIDAL_ERR_INVALID;
    const int Hi = num_index_heads;
    if (Hi != kv->num_q_heads && Hi != kv->num_kv_heads && Hi != 1) return TIDAL_ERR_INVALID;
    if (kv->kv_dtype != TIDAL_KV_BF16) return TIDAL_ERR_UNSUPPORTED;
    const long long rows = (long long)kv->batch * kv->num_q_heads;
    if (rows > NOALLOC_MAX_ROWS) return TIDAL_ERR_TOO_LARGE;
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) { cudaGetLastError(); return TIDAL_ERR_CUDA; }
    if (device < 0 || device >= NOALLOC_MAX_DEVICES) return TIDAL_ERR_UNSUPPORTED;
    const NoallocDevice* dev = nullptr;
    if ((rc = noalloc_setup(device, &dev)) != TIDAL_OK) return rc;

    // Every item (one query head, or one KV head's group) is shared by S CTAs through its pool
    // cursor; a row then needs S partial slots and the scratch holds NOALLOC_MAX_ROWS of them.
    const int per_batch = (Hi == kv->num_q_heads) ? kv->num_q_heads : kv->num_kv_heads;
    const int items = kv->batch * per_batch;
    const int tiles_item = (k + TILE - 1) / TILE;
    int S = std::max(1, std::min(dev->slots, GRID_MAX) / items);
    S = std::min(S, std::max(1, tiles_item / MIN_TILES_PER_CTA));
    while (S > 1 && rows * S > NOALLOC_MAX_ROWS) --S;

    unsigned char* base = dev->scratch;
    int* words = reinterpret_cast<int*>(base + NOALLOC_PART_O + NOALLOC_PART_ML);
    AttnParams a;
    std::memset(&a, 0, sizeof a);
    a.q = (const __nv_bfloat16*)q;
    a.k = (const __nv_bfloat16*)kv->k;
    a.v = (const __nv_bfloat16*)kv->v;
    a.out = out;
    a.stride_b = kv->stride_b; a.stride_pos = kv->stride_pos; a.stride_head = kv->stride_head;
    a.stride_page = kv->stride_page;
    a.page_table = kv->page_table; a.max_pages = kv->max_pages_per_seq; a.num_pages = kv->num_pages;
    a.paged = kv->kv_layout == TIDAL_KV_PAGED;
    a.ctx_lens = kv->ctx_lens;
    a.max_ctx = kv->max_ctx_len;
    a.Hq = kv->num_q_heads; a.Hkv = kv->num_kv_heads; a.G = a.Hq / a.Hkv;
    a.scale = kv->sm_scale > 0.f ? kv->sm_scale : 1.0f / std::sqrt((float)kv->head_dim);
    a.scale_log2 = a.scale * 1.4426950408889634f;
    a.batch = kv->batch;
    a.splits_per_item = S;
    a.idx = idx; a.idx_count = idx_count; a.budget = k; a.Hi = Hi;
    a.part_o = reinterpret_cast<float*>(base);
    a.part_ml = reinterpret_cast<float2*>(base + NOALLOC_PART_O);
    a.counters = words;
    a.tile_ctr = words + NOALLOC_MAX_ROWS;
    a.ctr_stride = 1;
    a.status = words + 2 * NOALLOC_MAX_ROWS;
    a.max_splits = S;
    a.hist_shift = 21;
    a.pdl = 0;
    a.wait_first = 1;

    cudaStream_t st = (cudaStream_t)stream;
    // The array keeps whatever the previous call left behind: the counters and cursors must read
    // zero when the kernel starts (the partial results are always written before they are read).
    if (cudaMemsetAsync(words, 0, NOALLOC_WORDS, st) != cudaSuccess) { cudaGetLastError(); return TIDAL_ERR_CUDA; }
    attn_kernel<MODE_SPARSE, SPARSE_NW, SPARSE_STAGES>
        <<<S * items, SPARSE_NW * 32, attn_smem<MODE_SPARSE, SPARSE_NW, SPARSE_STAGES>(), st>>>(a);
    return cudaGetLastError() == cudaSuccess ? TIDAL_OK : TIDAL_ERR_CUDA;
}
