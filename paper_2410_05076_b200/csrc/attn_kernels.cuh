// Split-context decode attention for one query token per sequence (sm_100a).
//
// One kernel template serves the three layer types of the paper's Algorithm 1:
//   MODE_FULL    FullAttention(q, C[:])                      (Eq. 1 over the whole cache)
//   MODE_SELECT  the same, and the scaled logits q.k/sqrt(d) are written out so
//                that the top-k kernel can rank them (Section 3: the inner
//                products are stored during full attention)
//   MODE_SPARSE  SparseAttention(q, C[rho]): Eq. 1 over the listed positions only
//
// Work decomposition. A CTA owns one (sequence, KV head [or query head], chunk of
// the context / of the index list). Its warps take 16-position tiles round
// robin; every warp runs a private cp.async ring (global -> shared, 16-byte
// copies, no L1 allocation) so no CTA-wide barrier sits on the streaming path.
// The bytes are consumed by bf16 mma.sync m16n8k16 with fp32 accumulation:
//   S^T[16 pos x 8 heads] = K[16 pos x 128] . Q^T[128 x 8 heads]
//   O^T[128 x 8 heads]   += V^T[128 x 16 pos] . P^T[16 pos x 8 heads]
// i.e. the GQA group's query heads are the N columns, so the K/V bytes are read
// once per KV head however large the group is. The path is HBM-bound (4 flop
// per byte at group 4); the tensor cores only keep the issue slots free.
// Because the contraction index of the first product (the head dimension) and
// the row index of the second (again the head dimension) are dummy / relabelable
// indices, every lane fetches plain 16-byte pieces of a row from shared memory;
// two byte-permutes per register pair build the V^T fragments.
// Softmax is the usual running-max form in base 2; each warp keeps (m, l, O),
// warps are merged in shared memory, CTAs write (m, l, O) partials and the last
// CTA of a (sequence, head group) to finish combines them — no second launch
// and no waiting on other CTAs.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace tidal {

enum { MODE_FULL = 0, MODE_SELECT = 1, MODE_SPARSE = 2 };
// Bits of the sticky device status word.
enum { STATUS_BAD_INDEX = 1, STATUS_BAD_PAGE = 2, STATUS_SPLIT_OVERFLOW = 4 };

constexpr int HEAD_DIM = 128;
constexpr int TILE = 16;                 // positions per tile == page size
constexpr int TILE_BYTES = TILE * HEAD_DIM * 2;   // 4 KB of K, same of V
constexpr int STAGE_BYTES = 2 * TILE_BYTES;
// 8-bit caches (FP8 E4M3 codes): rows are 128 bytes, a 16-position tile is 2 KB of K and 2 KB of V.
constexpr int ROW_BYTES8 = HEAD_DIM;
constexpr int TILE_BYTES8 = TILE * ROW_BYTES8;
constexpr int STAGE_BYTES8 = 2 * TILE_BYTES8;
constexpr int HIST_BINS = 2048;          // global histogram row: up to 11 top bits of the score key
constexpr int HIST_SMEM_WORDS = 8192;    // shared histogram: columns x bins <= 8192 counters (32 KB)
// Candidate compaction in the selection layer's kernel (layout of the 32 KB behind the rings):
constexpr int CAL_TILES = 3;             // tiles per warp whose scores are staged to estimate the threshold (one ring fill)
constexpr int CAND_COLS = 4;             // query heads per KV head it supports
constexpr int CAND_BUF = 64;             // per (warp, head) buffer of candidates in shared memory ...
constexpr int CAND_FLUSH = 32;           // ... written out once it holds this many (two more tiles add at most 32)
constexpr int GRAB_TILES = 4;            // tiles a warp takes from its item's pool at a time afterwards (gather kernel)
constexpr int GRAB_TILES_DENSE = 2;      // the same for the streaming kernels, whose items hold thousands of tiles

struct AttnParams {
    const __nv_bfloat16* q;
    const __nv_bfloat16* k;
    const __nv_bfloat16* v;
    float* out;                // [B, Hq, 128]; bf16 instead of fp32 when out_bf16 is set
    float* out_final;          // value pass of a two-pass selection layer: where the finished rows go (null: out itself)
    int out_bf16;
    long long stride_b, stride_pos, stride_head, stride_page;
    const int* page_table;
    int max_pages, num_pages, paged;
    const int* ctx_lens;
    int max_ctx;               // host bound of ctx_lens; larger device values are clamped to it
    int Hq, Hkv, G;
    float scale, scale_log2;
    const float* k_scale;      // 8-bit caches: per-KV-head dequantisation scales [Hkv] (null: 1)
    const float* v_scale;
    int batch;
    int splits_per_item;       // > 0: pooled mode, CTA c works on item c % items; an item is served by every CTA
                               // of the grid that maps to it (this many, or one more); 0: static flat split
    float* scores;             // MODE_SELECT: [B, Hq, score_stride], or [B, Hkv, score_stride] with agg
    int agg;                   // MODE_SELECT: store one row per KV head, the sum of its group's scaled logits
    long long score_stride;
    const int* idx;            // MODE_SPARSE: [B, Hi, k]
    const int* idx_count;      // MODE_SPARSE: [B] or null
    int budget, Hi;            // MODE_SPARSE: entries per index row, index heads
    unsigned* split_max;       // two-pass selection layer: [Hq] key of every head's largest logit (0 between layers)
    float* split_sum;          // ... and [Hq] the sum of its softmax weights relative to that logit (0 between layers)
    float* part_o;             // [B*Hq, max_splits, 128] un-normalised partial outputs
    float2* part_ml;           // [B*Hq, max_splits] (running max in base 2, sum)
    int* counters;             // one per (sequence, item), zero between launches
    int max_splits;            // partial slots per (sequence, head) row
    // MODE_SELECT, optional (one sequence, one token set per query head, groups of at most four): instead
    // of the histogram, every CTA estimates a threshold per head from its first tiles and appends the
    // (key, position) of every score at or above it to that head's candidate list; the largest threshold
    // any CTA used is recorded, so that the top-k can tell whether the list is complete down to the k-th score.
    int compact;
    uint2* cand;               // [B*Hq][cand_stride]
    long long cand_stride;
    int* cand_cursor;          // [B*Hq][ctr_stride] entries in the list, zero between launches
    unsigned* thr_max;         // [B*Hq][ctr_stride] largest threshold key used, zero between launches
    float margin;              // the threshold aims at this multiple of k' / N of the scores
    unsigned* hist;            // MODE_SELECT, optional: [B*Hq][HIST_BINS] += histogram of the top key bits
    int hist_shift;            // bin = key >> hist_shift (21: 2048 bins, 22: 1024 bins for groups above 4)
    int* tile_ctr;             // splits_per_item > 0: per-item pool cursor, zero between launches
    int ctr_stride;            // ints between the cursors of consecutive items (32: one 128-byte line each)
    int pdl;                   // launched with programmatic stream serialization: see pdl_wait()
    int wait_first;            // the preceding kernel may have written ctx_lens / idx: wait before reading anything
    int wait_late;             // every input (query, lengths, index list, cache rows) was complete before the
                               // preceding kernel started: stream the whole item first and wait for that kernel
                               // only before the first write to memory shared with it (partial results, counters)
    int trigger_early;         // with wait_late: let the next kernel's CTAs take the slots of ours as they retire,
                               // without first waiting for the kernel before us (see the host's launch rule)
    int* status;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// 16-byte global->shared copy that bypasses L1; src_bytes = 0 zero-fills.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes)
                 : "memory");
}
__device__ __forceinline__ void cp_async16_full(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(src) : "memory");
}
// The same with an L2 eviction hint: the KV stream is read once, so its lines should be the first
// to go and leave the scores, index lists and partial results of the step in L2.
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;\n" : "=l"(pol));
    return pol;
}
// Scores are written once and read back by the top-k right after: they are asked to stay in L2
// (evict-last), so that they are not written out to DRAM in between.
__device__ __forceinline__ uint64_t l2_evict_last_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;\n" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void st_keep(float* ptr, float v, uint64_t pol) {
    asm volatile("st.global.L2::cache_hint.f32 [%0], %1, %2;\n" ::"l"(ptr), "f"(v), "l"(pol) : "memory");
}
__device__ __forceinline__ void cp_async16_hint(uint32_t dst, const void* src, int src_bytes, uint64_t pol) {
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2, %3;\n" ::"r"(dst), "l"(src), "r"(src_bytes), "l"(pol) : "memory");
}
__device__ __forceinline__ void cp_async16_full_hint(uint32_t dst, const void* src, uint64_t pol) {
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "l"(pol) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}

// Programmatic dependent launch: this grid may start while the previous kernel of the stream
// is still draining. pdl_wait() blocks until that kernel has completed and its writes are
// visible; pdl_trigger() lets the next kernel start filling SMs as our CTAs retire.
// One output element: fp32, or rounded to bf16 (nearest even) for callers that feed a bf16 GEMM next.
__device__ __forceinline__ void store_out(const AttnParams& p, long long i, float v) {
    if (p.out_bf16) reinterpret_cast<__nv_bfloat16*>(p.out)[i] = __float2bfloat16_rn(v);
    else p.out[i] = v;
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }

__device__ __forceinline__ void lds128(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}

// Four 8x8 b16 matrices, transposed on the way in: register j of lane (gid, tig) holds
// elements (row 2*tig, col gid) and (row 2*tig+1, col gid) of matrix j.
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}

// Four 8x8 b16 matrices as they lie in memory: register j of lane (gid, tig) holds elements
// (row gid, cols 2*tig, 2*tig+1) of matrix j; lane l supplies the address of row l&7 of matrix l>>3.
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                               uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Transpose an 8x8 matrix of 16-bit elements held one 32-bit register per lane.
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(d) : "r"(a));
    return d;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;\n" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}

// Order-preserving key of a score: larger float <=> larger key, -0 counted as +0.
__device__ __forceinline__ uint32_t score_key_bits(float s) {
    uint32_t u = __float_as_uint(s);
    if (u == 0x80000000u) u = 0u;
    if ((u & 0x7fffffffu) > 0x7f800000u) return 0u;      // not a number: below every number
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Per-warp running softmax state. Columns of the MMA tiles are query heads:
// this lane owns heads 2*tig and 2*tig+1 of the group.
struct WarpAcc {
    float m[2];        // running max of logit*log2(e), identical in all lanes that share tig
    float l[2];        // this lane's share of the running sum
    float o[8][4];     // O^T fragments: o[t][0..1] d = 16*t+gid, o[t][2..3] d = 16*t+8+gid
};

// Consume one staged tile: 16 K rows at ks, 16 V rows at vs (swizzled, see
// the issue code), `vmask` bit r set when row r is a real cached token,
// pos_base + r its position (only used to store scores).
// What one warp needs to compact candidates while it consumes a tile (selection layers only).
struct CandWarp {
    uint32_t* stage;           // calibration: where this tile's keys go, [16 rows][CAND_COLS]; null afterwards
    float thr0, thr1;          // thresholds of this lane's two heads
    uint2* buf;                // this warp's candidate buffers [CAND_COLS][CAND_BUF]
    int* cnt;                  // ... and their fill counts [CAND_COLS]
};

template <int MODE>
__device__ __forceinline__ void consume_tile(const AttnParams& p, uint32_t ks, uint32_t vs,
                                             const uint32_t (&qf)[4][4], WarpAcc& acc, uint32_t vmask,
                                             int gid, int tig, float* score_row0, float* score_row1,
                                             int pos_base, uint32_t* hist, const CandWarp* cw = nullptr) {
    // ---- S^T = K . Q^T ------------------------------------------------------
    // Two independent accumulator chains (even / odd 32-element blocks of the head dimension).
    float s[4] = {0.f, 0.f, 0.f, 0.f};
    float s2[4] = {0.f, 0.f, 0.f, 0.f};
    const uint32_t krow = ks + gid * 256;
    const uint32_t kswz = (gid & 1) << 2;
#pragma unroll
    for (int j = 0; j < 4; j += 2) {
        uint32_t ka[4], kb[4], kc[4], kd[4];
        const uint32_t off0 = (((4 * j + tig) ^ kswz) << 4), off1 = (((4 * j + 4 + tig) ^ kswz) << 4);
        lds128(krow + off0, ka);                // row gid
        lds128(krow + 8 * 256 + off0, kb);      // row gid + 8
        lds128(krow + off1, kc);
        lds128(krow + 8 * 256 + off1, kd);
        mma_bf16_16816(s, ka[0], kb[0], ka[1], kb[1], qf[j][0], qf[j][1]);
        mma_bf16_16816(s2, kc[0], kd[0], kc[1], kd[1], qf[j + 1][0], qf[j + 1][1]);
        mma_bf16_16816(s, ka[2], kb[2], ka[3], kb[3], qf[j][2], qf[j][3]);
        mma_bf16_16816(s2, kc[2], kd[2], kc[3], kd[3], qf[j + 1][2], qf[j + 1][3]);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) s[i] += s2[i];
    const bool v0 = (vmask >> gid) & 1u, v1 = (vmask >> (gid + 8)) & 1u;
    if (MODE == MODE_SELECT) {
        // s[0],s[1]: (pos gid; heads 2tig, 2tig+1)   s[2],s[3]: (pos gid+8; same heads)
        const float f0 = s[0] * p.scale, f1 = s[1] * p.scale, f2 = s[2] * p.scale, f3 = s[3] * p.scale;
        const uint64_t keep = l2_evict_last_policy();
        if (p.agg) {
            // One ranking score per (position, KV head): the group's columns summed (unused columns
            // hold zeros). Lanes that differ only in tig hold the columns of one position.
            float a0 = f0 + f1, a1 = f2 + f3;
            a0 += __shfl_xor_sync(0xffffffffu, a0, 1);
            a1 += __shfl_xor_sync(0xffffffffu, a1, 1);
            a0 += __shfl_xor_sync(0xffffffffu, a0, 2);
            a1 += __shfl_xor_sync(0xffffffffu, a1, 2);
            if (tig == 0) {
                if (v0) st_keep(score_row0 + pos_base + gid, a0, keep);
                if (v1) st_keep(score_row0 + pos_base + gid + 8, a1, keep);
                if (hist) {
                    if (v0) atomicAdd(hist + (score_key_bits(a0) >> p.hist_shift), 1u);
                    if (v1) atomicAdd(hist + (score_key_bits(a1) >> p.hist_shift), 1u);
                }
            }
        } else {
        if (score_row0) {
            if (v0) st_keep(score_row0 + pos_base + gid, f0, keep);
            if (v1) st_keep(score_row0 + pos_base + gid + 8, f2, keep);
        }
        if (score_row1) {
            if (v0) st_keep(score_row1 + pos_base + gid, f1, keep);
            if (v1) st_keep(score_row1 + pos_base + gid + 8, f3, keep);
        }
        if (cw) {
            if (cw->stage) {
                // calibration tiles: keep the keys (0 where there is no token) for the threshold estimate
                if (score_row0) {
                    cw->stage[gid * CAND_COLS + 2 * tig] = v0 ? score_key_bits(f0) : 0u;
                    cw->stage[(gid + 8) * CAND_COLS + 2 * tig] = v1 ? score_key_bits(f2) : 0u;
                }
                if (score_row1) {
                    cw->stage[gid * CAND_COLS + 2 * tig + 1] = v0 ? score_key_bits(f1) : 0u;
                    cw->stage[(gid + 8) * CAND_COLS + 2 * tig + 1] = v1 ? score_key_bits(f3) : 0u;
                }
            } else {
                // Slots in the warp's per-head buffers come from ballots, not from atomics that return a
                // value (their round trips would stall the warp four times per tile): the lanes that share
                // a tig hold the scores of the same two heads.
                const bool c0 = score_row0 && v0 && f0 >= cw->thr0, c2 = score_row0 && v1 && f2 >= cw->thr0;
                const bool c1 = score_row1 && v0 && f1 >= cw->thr1, c3 = score_row1 && v1 && f3 >= cw->thr1;
                const unsigned m0 = __ballot_sync(0xffffffffu, c0), m2 = __ballot_sync(0xffffffffu, c2);
                const unsigned m1 = __ballot_sync(0xffffffffu, c1), m3 = __ballot_sync(0xffffffffu, c3);
                if (m0 | m1 | m2 | m3) {
                    const unsigned grp = 0x11111111u << tig, below = (1u << (gid * 4 + tig)) - 1u;
                    const int h0 = 2 * tig, h1 = h0 + 1;
                    const int base0 = score_row0 ? cw->cnt[h0] : 0, base1 = score_row1 ? cw->cnt[h1] : 0;
                    const int n00 = __popc(m0 & grp), n01 = __popc(m2 & grp), n10 = __popc(m1 & grp), n11 = __popc(m3 & grp);
                    if (c0) cw->buf[h0 * CAND_BUF + base0 + __popc(m0 & grp & below)] = make_uint2(score_key_bits(f0), pos_base + gid);
                    if (c2) cw->buf[h0 * CAND_BUF + base0 + n00 + __popc(m2 & grp & below)] = make_uint2(score_key_bits(f2), pos_base + gid + 8);
                    if (c1) cw->buf[h1 * CAND_BUF + base1 + __popc(m1 & grp & below)] = make_uint2(score_key_bits(f1), pos_base + gid);
                    if (c3) cw->buf[h1 * CAND_BUF + base1 + n10 + __popc(m3 & grp & below)] = make_uint2(score_key_bits(f3), pos_base + gid + 8);
                    __syncwarp();                     // every lane has read the counts it needs
                    if (gid == 0) {
                        if (score_row0 && (n00 | n01)) cw->cnt[h0] = base0 + n00 + n01;
                        if (score_row1 && (n10 | n11)) cw->cnt[h1] = base1 + n10 + n11;
                    }
                }
            }
        }
        if (hist) {      // histogram of the top key bits of every stored score, per head
            const int nb = 1 << (32 - p.hist_shift);
            uint32_t* h0 = hist + (2 * tig) * nb;
            uint32_t* h1 = h0 + nb;
            if (score_row0) {
                if (v0) atomicAdd(h0 + (score_key_bits(f0) >> p.hist_shift), 1u);
                if (v1) atomicAdd(h0 + (score_key_bits(f2) >> p.hist_shift), 1u);
            }
            if (score_row1) {
                if (v0) atomicAdd(h1 + (score_key_bits(f1) >> p.hist_shift), 1u);
                if (v1) atomicAdd(h1 + (score_key_bits(f3) >> p.hist_shift), 1u);
            }
        }
        }
    }
    // ---- running softmax (base 2) ---------------------------------------------
    const float NEG_INF = -INFINITY;
    float t0 = v0 ? s[0] * p.scale_log2 : NEG_INF, t1 = v0 ? s[1] * p.scale_log2 : NEG_INF;
    float t2 = v1 ? s[2] * p.scale_log2 : NEG_INF, t3 = v1 ? s[3] * p.scale_log2 : NEG_INF;
    float mx0 = fmaxf(t0, t2), mx1 = fmaxf(t1, t3);
    // The running max rarely grows after the first tiles: one vote decides whether the
    // cross-lane max and the rescale of the accumulators are needed at all.
    if (__any_sync(0xffffffffu, (mx0 > acc.m[0]) || (mx1 > acc.m[1]))) {
#pragma unroll
        for (int sh = 4; sh <= 16; sh <<= 1) {
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, sh));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, sh));
        }
        const float g0 = fmaxf(acc.m[0], mx0), g1 = fmaxf(acc.m[1], mx1);
        // exp2(-inf - finite) = 0; when both are -inf the accumulators are still 0.
        const float a0 = (g0 == NEG_INF) ? 1.f : fast_exp2(acc.m[0] - g0);
        const float a1 = (g1 == NEG_INF) ? 1.f : fast_exp2(acc.m[1] - g1);
        acc.l[0] *= a0;
        acc.l[1] *= a1;
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            acc.o[t][0] *= a0; acc.o[t][1] *= a1; acc.o[t][2] *= a0; acc.o[t][3] *= a1;
        }
        acc.m[0] = g0;
        acc.m[1] = g1;
    }
    const float mn0 = acc.m[0], mn1 = acc.m[1];
    const float ms0 = (mn0 == NEG_INF) ? 0.f : mn0, ms1 = (mn1 == NEG_INF) ? 0.f : mn1;
    const float p0 = fast_exp2(t0 - ms0), p1 = fast_exp2(t1 - ms1);
    const float p2 = fast_exp2(t2 - ms0), p3 = fast_exp2(t3 - ms1);
    acc.l[0] += p0 + p2;
    acc.l[1] += p1 + p3;
    // P^T as the B operand: transpose (pos x head) -> (head x pos) across the warp.
    const uint32_t pb0 = movmatrix_trans(pack_bf16(p0, p1));
    const uint32_t pb1 = movmatrix_trans(pack_bf16(p2, p3));
    // ---- O^T += V^T . P^T ------------------------------------------------------
    // ldmatrix.trans hands out V^T fragments directly: for the 16 head-dim rows of block t the
    // four matrices are (pos 0-7 | 8-15) x (16-byte pieces 2t | 2t+1) of the V tile. Lane l
    // addresses row (l&7) + 8*(l>>4) and piece 2t + ((l>>3)&1); piece c of row r sits at c ^ (r&7).
    const int lane = gid * 4 + tig;
    const int rr = lane & 7, mb = (lane >> 3) & 1;
    const uint32_t vlane = vs + (rr + ((lane >> 4) << 3)) * 256 + ((rr ^ mb) << 4);
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        uint32_t a[4];
        ldmatrix_x4_trans(vlane ^ (t << 5), a);       // ring slots are 256-byte aligned
        mma_bf16_16816(acc.o[t], a[0], a[1], a[2], a[3], pb0, pb1);
    }
}

__device__ __forceinline__ void mma_f16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                              uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// Four E4M3 codes in one word -> two fp16 pairs (exact: every E4M3 value is an fp16 value).
__device__ __forceinline__ void e4m3x4_to_f16x2x2(uint32_t w, uint32_t& lo, uint32_t& hi) {
    asm("{\n.reg .b16 l, h;\nmov.b32 {l, h}, %2;\ncvt.rn.f16x2.e4m3x2 %0, l;\ncvt.rn.f16x2.e4m3x2 %1, h;\n}\n"
        : "=r"(lo), "=r"(hi) : "r"(w));
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;\n" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
// Two bf16 in one word -> the same two numbers as fp16 (exact inside fp16's range).
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t w) {
    return pack_f16(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}

// The same step for a tile of an 8-bit cache: 16 key rows of 128 bytes at ks, 16 value rows at vs, both
// holding E4M3 codes (16-byte piece c of row r at piece c ^ ((r&1)<<2) for K, c ^ (r&7) for V). Codes
// are converted to fp16 in registers and both products run as fp16 MMAs; qf holds the query as fp16:
// qf[s][2i], qf[s][2i+1] are head-dim elements 16c + 4i .. 16c + 4i + 3 for this lane's piece c = tig + 4s.
// `scale` / `scale_log2` already contain the head's key scale. The O^T fragments come out with a
// different row order than in the 16-bit kernel: o[t][0..1] is d = 16t + 2gid, o[t][2..3] is d = 16t + 2gid + 1.
template <int MODE>
__device__ __forceinline__ void consume_tile8(const AttnParams& p, float scale, float scale_log2, uint32_t ks,
                                              uint32_t vs, const uint32_t (&qf)[2][8], WarpAcc& acc, uint32_t vmask,
                                              int gid, int tig, float* score_row0, float* score_row1,
                                              int pos_base, uint32_t* hist) {
    float s[4] = {0.f, 0.f, 0.f, 0.f};
    float s2[4] = {0.f, 0.f, 0.f, 0.f};
    const uint32_t krow = ks + gid * ROW_BYTES8;
    const uint32_t kswz = (gid & 1) << 2;
#pragma unroll
    for (int sl = 0; sl < 2; ++sl) {
        uint32_t ka[4], kb[4];
        const uint32_t off = ((uint32_t)((tig + 4 * sl) ^ kswz)) << 4;
        lds128(krow + off, ka);                        // row gid, 16 codes
        lds128(krow + 8 * ROW_BYTES8 + off, kb);       // row gid + 8
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint32_t a0, a2, a1, a3;
            e4m3x4_to_f16x2x2(ka[i], a0, a2);
            e4m3x4_to_f16x2x2(kb[i], a1, a3);
            if (i & 1) mma_f16_16816(s2, a0, a1, a2, a3, qf[sl][2 * i], qf[sl][2 * i + 1]);
            else mma_f16_16816(s, a0, a1, a2, a3, qf[sl][2 * i], qf[sl][2 * i + 1]);
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) s[i] += s2[i];
    const bool v0 = (vmask >> gid) & 1u, v1 = (vmask >> (gid + 8)) & 1u;
    if (MODE == MODE_SELECT) {
        const float f0 = s[0] * scale, f1 = s[1] * scale, f2 = s[2] * scale, f3 = s[3] * scale;
        const uint64_t keep = l2_evict_last_policy();
        if (p.agg) {
            float a0 = f0 + f1, a1 = f2 + f3;
            a0 += __shfl_xor_sync(0xffffffffu, a0, 1);
            a1 += __shfl_xor_sync(0xffffffffu, a1, 1);
            a0 += __shfl_xor_sync(0xffffffffu, a0, 2);
            a1 += __shfl_xor_sync(0xffffffffu, a1, 2);
            if (tig == 0) {
                if (v0) st_keep(score_row0 + pos_base + gid, a0, keep);
                if (v1) st_keep(score_row0 + pos_base + gid + 8, a1, keep);
                if (hist) {
                    if (v0) atomicAdd(hist + (score_key_bits(a0) >> p.hist_shift), 1u);
                    if (v1) atomicAdd(hist + (score_key_bits(a1) >> p.hist_shift), 1u);
                }
            }
        } else {
            if (score_row0) {
                if (v0) st_keep(score_row0 + pos_base + gid, f0, keep);
                if (v1) st_keep(score_row0 + pos_base + gid + 8, f2, keep);
            }
            if (score_row1) {
                if (v0) st_keep(score_row1 + pos_base + gid, f1, keep);
                if (v1) st_keep(score_row1 + pos_base + gid + 8, f3, keep);
            }
            if (hist) {
                const int nb = 1 << (32 - p.hist_shift);
                uint32_t* h0 = hist + (2 * tig) * nb;
                uint32_t* h1 = h0 + nb;
                if (score_row0) {
                    if (v0) atomicAdd(h0 + (score_key_bits(f0) >> p.hist_shift), 1u);
                    if (v1) atomicAdd(h0 + (score_key_bits(f2) >> p.hist_shift), 1u);
                }
                if (score_row1) {
                    if (v0) atomicAdd(h1 + (score_key_bits(f1) >> p.hist_shift), 1u);
                    if (v1) atomicAdd(h1 + (score_key_bits(f3) >> p.hist_shift), 1u);
                }
            }
        }
    }
    // ---- running softmax (base 2), as in the 16-bit kernel ------------------------------------------
    const float NEG_INF = -INFINITY;
    float t0 = v0 ? s[0] * scale_log2 : NEG_INF, t1 = v0 ? s[1] * scale_log2 : NEG_INF;
    float t2 = v1 ? s[2] * scale_log2 : NEG_INF, t3 = v1 ? s[3] * scale_log2 : NEG_INF;
    float mx0 = fmaxf(t0, t2), mx1 = fmaxf(t1, t3);
    if (__any_sync(0xffffffffu, (mx0 > acc.m[0]) || (mx1 > acc.m[1]))) {
#pragma unroll
        for (int sh = 4; sh <= 16; sh <<= 1) {
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, sh));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, sh));
        }
        const float g0 = fmaxf(acc.m[0], mx0), g1 = fmaxf(acc.m[1], mx1);
        const float a0 = (g0 == NEG_INF) ? 1.f : fast_exp2(acc.m[0] - g0);
        const float a1 = (g1 == NEG_INF) ? 1.f : fast_exp2(acc.m[1] - g1);
        acc.l[0] *= a0;
        acc.l[1] *= a1;
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            acc.o[t][0] *= a0; acc.o[t][1] *= a1; acc.o[t][2] *= a0; acc.o[t][3] *= a1;
        }
        acc.m[0] = g0;
        acc.m[1] = g1;
    }
    const float mn0 = acc.m[0], mn1 = acc.m[1];
    const float ms0 = (mn0 == NEG_INF) ? 0.f : mn0, ms1 = (mn1 == NEG_INF) ? 0.f : mn1;
    const float p0 = fast_exp2(t0 - ms0), p1 = fast_exp2(t1 - ms1);
    const float p2 = fast_exp2(t2 - ms0), p3 = fast_exp2(t3 - ms1);
    acc.l[0] += p0 + p2;
    acc.l[1] += p1 + p3;
    const uint32_t pb0 = movmatrix_trans(pack_f16(p0, p1));
    const uint32_t pb1 = movmatrix_trans(pack_f16(p2, p3));
    // ---- O^T += V^T . P^T ------------------------------------------------------------------------------
    // ldmatrix.trans moves 16-bit units, i.e. pairs of codes (d, d+1) of one position. Matrix (pos half
    // hp, piece c) hands lane (gid, tig) the word [V[p][d0], V[p][d1], V[p+1][d0], V[p+1][d1]] with
    // p = 8hp + 2tig, d0 = 16c + 2gid, d1 = d0 + 1. A byte permute regroups it into (V[p][d0], V[p+1][d0])
    // and (V[p][d1], V[p+1][d1]): the A fragments of rows d0 (MMA row gid) and d1 (MMA row gid + 8).
    const int lane = gid * 4 + tig;
    const int rr = lane & 7, mi = lane >> 3;
    const int vrow = rr + ((mi >> 1) << 3);
    const uint32_t vbase = vs + vrow * ROW_BYTES8;
    const uint32_t vswz = rr;                          // vrow & 7
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        uint32_t m[4];
        ldmatrix_x4_trans(vbase + ((uint32_t)((2 * u + (mi & 1)) ^ vswz) << 4), m);
        uint32_t x0, y0, x2, y2, x1, y1, x3, y3;
        e4m3x4_to_f16x2x2(__byte_perm(m[0], 0, 0x3120), x0, y0);      // piece 2u, positions 0-7
        e4m3x4_to_f16x2x2(__byte_perm(m[2], 0, 0x3120), x2, y2);      // piece 2u, positions 8-15
        mma_f16_16816(acc.o[2 * u], x0, y0, x2, y2, pb0, pb1);
        e4m3x4_to_f16x2x2(__byte_perm(m[1], 0, 0x3120), x1, y1);      // piece 2u + 1
        e4m3x4_to_f16x2x2(__byte_perm(m[3], 0, 0x3120), x3, y3);
        mma_f16_16816(acc.o[2 * u + 1], x1, y1, x3, y3, pb0, pb1);
    }
}

// Tiles of one (sequence, head group) item: at least one, so that an empty item still
// produces its (all-zero) output row.
__device__ __forceinline__ int item_tiles(int total) { return max(1, (total + TILE - 1) / TILE); }

// NEWEST (gather kernel only): every list has one more slot that stands for the newest token.
// COMPACT (selection kernel only): the instantiation that compacts top-k candidates; the default
// selection kernel carries none of that code.
// KV8: the cache holds FP8 E4M3 codes (128-byte rows, per-KV-head scales); same kernel, half-size ring
// slots, conversion to fp16 in front of the MMAs (consume_tile8).
template <int MODE, int NW, int STAGES, bool NEWEST = false, bool COMPACT = false, bool KV8 = false>
__global__ void __launch_bounds__(NW * 32, (MODE == MODE_SPARSE && KV8) ? 2 : 1) attn_kernel(const AttnParams p) {
    static_assert(!(COMPACT && KV8), "candidate compaction is built for 16-bit caches only");
    constexpr int SLOT_BYTES = KV8 ? STAGE_BYTES8 : STAGE_BYTES;
    constexpr int KPART_BYTES = KV8 ? TILE_BYTES8 : TILE_BYTES;       // the value rows of a slot start here
    extern __shared__ __align__(128) uint8_t smem_raw[];
    // Ring slots must be 256-byte aligned (the V fragment addressing XORs bits 5-7).
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    __shared__ uint32_t s_vmask[NW][STAGES];
    __shared__ int s_posbase[NW][STAGES];
    __shared__ int s_is_last;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gid = lane >> 2, tig = lane & 3;
    constexpr int RING_BYTES = NW * STAGES * SLOT_BYTES;
    uint32_t* hist = reinterpret_cast<uint32_t*>(smem + RING_BYTES);   // MODE_SELECT: [columns][bins] counters
    const bool hist_on = (MODE == MODE_SELECT) && p.hist != nullptr;

    bool waited = !p.pdl;
    if (p.pdl && p.wait_first) { pdl_wait(); pdl_trigger(); waited = true; }
    else if (p.pdl && p.wait_late && p.trigger_early) pdl_trigger();

    // ---- this CTA's share of the flattened (sequence, item, tile) space ---------------------------
    const bool per_qhead = (MODE == MODE_SPARSE) && (p.Hi == p.Hq);
    const int IY = per_qhead ? p.Hq : p.Hkv;            // items per sequence
    auto seq_total = [&](int b) -> int {
        const int N = min(p.ctx_lens[b], p.max_ctx);
        if (MODE != MODE_SPARSE) return max(N, 0);
        const int cnt = p.idx_count ? min(p.idx_count[b], p.budget) : p.budget;
        return max(cnt, 0) + (NEWEST ? 1 : 0);
    };
    long long per_cta, lo, hi, seq_start = 0;
    int b = 0, tiles_b;
    int part_idx = 0, item_ctas = 0;                   // pooled: which of the item's CTAs this is, out of how many
    if (p.splits_per_item > 0) {
        // Pooled split: S CTAs work on each item and share its tiles dynamically, so
        // that SMs that get less memory bandwidth simply take fewer tiles; no CTA spans two items.
        // CTA -> item round robin: the CTAs of one item are spread over the whole chip.
        const int n_items = p.batch * IY;
        const int item = blockIdx.x % n_items, part = blockIdx.x / n_items;
        b = item / IY;
        part_idx = part;
        item_ctas = ((int)gridDim.x - item + n_items - 1) / n_items;
        tiles_b = item_tiles(seq_total(b));
        per_cta = tiles_b;
        // flat index of the item's first tile relative to sequence b (seq_start stays 0); the
        // tiles themselves are handed out by the item's pool cursor
        lo = (long long)(item % IY) * tiles_b;
        hi = lo + 1;

    } else {
        long long T = 0;
        for (int bb = 0; bb < p.batch; ++bb) T += (long long)IY * item_tiles(seq_total(bb));
        per_cta = (T + gridDim.x - 1) / gridDim.x;
        lo = (long long)blockIdx.x * per_cta;
        hi = min(T, lo + per_cta);
        tiles_b = item_tiles(seq_total(0));
        if (lo < hi) {
            while (seq_start + (long long)IY * tiles_b <= lo) {
                seq_start += (long long)IY * tiles_b;
                ++b;
                tiles_b = item_tiles(seq_total(b));
            }
        }
    }
    if (lo >= hi && p.splits_per_item == 0) {
        // No work for this CTA. A late-waiting launch promises that none of its CTAs retires before the
        // kernel before it is complete (the host's early-trigger rule counts on it), so it waits too.
        if (!waited) pdl_wait();
        return;
    }
    if (hist_on) {
        for (int i = threadIdx.x; i < HIST_SMEM_WORDS; i += NW * 32) hist[i] = 0;
        __syncthreads();
    }
    // Candidate compaction (pooled launches only: a CTA serves one item). The 32 KB behind the rings hold
    //   stage    [NW][CAL_TILES][16][CAND_COLS] keys of the calibration tiles
    //   st_pos   [NW][CAL_TILES] first position of each staged tile (-1: none), st_vm: its valid rows
    //   thr_key  [CAND_COLS] the thresholds as keys, thr_val as values
    //   cbuf     [NW][CAND_COLS][CAND_BUF] candidates waiting to be written out, ccnt [NW][CAND_COLS] fill counts
    constexpr bool compact = (MODE == MODE_SELECT) && COMPACT;      // the host launches it for pooled grids only
    uint32_t* stage_all = hist;
    int* st_pos = reinterpret_cast<int*>(stage_all + NW * CAL_TILES * 16 * CAND_COLS);
    uint32_t* st_vm = reinterpret_cast<uint32_t*>(st_pos + NW * CAL_TILES);
    uint32_t* thr_key = st_vm + NW * CAL_TILES;
    float* thr_val = reinterpret_cast<float*>(thr_key + CAND_COLS);
    int* ccnt_all = reinterpret_cast<int*>(thr_val + CAND_COLS);
    uint2* cbuf_all = reinterpret_cast<uint2*>(ccnt_all + NW * CAND_COLS);        // 8-byte aligned: all counts above are even
    static_assert((NW * CAL_TILES * 16 * CAND_COLS + 2 * NW * CAL_TILES + 2 * CAND_COLS + NW * CAND_COLS) * 4 +
                  NW * CAND_COLS * CAND_BUF * 8 <= HIST_SMEM_WORDS * 4 || !COMPACT, "compaction scratch exceeds the histogram area");
    if (compact) {
        if (lane < CAL_TILES) st_pos[warp * CAL_TILES + lane] = -1;
        if (lane < CAND_COLS) ccnt_all[warp * CAND_COLS + lane] = 0;
        __syncwarp();
    }

    uint8_t* wbase = smem + (size_t)warp * STAGES * SLOT_BYTES;
    const uint32_t wbase_u32 = smem_u32(wbase);
    const int c16 = lane & 15, rhalf = lane >> 4;
    const long long lane_src = (long long)rhalf * p.stride_pos + c16 * 8;
    const long long two_rows = 2 * p.stride_pos;
    // Destination of this lane's piece inside a slot, row pair i adds 512 bytes:
    //   K: row rhalf+2i, piece c16 ^ (rhalf<<2);   V: row rhalf+2i, piece (c16^rhalf) ^ ((i&3)<<1).
    const uint32_t kdst = rhalf * 256 + ((c16 ^ (rhalf << 2)) << 4);
    const uint32_t vdst = rhalf * 256;
    const uint32_t vc = c16 ^ rhalf;
    // 8-bit caches: lane l copies piece l&7 of rows (l>>3) + 4i, i = 0..3 (one instruction moves four
    // whole 128-byte rows); K piece c of row r goes to c ^ ((r&1)<<2), V piece c to c ^ (r&7).
    const int piece8 = lane & 7, row8 = lane >> 3;
    const long long lane_src8 = (long long)row8 * p.stride_pos + piece8 * 16;
    const long long four_rows = 4 * p.stride_pos;
    const uint32_t kdst8 = row8 * ROW_BYTES8 + ((piece8 ^ ((row8 & 1) << 2)) << 4);
    const uint32_t vdst8 = row8 * ROW_BYTES8;
    const uint32_t vc8 = piece8 ^ row8;                                // row & 7 == row8 ^ ((i&1)<<2)
    const uint8_t* kbytes = reinterpret_cast<const uint8_t*>(p.k);
    const uint8_t* vbytes = reinterpret_cast<const uint8_t*>(p.v);
    const bool pooled = p.splits_per_item > 0;
    const uint64_t kv_policy = l2_evict_first_policy();

    do {
        // ---- one segment: tiles [t0, t1) of item y of sequence b (pooled: whatever the warps grab) --
        const int y = (int)((lo - seq_start) / tiles_b);
        const int t0 = (int)((lo - seq_start) % tiles_b);
        const int t1 = pooled ? tiles_b : (int)min((long long)tiles_b, t0 + (hi - lo));
        const int total = seq_total(b);
        const int N = max(min(p.ctx_lens[b], p.max_ctx), 0);
        int head0, ncols, g;
        if (per_qhead) { head0 = y; ncols = 1; g = y / p.G; }
        else { g = y; head0 = g * p.G; ncols = p.G; }
        const int* idx_row = nullptr;
        if (MODE == MODE_SPARSE) {
            const int hi_idx = per_qhead ? y : ((p.Hi == p.Hkv) ? g : 0);
            idx_row = p.idx + ((long long)b * p.Hi + hi_idx) * p.budget;
        }
        int* pool = pooled ? p.tile_ctr + ((long long)b * IY + y) * p.ctr_stride : nullptr;
        // Optional deviation from Algorithm 1: the newest token is attended even if it was not selected.
        // The reserved last slot of the list stands for it unless the (ascending) list already ends with it.
        int newest_pos = -1;
        if (MODE == MODE_SPARSE && NEWEST) {
            const int cnt = total - 1;
            const int last = cnt > 0 ? __ldg(idx_row + cnt - 1) : -1;
            if (N > 0 && last != N - 1) newest_pos = N - 1;
        }

        float* score_row0 = nullptr;
        float* score_row1 = nullptr;
        if (MODE == MODE_SELECT && p.agg) {
            score_row0 = p.scores + ((long long)b * p.Hkv + g) * p.score_stride;
        } else if (MODE == MODE_SELECT) {
            if (2 * tig < ncols) score_row0 = p.scores + ((long long)b * p.Hq + head0 + 2 * tig) * p.score_stride;
            if (2 * tig + 1 < ncols) score_row1 = p.scores + ((long long)b * p.Hq + head0 + 2 * tig + 1) * p.score_stride;
        }
        WarpAcc acc;
        acc.m[0] = acc.m[1] = -INFINITY;
        acc.l[0] = acc.l[1] = 0.f;
#pragma unroll
        for (int t = 0; t < 8; ++t) { acc.o[t][0] = acc.o[t][1] = acc.o[t][2] = acc.o[t][3] = 0.f; }

        const long long head_off = (long long)g * p.stride_head;
        const long long item_off = (p.paged ? 0 : (long long)b * p.stride_b) + head_off;

        // ---- this warp's tile sequence -----------------------------------------------------------------
        // static: t0 + warp, + NW, ... below t1.  pooled: a fixed first chunk, then GRAB_TILES consecutive
        // tiles at a time from the item's cursor; the next grab is requested one chunk ahead so that its
        // latency is hidden.
        int cur = t0 + warp, cur_end = t1;             // static walk
        int grab_raw = 0;                              // lane 0: value returned by the outstanding grab
        // The first chunk of every warp is fixed (no round trip before the first load); the pool
        // cursor hands out the tiles after those. Requests to one cursor are served one after the
        // other by the L2 (roughly 15-20 per microsecond), so chunks must not be too small: two-tile
        // and single-tile requests made the kernels slower, not better balanced.
        // Short items are spread evenly over all the item's warps instead (nothing left for the pool).
        const int item_warps = item_ctas * NW;
        // (fixed chunk: the ring's slots, all filled before the wait, plus the lookahead of two)
        constexpr int FIRST_TILES = STAGES + 2;
        const int first_tiles = (tiles_b <= item_warps * FIRST_TILES)
                                    ? max(1, (tiles_b + item_warps - 1) / max(item_warps, 1)) : FIRST_TILES;
        constexpr int GRAB = (MODE == MODE_SPARSE) ? GRAB_TILES : GRAB_TILES_DENSE;
        const int pool_base = item_warps * first_tiles;
        auto grab = [&]() { if (lane == 0) grab_raw = pool_base + atomicAdd(pool, GRAB); };
        if (pooled) {
            cur = (part_idx * NW + warp) * first_tiles;
            cur_end = min(tiles_b, cur + first_tiles);
        }
        auto next_tile = [&]() -> int {                // -1 when this warp has no more tiles
            if (!pooled) {
                if (cur >= cur_end) return -1;
                const int t = cur;
                cur += NW;
                return t;
            }
            if (cur >= cur_end) {
                if (cur_end >= tiles_b || pool_base >= tiles_b) return -1;   // nothing (left) in the pool
                cur = __shfl_sync(0xffffffffu, grab_raw, 0);
                if (cur >= tiles_b) { cur_end = tiles_b; return -1; }
                cur_end = min(tiles_b, cur + GRAB);
                grab();
            }
            return cur++;
        };

        // Tile queue with a lookahead of two: tA is issued next, tB after it. In the sparse mode the
        // row offset of tA is already resolved (offA / validA, including the page lookup) and the index
        // entry of tB is in flight (posB), so neither load ever delays a copy.
        int tA = next_tile();
        int tB = (tA >= 0) ? next_tile() : -1;
        auto load_pos = [&](int tile) -> int {
            if (MODE != MODE_SPARSE || tile < 0) return -1;
            const int e = tile * TILE + c16;
            if (NEWEST && e == total - 1) return newest_pos;
            return (e < total) ? __ldg(idx_row + e) : -1;
        };
        long long offA = 0;
        bool validA = false;
        auto resolve = [&](int pos) {
            validA = pos >= 0 && pos < N;
            if (pos >= N || pos < -1) atomicOr(p.status, STATUS_BAD_INDEX);   // -1 is padding, anything else is not a token
            offA = 0;
            if (validA) {
                if (p.paged) {
                    const int page = __ldg(p.page_table + (long long)b * p.max_pages + (pos >> 4));
                    if ((unsigned)page < (unsigned)p.num_pages) {
                        offA = (long long)page * p.stride_page + (long long)(pos & 15) * p.stride_pos + head_off;
                    } else {
                        validA = false;
                        atomicOr(p.status, STATUS_BAD_PAGE);
                    }
                } else {
                    offA = item_off + (long long)pos * p.stride_pos;
                }
            }
        };
        int posB = -1;
        if (MODE == MODE_SPARSE) {
            const int posA = load_pos(tA);
            posB = load_pos(tB);
            resolve(posA);
        }

        // Issue the copies of tile tA into ring slot `stage`, then advance the queue.
        // Shared layout of a slot: K rows then V rows, 256 B per row, 16-byte piece c of
        // row r stored at piece c ^ ((r&1)<<2) for K and c ^ (r&7) for V so that the
        // fragment reads in consume_tile are bank-conflict free. Lane l copies piece
        // l&15 of rows (l>>4) + 2i, i = 0..7: one instruction moves two whole rows.
        auto issue = [&](int stage) {
            const int tile = tA;
            const uint32_t ks = wbase_u32 + stage * SLOT_BYTES, vs = ks + KPART_BYTES;
            uint32_t vmask;
            if (MODE != MODE_SPARSE) {
                tA = tB;
                tB = (tA >= 0) ? next_tile() : -1;
                const int pos0 = tile * TILE;
                long long off;
                bool ok = true;
                if (p.paged) {
                    const int page = __ldg(p.page_table + (long long)b * p.max_pages + tile);
                    ok = (unsigned)page < (unsigned)p.num_pages;
                    if (!ok && lane == 0) atomicOr(p.status, STATUS_BAD_PAGE);
                    off = (ok ? (long long)page * p.stride_page : 0) + item_off + lane_src;
                } else {
                    off = item_off + (long long)pos0 * p.stride_pos + lane_src;
                }
                const int nvalid = ok ? max(0, min(TILE, total - pos0)) : 0;
                vmask = (1u << nvalid) - 1u;
                if constexpr (KV8) {
                    const long long off8 = off - lane_src + lane_src8;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const bool rv = row8 + 4 * i < nvalid;
                        const long long eo = rv ? off8 + i * four_rows : 0;
                        cp_async16_hint(ks + kdst8 + i * 512, kbytes + eo, rv ? 16 : 0, kv_policy);
                        cp_async16_hint(vs + vdst8 + i * 512 + ((vc8 ^ ((i & 1) << 2)) << 4), vbytes + eo, rv ? 16 : 0, kv_policy);
                    }
                    if (lane == 0) { s_vmask[warp][stage] = vmask; s_posbase[warp][stage] = pos0; }
                    return;
                }
                const __nv_bfloat16* ksrc = p.k + off;
                const __nv_bfloat16* vsrc = p.v + off;
                if (nvalid == TILE) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        cp_async16_full_hint(ks + kdst + i * 512, ksrc + i * two_rows, kv_policy);
                        cp_async16_full_hint(vs + vdst + i * 512 + ((vc ^ ((i & 3) << 1)) << 4), vsrc + i * two_rows, kv_policy);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const bool rv = rhalf + 2 * i < nvalid;
                        cp_async16(ks + kdst + i * 512, rv ? ksrc + i * two_rows : p.k, rv ? 16 : 0);
                        cp_async16(vs + vdst + i * 512 + ((vc ^ ((i & 3) << 1)) << 4), rv ? vsrc + i * two_rows : p.v, rv ? 16 : 0);
                    }
                }
                if (lane == 0) { s_vmask[warp][stage] = vmask; s_posbase[warp][stage] = pos0; }
            } else {
                const long long off = offA;
                const bool valid = validA;
                tA = tB;
                resolve(posB);                       // the page lookup of the next tile starts now
                tB = (tA >= 0) ? next_tile() : -1;
                posB = load_pos(tB);
                vmask = __ballot_sync(0xffffffffu, valid) & 0xffffu;
                if constexpr (KV8) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int r = row8 + 4 * i;
                        const long long ro = __shfl_sync(0xffffffffu, off, r);
                        const bool rv = (vmask >> r) & 1u;
                        const long long eo = rv ? ro + piece8 * 16 : 0;
                        cp_async16_hint(ks + kdst8 + i * 512, kbytes + eo, rv ? 16 : 0, kv_policy);
                        cp_async16_hint(vs + vdst8 + i * 512 + ((vc8 ^ ((i & 1) << 2)) << 4), vbytes + eo, rv ? 16 : 0, kv_policy);
                    }
                    if (lane == 0) { s_vmask[warp][stage] = vmask; s_posbase[warp][stage] = 0; }
                    return;
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int r = rhalf + 2 * i;
                    const long long ro = __shfl_sync(0xffffffffu, off, r);
                    const bool rv = (vmask >> r) & 1u;
                    const long long eo = rv ? ro + c16 * 8 : 0;
                    cp_async16_hint(ks + kdst + i * 512, p.k + eo, rv ? 16 : 0, kv_policy);
                    cp_async16_hint(vs + vdst + i * 512 + ((vc ^ ((i & 3) << 1)) << 4), p.v + eo, rv ? 16 : 0, kv_policy);
                }
                if (lane == 0) { s_vmask[warp][stage] = vmask; s_posbase[warp][stage] = 0; }
            }
        };

        // ---- private cp.async ring -----------------------------------------------------------------------
        // Until the grid dependency is resolved, only tiles that cannot hold the token appended for
        // this layer may be fetched: every tile but the last one of the item (index lists produced by
        // the selection kernel are ascending). The query and the scratch buffers belong to the kernels
        // before us and are touched only after the wait.
        int issued = 0, commits = 0;
        // The first pool request goes out at once, even before the grid dependency resolves: consecutive
        // launches use alternating sets of cursors, and the set of this launch was last touched two
        // launches ago (its last user reset it, and had finished before our predecessor could start us).
        // By the time the fixed chunk runs out the answer is there; asked for only after the wait, the
        // forty-odd warps of an item queue up on one address and stall at that point.
        if (pooled) grab();
        if (!waited && !p.wait_late) {
            while (commits < STAGES && tA >= 0 && tA < tiles_b - 1) {
                issue(issued % STAGES);
                ++issued;
                cp_async_commit();
                ++commits;
            }
            pdl_wait();
            pdl_trigger();
            waited = true;
        }

        // Q^T fragments: column gid is head head0+gid; this lane holds the 16-byte
        // pieces 4j+tig (j = 0..3) of that head's query row.
        uint32_t qf[4][4];
        uint32_t qf8[2][8];                             // 8-bit caches: the query as fp16, see consume_tile8
        {
            const uint4* qp = reinterpret_cast<const uint4*>(
                p.q + ((long long)b * p.Hq + head0 + min(gid, ncols - 1)) * HEAD_DIM);
            const bool on = gid < ncols;
            if constexpr (KV8) {
#pragma unroll
                for (int sl = 0; sl < 2; ++sl) {
                    const int c = tig + 4 * sl;         // this lane's 16-code piece of a key row = 32 bytes of the query row
                    const uint4 t0 = __ldg(qp + 2 * c), t1 = __ldg(qp + 2 * c + 1);
                    const uint32_t w[8] = {t0.x, t0.y, t0.z, t0.w, t1.x, t1.y, t1.z, t1.w};
#pragma unroll
                    for (int i = 0; i < 8; ++i) qf8[sl][i] = on ? bf16x2_to_f16x2(w[i]) : 0u;
                }
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint4 t = __ldg(qp + 4 * j + tig);
                    qf[j][0] = on ? t.x : 0u; qf[j][1] = on ? t.y : 0u; qf[j][2] = on ? t.z : 0u; qf[j][3] = on ? t.w : 0u;
                }
            }
        }
        // 8-bit caches: the key scale of this KV head goes into the logit scale, the value scale is applied
        // to the accumulators once, at the end
        const float kscale = (KV8 && p.k_scale) ? __ldg(p.k_scale + g) : 1.f;
        const float vscale = (KV8 && p.v_scale) ? __ldg(p.v_scale + g) : 1.f;
        const float seg_scale = p.scale * kscale, seg_scale_log2 = p.scale_log2 * kscale;


        // Before the grid dependency was resolved the whole ring may have been filled (one slot more
        // than the loop keeps in flight): the first iteration then has no free slot and issues nothing.
        const bool ring_full = commits == STAGES;
        while (commits < STAGES - 1) {
            if (tA >= 0) { issue(issued % STAGES); ++issued; }
            cp_async_commit();
            ++commits;
        }
        // ---- candidate compaction: helpers of this warp ---------------------------------------------------
        CandWarp cw;
        cw.stage = nullptr;
        cw.thr0 = cw.thr1 = INFINITY;
        cw.buf = cbuf_all + warp * CAND_COLS * CAND_BUF;
        cw.cnt = ccnt_all + warp * CAND_COLS;
        bool calibrated = false;
        // Write out the buffers of this warp that hold at least `least` candidates: one cursor bump per buffer.
        auto cand_flush = [&](int least) {
            __syncwarp();
            const int c = (lane < ncols) ? cw.cnt[lane] : 0;
            unsigned m = __ballot_sync(0xffffffffu, c >= least && c > 0);
            while (m) {
                const int col = __ffs(m) - 1;
                m &= m - 1;
                const int n = __shfl_sync(0xffffffffu, c, col);
                const long long row = (long long)b * p.Hq + head0 + col;
                int base = 0;
                if (lane == 0) base = atomicAdd(p.cand_cursor + row * p.ctr_stride, n);
                base = __shfl_sync(0xffffffffu, base, 0);
                uint2* dst = p.cand + row * p.cand_stride;
                for (int i = lane; i < n; i += 32)
                    if (base + i < p.cand_stride) dst[base + i] = cw.buf[col * CAND_BUF + i];
                if (lane == 0) cw.cnt[col] = 0;
            }
            __syncwarp();
        };
        // Once per CTA, by all warps together: thresholds from the staged scores of every warp's first tiles
        // (the r-th largest staged key of a head, r = margin * k' / N of the sample), then every warp
        // compacts its own staged tiles with them.
        auto calibrate = [&]() {
            __syncthreads();
            if (warp < ncols) {
                const int col = warp;
                constexpr int PER_LANE = (NW * CAL_TILES * 16 + 31) / 32;
                uint32_t keys[PER_LANE];
                int nvalid = 0;
#pragma unroll
                for (int u = 0; u < PER_LANE; ++u) {
                    const int e = lane + 32 * u, wt = e >> 4, r = e & 15;        // wt = warp * CAL_TILES + tile
                    const bool ok = wt < NW * CAL_TILES && st_pos[wt] >= 0 && ((st_vm[wt] >> r) & 1u);
                    keys[u] = ok ? stage_all[(wt * 16 + r) * CAND_COLS + col] : 0u;
                    nvalid += ok;
                }
#pragma unroll
                for (int sh = 16; sh >= 1; sh >>= 1) nvalid += __shfl_xor_sync(0xffffffffu, nvalid, sh);
                const int kk = min(p.budget, N);
                const float frac = p.margin * (float)kk / (float)max(N, 1);
                const int rank = (int)ceilf(frac * (float)nvalid) + 2;
                uint32_t tk = 0;                                            // 0: everything is a candidate
                if (nvalid >= 64 && rank < nvalid) {
                    // the rank-th largest staged key: the largest value that at least `rank` keys reach
                    for (int bit = 31; bit >= 12; --bit) {           // 20 bits: the threshold need not be finer
                        const uint32_t trial = tk | (1u << bit);
                        int cnt = 0;
#pragma unroll
                        for (int u = 0; u < PER_LANE; ++u) cnt += keys[u] >= trial;
#pragma unroll
                        for (int sh = 16; sh >= 1; sh >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, sh);
                        if (cnt >= rank) tk = trial;
                    }
                }
                if (lane == 0) {
                    thr_key[col] = tk;
                    // the value whose key is tk (key 0 belongs to no number: everything passes)
                    thr_val[col] = tk == 0 ? -INFINITY : __uint_as_float((tk & 0x80000000u) ? (tk & 0x7fffffffu) : ~tk);
                    atomicMax(p.thr_max + ((long long)b * p.Hq + head0 + col) * p.ctr_stride, tk);
                }
            }
            __syncthreads();
            cw.thr0 = (2 * tig < ncols) ? thr_val[2 * tig] : INFINITY;
            cw.thr1 = (2 * tig + 1 < ncols) ? thr_val[2 * tig + 1] : INFINITY;
            for (int t = 0; t < CAL_TILES; ++t) {
                const int wt = warp * CAL_TILES + t, pos0 = st_pos[wt];
                if (pos0 < 0) break;
                const uint32_t vm = st_vm[wt];
                static_assert(CAND_COLS == 4, "a lane's column below is its tig");
#pragma unroll
                for (int u = 0; u < 16 * CAND_COLS / 32; ++u) {
                    const int e = lane + 32 * u, r = e / CAND_COLS, col = tig;        // e % CAND_COLS == lane & 3
                    const uint32_t key = stage_all[(wt * 16 + r) * CAND_COLS + col];
                    const bool take = col < ncols && ((vm >> r) & 1u) && key >= thr_key[col];
                    const unsigned m = __ballot_sync(0xffffffffu, take) & (0x11111111u << tig);
                    const int base = (col < ncols) ? cw.cnt[col] : 0;
                    if (take) cw.buf[col * CAND_BUF + base + __popc(m & ((1u << lane) - 1u))] = make_uint2(key, (unsigned)(pos0 + r));
                    __syncwarp();
                    if (gid == 0 && m) cw.cnt[col] = base + __popc(m);
                    __syncwarp();
                }
                cand_flush(CAND_FLUSH);
            }
            calibrated = true;
        };

        for (int it = 0; it < issued; ++it) {
            if (it == 0 && ring_full) {
                cp_async_wait<STAGES - 1>();
                __syncwarp();
            } else {
                cp_async_wait<STAGES - 2>();      // tile `it` has landed (this lane's copies)
                __syncwarp();                     // ... and every other lane's; slot (it-1)%STAGES is free
                if (tA >= 0) { issue((it + STAGES - 1) % STAGES); ++issued; }
                cp_async_commit();
            }
            const int stage = it % STAGES;
            const uint32_t ks = wbase_u32 + stage * SLOT_BYTES;
            if constexpr (KV8) {
                consume_tile8<MODE>(p, seg_scale, seg_scale_log2, ks, ks + KPART_BYTES, qf8, acc, s_vmask[warp][stage],
                                    gid, tig, score_row0, score_row1, s_posbase[warp][stage], hist_on ? hist : nullptr);
            } else if constexpr (compact) {
                if (!calibrated && it == CAL_TILES) calibrate();
                cw.stage = nullptr;
                if (!calibrated) {
                    const int wt = warp * CAL_TILES + it;
                    cw.stage = stage_all + wt * 16 * CAND_COLS;
                    if (lane == 0) { st_pos[wt] = s_posbase[warp][stage]; st_vm[wt] = s_vmask[warp][stage]; }
                }
                // A buffer that has reached CAND_FLUSH entries reserves its place in the head's list now (lane
                // `col` asks for buffer `col`) and is written out after the tile, when the answer has arrived;
                // what the tile itself adds stays behind as the start of the next batch.
                int pend_n = 0, pend_base = 0;
                __syncwarp();                                         // the counts as the previous tile left them
                if (calibrated && lane < ncols) {
                    const int c = cw.cnt[lane];
                    if (c >= CAND_FLUSH) {
                        pend_n = c;
                        pend_base = atomicAdd(p.cand_cursor + ((long long)b * p.Hq + head0 + lane) * p.ctr_stride, c);
                    }
                }
                consume_tile<MODE>(p, ks, ks + TILE_BYTES, qf, acc, s_vmask[warp][stage], gid, tig,
                                   score_row0, score_row1, s_posbase[warp][stage], nullptr, &cw);
                __syncwarp();
                unsigned pend = __ballot_sync(0xffffffffu, pend_n > 0);
                while (pend) {
                    const int col = __ffs(pend) - 1;
                    pend &= pend - 1;
                    const int n = __shfl_sync(0xffffffffu, pend_n, col), base = __shfl_sync(0xffffffffu, pend_base, col);
                    uint2* dst = p.cand + ((long long)b * p.Hq + head0 + col) * p.cand_stride;
                    uint2* src = cw.buf + col * CAND_BUF;
                    const int total = cw.cnt[col];                    // n plus what this tile added (at most 16)
                    for (int i = lane; i < n; i += 32)
                        if (base + i < p.cand_stride) dst[base + i] = src[i];
                    const uint2 moved = (lane < total - n) ? src[n + lane] : make_uint2(0u, 0u);
                    __syncwarp();
                    if (lane < total - n) src[lane] = moved;
                    if (lane == 0) cw.cnt[col] = total - n;
                    __syncwarp();
                }
            } else {
                consume_tile<MODE>(p, ks, ks + TILE_BYTES, qf, acc, s_vmask[warp][stage], gid, tig,
                                   score_row0, score_row1, s_posbase[warp][stage], hist_on ? hist : nullptr);
            }
        }
        cp_async_wait<0>();
        __syncwarp();
        if constexpr (compact) {
            if (!calibrated) calibrate();         // fewer tiles than the calibration takes: every warp still meets here
            cand_flush(1);
        }
        // All of this item's tiles are in the accumulators. With a late wait the grid dependency is
        // resolved only now: everything below writes memory that the preceding kernel may still use.
        if (!waited) {
            pdl_wait();
            if (!p.trigger_early) pdl_trigger();
            waited = true;
        }

        if (hist_on) {                        // add this segment's histogram to the global one
            __syncthreads();
            const int nb = 1 << (32 - p.hist_shift);
            const long long hrow0 = p.agg ? (long long)b * p.Hkv + g : (long long)b * p.Hq + head0;
            for (int i = threadIdx.x; i < (p.agg ? 1 : ncols) * nb; i += NW * 32) {
                const uint32_t w = hist[i];
                if (w) {
                    atomicAdd(p.hist + (hrow0 + i / nb) * HIST_BINS + (i % nb), w);
                    hist[i] = 0;
                }
            }
            __syncthreads();
        }

        // ---- merge the warps of this CTA ---------------------------------------------------------------
#pragma unroll
        for (int sh = 4; sh <= 16; sh <<= 1) {
            acc.l[0] += __shfl_xor_sync(0xffffffffu, acc.l[0], sh);
            acc.l[1] += __shfl_xor_sync(0xffffffffu, acc.l[1], sh);
        }
        __syncthreads();                      // all rings drained; reuse the shared memory
        float* mo = reinterpret_cast<float*>(smem);                                // [NW][8][128]
        float2* mml = reinterpret_cast<float2*>(smem + NW * 8 * HEAD_DIM * 4);    // [NW][8]
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            float* w0 = mo + ((warp * 8 + 2 * tig) * HEAD_DIM);
            float* w1 = w0 + HEAD_DIM;
            if constexpr (KV8) {                      // rows of the O^T fragments are d = 16t + 2gid and + 1 here
                w0[16 * t + 2 * gid] = acc.o[t][0] * vscale;
                w1[16 * t + 2 * gid] = acc.o[t][1] * vscale;
                w0[16 * t + 2 * gid + 1] = acc.o[t][2] * vscale;
                w1[16 * t + 2 * gid + 1] = acc.o[t][3] * vscale;
            } else {
                w0[16 * t + gid] = acc.o[t][0];
                w1[16 * t + gid] = acc.o[t][1];
                w0[16 * t + 8 + gid] = acc.o[t][2];
                w1[16 * t + 8 + gid] = acc.o[t][3];
            }
        }
        if (gid == 0) {
            mml[warp * 8 + 2 * tig] = make_float2(acc.m[0], acc.l[0]);
            mml[warp * 8 + 2 * tig + 1] = make_float2(acc.m[1], acc.l[1]);
        }
        __syncthreads();

        // CTAs that share this item: those whose range meets [item_lo, item_lo + tiles_b).
        int nsplits, split;
        if (pooled) {
            nsplits = item_ctas;                  // every CTA of the item arrives, with or without tiles
            split = part_idx;
        } else {
            const long long item_lo = seq_start + (long long)y * tiles_b;
            const int first_cta = (int)(item_lo / per_cta);
            nsplits = (int)((item_lo + tiles_b - 1) / per_cta) - first_cta + 1;
            split = (int)blockIdx.x - first_cta;
        }
        const long long row0 = (long long)b * p.Hq + head0;
        for (int e = threadIdx.x; e < ncols * HEAD_DIM; e += NW * 32) {
            const int col = e >> 7, c = e & 127;
            float M = -INFINITY;
#pragma unroll
            for (int w = 0; w < NW; ++w) M = fmaxf(M, mml[w * 8 + col].x);
            float L = 0.f, O = 0.f;
            if (M != -INFINITY) {
#pragma unroll
                for (int w = 0; w < NW; ++w) {
                    const float2 ml = mml[w * 8 + col];
                    const float f = (ml.x == -INFINITY) ? 0.f : fast_exp2(ml.x - M);
                    L += ml.y * f;
                    O += mo[(w * 8 + col) * HEAD_DIM + c] * f;
                }
            }
            if (nsplits == 1) {
                store_out(p, (row0 + col) * HEAD_DIM + c, (L > 0.f) ? O / L : 0.f);
            } else if (split < p.max_splits) {
                const long long pr = (row0 + col) * p.max_splits + split;
                p.part_o[pr * HEAD_DIM + c] = O;
                if (c == 0) p.part_ml[pr] = make_float2(M, L);
            } else if (e == 0) {
                atomicOr(p.status, STATUS_SPLIT_OVERFLOW);    // the host's bound on splits per row was wrong: say so
            }
        }
        if (nsplits == 1 && pooled && threadIdx.x == 0) { *pool = 0; __threadfence(); }
        if (nsplits > 1) {
            // ---- the last CTA of this item to arrive combines the splits ---------------------------------
            __syncthreads();
            int* ctr = p.counters + ((long long)b * IY + y) * p.ctr_stride;
            if (threadIdx.x == 0) {
                // release: orders the whole CTA's partial stores (made visible to this thread by the barrier)
                // before the arrival; acquire: the last arrival sees every earlier part's stores
                int old;
                asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;\n" : "=r"(old) : "l"(ctr) : "memory");
                s_is_last = (old == nsplits - 1);
            }
            __syncthreads();
            if (s_is_last) {
                const int ns = min(nsplits, p.max_splits);
                // Every thread first puts the loads of its output elements in flight (up to 16 splits
                // at once), the warps meanwhile reduce the (max, sum) pairs to per-split scale factors
                // in shared memory: one round trip to L2 instead of three.
                float* fsc = reinterpret_cast<float*>(smem);              // [ncols][max_splits] exp2(m_s - M)
                float* linv = fsc + 8 * p.max_splits;                    // [ncols] 1 / sum
                constexpr int CB = 16;
                const int e0 = threadIdx.x;                               // first (col, c) element of this thread
                const bool has0 = e0 < ncols * HEAD_DIM;
                const float* po0 = p.part_o + ((row0 + (e0 >> 7)) * p.max_splits) * HEAD_DIM + (e0 & 127);
                float v0[CB];
#pragma unroll
                for (int u = 0; u < CB; ++u) v0[u] = (has0 && u < ns) ? __ldcg(po0 + (long long)u * HEAD_DIM) : 0.f;
                // The item's pool cursor is cleared for a later launch now, behind this thread's loads (the
                // fence then costs nothing extra: it returns when they do). The fence makes the cleared
                // cursor visible device-wide before this CTA can retire: a later launch may request tiles
                // from it without waiting for this grid (see the host's rule for early triggers), and cannot
                // start before this CTA is gone.
                if (pooled && threadIdx.x == NW * 32 - 1) { *pool = 0; __threadfence(); }
                for (int col = warp; col < ncols; col += NW) {
                    const long long pr = (row0 + col) * p.max_splits;
                    float M = -INFINITY;
                    for (int s = lane; s < ns; s += 32) M = fmaxf(M, __ldcg(&p.part_ml[pr + s].x));
#pragma unroll
                    for (int sh = 16; sh >= 1; sh >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, sh));
                    float L = 0.f;
                    for (int s = lane; s < ns; s += 32) {
                        const float2 ml = __ldcg(&p.part_ml[pr + s]);
                        const float f = (ml.x == -INFINITY || M == -INFINITY) ? 0.f : fast_exp2(ml.x - M);
                        fsc[col * p.max_splits + s] = f;
                        L += ml.y * f;
                    }
#pragma unroll
                    for (int sh = 16; sh >= 1; sh >>= 1) L += __shfl_xor_sync(0xffffffffu, L, sh);
                    if (lane == 0) linv[col] = (L > 0.f) ? 1.f / L : 0.f;
                }
                __syncthreads();
                for (int e = threadIdx.x; e < ncols * HEAD_DIM; e += NW * 32) {
                    const int col = e >> 7, c = e & 127;
                    const float* po = p.part_o + ((row0 + col) * p.max_splits) * HEAD_DIM + c;
                    const float* fs = fsc + col * p.max_splits;
                    float O = 0.f;
                    int s = 0;
                    if (e == e0) {
#pragma unroll
                        for (int u = 0; u < CB; ++u) if (u < ns) O += v0[u] * fs[u];
                        s = min(ns, CB);
                    }
                    for (; s + 8 <= ns; s += 8) {
                        float v[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u) v[u] = __ldcg(po + (long long)(s + u) * HEAD_DIM);
#pragma unroll
                        for (int u = 0; u < 8; ++u) O += v[u] * fs[s + u];
                    }
                    for (; s < ns; ++s) O += __ldcg(po + (long long)s * HEAD_DIM) * fs[s];
                    store_out(p, (row0 + col) * HEAD_DIM + c, O * linv[col]);
                }
                if (threadIdx.x == 0) *ctr = 0;       // ready for the next launch
            }
        }
        __syncthreads();                          // shared memory is reused by the next segment

        // ---- advance to the next segment -----------------------------------------------------------------
        if (pooled) break;
        lo += (t1 - t0);
        if (lo < hi && lo >= seq_start + (long long)IY * tiles_b) {
            seq_start += (long long)IY * tiles_b;
            ++b;
            tiles_b = item_tiles(seq_total(b));
        }
    } while (lo < hi);
}

// C.append(k, v): one warp per (sequence, KV head) copies the two 256-byte rows of the new token
// to position ctx_lens[b] - 1 of the cache.
struct AppendParams {
    __nv_bfloat16* k;
    __nv_bfloat16* v;
    const __nv_bfloat16* k_new;
    const __nv_bfloat16* v_new;
    long long stride_b, stride_pos, stride_head, stride_page;
    const int* page_table;
    int max_pages, num_pages, paged;
    const int* ctx_lens;
    int max_ctx, batch, Hkv;
    int elem_bytes;            // 2: bf16 rows of 256 bytes; 1: rows of 128 bytes of E4M3 codes
    int* status;
};

__device__ __forceinline__ void kv_append_rows(const AppendParams& p) {
    const int pair = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (pair >= p.batch * p.Hkv) return;
    const int b = pair / p.Hkv, g = pair % p.Hkv;
    const int pos = p.ctx_lens[b] - 1;
    if (pos < 0 || pos >= p.max_ctx) return;
    long long off;
    if (p.paged) {
        const int page = p.page_table[(long long)b * p.max_pages + (pos >> 4)];
        if ((unsigned)page >= (unsigned)p.num_pages) { if (lane == 0) atomicOr(p.status, STATUS_BAD_PAGE); return; }
        off = (long long)page * p.stride_page + (long long)(pos & 15) * p.stride_pos + (long long)g * p.stride_head;
    } else {
        off = (long long)b * p.stride_b + (long long)pos * p.stride_pos + (long long)g * p.stride_head;
    }
    const long long src = (long long)pair * HEAD_DIM;
    // lanes 0-15 move the key row, lanes 16-31 the value row, 16 bytes each (an 8-bit row takes 8 lanes)
    const int piece = lane & 15;
    if (piece * 16 >= HEAD_DIM * p.elem_bytes) return;
    const char* from = reinterpret_cast<const char*>(lane < 16 ? p.k_new : p.v_new) + src * p.elem_bytes + piece * 16;
    char* to = reinterpret_cast<char*>(lane < 16 ? p.k : p.v) + off * p.elem_bytes + piece * 16;
    *reinterpret_cast<uint4*>(to) = __ldg(reinterpret_cast<const uint4*>(from));
}

__global__ void __launch_bounds__(128) kv_append_kernel(const AppendParams p) { kv_append_rows(p); }

// The same for several layers in one launch: blockIdx.y picks the layer.
constexpr int APPEND_MAX_LAYERS = 24;
struct AppendBatchParams {
    AppendParams layer[APPEND_MAX_LAYERS];
};
__global__ void __launch_bounds__(128) kv_append_layers_kernel(const __grid_constant__ AppendBatchParams p) {
    kv_append_rows(p.layer[blockIdx.y]);
}

}  // namespace tidal
