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
enum { STATUS_BAD_INDEX = 1, STATUS_BAD_PAGE = 2 };

constexpr int HEAD_DIM = 128;
constexpr int TILE = 16;                 // positions per tile == page size
constexpr int TILE_BYTES = TILE * HEAD_DIM * 2;   // 4 KB of K, same of V
constexpr int STAGE_BYTES = 2 * TILE_BYTES;

struct AttnParams {
    const __nv_bfloat16* q;
    const __nv_bfloat16* k;
    const __nv_bfloat16* v;
    float* out;
    long long stride_b, stride_pos, stride_head, stride_page;
    const int* page_table;
    int max_pages, num_pages, paged;
    const int* ctx_lens;
    int max_ctx;               // host bound of ctx_lens; larger device values are clamped to it
    int Hq, Hkv, G;
    float scale, scale_log2;
    int chunk;                 // context positions (or index entries) per CTA, multiple of 16
    float* scores;             // MODE_SELECT: [B, Hq, score_stride]
    long long score_stride;
    const int* idx;            // MODE_SPARSE: [B, Hi, k]
    const int* idx_count;      // MODE_SPARSE: [B] or null
    int budget, Hi;            // MODE_SPARSE: entries per index row, index heads
    float* part_o;             // [B*Hq, max_splits, 128] un-normalised partial outputs
    float2* part_ml;           // [B*Hq, max_splits] (running max in base 2, sum)
    int* counters;             // [B * gridDim.y], zero between launches
    int max_splits;
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
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}

__device__ __forceinline__ void lds128(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n"
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

// Per-warp running softmax state. Columns of the MMA tiles are query heads:
// this lane owns heads 2*tig and 2*tig+1 of the group.
struct WarpAcc {
    float m[2];        // running max of logit*log2(e), identical in all lanes that share tig
    float l[2];        // this lane's share of the running sum
    float o[8][4];     // O^T fragments: o[t][0..1] d = 8*gid+t, o[t][2..3] d = 64+8*gid+t
};

// Consume one staged tile: 16 K rows at ks, 16 V rows at vs (swizzled, see
// the issue code), `vmask` bit r set when row r is a real cached token,
// pos_base + r its position (only used to store scores).
template <int MODE>
__device__ __forceinline__ void consume_tile(const AttnParams& p, uint32_t ks, uint32_t vs,
                                             const uint32_t (&qf)[4][4], WarpAcc& acc, uint32_t vmask,
                                             int gid, int tig, float* score_row0, float* score_row1,
                                             int pos_base) {
    // ---- S^T = K . Q^T ------------------------------------------------------
    float s[4] = {0.f, 0.f, 0.f, 0.f};
    const uint32_t krow = ks + gid * 256;
    const uint32_t kswz = (gid & 1) << 2;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        uint32_t ka[4], kb[4];
        const uint32_t off = (((4 * j + tig) ^ kswz) << 4);
        lds128(krow + off, ka);                 // row gid
        lds128(krow + 8 * 256 + off, kb);       // row gid + 8
        mma_bf16_16816(s, ka[0], kb[0], ka[1], kb[1], qf[j][0], qf[j][1]);
        mma_bf16_16816(s, ka[2], kb[2], ka[3], kb[3], qf[j][2], qf[j][3]);
    }
    const bool v0 = (vmask >> gid) & 1u, v1 = (vmask >> (gid + 8)) & 1u;
    if (MODE == MODE_SELECT) {
        // s[0],s[1]: (pos gid; heads 2tig, 2tig+1)   s[2],s[3]: (pos gid+8; same heads)
        if (score_row0) {
            if (v0) score_row0[pos_base + gid] = s[0] * p.scale;
            if (v1) score_row0[pos_base + gid + 8] = s[2] * p.scale;
        }
        if (score_row1) {
            if (v0) score_row1[pos_base + gid] = s[1] * p.scale;
            if (v1) score_row1[pos_base + gid + 8] = s[3] * p.scale;
        }
    }
    // ---- running softmax (base 2) ---------------------------------------------
    const float NEG_INF = -INFINITY;
    float t0 = v0 ? s[0] * p.scale_log2 : NEG_INF, t1 = v0 ? s[1] * p.scale_log2 : NEG_INF;
    float t2 = v1 ? s[2] * p.scale_log2 : NEG_INF, t3 = v1 ? s[3] * p.scale_log2 : NEG_INF;
    float mx0 = fmaxf(t0, t2), mx1 = fmaxf(t1, t3);
#pragma unroll
    for (int sh = 4; sh <= 16; sh <<= 1) {
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, sh));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, sh));
    }
    const float mn0 = fmaxf(acc.m[0], mx0), mn1 = fmaxf(acc.m[1], mx1);
    const bool grew = (mn0 > acc.m[0]) || (mn1 > acc.m[1]);
    if (__any_sync(0xffffffffu, grew)) {
        // exp2(-inf - finite) = 0; when both are -inf the accumulators are still 0.
        const float a0 = (mn0 == NEG_INF) ? 1.f : fast_exp2(acc.m[0] - mn0);
        const float a1 = (mn1 == NEG_INF) ? 1.f : fast_exp2(acc.m[1] - mn1);
        acc.l[0] *= a0;
        acc.l[1] *= a1;
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            acc.o[t][0] *= a0; acc.o[t][1] *= a1; acc.o[t][2] *= a0; acc.o[t][3] *= a1;
        }
        acc.m[0] = mn0;
        acc.m[1] = mn1;
    }
    const float ms0 = (mn0 == NEG_INF) ? 0.f : mn0, ms1 = (mn1 == NEG_INF) ? 0.f : mn1;
    const float p0 = fast_exp2(t0 - ms0), p1 = fast_exp2(t1 - ms1);
    const float p2 = fast_exp2(t2 - ms0), p3 = fast_exp2(t3 - ms1);
    acc.l[0] += p0 + p2;
    acc.l[1] += p1 + p3;
    // P^T as the B operand: transpose (pos x head) -> (head x pos) across the warp.
    const uint32_t pb0 = movmatrix_trans(pack_bf16(p0, p1));
    const uint32_t pb1 = movmatrix_trans(pack_bf16(p2, p3));
    // ---- O^T += V^T . P^T ------------------------------------------------------
    // This lane needs rows 2tig, 2tig+1, 2tig+8, 2tig+9 and the 16-byte pieces gid and gid+8.
    uint32_t vr[4][2][4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = 2 * tig + (i & 1) + ((i >> 1) << 3);
        const uint32_t vswz = ((r >> 1) & 3) << 1;
        lds128(vs + r * 256 + ((gid ^ vswz) << 4), vr[i][0]);
        lds128(vs + r * 256 + (((gid + 8) ^ vswz) << 4), vr[i][1]);
    }
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        const int u = t >> 1;
        const uint32_t sel = (t & 1) ? 0x7632u : 0x5410u;
        const uint32_t a0 = __byte_perm(vr[0][0][u], vr[1][0][u], sel);
        const uint32_t a1 = __byte_perm(vr[0][1][u], vr[1][1][u], sel);
        const uint32_t a2 = __byte_perm(vr[2][0][u], vr[3][0][u], sel);
        const uint32_t a3 = __byte_perm(vr[2][1][u], vr[3][1][u], sel);
        mma_bf16_16816(acc.o[t], a0, a1, a2, a3, pb0, pb1);
    }
}

template <int MODE, int NW, int STAGES>
__global__ void __launch_bounds__(NW * 32) attn_kernel(const AttnParams p) {
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ uint32_t s_vmask[NW][STAGES];
    __shared__ int s_posbase[NW][STAGES];
    __shared__ int s_is_last;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gid = lane >> 2, tig = lane & 3;
    const int b = blockIdx.z, item = blockIdx.y, split = blockIdx.x;

    int head0, ncols, g;
    if (MODE == MODE_SPARSE && p.Hi == p.Hq) { head0 = item; ncols = 1; g = item / p.G; }
    else { g = item; head0 = g * p.G; ncols = p.G; }

    const int N = min(p.ctx_lens[b], p.max_ctx);
    int total = N;
    const int* idx_row = nullptr;
    if (MODE == MODE_SPARSE) {
        int cnt = p.idx_count ? min(p.idx_count[b], p.budget) : p.budget;
        total = max(cnt, 0);
        const int hi = (p.Hi == p.Hq) ? item : ((p.Hi == p.Hkv) ? g : 0);
        idx_row = p.idx + ((long long)b * p.Hi + hi) * p.budget;
    }
    total = max(total, 0);
    const int nsplits = max(1, (total + p.chunk - 1) / p.chunk);
    if (split >= nsplits) return;
    const int e0 = split * p.chunk, e1 = min(total, e0 + p.chunk);
    const int ntiles = (max(e1 - e0, 0) + TILE - 1) / TILE;

    // Q^T fragments: column gid is head head0+gid; this lane holds the 16-byte
    // pieces 4j+tig (j = 0..3) of that head's query row.
    uint32_t qf[4][4];
    {
        const uint4* qp = reinterpret_cast<const uint4*>(p.q + ((long long)b * p.Hq + head0 + min(gid, ncols - 1)) * HEAD_DIM);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint4 t = __ldg(qp + 4 * j + tig);
            const bool on = gid < ncols;
            qf[j][0] = on ? t.x : 0u; qf[j][1] = on ? t.y : 0u; qf[j][2] = on ? t.z : 0u; qf[j][3] = on ? t.w : 0u;
        }
    }

    float* score_row0 = nullptr;
    float* score_row1 = nullptr;
    if (MODE == MODE_SELECT) {
        if (2 * tig < ncols) score_row0 = p.scores + ((long long)b * p.Hq + head0 + 2 * tig) * p.score_stride;
        if (2 * tig + 1 < ncols) score_row1 = p.scores + ((long long)b * p.Hq + head0 + 2 * tig + 1) * p.score_stride;
    }

    WarpAcc acc;
    acc.m[0] = acc.m[1] = -INFINITY;
    acc.l[0] = acc.l[1] = 0.f;
#pragma unroll
    for (int t = 0; t < 8; ++t) { acc.o[t][0] = acc.o[t][1] = acc.o[t][2] = acc.o[t][3] = 0.f; }

    uint8_t* wbase = smem + (size_t)warp * STAGES * STAGE_BYTES;
    const uint32_t wbase_u32 = smem_u32(wbase);
    const long long head_off = (long long)g * p.stride_head;
    const int my_tiles = (ntiles > warp) ? (ntiles - warp + NW - 1) / NW : 0;   // tiles warp, warp+NW, ...

    // Sparse: the index entry this lane will need for the next tile to be issued.
    int pref_pos = -1;
    auto prefetch_idx = [&](int it) {
        if (MODE == MODE_SPARSE) {
            const int e = e0 + (warp + it * NW) * TILE + (lane & 15);
            pref_pos = (it < my_tiles && e < e1) ? __ldg(idx_row + e) : -1;
        }
    };
    prefetch_idx(0);

    // Issue the copies of this warp's `it`-th tile into ring slot `stage`.
    // Shared layout of a slot: K rows then V rows, 256 B per row, 16-byte piece c of
    // row r stored at piece c ^ ((r&1)<<2) for K and c ^ (((r>>1)&3)<<1) for V so that
    // the fragment reads in consume_tile are bank-conflict free.
    auto issue = [&](int it, int stage) {
        const int tile = warp + it * NW;
        const uint32_t ks = wbase_u32 + stage * STAGE_BYTES, vs = ks + TILE_BYTES;
        const int c = lane & 15;
        uint32_t vmask;
        if (MODE != MODE_SPARSE) {
            const int pos0 = e0 + tile * TILE;
            long long off;
            bool ok = true;
            if (p.paged) {
                const int page = __ldg(p.page_table + (long long)b * p.max_pages + (pos0 >> 4));
                ok = (unsigned)page < (unsigned)p.num_pages;
                if (!ok && lane == 0) atomicOr(p.status, STATUS_BAD_PAGE);
                off = (ok ? (long long)page * p.stride_page : 0) + head_off;
            } else {
                off = (long long)b * p.stride_b + head_off + (long long)pos0 * p.stride_pos;
            }
            const int nvalid = ok ? min(TILE, e1 - pos0) : 0;
            vmask = (1u << nvalid) - 1u;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int r = (lane >> 4) + 2 * i;
                const bool rv = r < nvalid;
                const long long eo = rv ? off + (long long)r * p.stride_pos + c * 8 : 0;
                cp_async16(ks + r * 256 + ((c ^ ((r & 1) << 2)) << 4), p.k + eo, rv ? 16 : 0);
                cp_async16(vs + r * 256 + ((c ^ (((r >> 1) & 3) << 1)) << 4), p.v + eo, rv ? 16 : 0);
            }
            if (lane == 0) { s_vmask[warp][stage] = vmask; s_posbase[warp][stage] = pos0; }
        } else {
            const int pos = pref_pos;
            prefetch_idx(it + 1);
            bool valid = pos >= 0 && pos < N;
            if (pos >= N) atomicOr(p.status, STATUS_BAD_INDEX);
            long long off = 0;
            if (valid) {
                if (p.paged) {
                    const int page = __ldg(p.page_table + (long long)b * p.max_pages + (pos >> 4));
                    if ((unsigned)page < (unsigned)p.num_pages) {
                        off = (long long)page * p.stride_page + (long long)(pos & 15) * p.stride_pos + head_off;
                    } else {
                        valid = false;
                        atomicOr(p.status, STATUS_BAD_PAGE);
                    }
                } else {
                    off = (long long)b * p.stride_b + (long long)pos * p.stride_pos + head_off;
                }
            }
            vmask = __ballot_sync(0xffffffffu, valid) & 0xffffu;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int r = (lane >> 4) + 2 * i;
                const long long ro = __shfl_sync(0xffffffffu, off, r);
                const bool rv = (vmask >> r) & 1u;
                const long long eo = rv ? ro + c * 8 : 0;
                cp_async16(ks + r * 256 + ((c ^ ((r & 1) << 2)) << 4), p.k + eo, rv ? 16 : 0);
                cp_async16(vs + r * 256 + ((c ^ (((r >> 1) & 3) << 1)) << 4), p.v + eo, rv ? 16 : 0);
            }
            if (lane == 0) { s_vmask[warp][stage] = vmask; s_posbase[warp][stage] = 0; }
        }
    };

    // ---- private cp.async ring --------------------------------------------------
#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) {
        if (s < my_tiles) issue(s, s);
        cp_async_commit();
    }
    for (int it = 0; it < my_tiles; ++it) {
        cp_async_wait<STAGES - 2>();      // tile `it` has landed (this lane's copies)
        __syncwarp();                     // ... and every other lane's; slot (it-1)%STAGES is free
        const int nxt = it + STAGES - 1;
        if (nxt < my_tiles) issue(nxt, nxt % STAGES);
        cp_async_commit();
        const int stage = it % STAGES;
        const uint32_t ks = wbase_u32 + stage * STAGE_BYTES;
        consume_tile<MODE>(p, ks, ks + TILE_BYTES, qf, acc, s_vmask[warp][stage], gid, tig,
                           score_row0, score_row1, s_posbase[warp][stage]);
    }
    cp_async_wait<0>();

    // ---- merge the warps of this CTA ---------------------------------------------
#pragma unroll
    for (int sh = 4; sh <= 16; sh <<= 1) {
        acc.l[0] += __shfl_xor_sync(0xffffffffu, acc.l[0], sh);
        acc.l[1] += __shfl_xor_sync(0xffffffffu, acc.l[1], sh);
    }
    __syncthreads();                      // all rings drained; reuse the shared memory
    float* mo = reinterpret_cast<float*>(smem);                   // [NW][8][128]
    float2* mml = reinterpret_cast<float2*>(smem + NW * 8 * HEAD_DIM * 4);   // [NW][8]
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        float* w0 = mo + ((warp * 8 + 2 * tig) * HEAD_DIM);
        float* w1 = w0 + HEAD_DIM;
        w0[8 * gid + t] = acc.o[t][0];
        w1[8 * gid + t] = acc.o[t][1];
        w0[64 + 8 * gid + t] = acc.o[t][2];
        w1[64 + 8 * gid + t] = acc.o[t][3];
    }
    if (gid == 0) {
        mml[warp * 8 + 2 * tig] = make_float2(acc.m[0], acc.l[0]);
        mml[warp * 8 + 2 * tig + 1] = make_float2(acc.m[1], acc.l[1]);
    }
    __syncthreads();

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
            p.out[(row0 + col) * HEAD_DIM + c] = (L > 0.f) ? O / L : 0.f;
        } else {
            const long long pr = (row0 + col) * p.max_splits + split;
            p.part_o[pr * HEAD_DIM + c] = O;
            if (c == 0) p.part_ml[pr] = make_float2(M, L);
        }
    }
    if (nsplits == 1) return;

    // ---- the last CTA of this (sequence, head group) combines the splits -----------
    __threadfence();
    __syncthreads();
    int* ctr = p.counters + (long long)b * gridDim.y + item;
    if (threadIdx.x == 0) {
        const int old = atomicAdd(ctr, 1);
        s_is_last = (old == nsplits - 1);
    }
    __syncthreads();
    if (!s_is_last) return;
    __threadfence();
    for (int e = threadIdx.x; e < ncols * HEAD_DIM; e += NW * 32) {
        const int col = e >> 7, c = e & 127;
        const long long pr = (row0 + col) * p.max_splits;
        float M = -INFINITY;
        for (int s = 0; s < nsplits; ++s) M = fmaxf(M, __ldcg(&p.part_ml[pr + s].x));
        float L = 0.f, O = 0.f;
        if (M != -INFINITY) {
            for (int s = 0; s < nsplits; ++s) {
                const float2 ml = __ldcg(&p.part_ml[pr + s]);
                const float f = (ml.x == -INFINITY) ? 0.f : fast_exp2(ml.x - M);
                L += ml.y * f;
                O += __ldcg(&p.part_o[(pr + s) * HEAD_DIM + c]) * f;
            }
        }
        p.out[(row0 + col) * HEAD_DIM + c] = (L > 0.f) ? O / L : 0.f;
    }
    if (threadIdx.x == 0) *ctr = 0;       // ready for the next launch
}

}  // namespace tidal
