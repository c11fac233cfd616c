// A token selection layer in two passes over the cache (one sequence, one set per query head; bf16 caches,
// and at the end of this file caches of E4M3 codes).
//
// Algorithm 1's selection layer needs the scaled logits of every cached token twice: for the softmax
// of its own output and for argTopK. The fused kernel (attn_kernel<MODE_SELECT>) streams K and V
// together and the top-k can only start when all of it is done; the sparse layers after it then wait
// for the top-k, and for those 20 microseconds the memory system idles. Here the layer is split:
//
//   score_pass_kernel  streams the KEY rows only: logits, their histogram (for the top-k) and the largest
//                      logit M of every head (one atomicMax per CTA and head); the first CTA of a KV head
//                      clears the layer's output rows. No partial results, no combine.
//   value_pass_kernel  streams the VALUE rows only: softmax weights exp(s - M) come from the stored logits
//                      and the final M, so every partial result has the same scale and CTAs simply add
//                      their part of sum_j p_j v_j and of sum_j p_j to the output row and to the head's sum
//                      with reductions; the last CTA of a KV head to finish divides the rows by the sums.
//
// The step driver launches the value pass on a second stream, so that it runs beside the top-k: the layer
// then costs what its two streaming passes cost, the top-k's latency chain hides behind the second. Key and value rows interleave in memory at 256-byte granularity; reading every
// other 256-byte row costs HBM nothing (measured: the same useful bandwidth as the dense stream).
#pragma once

#include "attn_kernels.cuh"

namespace tidal {

constexpr float LOG2E = 1.4426950408889634f;

// Tile sequence of one warp of a pooled launch (see attn_kernel): a fixed first chunk, then GRAB
// tiles at a time from the item's cursor, requested one chunk ahead.
struct PoolWalk {
    int cur, cur_end, grab_raw, tiles, pool_base, lane;
    int* pool;
    template <int GRAB>
    __device__ __forceinline__ void start(int* cursor, int tiles_, int item_warps, int my_warp, int first_tiles_max, int lane_) {
        pool = cursor; tiles = tiles_; lane = lane_; grab_raw = 0;
        const int first = (tiles <= item_warps * first_tiles_max) ? max(1, (tiles + item_warps - 1) / max(item_warps, 1))
                                                                  : first_tiles_max;
        pool_base = item_warps * first;
        cur = my_warp * first;
        cur_end = min(tiles, cur + first);
        if (lane == 0) grab_raw = pool_base + atomicAdd(pool, GRAB);
    }
    template <int GRAB>
    __device__ __forceinline__ int next() {
        if (cur >= cur_end) {
            if (cur_end >= tiles || pool_base >= tiles) return -1;
            cur = __shfl_sync(0xffffffffu, grab_raw, 0);
            if (cur >= tiles) { cur_end = tiles; return -1; }
            cur_end = min(tiles, cur + GRAB);
            if (lane == 0) grab_raw = pool_base + atomicAdd(pool, GRAB);
        }
        return cur++;
    }
};

// ---- pass 1: logits, histogram, softmax statistics -------------------------------------------------------
// Uses of AttnParams: q, k, strides, page table, ctx_lens, scale, scores / score_stride, hist / hist_shift,
// tile_ctr / ctr_stride (a cursor set of the main stream's rotation), split_max (per head: the order-preserving
// key of the largest logit, 0 = none yet), out (cleared), pdl / wait_first / wait_late / trigger_early, status.
// batch must be 1, splits_per_item > 0. The loop is written for few instructions per tile (a tile is only 4 KB
// here): constant ring-slot numbers, tile numbers in registers, one unmasked path for whole tiles of eight heads.
// ROW512: consecutive positions of a head lie 512 bytes apart (K and V rows interleaved, contiguous or paged),
// so that the sixteen rows of a tile are reached with constant offsets from one pointer.
template <int NW, int STAGES, bool ROW512>
__global__ void __launch_bounds__(NW * 32, 1) score_pass_kernel(const AttnParams p) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    __shared__ float s_max[NW][8];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gid = lane >> 2, tig = lane & 3;
    constexpr int RING_BYTES = NW * STAGES * TILE_BYTES;
    uint32_t* hist = reinterpret_cast<uint32_t*>(smem + RING_BYTES);
    const bool hist_on = p.hist != nullptr;

    bool waited = !p.pdl;
    if (p.pdl && p.wait_first) { pdl_wait(); pdl_trigger(); waited = true; }
    else if (p.pdl && p.wait_late && p.trigger_early) pdl_trigger();

    const int n_items = p.Hkv;                               // one sequence
    const int g = blockIdx.x % n_items, part = blockIdx.x / n_items;
    const int item_ctas = ((int)gridDim.x - g + n_items - 1) / n_items;
    const int N = max(min(p.ctx_lens[0], p.max_ctx), 0);
    const int tiles = item_tiles(N);
    const int head0 = g * p.G, ncols = p.G;
    // this lane's two heads (2 tig, 2 tig + 1; clamped to the group, masked where they are used) and its row gid
    const bool col0 = 2 * tig < ncols, col1 = 2 * tig + 1 < ncols;
    float* const score_row0 = p.scores + (long long)(head0 + min(2 * tig, ncols - 1)) * p.score_stride + gid;
    float* const score_row1 = p.scores + (long long)(head0 + min(2 * tig + 1, ncols - 1)) * p.score_stride + gid;
    const int hshift = p.hist_shift;
    uint32_t* const h0 = hist + ((2 * tig) << (32 - hshift));
    uint32_t* const h1 = hist + ((2 * tig + 1) << (32 - hshift));

    const uint32_t wbase = smem_u32(smem + (size_t)warp * STAGES * TILE_BYTES);
    const int c16 = lane & 15, rhalf = lane >> 4;
    const long long two_rows = 2 * p.stride_pos;
    const long long tile_step = (long long)TILE * p.stride_pos;
    // key rows in a ring slot: row r at r * 256, its 16-byte piece c at position c ^ (r & 7), so that the eight
    // rows of an ldmatrix fall into different banks; this lane copies piece c16 of rows rhalf + 2 i
    uint32_t kdst[4];                                        // rows i and i + 4 share a swizzle
#pragma unroll
    for (int i = 0; i < 4; ++i) kdst[i] = (rhalf + 2 * i) * 256 + ((c16 ^ (rhalf + 2 * i)) << 4);
    const __nv_bfloat16* const kbase = p.k + (long long)g * p.stride_head + (long long)rhalf * p.stride_pos + c16 * 8;
    const uint64_t kv_policy = l2_evict_first_policy();
    const uint64_t keep = l2_evict_last_policy();

    int* pool = p.tile_ctr + (long long)g * p.ctr_stride;
    PoolWalk walk;
    constexpr int GRAB = GRAB_TILES_DENSE;
    walk.template start<GRAB>(pool, tiles, item_ctas * NW, part * NW + warp, STAGES + 2, lane);

    // A ring slot's tile number stays in a register (the ring is walked with constant slot numbers); a tile
    // whose page id is outside the pool is marked and counts as empty.
    constexpr int BAD_TILE = 1 << 30;
    auto issue = [&](uint32_t ks, int& tile) {
        const __nv_bfloat16* src;
        if (p.paged) {
            const int page = __ldg(p.page_table + tile);
            const bool ok = (unsigned)page < (unsigned)p.num_pages;
            if (!ok) {
                if (lane == 0) atomicOr(p.status, STATUS_BAD_PAGE);
                tile |= BAD_TILE;
            }
            src = kbase + (ok ? (long long)page * p.stride_page : 0);
        } else {
            src = kbase + tile * tile_step;
        }
        const int nvalid = (tile & BAD_TILE) ? 0 : max(0, min(TILE, N - tile * TILE));
        if (nvalid == TILE) {
            if (ROW512) {
#pragma unroll
                for (int i = 0; i < 8; ++i) cp_async16_full_hint(ks + kdst[i & 3] + (i >> 2) * 2048, src + i * (4 * HEAD_DIM), kv_policy);
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i) cp_async16_full_hint(ks + kdst[i & 3] + (i >> 2) * 2048, src + i * two_rows, kv_policy);
            }
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const bool rv = rhalf + 2 * i < nvalid;
                cp_async16_hint(ks + kdst[i & 3] + (i >> 2) * 2048, rv ? src + i * two_rows : p.k, rv ? 16 : 0, kv_policy);
            }
        }
    };

    int tl[STAGES];
#pragma unroll
    for (int s = 0; s < STAGES; ++s) tl[s] = -1;
    // fill all but one slot; a kernel that may read ahead of its wait still leaves the last tile (the newest
    // token's row) for afterwards
#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) {
        int t = walk.template next<GRAB>();
        if (t >= 0) {
            if (!waited && !p.wait_late && t == tiles - 1) { pdl_wait(); pdl_trigger(); waited = true; }
            issue(wbase + s * TILE_BYTES, t);
        }
        tl[s] = t;
        cp_async_commit();
    }
    if (!waited && !p.wait_late) { pdl_wait(); pdl_trigger(); waited = true; }
    if (hist_on) {                                     // (the first tiles are on their way meanwhile)
        for (int i = threadIdx.x; i < HIST_SMEM_WORDS; i += NW * 32) hist[i] = 0;
        __syncthreads();
    }
    // a selection layer that waits late writes its scores ahead of the wait: the host allows that only
    // when nothing can still be reading the score buffer
    // B fragments of the eight k-steps: head gid's elements 16 j + 2 tig (+1) and 16 j + 8 + 2 tig (+1)
    uint32_t qf[8][2];
    {
        const uint32_t* qw = reinterpret_cast<const uint32_t*>(p.q + (long long)(head0 + min(gid, ncols - 1)) * HEAD_DIM);
        const bool on = gid < ncols;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t w0 = __ldg(qw + 8 * j + tig), w1 = __ldg(qw + 8 * j + 4 + tig);
            qf[j][0] = on ? w0 : 0u;
            qf[j][1] = on ? w1 : 0u;
        }
    }
    float m0 = -INFINITY, m1 = -INFINITY;              // largest logit this lane has seen of heads 2tig, 2tig+1
    // ldmatrix: lane l addresses row (l & 7) + 8 * ((l >> 3) & 1), piece 2 j + (l >> 4) of the tile
    const int lrow = (lane & 7) + ((lane >> 3) & 1) * 8;
    const uint32_t klane = lrow * 256 + ((((lane >> 4) & 1) ^ (lane & 7)) << 4);

    auto consume = [&](uint32_t ks, int tile) {
        const int pos_base = (tile & ~BAD_TILE) * TILE;
        const int nvalid = (tile & BAD_TILE) ? 0 : max(0, min(TILE, N - pos_base));
        // S^T = K . Q^T: positions are the rows of the MMA, the group's heads its columns; two accumulator chains
        float s[4] = {0.f, 0.f, 0.f, 0.f}, s2[4] = {0.f, 0.f, 0.f, 0.f};
        const uint32_t kl = ks + klane;
#pragma unroll
        for (int j = 0; j < 8; j += 2) {
            uint32_t a[4], b[4];
            ldmatrix_x4(kl ^ (j << 5), a);             // ring slots are 256-byte aligned
            ldmatrix_x4(kl ^ ((j + 1) << 5), b);
            mma_bf16_16816(s, a[0], a[1], a[2], a[3], qf[j][0], qf[j][1]);
            mma_bf16_16816(s2, b[0], b[1], b[2], b[3], qf[j + 1][0], qf[j + 1][1]);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) s[i] += s2[i];
        const float f0 = s[0] * p.scale, f1 = s[1] * p.scale, f2 = s[2] * p.scale, f3 = s[3] * p.scale;
        if (nvalid == TILE) {
            // the common case: sixteen cached tokens, no row to mask (lanes beyond the group's heads sit out)
            if (col0) {
                st_keep(score_row0 + pos_base, f0, keep);
                st_keep(score_row0 + pos_base + 8, f2, keep);
                if (hist_on) {
                    atomicAdd(h0 + (score_key_bits(f0) >> hshift), 1u);
                    atomicAdd(h0 + (score_key_bits(f2) >> hshift), 1u);
                }
                m0 = fmaxf(m0, fmaxf(f0, f2));
            }
            if (col1) {
                st_keep(score_row1 + pos_base, f1, keep);
                st_keep(score_row1 + pos_base + 8, f3, keep);
                if (hist_on) {
                    atomicAdd(h1 + (score_key_bits(f1) >> hshift), 1u);
                    atomicAdd(h1 + (score_key_bits(f3) >> hshift), 1u);
                }
                m1 = fmaxf(m1, fmaxf(f1, f3));
            }
        } else {
            const bool v0 = gid < nvalid, v1 = gid + 8 < nvalid;
            if (col0) {
                if (v0) st_keep(score_row0 + pos_base, f0, keep);
                if (v1) st_keep(score_row0 + pos_base + 8, f2, keep);
            }
            if (col1) {
                if (v0) st_keep(score_row1 + pos_base, f1, keep);
                if (v1) st_keep(score_row1 + pos_base + 8, f3, keep);
            }
            if (hist_on) {
                if (col0) {
                    if (v0) atomicAdd(h0 + (score_key_bits(f0) >> hshift), 1u);
                    if (v1) atomicAdd(h0 + (score_key_bits(f2) >> hshift), 1u);
                }
                if (col1) {
                    if (v0) atomicAdd(h1 + (score_key_bits(f1) >> hshift), 1u);
                    if (v1) atomicAdd(h1 + (score_key_bits(f3) >> hshift), 1u);
                }
            }
            if (v0) { m0 = fmaxf(m0, f0); m1 = fmaxf(m1, f1); }
            if (v1) { m0 = fmaxf(m0, f2); m1 = fmaxf(m1, f3); }
        }
    };

    for (bool live = true; live;) {
#pragma unroll
        for (int s = 0; s < STAGES; ++s) {
            if (tl[s] < 0) { live = false; break; }
            cp_async_wait<STAGES - 2>();
            __syncwarp();                              // every lane is done with the slot that is refilled next
            const int sn = (s + STAGES - 1) % STAGES;
            int t = walk.template next<GRAB>();
            if (t >= 0) issue(wbase + sn * TILE_BYTES, t);
            tl[sn] = t;
            cp_async_commit();
            consume(wbase + s * TILE_BYTES, tl[s]);
        }
    }
    cp_async_wait<0>();
    __syncwarp();
    if (!waited) {
        pdl_wait();
        if (!p.trigger_early) pdl_trigger();
        waited = true;
    }
    if (hist_on) {
        __syncthreads();
        const int nb = 1 << (32 - p.hist_shift);
        for (int i = threadIdx.x; i < ncols * nb; i += NW * 32) {
            const uint32_t w = hist[i];
            if (w) atomicAdd(p.hist + (long long)(head0 + i / nb) * HIST_BINS + (i % nb), w);
        }
    }
    // ---- the largest logit of this CTA per head, then of the head: one atomicMax on its key -------------
#pragma unroll
    for (int sh = 4; sh <= 16; sh <<= 1) {
        m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, sh));
        m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, sh));
    }
    if (gid == 0) { s_max[warp][2 * tig] = m0; s_max[warp][2 * tig + 1] = m1; }
    __syncthreads();
    if (threadIdx.x < ncols) {
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < NW; ++w) M = fmaxf(M, s_max[w][threadIdx.x]);
        if (M != -INFINITY) atomicMax(p.split_max + head0 + threadIdx.x, score_key_bits(M));
    }
    // the value pass adds its parts to the output rows: they start at zero (this pass ends before it starts)
    if (part == 0)
        for (int e = threadIdx.x; e < ncols * HEAD_DIM; e += NW * 32) p.out[(long long)head0 * HEAD_DIM + e] = 0.f;
    // the pool cursor of this launch's set is cleared by the item's last CTA to get here
    if (threadIdx.x == 0) {
        int* ctr = p.counters + (long long)g * p.ctr_stride;
        int old;
        asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;\n" : "=r"(old) : "l"(ctr) : "memory");
        if (old == item_ctas - 1) { *ctr = 0; *pool = 0; __threadfence(); }
    }
}

// ---- pass 2: sum_j softmax_j v_j from the stored logits ------------------------------------------------------
// Uses of AttnParams: v, strides, page table, ctx_lens, scores / score_stride, split_max, split_sum (per head,
// zero between launches), out (+= with reductions, then divided, the quotient written to out_final if given),
// counters / tile_ctr / ctr_stride (arrays of its
// own: it runs beside the main stream's kernels), status.
template <int NW, int STAGES, bool ROW512>
__global__ void __launch_bounds__(NW * 32, 2) value_pass_kernel(const AttnParams p) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    constexpr int SLOT = TILE_BYTES + 512;                   // 16 value rows, then 16 logits of up to 8 heads

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gid = lane >> 2, tig = lane & 3;
    const int n_items = p.Hkv;
    const int g = blockIdx.x % n_items, part = blockIdx.x / n_items;
    const int item_ctas = ((int)gridDim.x - g + n_items - 1) / n_items;
    const int N = max(min(p.ctx_lens[0], p.max_ctx), 0);
    const int tiles = item_tiles(N);
    const int head0 = g * p.G, ncols = p.G;

    const uint32_t wbase = smem_u32(smem + (size_t)warp * STAGES * SLOT);
    const int c16 = lane & 15, rhalf = lane >> 4;
    const long long two_rows = 2 * p.stride_pos;
    const long long tile_step = (long long)TILE * p.stride_pos;
    const uint32_t vc = c16 ^ rhalf;
    uint32_t vdst[4];                                        // row pairs i and i + 4 share a swizzle
#pragma unroll
    for (int i = 0; i < 4; ++i) vdst[i] = rhalf * 256 + i * 512 + ((vc ^ (i << 1)) << 4);
    const __nv_bfloat16* const vbase = p.v + (long long)g * p.stride_head + (long long)rhalf * p.stride_pos + c16 * 8;
    const uint64_t kv_policy = l2_evict_first_policy();
    // lane l < 4 * ncols fetches 16 bytes (four positions) of head l >> 2's logits
    const bool score_lane = lane < 4 * ncols;
    const float* const score_src = p.scores + (long long)(head0 + min(lane >> 2, ncols - 1)) * p.score_stride + 4 * (lane & 3);
    const uint32_t score_dst = TILE_BYTES + lane * 16;

    int* pool = p.tile_ctr + (long long)g * p.ctr_stride;
    PoolWalk walk;
    constexpr int GRAB = GRAB_TILES_DENSE;
    walk.template start<GRAB>(pool, tiles, item_ctas * NW, part * NW + warp, STAGES + 2, lane);

    constexpr int BAD_TILE = 1 << 30;
    auto issue = [&](uint32_t vs, int& tile) {
        const __nv_bfloat16* src;
        if (p.paged) {
            const int page = __ldg(p.page_table + tile);
            const bool ok = (unsigned)page < (unsigned)p.num_pages;
            if (!ok) {
                if (lane == 0) atomicOr(p.status, STATUS_BAD_PAGE);
                tile |= BAD_TILE;
            }
            src = vbase + (ok ? (long long)page * p.stride_page : 0);
        } else {
            src = vbase + tile * tile_step;
        }
        const int pos0 = (tile & ~BAD_TILE) * TILE;
        const int nvalid = (tile & BAD_TILE) ? 0 : max(0, min(TILE, N - pos0));
        if (nvalid == TILE) {
#pragma unroll
            for (int i = 0; i < 8; ++i)
                cp_async16_full_hint(vs + vdst[i & 3] + (i >> 2) * 2048, ROW512 ? src + i * (4 * HEAD_DIM) : src + i * two_rows, kv_policy);
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const bool rv = rhalf + 2 * i < nvalid;
                cp_async16_hint(vs + vdst[i & 3] + (i >> 2) * 2048, rv ? src + i * two_rows : p.v, rv ? 16 : 0, kv_policy);
            }
        }
        // (logits past the end of the sequence are never used: their rows are masked)
        if (score_lane) cp_async16(vs + score_dst, score_src + pos0, 16);
    };

    // the largest logit of this lane's two heads, in base-2 units (key 0: the head has no token at all)
    float M0 = -INFINITY, M1 = -INFINITY;
    {
        const uint32_t k0 = (2 * tig < ncols) ? __ldcg(p.split_max + head0 + 2 * tig) : 0u;
        const uint32_t k1 = (2 * tig + 1 < ncols) ? __ldcg(p.split_max + head0 + 2 * tig + 1) : 0u;
        if (k0) M0 = __uint_as_float((k0 & 0x80000000u) ? (k0 & 0x7fffffffu) : ~k0) * LOG2E;
        if (k1) M1 = __uint_as_float((k1 & 0x80000000u) ? (k1 & 0x7fffffffu) : ~k1) * LOG2E;
    }
    const bool h0 = 2 * tig < ncols && M0 != -INFINITY, h1 = 2 * tig + 1 < ncols && M1 != -INFINITY;
    const bool col0 = 2 * tig < ncols, col1 = 2 * tig + 1 < ncols;
    const bool plain = __all_sync(0xffffffffu, (h0 || !col0) && (h1 || !col1));   // every head of the group has a finite maximum
    float l0 = 0.f, l1 = 0.f;                          // this lane's share of sum_j p_j
    float o[8][4];
#pragma unroll
    for (int t = 0; t < 8; ++t) { o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f; }
    // logits of (position gid | gid + 8, heads 2tig | 2tig + 1): head h's 16 floats start at 64 * h
    const uint32_t slane = TILE_BYTES + (2 * tig) * 64 + gid * 4;
    const int rr = lane & 7, mb = (lane >> 3) & 1;
    const uint32_t vlane = (rr + ((lane >> 4) << 3)) * 256 + ((rr ^ mb) << 4);

    auto consume = [&](uint32_t vs, int tile) {
        const int nvalid = (tile & BAD_TILE) ? 0 : max(0, min(TILE, N - (tile & ~BAD_TILE) * TILE));
        float f0, f1, f2, f3;
        asm volatile("ld.shared.f32 %0, [%1];\n" : "=f"(f0) : "r"(vs + slane));
        asm volatile("ld.shared.f32 %0, [%1];\n" : "=f"(f2) : "r"(vs + slane + 32));
        asm volatile("ld.shared.f32 %0, [%1];\n" : "=f"(f1) : "r"(vs + slane + 64));
        asm volatile("ld.shared.f32 %0, [%1];\n" : "=f"(f3) : "r"(vs + slane + 96));
        float p0, p1, p2, p3;
        if (nvalid == TILE && plain) {
            p0 = col0 ? fast_exp2(f0 * LOG2E - M0) : 0.f; p1 = col1 ? fast_exp2(f1 * LOG2E - M1) : 0.f;
            p2 = col0 ? fast_exp2(f2 * LOG2E - M0) : 0.f; p3 = col1 ? fast_exp2(f3 * LOG2E - M1) : 0.f;
        } else {
            const bool v0 = gid < nvalid, v1 = gid + 8 < nvalid;
            p0 = (v0 && h0) ? fast_exp2(f0 * LOG2E - M0) : 0.f; p1 = (v0 && h1) ? fast_exp2(f1 * LOG2E - M1) : 0.f;
            p2 = (v1 && h0) ? fast_exp2(f2 * LOG2E - M0) : 0.f; p3 = (v1 && h1) ? fast_exp2(f3 * LOG2E - M1) : 0.f;
        }
        l0 += p0 + p2;
        l1 += p1 + p3;
        const uint32_t pb0 = movmatrix_trans(pack_bf16(p0, p1));
        const uint32_t pb1 = movmatrix_trans(pack_bf16(p2, p3));
        const uint32_t vl = vs + vlane;
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            uint32_t a[4];
            ldmatrix_x4_trans(vl ^ (t << 5), a);
            mma_bf16_16816(o[t], a[0], a[1], a[2], a[3], pb0, pb1);
        }
    };

    int tl[STAGES];
#pragma unroll
    for (int s = 0; s < STAGES; ++s) tl[s] = -1;
#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) {
        int t = walk.template next<GRAB>();
        if (t >= 0) issue(wbase + s * SLOT, t);
        tl[s] = t;
        cp_async_commit();
    }
    for (bool live = true; live;) {
#pragma unroll
        for (int s = 0; s < STAGES; ++s) {
            if (tl[s] < 0) { live = false; break; }
            cp_async_wait<STAGES - 2>();
            __syncwarp();                              // every lane is done with the slot that is refilled next
            const int sn = (s + STAGES - 1) % STAGES;
            int t = walk.template next<GRAB>();
            if (t >= 0) issue(wbase + sn * SLOT, t);
            tl[sn] = t;
            cp_async_commit();
            consume(wbase + s * SLOT, tl[s]);
        }
    }
    cp_async_wait<0>();
#pragma unroll
    for (int sh = 4; sh <= 16; sh <<= 1) {
        l0 += __shfl_xor_sync(0xffffffffu, l0, sh);
        l1 += __shfl_xor_sync(0xffffffffu, l1, sh);
    }
    __syncthreads();                                   // all rings drained; reuse the shared memory
    // ---- sum the warps of this CTA and add the CTA's part to the output rows and to the heads' sums ------
    float* mo = reinterpret_cast<float*>(smem);       // [NW][8][128]
    float* ml = mo + NW * 8 * HEAD_DIM;               // [NW][8]
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        float* w0 = mo + ((warp * 8 + 2 * tig) * HEAD_DIM);
        float* w1 = w0 + HEAD_DIM;
        w0[16 * t + gid] = o[t][0];
        w1[16 * t + gid] = o[t][1];
        w0[16 * t + 8 + gid] = o[t][2];
        w1[16 * t + 8 + gid] = o[t][3];
    }
    if (gid == 0) { ml[warp * 8 + 2 * tig] = l0; ml[warp * 8 + 2 * tig + 1] = l1; }
    __syncthreads();
    for (int e = threadIdx.x; e < ncols * (HEAD_DIM / 4); e += NW * 32) {      // four output elements per reduction
        const int col = e >> 5, c = (e & 31) * 4;
        float4 O = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int w = 0; w < NW; ++w) {
            const float4 t = *reinterpret_cast<const float4*>(mo + (w * 8 + col) * HEAD_DIM + c);
            O.x += t.x; O.y += t.y; O.z += t.z; O.w += t.w;
        }
        if (O.x != 0.f || O.y != 0.f || O.z != 0.f || O.w != 0.f)
            asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};\n" ::"l"(p.out + (long long)(head0 + col) * HEAD_DIM + c),
                         "f"(O.x), "f"(O.y), "f"(O.z), "f"(O.w) : "memory");
    }
    if (threadIdx.x < ncols) {
        float L = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) L += ml[w * 8 + threadIdx.x];
        if (L != 0.f) atomicAdd(p.split_sum + head0 + threadIdx.x, L);
    }
    // ---- the last CTA of this KV head to arrive divides the rows by the sums and cleans up --------------------
    __shared__ int s_last;
    __syncthreads();
    int* ctr = p.counters + (long long)g * p.ctr_stride;
    if (threadIdx.x == 0) {
        int old;
        asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;\n" : "=r"(old) : "l"(ctr) : "memory");
        s_last = (old == item_ctas - 1);
    }
    __syncthreads();
    if (s_last) {
        float* const rows = p.out_final ? p.out_final : p.out;
        for (int e = threadIdx.x; e < ncols * HEAD_DIM; e += NW * 32) {
            const float L = __ldcg(p.split_sum + head0 + (e >> 7));
            const float O = __ldcg(p.out + (long long)head0 * HEAD_DIM + e);
            rows[(long long)head0 * HEAD_DIM + e] = (L > 0.f) ? O / L : 0.f;
        }
        __syncthreads();
        if (threadIdx.x < ncols) { p.split_sum[head0 + threadIdx.x] = 0.f; p.split_max[head0 + threadIdx.x] = 0u; }
        if (threadIdx.x == 0) { *ctr = 0; *pool = 0; }
    }
}

// ---- the same two passes for a batch -------------------------------------------------------------------------
// Sequences of a batch differ in length, so the (sequence, KV head, tile) space is cut into equal contiguous
// ranges, one per CTA (the static flat split of attn_kernel). A CTA walks its range item by item; within an
// item its warps take tiles t0 + warp, t0 + warp + NW, ...; the per-item work of the pooled kernels (histogram
// flush, largest logits, clearing the output rows; sums, arrival, division) happens at the end of every
// segment. bf16 caches. Row indices: query head h of sequence b is row b * Hq + h of the scores, of split_max
// and of split_sum; item (b, g) owns counter b * Hkv + g.
struct FlatWalk {
    long long lo, hi, per_cta, seq_start;
    int b, tiles_b;
    // the range of CTA `cta` and the sequence its first tile lies in; false: no tile for this CTA
    __device__ __forceinline__ bool start(const AttnParams& p, int cta, int n_ctas) {
        long long T = 0;
        for (int bb = 0; bb < p.batch; ++bb) T += (long long)p.Hkv * item_tiles(max(min(p.ctx_lens[bb], p.max_ctx), 0));
        per_cta = (T + n_ctas - 1) / n_ctas;
        lo = (long long)cta * per_cta;
        hi = min(T, lo + per_cta);
        b = 0; seq_start = 0;
        tiles_b = item_tiles(max(min(p.ctx_lens[0], p.max_ctx), 0));
        if (lo >= hi) return false;
        while (seq_start + (long long)p.Hkv * tiles_b <= lo) {
            seq_start += (long long)p.Hkv * tiles_b;
            ++b;
            tiles_b = item_tiles(max(min(p.ctx_lens[b], p.max_ctx), 0));
        }
        return true;
    }
    // the segment at lo: KV head g, tiles [t0, t1) of sequence b
    __device__ __forceinline__ void segment(int& g, int& t0, int& t1) const {
        g = (int)((lo - seq_start) / tiles_b);
        t0 = (int)((lo - seq_start) % tiles_b);
        t1 = (int)min((long long)tiles_b, t0 + (hi - lo));
    }
    __device__ __forceinline__ void advance(const AttnParams& p, int done) {
        lo += done;
        if (lo < hi && lo >= seq_start + (long long)p.Hkv * tiles_b) {
            seq_start += (long long)p.Hkv * tiles_b;
            ++b;
            tiles_b = item_tiles(max(min(p.ctx_lens[b], p.max_ctx), 0));
        }
    }
};

template <int NW, int STAGES, bool ROW512>
__global__ void __launch_bounds__(NW * 32, 1) score_pass_flat_kernel(const AttnParams p) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    __shared__ float s_max[NW][8];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gid = lane >> 2, tig = lane & 3;
    constexpr int RING_BYTES = NW * STAGES * TILE_BYTES;
    uint32_t* hist = reinterpret_cast<uint32_t*>(smem + RING_BYTES);
    const bool hist_on = p.hist != nullptr;

    bool waited = !p.pdl;
    if (p.pdl && p.wait_first) { pdl_wait(); pdl_trigger(); waited = true; }
    else if (p.pdl && p.wait_late && p.trigger_early) pdl_trigger();

    FlatWalk fw;
    if (!fw.start(p, blockIdx.x, gridDim.x)) {
        if (!waited) pdl_wait();                     // (no CTA of a late-waiting launch retires before its predecessor is complete)
        return;
    }
    const int ncols = p.G;
    const bool col0 = 2 * tig < ncols, col1 = 2 * tig + 1 < ncols;
    const int hshift = p.hist_shift;
    uint32_t* const h0 = hist + ((2 * tig) << (32 - hshift));
    uint32_t* const h1 = hist + ((2 * tig + 1) << (32 - hshift));
    const uint32_t wbase = smem_u32(smem + (size_t)warp * STAGES * TILE_BYTES);
    const int c16 = lane & 15, rhalf = lane >> 4;
    const long long two_rows = 2 * p.stride_pos;
    const long long tile_step = (long long)TILE * p.stride_pos;
    uint32_t kdst[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) kdst[i] = (rhalf + 2 * i) * 256 + ((c16 ^ (rhalf + 2 * i)) << 4);
    const long long lane_off = (long long)rhalf * p.stride_pos + c16 * 8;
    const uint64_t kv_policy = l2_evict_first_policy();
    const uint64_t keep = l2_evict_last_policy();
    const int lrow = (lane & 7) + ((lane >> 3) & 1) * 8;
    const uint32_t klane = lrow * 256 + ((((lane >> 4) & 1) ^ (lane & 7)) << 4);
    constexpr int BAD_TILE = 1 << 30;

    while (fw.lo < fw.hi) {
        int g, t0, t1;
        fw.segment(g, t0, t1);
        const int b = fw.b;
        const int N = max(min(p.ctx_lens[b], p.max_ctx), 0);
        const long long row0 = (long long)b * p.Hq + g * p.G;          // first query head of the item, as a row index
        float* const score_row0 = p.scores + (row0 + min(2 * tig, ncols - 1)) * p.score_stride + gid;
        float* const score_row1 = p.scores + (row0 + min(2 * tig + 1, ncols - 1)) * p.score_stride + gid;
        const __nv_bfloat16* const kbase = p.k + (p.paged ? 0 : (long long)b * p.stride_b) + (long long)g * p.stride_head + lane_off;
        const int* const pages = p.page_table + (long long)b * p.max_pages;
        if (hist_on) {
            for (int i = threadIdx.x; i < HIST_SMEM_WORDS; i += NW * 32) hist[i] = 0;
            __syncthreads();
        }
        uint32_t qf[8][2];
        {
            const uint32_t* qw = reinterpret_cast<const uint32_t*>(p.q + (row0 + min(gid, ncols - 1)) * HEAD_DIM);
            const bool on = gid < ncols;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint32_t w0 = __ldg(qw + 8 * j + tig), w1 = __ldg(qw + 8 * j + 4 + tig);
                qf[j][0] = on ? w0 : 0u;
                qf[j][1] = on ? w1 : 0u;
            }
        }
        float m0 = -INFINITY, m1 = -INFINITY;

        auto issue = [&](uint32_t ks, int& tile) {
            const __nv_bfloat16* src;
            if (p.paged) {
                const int page = __ldg(pages + tile);
                const bool ok = (unsigned)page < (unsigned)p.num_pages;
                if (!ok) {
                    if (lane == 0) atomicOr(p.status, STATUS_BAD_PAGE);
                    tile |= BAD_TILE;
                }
                src = kbase + (ok ? (long long)page * p.stride_page : 0);
            } else {
                src = kbase + tile * tile_step;
            }
            const int nvalid = (tile & BAD_TILE) ? 0 : max(0, min(TILE, N - tile * TILE));
            if (nvalid == TILE) {
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    cp_async16_full_hint(ks + kdst[i & 3] + (i >> 2) * 2048, ROW512 ? src + i * (4 * HEAD_DIM) : src + i * two_rows, kv_policy);
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const bool rv = rhalf + 2 * i < nvalid;
                    cp_async16_hint(ks + kdst[i & 3] + (i >> 2) * 2048, rv ? src + i * two_rows : p.k, rv ? 16 : 0, kv_policy);
                }
            }
        };
        auto consume = [&](uint32_t ks, int tile) {
            const int pos_base = (tile & ~BAD_TILE) * TILE;
            const int nvalid = (tile & BAD_TILE) ? 0 : max(0, min(TILE, N - pos_base));
            float s[4] = {0.f, 0.f, 0.f, 0.f}, s2[4] = {0.f, 0.f, 0.f, 0.f};
            const uint32_t kl = ks + klane;
#pragma unroll
            for (int j = 0; j < 8; j += 2) {
                uint32_t a[4], bb[4];
                ldmatrix_x4(kl ^ (j << 5), a);
                ldmatrix_x4(kl ^ ((j + 1) << 5), bb);
                mma_bf16_16816(s, a[0], a[1], a[2], a[3], qf[j][0], qf[j][1]);
                mma_bf16_16816(s2, bb[0], bb[1], bb[2], bb[3], qf[j + 1][0], qf[j + 1][1]);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) s[i] += s2[i];
            const float f0 = s[0] * p.scale, f1 = s[1] * p.scale, f2 = s[2] * p.scale, f3 = s[3] * p.scale;
            const bool v0 = gid < nvalid, v1 = gid + 8 < nvalid;
            if (col0) {
                if (v0) st_keep(score_row0 + pos_base, f0, keep);
                if (v1) st_keep(score_row0 + pos_base + 8, f2, keep);
                if (hist_on) {
                    if (v0) atomicAdd(h0 + (score_key_bits(f0) >> hshift), 1u);
                    if (v1) atomicAdd(h0 + (score_key_bits(f2) >> hshift), 1u);
                }
                if (v0) m0 = fmaxf(m0, f0);
                if (v1) m0 = fmaxf(m0, f2);
            }
            if (col1) {
                if (v0) st_keep(score_row1 + pos_base, f1, keep);
                if (v1) st_keep(score_row1 + pos_base + 8, f3, keep);
                if (hist_on) {
                    if (v0) atomicAdd(h1 + (score_key_bits(f1) >> hshift), 1u);
                    if (v1) atomicAdd(h1 + (score_key_bits(f3) >> hshift), 1u);
                }
                if (v0) m1 = fmaxf(m1, f1);
                if (v1) m1 = fmaxf(m1, f3);
            }
        };

        // this warp's tiles of the segment: t0 + warp, + NW, ... below t1
        int nxt = t0 + warp;
        auto take = [&]() { const int t = nxt < t1 ? nxt : -1; nxt += NW; return t; };
        int tl[STAGES];
#pragma unroll
        for (int s = 0; s < STAGES; ++s) tl[s] = -1;
#pragma unroll
        for (int s = 0; s < STAGES - 1; ++s) {
            int t = take();
            if (t >= 0) {
                // a kernel that may read ahead of its wait leaves a sequence's last tile (the newest token's row) for afterwards
                if (!waited && !p.wait_late && t == fw.tiles_b - 1) { pdl_wait(); pdl_trigger(); waited = true; }
                issue(wbase + s * TILE_BYTES, t);
            }
            tl[s] = t;
            cp_async_commit();
        }
        if (!waited && !p.wait_late) { pdl_wait(); pdl_trigger(); waited = true; }
        for (bool live = true; live;) {
#pragma unroll
            for (int s = 0; s < STAGES; ++s) {
                if (tl[s] < 0) { live = false; break; }
                cp_async_wait<STAGES - 2>();
                __syncwarp();
                const int sn = (s + STAGES - 1) % STAGES;
                int t = take();
                if (t >= 0) issue(wbase + sn * TILE_BYTES, t);
                tl[sn] = t;
                cp_async_commit();
                consume(wbase + s * TILE_BYTES, tl[s]);
            }
        }
        cp_async_wait<0>();
        __syncwarp();
        if (!waited) {
            pdl_wait();
            if (!p.trigger_early) pdl_trigger();
            waited = true;
        }
        __syncthreads();                               // every warp's counts of this segment are in
        if (hist_on) {
            const int nb = 1 << (32 - hshift);
            for (int i = threadIdx.x; i < ncols * nb; i += NW * 32) {
                const uint32_t w = hist[i];
                if (w) atomicAdd(p.hist + (row0 + i / nb) * HIST_BINS + (i % nb), w);
            }
        }
#pragma unroll
        for (int sh = 4; sh <= 16; sh <<= 1) {
            m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, sh));
            m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, sh));
        }
        if (gid == 0) { s_max[warp][2 * tig] = m0; s_max[warp][2 * tig + 1] = m1; }
        __syncthreads();
        if (threadIdx.x < ncols) {
            float M = -INFINITY;
#pragma unroll
            for (int w = 0; w < NW; ++w) M = fmaxf(M, s_max[w][threadIdx.x]);
            if (M != -INFINITY) atomicMax(p.split_max + row0 + threadIdx.x, score_key_bits(M));
        }
        // the CTA that holds an item's first tile clears its output rows (the value pass adds to them)
        if (t0 == 0)
            for (int e = threadIdx.x; e < ncols * HEAD_DIM; e += NW * 32) p.out[row0 * HEAD_DIM + e] = 0.f;
        __syncthreads();                               // the histogram and s_max are reused by the next segment
        fw.advance(p, t1 - t0);
    }
}

template <int NW, int STAGES, bool ROW512>
__global__ void __launch_bounds__(NW * 32, 2) value_pass_flat_kernel(const AttnParams p) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    constexpr int SLOT = TILE_BYTES + 512;                   // 16 value rows, then 16 logits of up to 8 heads
    __shared__ int s_last;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gid = lane >> 2, tig = lane & 3;
    FlatWalk fw;
    if (!fw.start(p, blockIdx.x, gridDim.x)) return;
    const int ncols = p.G;
    const bool col0 = 2 * tig < ncols, col1 = 2 * tig + 1 < ncols;

    const uint32_t wbase = smem_u32(smem + (size_t)warp * STAGES * SLOT);
    const int c16 = lane & 15, rhalf = lane >> 4;
    const long long two_rows = 2 * p.stride_pos;
    const long long tile_step = (long long)TILE * p.stride_pos;
    const uint32_t vc = c16 ^ rhalf;
    uint32_t vdst[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) vdst[i] = rhalf * 256 + i * 512 + ((vc ^ (i << 1)) << 4);
    const long long lane_off = (long long)rhalf * p.stride_pos + c16 * 8;
    const uint64_t kv_policy = l2_evict_first_policy();
    const bool score_lane = lane < 4 * ncols;
    const uint32_t score_dst = TILE_BYTES + lane * 16;
    const uint32_t slane = TILE_BYTES + (2 * tig) * 64 + gid * 4;
    const int rr = lane & 7, mb = (lane >> 3) & 1;
    const uint32_t vlane = (rr + ((lane >> 4) << 3)) * 256 + ((rr ^ mb) << 4);
    constexpr int BAD_TILE = 1 << 30;

    while (fw.lo < fw.hi) {
        int g, t0, t1;
        fw.segment(g, t0, t1);
        const int b = fw.b;
        const int N = max(min(p.ctx_lens[b], p.max_ctx), 0);
        const long long row0 = (long long)b * p.Hq + g * p.G;
        const __nv_bfloat16* const vbase = p.v + (p.paged ? 0 : (long long)b * p.stride_b) + (long long)g * p.stride_head + lane_off;
        const int* const pages = p.page_table + (long long)b * p.max_pages;
        const float* const score_src = p.scores + (row0 + min(lane >> 2, ncols - 1)) * p.score_stride + 4 * (lane & 3);
        float M0 = -INFINITY, M1 = -INFINITY;
        {
            const uint32_t k0 = col0 ? __ldcg(p.split_max + row0 + 2 * tig) : 0u;
            const uint32_t k1 = col1 ? __ldcg(p.split_max + row0 + 2 * tig + 1) : 0u;
            if (k0) M0 = __uint_as_float((k0 & 0x80000000u) ? (k0 & 0x7fffffffu) : ~k0) * LOG2E;
            if (k1) M1 = __uint_as_float((k1 & 0x80000000u) ? (k1 & 0x7fffffffu) : ~k1) * LOG2E;
        }
        const bool h0 = col0 && M0 != -INFINITY, h1 = col1 && M1 != -INFINITY;
        float l0 = 0.f, l1 = 0.f;
        float o[8][4];
#pragma unroll
        for (int t = 0; t < 8; ++t) { o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f; }

        auto issue = [&](uint32_t vs, int& tile) {
            const __nv_bfloat16* src;
            if (p.paged) {
                const int page = __ldg(pages + tile);
                const bool ok = (unsigned)page < (unsigned)p.num_pages;
                if (!ok) {
                    if (lane == 0) atomicOr(p.status, STATUS_BAD_PAGE);
                    tile |= BAD_TILE;
                }
                src = vbase + (ok ? (long long)page * p.stride_page : 0);
            } else {
                src = vbase + tile * tile_step;
            }
            const int pos0 = (tile & ~BAD_TILE) * TILE;
            const int nvalid = (tile & BAD_TILE) ? 0 : max(0, min(TILE, N - pos0));
            if (nvalid == TILE) {
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    cp_async16_full_hint(vs + vdst[i & 3] + (i >> 2) * 2048, ROW512 ? src + i * (4 * HEAD_DIM) : src + i * two_rows, kv_policy);
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const bool rv = rhalf + 2 * i < nvalid;
                    cp_async16_hint(vs + vdst[i & 3] + (i >> 2) * 2048, rv ? src + i * two_rows : p.v, rv ? 16 : 0, kv_policy);
                }
            }
            if (score_lane) cp_async16(vs + score_dst, score_src + pos0, 16);
        };
        auto consume = [&](uint32_t vs, int tile) {
            const int nvalid = (tile & BAD_TILE) ? 0 : max(0, min(TILE, N - (tile & ~BAD_TILE) * TILE));
            float f0, f1, f2, f3;
            asm volatile("ld.shared.f32 %0, [%1];\n" : "=f"(f0) : "r"(vs + slane));
            asm volatile("ld.shared.f32 %0, [%1];\n" : "=f"(f2) : "r"(vs + slane + 32));
            asm volatile("ld.shared.f32 %0, [%1];\n" : "=f"(f1) : "r"(vs + slane + 64));
            asm volatile("ld.shared.f32 %0, [%1];\n" : "=f"(f3) : "r"(vs + slane + 96));
            const bool v0 = gid < nvalid, v1 = gid + 8 < nvalid;
            const float p0 = (v0 && h0) ? fast_exp2(f0 * LOG2E - M0) : 0.f, p1 = (v0 && h1) ? fast_exp2(f1 * LOG2E - M1) : 0.f;
            const float p2 = (v1 && h0) ? fast_exp2(f2 * LOG2E - M0) : 0.f, p3 = (v1 && h1) ? fast_exp2(f3 * LOG2E - M1) : 0.f;
            l0 += p0 + p2;
            l1 += p1 + p3;
            const uint32_t pb0 = movmatrix_trans(pack_bf16(p0, p1));
            const uint32_t pb1 = movmatrix_trans(pack_bf16(p2, p3));
            const uint32_t vl = vs + vlane;
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                uint32_t a[4];
                ldmatrix_x4_trans(vl ^ (t << 5), a);
                mma_bf16_16816(o[t], a[0], a[1], a[2], a[3], pb0, pb1);
            }
        };

        int nxt = t0 + warp;
        auto take = [&]() { const int t = nxt < t1 ? nxt : -1; nxt += NW; return t; };
        int tl[STAGES];
#pragma unroll
        for (int s = 0; s < STAGES; ++s) tl[s] = -1;
#pragma unroll
        for (int s = 0; s < STAGES - 1; ++s) {
            int t = take();
            if (t >= 0) issue(wbase + s * SLOT, t);
            tl[s] = t;
            cp_async_commit();
        }
        for (bool live = true; live;) {
#pragma unroll
            for (int s = 0; s < STAGES; ++s) {
                if (tl[s] < 0) { live = false; break; }
                cp_async_wait<STAGES - 2>();
                __syncwarp();
                const int sn = (s + STAGES - 1) % STAGES;
                int t = take();
                if (t >= 0) issue(wbase + sn * SLOT, t);
                tl[sn] = t;
                cp_async_commit();
                consume(wbase + s * SLOT, tl[s]);
            }
        }
        cp_async_wait<0>();
#pragma unroll
        for (int sh = 4; sh <= 16; sh <<= 1) {
            l0 += __shfl_xor_sync(0xffffffffu, l0, sh);
            l1 += __shfl_xor_sync(0xffffffffu, l1, sh);
        }
        __syncthreads();                               // all rings drained; reuse the shared memory
        float* mo = reinterpret_cast<float*>(smem);   // [NW][8][128]
        float* ml = mo + NW * 8 * HEAD_DIM;           // [NW][8]
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            float* w0 = mo + ((warp * 8 + 2 * tig) * HEAD_DIM);
            float* w1 = w0 + HEAD_DIM;
            w0[16 * t + gid] = o[t][0];
            w1[16 * t + gid] = o[t][1];
            w0[16 * t + 8 + gid] = o[t][2];
            w1[16 * t + 8 + gid] = o[t][3];
        }
        if (gid == 0) { ml[warp * 8 + 2 * tig] = l0; ml[warp * 8 + 2 * tig + 1] = l1; }
        __syncthreads();
        for (int e = threadIdx.x; e < ncols * (HEAD_DIM / 4); e += NW * 32) {
            const int col = e >> 5, c = (e & 31) * 4;
            float4 O = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int w = 0; w < NW; ++w) {
                const float4 t = *reinterpret_cast<const float4*>(mo + (w * 8 + col) * HEAD_DIM + c);
                O.x += t.x; O.y += t.y; O.z += t.z; O.w += t.w;
            }
            if (O.x != 0.f || O.y != 0.f || O.z != 0.f || O.w != 0.f)
                asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};\n" ::"l"(p.out + (row0 + col) * HEAD_DIM + c),
                             "f"(O.x), "f"(O.y), "f"(O.z), "f"(O.w) : "memory");
        }
        if (threadIdx.x < ncols) {
            float L = 0.f;
#pragma unroll
            for (int w = 0; w < NW; ++w) L += ml[w * 8 + threadIdx.x];
            if (L != 0.f) atomicAdd(p.split_sum + row0 + threadIdx.x, L);
        }
        // ---- the last of the CTAs whose ranges meet this item divides the rows by the sums and cleans up -----
        const long long item_lo = fw.seq_start + (long long)g * fw.tiles_b;
        const int first_cta = (int)(item_lo / fw.per_cta);
        const int nsplits = (int)((item_lo + fw.tiles_b - 1) / fw.per_cta) - first_cta + 1;
        __syncthreads();
        int* ctr = p.counters + ((long long)b * p.Hkv + g) * p.ctr_stride;
        if (threadIdx.x == 0) {
            int old;
            asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;\n" : "=r"(old) : "l"(ctr) : "memory");
            s_last = (old == nsplits - 1);
        }
        __syncthreads();
        if (s_last) {
            float* const rows = p.out_final ? p.out_final : p.out;
            for (int e = threadIdx.x; e < ncols * HEAD_DIM; e += NW * 32) {
                const float L = __ldcg(p.split_sum + row0 + (e >> 7));
                const float O = __ldcg(p.out + row0 * HEAD_DIM + e);
                rows[row0 * HEAD_DIM + e] = (L > 0.f) ? O / L : 0.f;
            }
            __syncthreads();
            if (threadIdx.x < ncols) { p.split_sum[row0 + threadIdx.x] = 0.f; p.split_max[row0 + threadIdx.x] = 0u; }
            if (threadIdx.x == 0) *ctr = 0;
        }
        __syncthreads();                               // shared memory is reused by the next segment
        fw.advance(p, t1 - t0);
    }
}

// ---- the same two passes over an 8-bit cache -------------------------------------------------------------------
// A 16-position tile of E4M3 codes is 2 KB: half the bytes for the same per-tile cost. Both passes therefore
// work on units of 32 positions (two tiles, 4 KB per ring slot; with pages, two lookups). Row and fragment
// layouts, the conversion to fp16 in front of the MMAs and the order of the O^T fragments are those of
// consume_tile8; the key scale goes into the logit scale, the value scale into the partial sums.
constexpr int UNIT8_TILES = 2;
constexpr int UNIT8_BYTES = UNIT8_TILES * TILE_BYTES8;       // 4 KB

// ROWC: consecutive positions of a head lie 256 bytes apart (K and V code rows interleaved).
template <int NW, int STAGES, bool ROWC>
__global__ void __launch_bounds__(NW * 32, 1) score_pass8_kernel(const AttnParams p) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    __shared__ float s_max[NW][8];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gid = lane >> 2, tig = lane & 3;
    constexpr int RING_BYTES = NW * STAGES * UNIT8_BYTES;
    uint32_t* hist = reinterpret_cast<uint32_t*>(smem + RING_BYTES);
    const bool hist_on = p.hist != nullptr;

    bool waited = !p.pdl;
    if (p.pdl && p.wait_first) { pdl_wait(); pdl_trigger(); waited = true; }
    else if (p.pdl && p.wait_late && p.trigger_early) pdl_trigger();

    const int n_items = p.Hkv;                               // one sequence
    const int g = blockIdx.x % n_items, part = blockIdx.x / n_items;
    const int item_ctas = ((int)gridDim.x - g + n_items - 1) / n_items;
    const int N = max(min(p.ctx_lens[0], p.max_ctx), 0);
    const int tiles = item_tiles(N);
    const int units = (tiles + UNIT8_TILES - 1) / UNIT8_TILES;
    const int head0 = g * p.G, ncols = p.G;
    const bool col0 = 2 * tig < ncols, col1 = 2 * tig + 1 < ncols;
    float* const score_row0 = p.scores + (long long)(head0 + min(2 * tig, ncols - 1)) * p.score_stride + gid;
    float* const score_row1 = p.scores + (long long)(head0 + min(2 * tig + 1, ncols - 1)) * p.score_stride + gid;
    const int hshift = p.hist_shift;
    uint32_t* const h0 = hist + ((2 * tig) << (32 - hshift));
    uint32_t* const h1 = hist + ((2 * tig + 1) << (32 - hshift));

    const uint32_t wbase = smem_u32(smem + (size_t)warp * STAGES * UNIT8_BYTES);
    // this lane copies the 16-byte piece piece8 of rows row8 + 4 i of a tile (strides count bytes here)
    const int piece8 = lane & 7, row8 = lane >> 3;
    const long long four_rows = 4 * p.stride_pos;
    const long long tile_step = (long long)TILE * p.stride_pos;
    const uint32_t kdst8 = row8 * ROW_BYTES8 + ((piece8 ^ ((row8 & 1) << 2)) << 4);
    const uint8_t* const kbase = reinterpret_cast<const uint8_t*>(p.k) + (long long)g * p.stride_head + (long long)row8 * p.stride_pos + piece8 * 16;
    const uint64_t kv_policy = l2_evict_first_policy();
    const uint64_t keep = l2_evict_last_policy();

    int* pool = p.tile_ctr + (long long)g * p.ctr_stride;
    PoolWalk walk;
    constexpr int GRAB = GRAB_TILES_DENSE;
    walk.template start<GRAB>(pool, units, item_ctas * NW, part * NW + warp, STAGES + 2, lane);

    constexpr int BAD_A = 1 << 30, BAD_B = 1 << 29, UNIT_MASK = BAD_B - 1;
    auto tile_valid = [&](int tile) { return max(0, min(TILE, N - tile * TILE)); };
    // one tile's sixteen code rows into a ring slot half; returns false for a page id outside the pool
    auto load_tile = [&](uint32_t dst, int tile) -> bool {
        const uint8_t* src;
        bool ok = true;
        if (p.paged) {
            const int page = __ldg(p.page_table + tile);
            ok = (unsigned)page < (unsigned)p.num_pages;
            if (!ok && lane == 0) atomicOr(p.status, STATUS_BAD_PAGE);
            src = kbase + (ok ? (long long)page * p.stride_page : 0);
        } else {
            src = kbase + tile * tile_step;
        }
        const int nvalid = ok ? tile_valid(tile) : 0;
        if (nvalid == TILE) {
#pragma unroll
            for (int i = 0; i < 4; ++i)
                cp_async16_full_hint(dst + kdst8 + i * 512, ROWC ? src + i * (8 * HEAD_DIM) : src + i * four_rows, kv_policy);
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const bool rv = row8 + 4 * i < nvalid;
                cp_async16_hint(dst + kdst8 + i * 512, rv ? src + i * four_rows : reinterpret_cast<const uint8_t*>(p.k), rv ? 16 : 0, kv_policy);
            }
        }
        return ok;
    };
    auto issue = [&](uint32_t ks, int& u) {
        const int ta = UNIT8_TILES * u;
        int flags = load_tile(ks, ta) ? 0 : BAD_A;
        if (ta + 1 < tiles && !load_tile(ks + TILE_BYTES8, ta + 1)) flags |= BAD_B;
        u |= flags;
    };

    int tl[STAGES];
#pragma unroll
    for (int s = 0; s < STAGES; ++s) tl[s] = -1;
#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) {
        int t = walk.template next<GRAB>();
        if (t >= 0) {
            if (!waited && !p.wait_late && t == units - 1) { pdl_wait(); pdl_trigger(); waited = true; }
            issue(wbase + s * UNIT8_BYTES, t);
        }
        tl[s] = t;
        cp_async_commit();
    }
    if (!waited && !p.wait_late) { pdl_wait(); pdl_trigger(); waited = true; }
    if (hist_on) {
        for (int i = threadIdx.x; i < HIST_SMEM_WORDS; i += NW * 32) hist[i] = 0;
        __syncthreads();
    }
    uint32_t qf8[2][8];                                 // the query as fp16, see consume_tile8
    {
        const uint4* qp = reinterpret_cast<const uint4*>(p.q + (long long)(head0 + min(gid, ncols - 1)) * HEAD_DIM);
        const bool on = gid < ncols;
#pragma unroll
        for (int sl = 0; sl < 2; ++sl) {
            const int c = tig + 4 * sl;
            const uint4 t0 = __ldg(qp + 2 * c), t1 = __ldg(qp + 2 * c + 1);
            const uint32_t w[8] = {t0.x, t0.y, t0.z, t0.w, t1.x, t1.y, t1.z, t1.w};
#pragma unroll
            for (int i = 0; i < 8; ++i) qf8[sl][i] = on ? bf16x2_to_f16x2(w[i]) : 0u;
        }
    }
    const float scale = p.scale * (p.k_scale ? __ldg(p.k_scale + g) : 1.f);
    float m0 = -INFINITY, m1 = -INFINITY;
    const uint32_t klane = gid * ROW_BYTES8;
    const uint32_t kswz = (gid & 1) << 2;

    auto key_part = [&](uint32_t ks, int pos_base, int nvalid) {
        float s[4] = {0.f, 0.f, 0.f, 0.f}, s2[4] = {0.f, 0.f, 0.f, 0.f};
        const uint32_t krow = ks + klane;
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
                if (i & 1) mma_f16_16816(s2, a0, a1, a2, a3, qf8[sl][2 * i], qf8[sl][2 * i + 1]);
                else mma_f16_16816(s, a0, a1, a2, a3, qf8[sl][2 * i], qf8[sl][2 * i + 1]);
            }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) s[i] += s2[i];
        const float f0 = s[0] * scale, f1 = s[1] * scale, f2 = s[2] * scale, f3 = s[3] * scale;
        if (nvalid == TILE) {
            if (col0) {
                st_keep(score_row0 + pos_base, f0, keep);
                st_keep(score_row0 + pos_base + 8, f2, keep);
                if (hist_on) {
                    atomicAdd(h0 + (score_key_bits(f0) >> hshift), 1u);
                    atomicAdd(h0 + (score_key_bits(f2) >> hshift), 1u);
                }
                m0 = fmaxf(m0, fmaxf(f0, f2));
            }
            if (col1) {
                st_keep(score_row1 + pos_base, f1, keep);
                st_keep(score_row1 + pos_base + 8, f3, keep);
                if (hist_on) {
                    atomicAdd(h1 + (score_key_bits(f1) >> hshift), 1u);
                    atomicAdd(h1 + (score_key_bits(f3) >> hshift), 1u);
                }
                m1 = fmaxf(m1, fmaxf(f1, f3));
            }
        } else {
            const bool v0 = gid < nvalid, v1 = gid + 8 < nvalid;
            if (col0) {
                if (v0) st_keep(score_row0 + pos_base, f0, keep);
                if (v1) st_keep(score_row0 + pos_base + 8, f2, keep);
            }
            if (col1) {
                if (v0) st_keep(score_row1 + pos_base, f1, keep);
                if (v1) st_keep(score_row1 + pos_base + 8, f3, keep);
            }
            if (hist_on) {
                if (col0) {
                    if (v0) atomicAdd(h0 + (score_key_bits(f0) >> hshift), 1u);
                    if (v1) atomicAdd(h0 + (score_key_bits(f2) >> hshift), 1u);
                }
                if (col1) {
                    if (v0) atomicAdd(h1 + (score_key_bits(f1) >> hshift), 1u);
                    if (v1) atomicAdd(h1 + (score_key_bits(f3) >> hshift), 1u);
                }
            }
            if (v0) { m0 = fmaxf(m0, f0); m1 = fmaxf(m1, f1); }
            if (v1) { m0 = fmaxf(m0, f2); m1 = fmaxf(m1, f3); }
        }
    };
    auto consume = [&](uint32_t ks, int uf) {
        const int ta = UNIT8_TILES * (uf & UNIT_MASK);
        key_part(ks, ta * TILE, (uf & BAD_A) ? 0 : tile_valid(ta));
        if (ta + 1 < tiles) key_part(ks + TILE_BYTES8, (ta + 1) * TILE, (uf & BAD_B) ? 0 : tile_valid(ta + 1));
    };

    for (bool live = true; live;) {
#pragma unroll
        for (int s = 0; s < STAGES; ++s) {
            if (tl[s] < 0) { live = false; break; }
            cp_async_wait<STAGES - 2>();
            __syncwarp();
            const int sn = (s + STAGES - 1) % STAGES;
            int t = walk.template next<GRAB>();
            if (t >= 0) issue(wbase + sn * UNIT8_BYTES, t);
            tl[sn] = t;
            cp_async_commit();
            consume(wbase + s * UNIT8_BYTES, tl[s]);
        }
    }
    cp_async_wait<0>();
    __syncwarp();
    if (!waited) {
        pdl_wait();
        if (!p.trigger_early) pdl_trigger();
        waited = true;
    }
    if (hist_on) {
        __syncthreads();
        const int nb = 1 << (32 - p.hist_shift);
        for (int i = threadIdx.x; i < ncols * nb; i += NW * 32) {
            const uint32_t w = hist[i];
            if (w) atomicAdd(p.hist + (long long)(head0 + i / nb) * HIST_BINS + (i % nb), w);
        }
    }
#pragma unroll
    for (int sh = 4; sh <= 16; sh <<= 1) {
        m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, sh));
        m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, sh));
    }
    if (gid == 0) { s_max[warp][2 * tig] = m0; s_max[warp][2 * tig + 1] = m1; }
    __syncthreads();
    if (threadIdx.x < ncols) {
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < NW; ++w) M = fmaxf(M, s_max[w][threadIdx.x]);
        if (M != -INFINITY) atomicMax(p.split_max + head0 + threadIdx.x, score_key_bits(M));
    }
    if (part == 0)
        for (int e = threadIdx.x; e < ncols * HEAD_DIM; e += NW * 32) p.out[(long long)head0 * HEAD_DIM + e] = 0.f;
    if (threadIdx.x == 0) {
        int* ctr = p.counters + (long long)g * p.ctr_stride;
        int old;
        asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;\n" : "=r"(old) : "l"(ctr) : "memory");
        if (old == item_ctas - 1) { *ctr = 0; *pool = 0; __threadfence(); }
    }
}

template <int NW, int STAGES, bool ROWC>
__global__ void __launch_bounds__(NW * 32, 2) value_pass8_kernel(const AttnParams p) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    constexpr int SLOT = UNIT8_BYTES + 1024;                // 32 value rows, then 32 logits of up to 8 heads

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gid = lane >> 2, tig = lane & 3;
    const int n_items = p.Hkv;
    const int g = blockIdx.x % n_items, part = blockIdx.x / n_items;
    const int item_ctas = ((int)gridDim.x - g + n_items - 1) / n_items;
    const int N = max(min(p.ctx_lens[0], p.max_ctx), 0);
    const int tiles = item_tiles(N);
    const int units = (tiles + UNIT8_TILES - 1) / UNIT8_TILES;
    const int head0 = g * p.G, ncols = p.G;

    const uint32_t wbase = smem_u32(smem + (size_t)warp * STAGES * SLOT);
    const int piece8 = lane & 7, row8 = lane >> 3;
    const long long four_rows = 4 * p.stride_pos;
    const long long tile_step = (long long)TILE * p.stride_pos;
    const uint32_t vc8 = piece8 ^ row8;                   // row & 7 == row8 ^ ((i & 1) << 2) for rows row8 + 4 i
    uint32_t vdst8[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) vdst8[i] = row8 * ROW_BYTES8 + i * 512 + ((vc8 ^ (i << 2)) << 4);
    const uint8_t* const vbase = reinterpret_cast<const uint8_t*>(p.v) + (long long)g * p.stride_head + (long long)row8 * p.stride_pos + piece8 * 16;
    const uint64_t kv_policy = l2_evict_first_policy();
    // lane l < 4 * ncols fetches twice 16 bytes (positions 4 (l & 3) .. + 3 of either tile) of head l >> 2's logits
    const bool score_lane = lane < 4 * ncols;
    const float* const score_src = p.scores + (long long)(head0 + min(lane >> 2, ncols - 1)) * p.score_stride + 4 * (lane & 3);
    const uint32_t score_dst = UNIT8_BYTES + (lane >> 2) * 128 + (lane & 3) * 16;

    int* pool = p.tile_ctr + (long long)g * p.ctr_stride;
    PoolWalk walk;
    constexpr int GRAB = GRAB_TILES_DENSE;
    walk.template start<GRAB>(pool, units, item_ctas * NW, part * NW + warp, STAGES + 2, lane);

    constexpr int BAD_A = 1 << 30, BAD_B = 1 << 29, UNIT_MASK = BAD_B - 1;
    auto tile_valid = [&](int tile) { return max(0, min(TILE, N - tile * TILE)); };
    auto load_tile = [&](uint32_t dst, int tile) -> bool {
        const uint8_t* src;
        bool ok = true;
        if (p.paged) {
            const int page = __ldg(p.page_table + tile);
            ok = (unsigned)page < (unsigned)p.num_pages;
            if (!ok && lane == 0) atomicOr(p.status, STATUS_BAD_PAGE);
            src = vbase + (ok ? (long long)page * p.stride_page : 0);
        } else {
            src = vbase + tile * tile_step;
        }
        const int nvalid = ok ? tile_valid(tile) : 0;
        if (nvalid == TILE) {
#pragma unroll
            for (int i = 0; i < 4; ++i)
                cp_async16_full_hint(dst + vdst8[i & 1] + (i >> 1) * 1024, ROWC ? src + i * (8 * HEAD_DIM) : src + i * four_rows, kv_policy);
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const bool rv = row8 + 4 * i < nvalid;
                cp_async16_hint(dst + vdst8[i & 1] + (i >> 1) * 1024, rv ? src + i * four_rows : reinterpret_cast<const uint8_t*>(p.v), rv ? 16 : 0, kv_policy);
            }
        }
        return ok;
    };
    auto issue = [&](uint32_t vs, int& u) {
        const int ta = UNIT8_TILES * u;
        int flags = load_tile(vs, ta) ? 0 : BAD_A;
        if (ta + 1 < tiles && !load_tile(vs + TILE_BYTES8, ta + 1)) flags |= BAD_B;
        // (logits past the end of the sequence are never used: their rows are masked)
        if (score_lane) {
            cp_async16(vs + score_dst, score_src + ta * TILE, 16);
            if (ta + 1 < tiles) cp_async16(vs + score_dst + 64, score_src + ta * TILE + TILE, 16);
        }
        u |= flags;
    };

    float M0 = -INFINITY, M1 = -INFINITY;
    {
        const uint32_t k0 = (2 * tig < ncols) ? __ldcg(p.split_max + head0 + 2 * tig) : 0u;
        const uint32_t k1 = (2 * tig + 1 < ncols) ? __ldcg(p.split_max + head0 + 2 * tig + 1) : 0u;
        if (k0) M0 = __uint_as_float((k0 & 0x80000000u) ? (k0 & 0x7fffffffu) : ~k0) * LOG2E;
        if (k1) M1 = __uint_as_float((k1 & 0x80000000u) ? (k1 & 0x7fffffffu) : ~k1) * LOG2E;
    }
    const bool h0 = 2 * tig < ncols && M0 != -INFINITY, h1 = 2 * tig + 1 < ncols && M1 != -INFINITY;
    float l0 = 0.f, l1 = 0.f;
    float o[8][4];
#pragma unroll
    for (int t = 0; t < 8; ++t) { o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f; }
    // logits of (position gid | gid + 8 of a tile, heads 2tig | 2tig + 1): head h's 32 floats start at 128 * h
    const uint32_t slane = UNIT8_BYTES + (2 * tig) * 128 + gid * 4;
    const int rr = lane & 7, mi = lane >> 3;
    const uint32_t vlane = (rr + ((mi >> 1) << 3)) * ROW_BYTES8;
    const uint32_t vswz = rr;

    auto value_part = [&](uint32_t vs, uint32_t sl, int nvalid) {
        float f0, f1, f2, f3;
        asm volatile("ld.shared.f32 %0, [%1];\n" : "=f"(f0) : "r"(sl));
        asm volatile("ld.shared.f32 %0, [%1];\n" : "=f"(f2) : "r"(sl + 32));
        asm volatile("ld.shared.f32 %0, [%1];\n" : "=f"(f1) : "r"(sl + 128));
        asm volatile("ld.shared.f32 %0, [%1];\n" : "=f"(f3) : "r"(sl + 160));
        const bool v0 = gid < nvalid, v1 = gid + 8 < nvalid;
        const float p0 = (v0 && h0) ? fast_exp2(f0 * LOG2E - M0) : 0.f, p1 = (v0 && h1) ? fast_exp2(f1 * LOG2E - M1) : 0.f;
        const float p2 = (v1 && h0) ? fast_exp2(f2 * LOG2E - M0) : 0.f, p3 = (v1 && h1) ? fast_exp2(f3 * LOG2E - M1) : 0.f;
        l0 += p0 + p2;
        l1 += p1 + p3;
        const uint32_t pb0 = movmatrix_trans(pack_f16(p0, p1));
        const uint32_t pb1 = movmatrix_trans(pack_f16(p2, p3));
        const uint32_t vb = vs + vlane;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            uint32_t m[4];
            ldmatrix_x4_trans(vb + ((uint32_t)((2 * u + (mi & 1)) ^ vswz) << 4), m);
            uint32_t x0, y0, x2, y2, x1, y1, x3, y3;
            e4m3x4_to_f16x2x2(__byte_perm(m[0], 0, 0x3120), x0, y0);
            e4m3x4_to_f16x2x2(__byte_perm(m[2], 0, 0x3120), x2, y2);
            mma_f16_16816(o[2 * u], x0, y0, x2, y2, pb0, pb1);
            e4m3x4_to_f16x2x2(__byte_perm(m[1], 0, 0x3120), x1, y1);
            e4m3x4_to_f16x2x2(__byte_perm(m[3], 0, 0x3120), x3, y3);
            mma_f16_16816(o[2 * u + 1], x1, y1, x3, y3, pb0, pb1);
        }
    };
    auto consume = [&](uint32_t vs, int uf) {
        const int ta = UNIT8_TILES * (uf & UNIT_MASK);
        value_part(vs, vs + slane, (uf & BAD_A) ? 0 : tile_valid(ta));
        if (ta + 1 < tiles) value_part(vs + TILE_BYTES8, vs + slane + 64, (uf & BAD_B) ? 0 : tile_valid(ta + 1));
    };

    int tl[STAGES];
#pragma unroll
    for (int s = 0; s < STAGES; ++s) tl[s] = -1;
#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) {
        int t = walk.template next<GRAB>();
        if (t >= 0) issue(wbase + s * SLOT, t);
        tl[s] = t;
        cp_async_commit();
    }
    for (bool live = true; live;) {
#pragma unroll
        for (int s = 0; s < STAGES; ++s) {
            if (tl[s] < 0) { live = false; break; }
            cp_async_wait<STAGES - 2>();
            __syncwarp();
            const int sn = (s + STAGES - 1) % STAGES;
            int t = walk.template next<GRAB>();
            if (t >= 0) issue(wbase + sn * SLOT, t);
            tl[sn] = t;
            cp_async_commit();
            consume(wbase + s * SLOT, tl[s]);
        }
    }
    cp_async_wait<0>();
#pragma unroll
    for (int sh = 4; sh <= 16; sh <<= 1) {
        l0 += __shfl_xor_sync(0xffffffffu, l0, sh);
        l1 += __shfl_xor_sync(0xffffffffu, l1, sh);
    }
    __syncthreads();                                   // all rings drained; reuse the shared memory
    const float vscale = p.v_scale ? __ldg(p.v_scale + g) : 1.f;
    float* mo = reinterpret_cast<float*>(smem);       // [NW][8][128]
    float* ml = mo + NW * 8 * HEAD_DIM;               // [NW][8]
#pragma unroll
    for (int t = 0; t < 8; ++t) {                     // rows of the O^T fragments are d = 16t + 2gid and + 1 here
        float* w0 = mo + ((warp * 8 + 2 * tig) * HEAD_DIM);
        float* w1 = w0 + HEAD_DIM;
        w0[16 * t + 2 * gid] = o[t][0] * vscale;
        w1[16 * t + 2 * gid] = o[t][1] * vscale;
        w0[16 * t + 2 * gid + 1] = o[t][2] * vscale;
        w1[16 * t + 2 * gid + 1] = o[t][3] * vscale;
    }
    if (gid == 0) { ml[warp * 8 + 2 * tig] = l0; ml[warp * 8 + 2 * tig + 1] = l1; }
    __syncthreads();
    for (int e = threadIdx.x; e < ncols * (HEAD_DIM / 4); e += NW * 32) {
        const int col = e >> 5, c = (e & 31) * 4;
        float4 O = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int w = 0; w < NW; ++w) {
            const float4 t = *reinterpret_cast<const float4*>(mo + (w * 8 + col) * HEAD_DIM + c);
            O.x += t.x; O.y += t.y; O.z += t.z; O.w += t.w;
        }
        if (O.x != 0.f || O.y != 0.f || O.z != 0.f || O.w != 0.f)
            asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};\n" ::"l"(p.out + (long long)(head0 + col) * HEAD_DIM + c),
                         "f"(O.x), "f"(O.y), "f"(O.z), "f"(O.w) : "memory");
    }
    if (threadIdx.x < ncols) {
        float L = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) L += ml[w * 8 + threadIdx.x];
        if (L != 0.f) atomicAdd(p.split_sum + head0 + threadIdx.x, L);
    }
    __shared__ int s_last;
    __syncthreads();
    int* ctr = p.counters + (long long)g * p.ctr_stride;
    if (threadIdx.x == 0) {
        int old;
        asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;\n" : "=r"(old) : "l"(ctr) : "memory");
        s_last = (old == item_ctas - 1);
    }
    __syncthreads();
    if (s_last) {
        float* const rows = p.out_final ? p.out_final : p.out;
        for (int e = threadIdx.x; e < ncols * HEAD_DIM; e += NW * 32) {
            const float L = __ldcg(p.split_sum + head0 + (e >> 7));
            const float O = __ldcg(p.out + (long long)head0 * HEAD_DIM + e);
            rows[(long long)head0 * HEAD_DIM + e] = (L > 0.f) ? O / L : 0.f;
        }
        __syncthreads();
        if (threadIdx.x < ncols) { p.split_sum[head0 + threadIdx.x] = 0.f; p.split_max[head0 + threadIdx.x] = 0u; }
        if (threadIdx.x == 0) { *ctr = 0; *pool = 0; }
    }
}

}  // namespace tidal
