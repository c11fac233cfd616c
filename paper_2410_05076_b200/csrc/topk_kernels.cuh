// argTopK of Algorithm 1: for every (sequence, index head) pick the
// k' = min(k, N) positions with the largest score, equal scores resolved
// toward the lower position, and write them in ascending position order.
//
// Scores become order-preserving 32-bit keys. The exact k'-th largest key is
// found by a most-significant-digit radix select (11 + 11 + 10 bits, or 10 + 11 + 11):
//   1. The histogram of the first digit comes from the selection layer's attention
//      kernel (fused, per query head) or from topk_hist_kernel (summed scores of a
//      head group).
//   2. topk_select_kernel, all SMs: every CTA derives the threshold bin from that
//      histogram; positions in higher bins are winners outright and go straight
//      into a position bitmap (each CTA owns whole words of it), positions in the
//      threshold bin itself — one bin's population — are appended to a
//      candidate list. The last CTA of an index head to finish resolves the
//      remaining 21 bits on the candidate list alone (in shared memory), adds the
//      candidates above the final threshold and as many equal to it as are still
//      needed (lowest positions first) to the bitmap, and enumerates the bitmap in
//      order. The result is the unique set that a full sort by (score desc,
//      position asc) gives.
// No CTA ever waits for another one; the per-head histogram, cursor and
// arrival counter are cleared by the CTA that used them last.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace tidal {

constexpr int TK_THREADS = 512;
constexpr int TK_BINS = 2048;          // first digit: up to 11 top bits of the key
constexpr int TK_VEC = 4;              // float4 loads per thread per slice
constexpr int TK_SLICE = TK_THREADS * TK_VEC * 4;   // positions per CTA (8192)
constexpr int TK_KEYS = TK_VEC * 4;    // keys per thread per slice
constexpr int TK_BATCHES = 2;          // slices a CTA of the select kernel walks through, one after the other
constexpr int TK_SPAN = TK_BATCHES * TK_SLICE;      // positions per CTA of the select kernel

struct TopkParams {
    const float* scores;       // [B, Hq, score_stride]
    long long score_stride;
    const int* ctx_lens;
    int max_ctx;
    int Hq, Hi;                // index head hi ranks the sum over its Hq/Hi member heads
    int k;
    int* idx;                  // [B, Hi, k]
    int* idx_count;            // [B] or null
    unsigned* hist;            // [items, TK_BINS], zero between calls
    int* cursor;               // [items][ctr_stride], zero between calls
    int* done;                 // [items][ctr_stride], zero between calls
    int ctr_stride;            // ints between consecutive items' counters (one 128-byte line each)
    uint2* cand;               // [items, cand_stride] (key, position) of the threshold bin
    long long cand_stride;
    unsigned* bitmap;          // [items, bitmap_stride] winners above the threshold bin, one bit per position
    long long bitmap_stride;   // words per item (covers max_ctx rounded up to a whole slice)
    int cand_smem;             // candidates the last CTA can hold in shared memory
    int solo_cand;             // > 0: rows of at most TK_SPAN positions are resolved by their single CTA entirely in
                               // shared memory, which then holds this many candidates behind the staged scores
    int vec_ok;                // score rows are 16-byte aligned: float4 loads allowed
    int shift;                 // first digit = key >> shift (21 or 22); the rest is split 11 + (shift-11) bits
    int pdl;                   // launched with programmatic stream serialization: wait for the producer of the scores
    unsigned* thr_max;         // topk_compact_kernel: [items][ctr_stride] largest provisional threshold key, zero between calls
    int list_smem;             // topk_compact_kernel: candidates its shared memory holds
};

// Larger float <=> larger key; -0 and +0 map to the same key.
// A score that is not a number gets key 0, below every number (the float comparisons used elsewhere
// in the selection are false for it as well, so it is never ranked above anything).
__device__ __forceinline__ uint32_t score_key(float s) {
    uint32_t u = __float_as_uint(s);
    if (u == 0x80000000u) u = 0u;
    if ((u & 0x7fffffffu) > 0x7f800000u) return 0u;
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Keys of (key, position) pairs or of a row of scores, behind one interface, so that the exact
// selection below can run on a compacted candidate list or, when that list turns out to be
// incomplete, on all scores of the row.
struct PairSource {
    const uint2* c;
    int n;
    __device__ __forceinline__ uint2 get(int i) const { return c[i]; }
};
struct ScoreSource {
    const float* s;
    int n;
    __device__ __forceinline__ uint2 get(int i) const { return make_uint2(score_key(__ldcg(s + i)), (unsigned)i); }
};

// The value whose key is `key` (inverse of score_key; -0 never occurs as a key).
__device__ __forceinline__ float key_score(uint32_t key) {
    return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

// Keys of this thread's positions of the slice starting at s0: TK_VEC groups of four
// consecutive positions, group j at s0 + 4*(j*TK_THREADS + tid). All loads are issued
// before any is used. Positions at or beyond n get key 0 and valid bit 0.
__device__ __forceinline__ unsigned load_slice_keys(const TopkParams& p, const float* srow, int members,
                                                    int s0, int n, uint32_t (&key)[TK_KEYS]) {
    float v[TK_KEYS];
#pragma unroll
    for (int j = 0; j < TK_VEC; ++j) {
        const int pos = s0 + 4 * (j * TK_THREADS + (int)threadIdx.x);
        if (p.vec_ok && pos + 3 < n) {
            float4 t = __ldcg(reinterpret_cast<const float4*>(srow + pos));
#pragma unroll 4
            for (int m = 1; m < members; ++m) {
                const float4 u = __ldcg(reinterpret_cast<const float4*>(srow + m * p.score_stride + pos));
                t.x += u.x; t.y += u.y; t.z += u.z; t.w += u.w;
            }
            v[4 * j] = t.x; v[4 * j + 1] = t.y; v[4 * j + 2] = t.z; v[4 * j + 3] = t.w;
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float t = 0.f;
                if (pos + e < n) {
                    t = __ldcg(srow + pos + e);
#pragma unroll 1
                    for (int m = 1; m < members; ++m) t += __ldcg(srow + m * p.score_stride + pos + e);
                }
                v[4 * j + e] = t;
            }
        }
    }
    unsigned valid = 0;
#pragma unroll
    for (int j = 0; j < TK_VEC; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int pos = s0 + 4 * (j * TK_THREADS + (int)threadIdx.x) + e;
            const bool ok = pos < n;
            key[4 * j + e] = ok ? score_key(v[4 * j + e]) : 0u;
            valid |= (ok ? 1u : 0u) << (4 * j + e);
        }
    return valid;
}

// Inclusive scan of one value per thread over a TK_THREADS block.
// (Not inlined, like pick_digit below: these kernels run most of their code exactly once, so their speed
// is set by instruction fetch and every repeated copy of a helper costs more misses than a call.)
template <typename T>
__device__ __noinline__ T block_scan_incl(T v, T* warp_sums, T& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const T t = __shfl_up_sync(0xffffffffu, v, d);
        if (lane >= d) v += t;
    }
    __syncthreads();                       // warp_sums may still be read from a previous call
    if (lane == 31) warp_sums[warp] = v;
    __syncthreads();
    T before = 0, all = 0;
#pragma unroll
    for (int w = 0; w < TK_THREADS / 32; ++w) {
        const T s = warp_sums[w];
        if (w < warp) before += s;
        all += s;
    }
    total = all;
    return v + before;
}

// Given a histogram of `nbins` digits (shared memory), find the digit holding
// the `need`-th largest remaining key; on return `need` is reduced by the number
// of keys in higher digits. Identical result in every thread.
__device__ __noinline__ int pick_digit(const unsigned* hist, int nbins, int* warp_sums, int* bcast,
                                       int& need) {
    const int per = (nbins + TK_THREADS - 1) / TK_THREADS;
    const int hi_bin = nbins - 1 - (int)threadIdx.x * per;      // this thread's highest bin
    int mine = 0;
    for (int i = 0; i < per; ++i) {
        const int bin = hi_bin - i;
        if (bin >= 0) mine += (int)hist[bin];
    }
    int total;
    const int incl = block_scan_incl<int>(mine, warp_sums, total);
    const int excl = incl - mine;
    if (excl < need && need <= incl) {
        int above = excl;
        for (int i = 0; i < per; ++i) {
            const int bin = hi_bin - i;
            const int c = (bin >= 0) ? (int)hist[bin] : 0;
            if (above + c >= need) { bcast[0] = bin; bcast[1] = need - above; break; }
            above += c;
        }
    }
    __syncthreads();
    const int digit = bcast[0];
    need = bcast[1];
    __syncthreads();
    return digit;
}

// Histogram of the first digit for rankings that sum several heads' scores (the attention
// kernel cannot build those: the member heads live in different CTAs).
__global__ void __launch_bounds__(TK_THREADS) topk_hist_kernel(const TopkParams p) {
    __shared__ unsigned sh[TK_BINS];
    const int item = blockIdx.y, b = item / p.Hi, hi = item % p.Hi, tid = threadIdx.x;
    if (p.pdl) {
        asm volatile("griddepcontrol.wait;\n" ::: "memory");
        asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
    }
    const int N = max(0, min(p.ctx_lens[b], p.max_ctx));
    if (min(p.k, N) == N) return;                      // everything is kept: no ranking needed
    const int s0 = blockIdx.x * TK_SLICE;
    if (s0 >= N) return;
    for (int i = tid; i < TK_BINS; i += TK_THREADS) sh[i] = 0;
    const int members = p.Hq / p.Hi;
    const float* srow = p.scores + ((long long)b * p.Hq + (long long)hi * members) * p.score_stride;
    uint32_t key[TK_KEYS];
    const unsigned valid = load_slice_keys(p, srow, members, s0, N, key);
    __syncthreads();
#pragma unroll
    for (int e = 0; e < TK_KEYS; ++e)
        if ((valid >> e) & 1u) atomicAdd(&sh[key[e] >> p.shift], 1u);
    __syncthreads();
    unsigned* gh = p.hist + (long long)item * TK_BINS;
    for (int i = tid; i < TK_BINS; i += TK_THREADS) {
        const unsigned c = sh[i];
        if (c) atomicAdd(&gh[i], c);
    }
}

__global__ void __launch_bounds__(TK_THREADS) topk_select_kernel(const TopkParams p) {
    extern __shared__ __align__(16) uint8_t tk_smem[];
    __shared__ __align__(16) unsigned sh_hist[TK_BINS];
    static_assert(TK_BINS == 4 * TK_THREADS, "one uint4 of the histogram per thread");
    __shared__ int warp_sums[TK_THREADS / 32];
    __shared__ unsigned long long warp_sums64[TK_THREADS / 32];
    __shared__ int bcast[2];
    __shared__ int s_last;

    const int item = blockIdx.y, b = item / p.Hi, hi = item % p.Hi, tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5;
    if (p.pdl) {
        // resident early, but nothing is read before the kernel that produced scores and histogram is done
        asm volatile("griddepcontrol.wait;\n" ::: "memory");
        asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
    }
    const int N = max(0, min(p.ctx_lens[b], p.max_ctx));
    const int kk = min(p.k, N);
    int* out = p.idx + (long long)item * p.k;
    const int s0 = blockIdx.x * TK_SPAN, s1 = min(N, s0 + TK_SPAN);
    if (blockIdx.x == 0 && hi == 0 && tid == 0 && p.idx_count) p.idx_count[b] = kk;
    unsigned* gh = p.hist + (long long)item * TK_BINS;

    if (kk == N) {                                     // identity list, then padding
        for (int i = s0 + tid; i < s1; i += TK_THREADS) out[i] = i;
        if (blockIdx.x == 0) {
            for (int i = N + tid; i < p.k; i += TK_THREADS) out[i] = -1;
            // a selection layer's attention kernel may have filled the histogram regardless of k
            for (int i = tid; i < TK_BINS; i += TK_THREADS) gh[i] = 0;
        }
        return;
    }
    if (s0 >= s1) return;
    const int nparts = (N + TK_SPAN - 1) / TK_SPAN;    // CTAs that reach the arrival counter

    // ---- stage this CTA's scores in shared memory, every load in flight at once -------------------------
    // (the staging area is the head of the dynamic shared memory, which only the last CTA of an
    // index head uses again later, for other things)
    const int members = p.Hq / p.Hi;
    const float* srow = p.scores + ((long long)b * p.Hq + (long long)hi * members) * p.score_stride;
    float* raw = reinterpret_cast<float*>(tk_smem);                // [TK_SPAN]
    if (p.vec_ok && members == 1) {
        // The attention kernel asked L2 to keep the scores (evict-last) until they were read back: this is
        // that read, and it hands the lines back (evict-first), so that they do not crowd the caller's
        // next kernels out of the cache.
        uint64_t done_with;
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;\n" : "=l"(done_with));
#pragma unroll
        for (int j = 0; j < TK_BATCHES * TK_VEC; ++j) {
            const int off = 4 * (j * TK_THREADS + tid);
            const int pos = s0 + off;
            const int nbytes = max(0, min(4, N - pos)) * 4;        // zero-fill past the end of the cache
            const uint32_t dst = static_cast<uint32_t>(__cvta_generic_to_shared(raw + off));
            asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2, %3;\n"
                         ::"r"(dst), "l"(nbytes ? srow + pos : srow), "r"(nbytes), "l"(done_with) : "memory");
        }
        asm volatile("cp.async.commit_group;\n" ::: "memory");
    } else if (p.vec_ok) {
        // summed member heads: the same groups of four positions, the members' rows added up
#pragma unroll 2
        for (int j = 0; j < TK_BATCHES * TK_VEC; ++j) {
            const int off = 4 * (j * TK_THREADS + tid);
            const int pos = s0 + off;
            float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
            if (pos < N) {                                         // rows are padded to a multiple of four
                t = __ldcg(reinterpret_cast<const float4*>(srow + pos));
#pragma unroll 4
                for (int m = 1; m < members; ++m) {
                    const float4 u = __ldcg(reinterpret_cast<const float4*>(srow + m * p.score_stride + pos));
                    t.x += u.x; t.y += u.y; t.z += u.z; t.w += u.w;
                }
            }
            *reinterpret_cast<float4*>(raw + off) = t;
        }
    } else {
        // unaligned score rows (a caller's buffer): one position at a time
#pragma unroll 1
        for (int i = tid; i < TK_SPAN; i += TK_THREADS) {
            const int pos = s0 + i;
            float t = 0.f;
            if (pos < N) {
#pragma unroll 1
                for (int m = 0; m < members; ++m) t += __ldcg(srow + m * p.score_stride + pos);
            }
            raw[i] = t;
        }
    }
    {
        const uint4 h4 = __ldcg(reinterpret_cast<const uint4*>(gh) + tid);
        reinterpret_cast<uint4*>(sh_hist)[tid] = h4;
    }
    __syncthreads();
    int need = kk;
    const int b1 = pick_digit(sh_hist, TK_BINS, warp_sums, bcast, need);
    // `need` of the keys in bin b1 are still to be taken; every key in a higher bin is a winner.
    asm volatile("cp.async.wait_group 0;\n" ::: "memory");
    __syncthreads();

    // ---- winners above the threshold bin: straight into the position bitmap ------------------------
    // Group j of a warp covers 128 consecutive positions, lane l the four at 4l: the 8 lanes of a
    // word OR their nibbles together and one of them stores the word (zeros included, so the
    // bitmap needs no clearing). Keys of the threshold bin itself are only marked here.
    // A row that fits one CTA never leaves shared memory: bitmap and candidates are built behind the
    // staged scores, and the arrival protocol is skipped.
    const bool solo = p.solo_cand > 0 && nparts == 1;
    unsigned* solo_bm = reinterpret_cast<unsigned*>(tk_smem + (size_t)TK_SPAN * sizeof(float));
    const int solo_words = TK_SPAN / 32;
    uint2* solo_cand = reinterpret_cast<uint2*>(solo_bm + 2 * solo_words);
    unsigned* bm = solo ? solo_bm : p.bitmap + (long long)item * p.bitmap_stride;
    const int bm_base = solo ? 0 : (s0 >> 5);
    unsigned eq_mask = 0;                                          // bit 4j+e: group j, element e
    // the values whose keys open bin b1 and bin b1 + 1 (nothing lies above the last bin: NaN compares false)
    const float f_lo = key_score((uint32_t)b1 << p.shift);
    const float f_hi = (b1 + 1 >= (1 << (32 - p.shift))) ? __uint_as_float(0x7fc00000u) : key_score((uint32_t)(b1 + 1) << p.shift);
#pragma unroll
    for (int j = 0; j < TK_BATCHES * TK_VEC; ++j) {
        const int off = 4 * (j * TK_THREADS + tid);
        const float4 f = *reinterpret_cast<const float4*>(raw + off);
        // bin > b1 <=> f >= f_hi and bin >= b1 <=> f >= f_lo: the key is monotone in the value, so two
        // float comparisons per score replace the key transform
        const unsigned ok = (1u << max(0, min(4, N - (s0 + off)))) - 1u;
        const unsigned hi4 = (f.x >= f_hi ? 1u : 0u) | (f.y >= f_hi ? 2u : 0u) | (f.z >= f_hi ? 4u : 0u) | (f.w >= f_hi ? 8u : 0u);
        const unsigned lo4 = (f.x >= f_lo ? 1u : 0u) | (f.y >= f_lo ? 2u : 0u) | (f.z >= f_lo ? 4u : 0u) | (f.w >= f_lo ? 8u : 0u);
        const unsigned nib = hi4 & ok;
        eq_mask |= (lo4 & ~hi4 & ok) << (4 * j);
        unsigned word = nib << (4 * (lane & 7));
        word |= __shfl_xor_sync(0xffffffffu, word, 1);
        word |= __shfl_xor_sync(0xffffffffu, word, 2);
        word |= __shfl_xor_sync(0xffffffffu, word, 4);
        if ((lane & 7) == 0) bm[bm_base + j * (TK_THREADS / 8) + warp * 4 + (lane >> 3)] = word;
    }

    // ---- the threshold bin's own keys: append to the candidate list, one cursor bump per CTA -------
    int cta_total;
    const int mine = __popc(eq_mask);
    int slot = block_scan_incl<int>(mine, warp_sums, cta_total) - mine;
    const bool solo_cands = solo && cta_total <= p.solo_cand;      // else the list goes through global memory
    if (tid == 0) bcast[0] = (cta_total && !solo) ? atomicAdd(&p.cursor[(size_t)item * p.ctr_stride], cta_total) : 0;
    __syncthreads();
    slot += bcast[0];
    uint2* cand = solo_cands ? solo_cand : p.cand + (long long)item * p.cand_stride;
    if (solo_cands) {
        unsigned m = eq_mask;
        while (m) {
            const int e = __ffs(m) - 1;
            m &= m - 1;
            const int off = 4 * ((e >> 2) * TK_THREADS + tid) + (e & 3);
            cand[slot++] = make_uint2(score_key(raw[off]), (unsigned)(s0 + off));
        }
    } else {
        unsigned m = eq_mask;
        while (m) {
            const int e = __ffs(m) - 1;
            m &= m - 1;
            const int off = 4 * ((e >> 2) * TK_THREADS + tid) + (e & 3);
            if (slot < p.cand_stride) cand[slot] = make_uint2(score_key(raw[off]), (unsigned)(s0 + off));
            ++slot;
        }
    }

    // ---- the last CTA of this index head resolves the rest ------------------------------------------
    __syncthreads();
    const int words = (N + 31) >> 5;
    const int per = (words + TK_THREADS - 1) / TK_THREADS;
    const int w0 = min(words, tid * per), w1 = min(words, w0 + per);
    unsigned* cgt;                                                  // [words] winners: higher bins + winning candidates
    unsigned* ceq;                                                  // [words] candidates equal to the threshold key
    const uint2* c;
    int M;
    if (solo) {
        cgt = solo_bm;
        ceq = solo_bm + solo_words;
        M = solo_cands ? cta_total : (int)min((long long)cta_total, p.cand_stride);
        c = cand;                                                   // shared memory, or this CTA's own global list
        for (int i = tid; i < words; i += TK_THREADS) ceq[i] = 0;
        for (int i = tid; i < TK_BINS; i += TK_THREADS) sh_hist[i] = 0;
        __syncthreads();
    } else {
        if (tid == 0) {
            // release: orders the CTA's bitmap and candidate stores (seen by this thread through the barrier)
            // before the arrival; acquire: the last arrival sees every other CTA's
            int old;
            asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;\n" : "=r"(old) : "l"(&p.done[(size_t)item * p.ctr_stride]) : "memory");
            s_last = (old == nparts - 1);
        }
        __syncthreads();
        if (!s_last) return;

        // One round trip for everything the last CTA needs: the candidate count, the winners' bitmap
        // written by all CTAs of this head (pulled into shared memory; candidates that turn out to be
        // winners are ORed into the same words) and, without waiting for the count, the first 2048
        // candidate slots (a usual threshold bin holds about that many; unused slots are in bounds).
        constexpr int BM_REGS = 16, CAND_REGS = 4;             // 16 x 512 words = the longest supported context
        cgt = reinterpret_cast<unsigned*>(tk_smem);
        ceq = cgt + words;
        uint2* scand = reinterpret_cast<uint2*>(ceq + words);      // [cand_smem]; 8*words bytes in: 8-byte aligned
        unsigned bmreg[BM_REGS];
        uint2 creg[CAND_REGS];
#pragma unroll
        for (int j = 0; j < BM_REGS; ++j) {
            const int i = tid + j * TK_THREADS;
            bmreg[j] = (i < words) ? __ldcg(&bm[i]) : 0u;
        }
#pragma unroll
        for (int j = 0; j < CAND_REGS; ++j) {
            const int i = tid + j * TK_THREADS;
            creg[j] = (i < p.cand_stride && i < p.cand_smem) ? __ldcg(&cand[i]) : make_uint2(0u, 0u);
        }
        M = (int)min((long long)__ldcg(&p.cursor[(size_t)item * p.ctr_stride]), p.cand_stride);
        c = cand;
        if (M <= p.cand_smem) {
#pragma unroll
            for (int j = 0; j < CAND_REGS; ++j) {
                const int i = tid + j * TK_THREADS;
                if (i < M) scand[i] = creg[j];
            }
#pragma unroll 4
            for (int i = tid + CAND_REGS * TK_THREADS; i < M; i += TK_THREADS) scand[i] = __ldcg(&cand[i]);
            c = scand;
        }
#pragma unroll
        for (int j = 0; j < BM_REGS; ++j) {
            const int i = tid + j * TK_THREADS;
            if (i < words) { cgt[i] = bmreg[j]; ceq[i] = 0; }
        }
        for (int i = tid; i < TK_BINS; i += TK_THREADS) sh_hist[i] = 0;
        __syncthreads();
    }

    // second digit: the next 11 key bits (every candidate already has first digit b1)
    const int s2 = p.shift - 11;                       // bits left for the third digit (10 or 11)
    for (int i = tid; i < M; i += TK_THREADS) atomicAdd(&sh_hist[(c[i].x >> s2) & 0x7ffu], 1u);
    __syncthreads();
    const int d2 = pick_digit(sh_hist, TK_BINS, warp_sums, bcast, need);
    const uint32_t prefix2 = ((uint32_t)b1 << p.shift) | ((uint32_t)d2 << s2);
    const int in_bin = (int)sh_hist[d2];               // candidates that share both digits with the threshold key
    __syncthreads();                                   // sh_hist is recycled below

    constexpr int SMALL = 64;
    if (in_bin <= SMALL) {
        // A handful of keys are left: rank them directly. Entry i is taken iff fewer than `need` of the
        // others beat it (larger key, or equal key at a lower position).
        uint2* few = reinterpret_cast<uint2*>(sh_hist);            // [SMALL]
        int* nfew = &bcast[0];
        if (tid == 0) *nfew = 0;
        __syncthreads();
        for (int i = tid; i < M; i += TK_THREADS) {
            const uint2 e = c[i];
            if ((e.x >> s2) == (prefix2 >> s2)) few[atomicAdd(nfew, 1)] = e;
            else if ((e.x >> s2) > (prefix2 >> s2)) atomicOr(&cgt[e.y >> 5], 1u << (e.y & 31));
        }
        __syncthreads();
        const int n = *nfew;
        if (tid < n) {
            const uint2 me = few[tid];
            int beaten_by = 0;
            for (int j = 0; j < n; ++j) {
                const uint2 o = few[j];
                beaten_by += (o.x > me.x) || (o.x == me.x && o.y < me.y);
            }
            if (beaten_by < need) atomicOr(&cgt[me.y >> 5], 1u << (me.y & 31));
        }
        need = 0;                                      // nothing is taken through the equal-key bitmap
        __syncthreads();
    } else {
        // third digit: the remaining low bits
        for (int i = tid; i < TK_BINS; i += TK_THREADS) sh_hist[i] = 0;
        __syncthreads();
        for (int i = tid; i < M; i += TK_THREADS) {
            const uint32_t k32 = c[i].x;
            if ((k32 >> s2) == (prefix2 >> s2)) atomicAdd(&sh_hist[k32 & ((1u << s2) - 1u)], 1u);
        }
        __syncthreads();
        const int d3 = pick_digit(sh_hist, 1 << s2, warp_sums, bcast, need);
        const uint32_t thr = prefix2 | (uint32_t)d3;   // the k'-th largest key; `need` keys equal to it are taken
        // candidates above / equal to the threshold, as position bitmaps
        for (int i = tid; i < M; i += TK_THREADS) {
            const uint2 e = c[i];
            if (e.x > thr) atomicOr(&cgt[e.y >> 5], 1u << (e.y & 31));
            else if (e.x == thr) atomicOr(&ceq[e.y >> 5], 1u << (e.y & 31));
        }
        __syncthreads();
    }

    if (need == 0 && (per & 3) == 0 && words == per * TK_THREADS) {
        // No equal-key positions are pending (the usual case) and the words divide evenly: only the
        // winners' bitmap is enumerated, fetched as 16-byte pieces (consecutive threads are `per` words
        // apart, which scalar reads turn into an 8-way bank conflict). The loops stay rolled: this
        // code runs once, so every instruction costs a fetch.
        const uint4* src = reinterpret_cast<const uint4*>(cgt + w0);
        int mine = 0;
#pragma unroll 1
        for (int j = 0; j < per / 4; ++j) {
            const uint4 t = src[j];
            mine += __popc(t.x) + __popc(t.y) + __popc(t.z) + __popc(t.w);
        }
        int tot;
        int at = block_scan_incl<int>(mine, warp_sums, tot) - mine;
#pragma unroll 1
        for (int j = 0; j < per; ++j) {
            unsigned bits = cgt[w0 + j];
            while (bits) {
                const int pbit = __ffs(bits) - 1;
                if (at < p.k) out[at] = ((w0 + j) << 5) + pbit;
                ++at;
                bits &= bits - 1;
            }
        }
        // (scores that are not numbers are counted but never taken: the list may then come out short)
        for (int i = min(tot, kk) + tid; i < kk; i += TK_THREADS) out[i] = -1;
    } else {
    // ordered enumeration: (winner count, equal count) scanned together in one 64-bit value
    unsigned long long cnt = 0;
    for (int w = w0; w < w1; ++w)
        cnt += ((unsigned long long)__popc(cgt[w]) << 32) | (unsigned long long)__popc(ceq[w]);
    unsigned long long tot;
    const unsigned long long excl = block_scan_incl<unsigned long long>(cnt, warp_sums64, tot) - cnt;
    int eq_seen = (int)(excl & 0xffffffffu);
    int at = (int)(excl >> 32) + min(eq_seen, need);
    for (int w = w0; w < w1; ++w) {
        unsigned e = ceq[w];
        const int ne = __popc(e);
        const int keep = min(max(need - eq_seen, 0), ne);   // lowest `keep` equal-key positions of this word
        eq_seen += ne;
        while (__popc(e) > keep) e &= ~(0x80000000u >> __clz(e));
        unsigned bits = cgt[w] | e;
        while (bits) {
            const int pbit = __ffs(bits) - 1;
            if (at < p.k) out[at] = (w << 5) + pbit;
            ++at;
            bits &= bits - 1;
        }
    }
    const int taken = (int)(tot >> 32) + min((int)(tot & 0xffffffffu), need);
    for (int i = min(taken, kk) + tid; i < kk; i += TK_THREADS) out[i] = -1;
    }
    for (int i = kk + tid; i < p.k; i += TK_THREADS) out[i] = -1;

    // leave the shared state clean for the next call
    for (int i = tid; i < TK_BINS; i += TK_THREADS) gh[i] = 0;
    if (tid == 0 && !solo) { p.cursor[(size_t)item * p.ctr_stride] = 0; p.done[(size_t)item * p.ctr_stride] = 0; }
}

// The k'-th largest key of a source by three digit passes (most significant first); on return `need`
// is how many keys equal to it are to be taken. Every thread gets the same result.
template <typename Src>
__device__ __noinline__ uint32_t kth_largest_key(const Src src, int shift, int& need, unsigned* sh_hist,
                                                 int* warp_sums, int* bcast) {
    const int tid = threadIdx.x;
    const int s2 = shift - 11;
    for (int i = tid; i < TK_BINS; i += TK_THREADS) sh_hist[i] = 0;
    __syncthreads();
    for (int i = tid; i < src.n; i += TK_THREADS) atomicAdd(&sh_hist[src.get(i).x >> shift], 1u);
    __syncthreads();
    const int b1 = pick_digit(sh_hist, TK_BINS, warp_sums, bcast, need);
    for (int i = tid; i < TK_BINS; i += TK_THREADS) sh_hist[i] = 0;
    __syncthreads();
    for (int i = tid; i < src.n; i += TK_THREADS) {
        const uint32_t k32 = src.get(i).x;
        if ((int)(k32 >> shift) == b1) atomicAdd(&sh_hist[(k32 >> s2) & 0x7ffu], 1u);
    }
    __syncthreads();
    const int d2 = pick_digit(sh_hist, TK_BINS, warp_sums, bcast, need);
    const uint32_t prefix2 = ((uint32_t)b1 << shift) | ((uint32_t)d2 << s2);
    for (int i = tid; i < TK_BINS; i += TK_THREADS) sh_hist[i] = 0;
    __syncthreads();
    for (int i = tid; i < src.n; i += TK_THREADS) {
        const uint32_t k32 = src.get(i).x;
        if ((k32 >> s2) == (prefix2 >> s2)) atomicAdd(&sh_hist[k32 & ((1u << s2) - 1u)], 1u);
    }
    __syncthreads();
    const int d3 = pick_digit(sh_hist, 1 << s2, warp_sums, bcast, need);
    return prefix2 | (uint32_t)d3;
}

// Positions of a source whose key exceeds `thr` into the bitmap cgt, those equal to it into ceq.
template <typename Src>
__device__ __noinline__ void mark_winners(const Src src, uint32_t thr, unsigned* cgt, unsigned* ceq) {
    for (int i = threadIdx.x; i < src.n; i += TK_THREADS) {
        const uint2 e = src.get(i);
        if (e.x > thr) atomicOr(&cgt[e.y >> 5], 1u << (e.y & 31));
        else if (e.x == thr) atomicOr(&ceq[e.y >> 5], 1u << (e.y & 31));
    }
}

// argTopK on the candidate lists that the selection layer's attention kernel compacted: one CTA per
// (sequence, head). The list holds every score at or above a provisional threshold chosen by each CTA
// of that kernel; thr_max is the largest threshold any of them used, so the list is complete for all
// keys >= thr_max. If the k'-th largest key of the list is at least thr_max it is the k'-th largest of
// the row and the list decides everything; otherwise (a threshold was too optimistic, or the list
// outgrew its buffer) the same exact selection runs on the row's scores instead: slower, same result.
__global__ void __launch_bounds__(TK_THREADS) topk_compact_kernel(const TopkParams p) {
    extern __shared__ __align__(16) uint8_t tk_smem[];
    __shared__ __align__(16) unsigned sh_hist[TK_BINS];
    __shared__ int warp_sums[TK_THREADS / 32];
    __shared__ unsigned long long warp_sums64[TK_THREADS / 32];
    __shared__ int bcast[2];

    const int item = blockIdx.x, b = item / p.Hi, tid = threadIdx.x;
    if (p.pdl) {
        asm volatile("griddepcontrol.wait;\n" ::: "memory");
        asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
    }
    const int N = max(0, min(p.ctx_lens[b], p.max_ctx));
    const int kk = min(p.k, N);
    int* out = p.idx + (long long)item * p.k;
    if (item % p.Hi == 0 && tid == 0 && p.idx_count) p.idx_count[b] = kk;
    int* cursor = p.cursor + (size_t)item * p.ctr_stride;
    unsigned* tmax = p.thr_max + (size_t)item * p.ctr_stride;
    const int M_raw = __ldcg(cursor);
    const uint32_t t_max = __ldcg(tmax);
    __syncthreads();                                   // everybody has read them: they can be cleared for the next call
    if (tid == 0) { *cursor = 0; *tmax = 0; }
    if (kk == N) {                                     // everything is kept
        for (int i = tid; i < N; i += TK_THREADS) out[i] = i;
        for (int i = N + tid; i < p.k; i += TK_THREADS) out[i] = -1;
        return;
    }
    const int words = (N + 31) >> 5;
    unsigned* cgt = reinterpret_cast<unsigned*>(tk_smem);
    unsigned* ceq = cgt + words;
    uint2* slist = reinterpret_cast<uint2*>(ceq + words);                  // 8 * words bytes in: 8-byte aligned
    for (int i = tid; i < 2 * words; i += TK_THREADS) cgt[i] = 0;

    const float* srow = p.scores + (long long)item * p.score_stride;
    const uint2* glist = p.cand + (long long)item * p.cand_stride;
    bool from_list = M_raw >= kk && M_raw <= p.cand_stride;
    int need = kk;
    if (from_list) {
        // ---- the list: into shared memory if it fits, its smallest and largest key on the way ----------
        PairSource src{glist, M_raw};
        const bool in_smem = M_raw <= p.list_smem;
        uint32_t kmin = 0xffffffffu, kmax = 0u;
        constexpr int LD = 8;                          // loads in flight per thread
        for (int i0 = 0; i0 < M_raw; i0 += LD * TK_THREADS) {
            uint2 r[LD];
#pragma unroll
            for (int u = 0; u < LD; ++u) {
                const int i = i0 + u * TK_THREADS + tid;
                r[u] = (i < M_raw) ? __ldcg(glist + i) : make_uint2(0u, 0u);
            }
#pragma unroll
            for (int u = 0; u < LD; ++u) {
                const int i = i0 + u * TK_THREADS + tid;
                if (i < M_raw) {
                    if (in_smem) slist[i] = r[u];
                    kmin = min(kmin, r[u].x);
                    kmax = max(kmax, r[u].x);
                }
            }
        }
        if (in_smem) src.c = slist;
#pragma unroll
        for (int sh = 16; sh >= 1; sh >>= 1) {
            kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, sh));
            kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, sh));
        }
        unsigned* red = reinterpret_cast<unsigned*>(warp_sums64);     // [32] words
        if ((tid & 31) == 0) { red[tid >> 5] = kmin; red[16 + (tid >> 5)] = kmax; }
        for (int i = tid; i < TK_BINS; i += TK_THREADS) sh_hist[i] = 0;
        __syncthreads();
#pragma unroll
        for (int w = 0; w < TK_THREADS / 32; ++w) { kmin = min(kmin, red[w]); kmax = max(kmax, red[16 + w]); }
        // ---- one digit of 11 bits over the list's own key range (the candidates of a head share their
        // top key bits, so the usual most-significant digit would put them all into a few bins) --------
        const uint32_t range = kmax - kmin;
        const int dsh = max(0, 21 - __clz(range | 1u));               // (range >> dsh) < 2048
        for (int i = tid; i < M_raw; i += TK_THREADS) atomicAdd(&sh_hist[(src.get(i).x - kmin) >> dsh], 1u);
        __syncthreads();
        const int b1 = pick_digit(sh_hist, TK_BINS, warp_sums, bcast, need);
        const int in_bin = (int)sh_hist[b1];
        __syncthreads();                               // sh_hist is recycled below
        constexpr int FEW = TK_BINS / 2;               // (key, position) pairs that fit the histogram's memory
        uint32_t thr = 0;
        if (in_bin <= FEW) {
            // everything above the threshold bin wins; the bin's own entries are ranked directly
            uint2* few = reinterpret_cast<uint2*>(sh_hist);
            if (tid == 0) { bcast[0] = 0; bcast[1] = (int)0xffffffffu; }
            __syncthreads();
            for (int i = tid; i < M_raw; i += TK_THREADS) {
                const uint2 e = src.get(i);
                const int d = (int)((e.x - kmin) >> dsh);
                if (d > b1) atomicOr(&cgt[e.y >> 5], 1u << (e.y & 31));
                else if (d == b1) few[atomicAdd(&bcast[0], 1)] = e;
            }
            __syncthreads();
            const int n = bcast[0];
            for (int t = tid; t < n; t += TK_THREADS) {
                const uint2 me = few[t];
                int beaten_by = 0;
                for (int j = 0; j < n; ++j) {
                    const uint2 o = few[j];
                    beaten_by += (o.x > me.x) || (o.x == me.x && o.y < me.y);
                }
                if (beaten_by < need) {
                    atomicOr(&cgt[me.y >> 5], 1u << (me.y & 31));
                    atomicMin(reinterpret_cast<unsigned*>(&bcast[1]), me.x);      // the smallest key taken is the k'-th largest
                }
            }
            __syncthreads();
            thr = (uint32_t)bcast[1];
            need = 0;                                  // equal keys were resolved by the ranking
            __syncthreads();
        } else {
            // many equal or nearly equal keys: the general digit-by-digit selection
            need = kk;
            thr = kth_largest_key(src, p.shift, need, sh_hist, warp_sums, bcast);
            mark_winners(src, thr, cgt, ceq);
        }
        from_list = thr >= t_max;                      // complete down to the k'-th key?
    }
    if (!from_list) {
        ScoreSource src{srow, N};
        __syncthreads();
        for (int i = tid; i < 2 * words; i += TK_THREADS) cgt[i] = 0;
        need = kk;
        __syncthreads();
        const uint32_t thr = kth_largest_key(src, p.shift, need, sh_hist, warp_sums, bcast);
        mark_winners(src, thr, cgt, ceq);
    }
    __syncthreads();

    // ordered enumeration: (winner count, equal count) scanned together in one 64-bit value; of the
    // positions whose key equals the threshold the lowest `need` are taken
    const int per = (words + TK_THREADS - 1) / TK_THREADS;
    const int w0 = min(words, tid * per), w1 = min(words, w0 + per);
    unsigned long long cnt = 0;
    for (int w = w0; w < w1; ++w)
        cnt += ((unsigned long long)__popc(cgt[w]) << 32) | (unsigned long long)__popc(ceq[w]);
    unsigned long long tot;
    const unsigned long long excl = block_scan_incl<unsigned long long>(cnt, warp_sums64, tot) - cnt;
    int eq_seen = (int)(excl & 0xffffffffu);
    int at = (int)(excl >> 32) + min(eq_seen, need);
    for (int w = w0; w < w1; ++w) {
        unsigned e = ceq[w];
        const int ne = __popc(e);
        const int keep = min(max(need - eq_seen, 0), ne);
        eq_seen += ne;
        while (__popc(e) > keep) e &= ~(0x80000000u >> __clz(e));
        unsigned bits = cgt[w] | e;
        while (bits) {
            const int pbit = __ffs(bits) - 1;
            if (at < p.k) out[at] = (w << 5) + pbit;
            ++at;
            bits &= bits - 1;
        }
    }
    // scores that are not numbers rank below everything and may leave the list short: pad, never stale
    const int taken = (int)(tot >> 32) + min((int)(tot & 0xffffffffu), need);
    for (int i = min(taken, kk) + tid; i < p.k; i += TK_THREADS) out[i] = -1;
}

}  // namespace tidal
