// argTopK of Algorithm 1: for every (sequence, index head) pick the
// k' = min(k, N) positions with the largest score, equal scores resolved
// toward the lower position, and write them in ascending position order.
//
// One thread-block CLUSTER works on one (sequence, index head). Each CTA of the
// cluster owns a contiguous slice of the positions, converts its scores to
// order-preserving 32-bit keys once and keeps them in shared memory; the exact
// k'-th largest key is then found by a most-significant-digit radix select
// (12 + 12 + 8 bits) whose per-digit histograms are built in shared memory and
// summed across the cluster through distributed shared memory. The final pass
// emits positions in order using block- and cluster-wide prefix counts, taking
// only as many keys equal to the threshold as are still needed (lowest positions
// first), so the result is the unique set a full sort with a (score desc,
// position asc) order would give.
#pragma once

#include <cooperative_groups.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace tidal {
namespace cg = cooperative_groups;

constexpr int TOPK_THREADS = 1024;
constexpr int TOPK_BINS = 4096;

struct TopkParams {
    const float* scores;       // [B, Hq, score_stride]
    long long score_stride;
    const int* ctx_lens;
    int max_ctx;
    int Hq, Hi;                // index head hi ranks the sum over its Hq/Hi member heads
    int k;
    int* idx;                  // [B, Hi, k]
    int* idx_count;            // [B] or null
    int slice_cap;             // keys a CTA can hold
};

// Larger float <=> larger key; -0 and +0 map to the same key.
__device__ __forceinline__ uint32_t score_key(float s) {
    uint32_t u = __float_as_uint(s);
    if (u == 0x80000000u) u = 0u;
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Inclusive scan over the block of one int per thread (TOPK_THREADS threads);
// returns this thread's inclusive prefix and the block total.
__device__ __forceinline__ int block_scan_incl(int v, int* warp_sums, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, v, d);
        if (lane >= d) v += t;
    }
    __syncthreads();                       // warp_sums may still be read from a previous call
    if (lane == 31) warp_sums[warp] = v;
    __syncthreads();
    if (warp == 0) {
        int w = warp_sums[lane];
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, w, d);
            if (lane >= d) w += t;
        }
        warp_sums[lane] = w;
    }
    __syncthreads();
    total = warp_sums[31];
    return v + (warp ? warp_sums[warp - 1] : 0);
}

// Sum the CTAs' histograms (nbins bins) over the cluster into `merged`, then
// find the digit that holds the `need`-th largest remaining key.
// On return (identical in every thread of every CTA): digit, and `need` reduced
// by the number of keys in higher digits.
__device__ __forceinline__ void cluster_pick_digit(cg::cluster_group& cluster, int* hist, int* merged,
                                                   int nbins, int* warp_sums, int* bcast, int& digit,
                                                   int& need) {
    const int cs = cluster.num_blocks();
    cluster.sync();                                    // every CTA's histogram is complete
    for (int bin = threadIdx.x; bin < nbins; bin += TOPK_THREADS) {
        int s = 0;
        for (int r = 0; r < cs; ++r) s += cluster.map_shared_rank(hist, r)[bin];
        merged[bin] = s;
    }
    cluster.sync();                                    // remote reads done: hist may be reused
    // Each thread owns a run of bins, highest digits first.
    const int per = (nbins + TOPK_THREADS - 1) / TOPK_THREADS;
    const int hi_bin = nbins - 1 - threadIdx.x * per;  // this thread's highest bin
    int mine = 0;
    for (int i = 0; i < per; ++i) {
        const int bin = hi_bin - i;
        if (bin >= 0) mine += merged[bin];
    }
    int total;
    const int incl = block_scan_incl(mine, warp_sums, total);
    const int excl = incl - mine;                      // keys in strictly higher runs
    if (excl < need && need <= incl) {                 // the threshold digit is in this run
        int above = excl;
        for (int i = 0; i < per; ++i) {
            const int bin = hi_bin - i;
            const int c = (bin >= 0) ? merged[bin] : 0;
            if (above + c >= need) { bcast[0] = bin; bcast[1] = need - above; break; }
            above += c;
        }
    }
    __syncthreads();
    digit = bcast[0];
    need = bcast[1];
    __syncthreads();
}

__global__ void __launch_bounds__(TOPK_THREADS, 1) topk_kernel(const TopkParams p) {
    extern __shared__ __align__(128) uint8_t smem[];
    uint32_t* keys = reinterpret_cast<uint32_t*>(smem);                        // [slice_cap]
    int* hist = reinterpret_cast<int*>(smem + (size_t)p.slice_cap * 4);        // [TOPK_BINS]
    int* merged = hist + TOPK_BINS;                                            // [TOPK_BINS]
    __shared__ int warp_sums[32];
    __shared__ int bcast[2];
    __shared__ int cta_counts[2];          // (keys above the threshold, keys equal to it) in this slice

    cg::cluster_group cluster = cg::this_cluster();
    const int cs = cluster.num_blocks();
    const int rank = cluster.block_rank();
    const int item = blockIdx.x / cs;      // cluster index = b * Hi + hi
    const int b = item / p.Hi, hi = item % p.Hi;
    const int tid = threadIdx.x;

    const int N = max(0, min(p.ctx_lens[b], p.max_ctx));
    const int kk = min(p.k, N);
    int* out = p.idx + (long long)item * p.k;
    if (hi == 0 && rank == 0 && tid == 0 && p.idx_count) p.idx_count[b] = kk;

    // Slice of this CTA: [s0, s1), slice length a multiple of 4 except the last.
    int slice = ((N + cs - 1) / cs + 3) & ~3;
    slice = min(slice, p.slice_cap);
    const int s0 = min(N, rank * slice), s1 = min(N, s0 + slice);
    const int n_local = s1 - s0;

    if (kk == N) {                         // everything is kept: identity list, then padding
        for (int i = s0 + tid; i < s1; i += TOPK_THREADS) out[i] = i;
        if (rank == 0)
            for (int i = N + tid; i < p.k; i += TOPK_THREADS) out[i] = -1;
        return;                            // uniform over the cluster: nobody waits
    }

    // ---- load scores, build keys and the first (top 12 bits) histogram ----------------
    for (int i = tid; i < TOPK_BINS; i += TOPK_THREADS) hist[i] = 0;
    __syncthreads();
    const int members = p.Hq / p.Hi;
    const float* srow = p.scores + ((long long)b * p.Hq + (long long)hi * members) * p.score_stride;
    for (int i = tid; i < n_local; i += TOPK_THREADS) {
        float s = __ldcg(srow + s0 + i);
        for (int m = 1; m < members; ++m) s += __ldcg(srow + m * p.score_stride + s0 + i);
        const uint32_t key = score_key(s);
        keys[i] = key;
        atomicAdd(&hist[key >> 20], 1);
    }
    __syncthreads();

    int need = kk, digit;
    cluster_pick_digit(cluster, hist, merged, TOPK_BINS, warp_sums, bcast, digit, need);
    uint32_t prefix = (uint32_t)digit << 20;           // top 12 bits of the threshold key

    // ---- second digit: bits 19..8 among keys whose top 12 bits match -------------------
    for (int i = tid; i < TOPK_BINS; i += TOPK_THREADS) hist[i] = 0;
    __syncthreads();
    for (int i = tid; i < n_local; i += TOPK_THREADS) {
        const uint32_t key = keys[i];
        if ((key >> 20) == (prefix >> 20)) atomicAdd(&hist[(key >> 8) & 0xfffu], 1);
    }
    __syncthreads();
    cluster_pick_digit(cluster, hist, merged, TOPK_BINS, warp_sums, bcast, digit, need);
    prefix |= (uint32_t)digit << 8;

    // ---- third digit: bits 7..0 ---------------------------------------------------------
    for (int i = tid; i < 256; i += TOPK_THREADS) hist[i] = 0;
    __syncthreads();
    for (int i = tid; i < n_local; i += TOPK_THREADS) {
        const uint32_t key = keys[i];
        if ((key >> 8) == (prefix >> 8)) atomicAdd(&hist[key & 0xffu], 1);
    }
    __syncthreads();
    cluster_pick_digit(cluster, hist, merged, 256, warp_sums, bcast, digit, need);
    const uint32_t thr = prefix | (uint32_t)digit;     // the k'-th largest key
    // `need` keys equal to thr are taken, lowest positions first.

    // ---- ordered output --------------------------------------------------------------------
    const int per = (n_local + TOPK_THREADS - 1) / TOPK_THREADS;
    const int r0 = min(n_local, tid * per), r1 = min(n_local, r0 + per);
    int gt = 0, eq = 0;
    for (int i = r0; i < r1; ++i) {
        const uint32_t key = keys[i];
        gt += key > thr;
        eq += key == thr;
    }
    int gt_total, eq_total;
    const int gt_excl = block_scan_incl(gt, warp_sums, gt_total) - gt;
    const int eq_excl = block_scan_incl(eq, warp_sums, eq_total) - eq;
    if (tid == 0) { cta_counts[0] = gt_total; cta_counts[1] = eq_total; }
    cluster.sync();
    int gt_base = 0, eq_base = 0;
    for (int r = 0; r < rank; ++r) {
        const int* rc = cluster.map_shared_rank(cta_counts, r);
        gt_base += rc[0];
        eq_base += rc[1];
    }
    int eq_seen = eq_base + eq_excl;                   // equal keys at lower positions
    int at = gt_base + gt_excl + min(eq_seen, need);   // selected entries at lower positions
    for (int i = r0; i < r1; ++i) {
        const uint32_t key = keys[i];
        bool take = key > thr;
        if (key == thr) { take = eq_seen < need; ++eq_seen; }
        if (take) { if (at < p.k) out[at] = s0 + i; ++at; }
    }
    if (rank == 0)
        for (int i = kk + tid; i < p.k; i += TOPK_THREADS) out[i] = -1;
    cluster.sync();                                    // keep shared memory alive until peers have read it
}

}  // namespace tidal
