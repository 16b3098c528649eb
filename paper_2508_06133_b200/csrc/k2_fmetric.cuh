// K2 -- F-metric batch selection over a sorted list (Algorithm 1, Phase 1, restricted to prefixes).
//
// Section 3: F(X) = (sum of o over X) / |X|^2; the batch with the smallest F is taken next, ties go
// to the larger batch.  Candidates here are the prefixes of the not-yet-selected requests in
// ascending (s+o, o, index) order (the order Algorithm 3 builds its first batch from), subject to
// Algorithms 2/3/4's memory test  sum (s_i + o_i) <= M.  With inclusive prefix sums P (of s+o) and
// O (of o) over the sorted list, the batch that starts at offset a is
//     k_max = max { k : P[a+k] - P[a] <= M },    k* = argmin_{1 <= k <= k_max} (O[a+k] - O[a]) / k^2,
// and the next batch starts at a + k*.  F values are compared exactly: A/ka^2 < B/kb^2 iff
// A*kb^2 < B*ka^2, evaluated on 128-bit products.
//
// The device routines work for any block size that is a multiple of 32: lanes stride over k, the
// best (sum, k) pair is reduced with warp shuffles and, for more than one warp, through shared
// memory.
#pragma once

#include "common.cuh"

// true iff batch (sumA, kA) is strictly preferred to (sumB, kB); kB == 0 means "no batch yet".
__device__ __forceinline__ bool k2_f_better(u64 sumA, u64 kA, u64 sumB, u64 kB) {
    if (kA == 0) return false;
    if (kB == 0) return true;
    const u64 a2 = kA * kA, b2 = kB * kB;
    const u64 l_hi = __umul64hi(sumA, b2), l_lo = sumA * b2;
    const u64 r_hi = __umul64hi(sumB, a2), r_lo = sumB * a2;
    if (l_hi != r_hi) return l_hi < r_hi;
    if (l_lo != r_lo) return l_lo < r_lo;
    return kA > kB;
}

// Inclusive-to-exclusive prefix sums of T = s+o and o over `ids` (list order):
// P[0] = O[0] = 0, P[q+1] = P[q] + T(ids[q]).  Block-wide, chunked; `carry` is 2 shared words.
// With a prefill weight alpha = a_num / a_den (Section 7's G-metric, alpha = 0 is F) the second sum
// runs over a_num * s + a_den * o instead of o.
// PT is the type the sums are stored in (int64, or int32 where the caller knows they fit); IT the
// type of the ids.
template <typename PT = i64, typename IT = int>
__device__ void k2_prefix_sums(const int* __restrict__ s, const int* __restrict__ o,
                               const IT* __restrict__ ids, int n, PT* P, PT* O,
                               i64* sh_warp /* [2 * 32] */, i64* carry /* [2] */,
                               i64 a_num = 0, i64 a_den = 1) {
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5, nw = blockDim.x >> 5;
    if (tid == 0) { carry[0] = 0; carry[1] = 0; P[0] = 0; O[0] = 0; }
    __syncthreads();
    for (int base = 0; base < n; base += blockDim.x) {
        const int q = base + tid;
        i64 vt = 0, vo = 0;
        if (q < n) { int id = ids[q]; vt = (i64)s[id] + o[id]; vo = a_num * s[id] + a_den * o[id]; }
        i64 it = vt, io = vo;
        for (int d = 1; d < 32; d <<= 1) {
            i64 yt = __shfl_up_sync(KV_FULL, it, d), yo = __shfl_up_sync(KV_FULL, io, d);
            if (lane >= d) { it += yt; io += yo; }
        }
        if (lane == 31) { sh_warp[w] = it; sh_warp[32 + w] = io; }
        __syncthreads();
        i64 bt = carry[0], bo = carry[1];
        for (int k = 0; k < w; ++k) { bt += sh_warp[k]; bo += sh_warp[32 + k]; }
        if (q < n) { P[q + 1] = (PT)(bt + it); O[q + 1] = (PT)(bo + io); }
        __syncthreads();
        if (tid == blockDim.x - 1) {
            i64 tt = 0, to = 0;
            for (int k = 0; k < nw; ++k) { tt += sh_warp[k]; to += sh_warp[32 + k]; }
            carry[0] += tt; carry[1] += to;
        }
        __syncthreads();
    }
}

// Batch boundaries by the rule above.  Writes batch_off[0..nb] and returns nb (same in all
// threads).  sh_best: 2 * 32 + 2 shared 64-bit words.
template <typename PT = i64>
__device__ int k2_select_batches(const PT* P, const PT* O, int n, i64 M, int* batch_off, u64* sh_best) {
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5, nw = blockDim.x >> 5;
    int a = 0, nb = 0;
    if (tid == 0) batch_off[0] = 0;
    while (a < n) {
        // k_max by binary search on P (every thread does the same search)
        int lo_k = 1, hi_k = n - a;
        const i64 Pa = (i64)P[a], Oa = (i64)O[a];
        while (lo_k < hi_k) {
            int mid = (lo_k + hi_k + 1) >> 1;
            if ((i64)P[a + mid] - Pa <= M) lo_k = mid; else hi_k = mid - 1;
        }
        const int kmax = lo_k;                      // >= 1 because every request fits on its own
        u64 bs = 0, bk = 0;
        for (int k = 1 + tid; k <= kmax; k += blockDim.x) {
            u64 sum = (u64)((i64)O[a + k] - Oa);
            if (k2_f_better(sum, (u64)k, bs, bk)) { bs = sum; bk = (u64)k; }
        }
        for (int d = 16; d >= 1; d >>= 1) {
            u64 os = __shfl_xor_sync(KV_FULL, bs, d), ok = __shfl_xor_sync(KV_FULL, bk, d);
            if (k2_f_better(os, ok, bs, bk)) { bs = os; bk = ok; }
        }
        if (nw > 1) {
            if (lane == 0) { sh_best[w] = bs; sh_best[32 + w] = bk; }
            __syncthreads();
            if (w == 0) {
                bs = lane < nw ? sh_best[lane] : 0; bk = lane < nw ? sh_best[32 + lane] : 0;
                for (int d = 16; d >= 1; d >>= 1) {
                    u64 os = __shfl_xor_sync(KV_FULL, bs, d), ok = __shfl_xor_sync(KV_FULL, bk, d);
                    if (k2_f_better(os, ok, bs, bk)) { bs = os; bk = ok; }
                }
                if (lane == 0) sh_best[64] = bk;
            }
            __syncthreads();
            bk = sh_best[64];
            __syncthreads();
        }
        a += (int)bk;
        ++nb;
        if (tid == 0) batch_off[KV_IDX(nb, n + 1, 801)] = a;
    }
    return nb;
}

// One CTA: prefix sums over the sorted ids, then the batch loop.  P, O: global int64[n+1].
__global__ void __launch_bounds__(1024)
k2_prefix_f(const int* __restrict__ s, const int* __restrict__ o, const int* __restrict__ sorted_ids,
            int n, i64 M, i64* __restrict__ P, i64* __restrict__ O,
            int* __restrict__ batch_off, int* __restrict__ num_batches, i64 a_num, i64 a_den) {
    __shared__ i64 sh_warp[64];
    __shared__ i64 carry[2];
    __shared__ u64 sh_best[66];
    k2_prefix_sums(s, o, sorted_ids, n, P, O, sh_warp, carry, a_num, a_den);
    __syncthreads();
    int nb = k2_select_batches(P, O, n, M, batch_off, sh_best);
    if (threadIdx.x == 0) *num_batches = nb;
}
