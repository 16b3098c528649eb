// K5 -- best move of a sweep: arg-min over per-candidate TELs, keyed (TEL, index).
//
// Each candidate's TEL = sum of completion times (Section 2.2) has already been accumulated by the
// warp that simulated it; this kernel reduces the TEL array to the smallest value and, among equal
// values, the smallest index -- the pair never depends on the order in which threads arrive.
// TELs are read as 16-byte vectors, reduced per warp with shuffles, per block through shared
// memory, and the last block to finish (ticket counter) folds the per-block partials and an
// optional earlier result (`prior`, for sweeps evaluated in several launches).  With `index_map` the
// array is in launch-slot order and element k belongs to index index_base + index_map[k].
#pragma once

#include "common.cuh"

#define K5_THREADS 256

__device__ __forceinline__ void k5_take(i64& bv, i64& bi, i64 v, i64 i) {
    if (v < bv || (v == bv && i < bi)) { bv = v; bi = i; }
}

__global__ void __launch_bounds__(K5_THREADS)
k5_argmin(const i64* __restrict__ tel, i64 count, i64 index_base, const int* __restrict__ index_map, const i64* prior,
          i64* __restrict__ partials, unsigned int* ticket, i64* __restrict__ best_out) {
    __shared__ i64 sh_v[K5_THREADS / 32], sh_i[K5_THREADS / 32];
    __shared__ bool is_last;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    i64 bv = INT64_MAX, bi = INT64_MAX;
    // the array may start on any 8-byte boundary: an odd first element is taken alone so that the
    // 16-byte loads behind it are aligned
    const int head = (count > 0 && ((unsigned long long)tel & 8ull)) ? 1 : 0;
    const i64 pairs = (count - head) >> 1;
    const longlong2* tel2 = reinterpret_cast<const longlong2*>(tel + head);
    for (i64 k = (i64)blockIdx.x * K5_THREADS + tid; k < pairs; k += (i64)gridDim.x * K5_THREADS) {
        const longlong2 v = tel2[k];
        const i64 e = head + 2 * k;
        k5_take(bv, bi, v.x, index_base + (index_map ? (i64)index_map[e] : e));
        k5_take(bv, bi, v.y, index_base + (index_map ? (i64)index_map[e + 1] : e + 1));
    }
    if (blockIdx.x == 0 && tid == 0) {
        if (head) k5_take(bv, bi, tel[0], index_base + (index_map ? (i64)index_map[0] : 0));
        if ((count - head) & 1)
            k5_take(bv, bi, tel[count - 1], index_base + (index_map ? (i64)index_map[count - 1] : count - 1));
    }
    for (int d = 16; d >= 1; d >>= 1) {
        const i64 ov = __shfl_xor_sync(KV_FULL, bv, d), oi = __shfl_xor_sync(KV_FULL, bi, d);
        k5_take(bv, bi, ov, oi);
    }
    if (lane == 0) { sh_v[w] = bv; sh_i[w] = bi; }
    __syncthreads();
    if (tid == 0) {
        for (int k = 1; k < K5_THREADS / 32; ++k) k5_take(bv, bi, sh_v[k], sh_i[k]);
        partials[2 * blockIdx.x] = bv;
        partials[2 * blockIdx.x + 1] = bi;
        __threadfence();
        const unsigned t = atomicAdd(ticket, 1u);
        is_last = (t == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    bv = INT64_MAX; bi = INT64_MAX;
    for (int k = tid; k < (int)gridDim.x; k += K5_THREADS) {
        const volatile i64* pp = partials;
        k5_take(bv, bi, pp[2 * k], pp[2 * k + 1]);
    }
    for (int d = 16; d >= 1; d >>= 1) {
        const i64 ov = __shfl_xor_sync(KV_FULL, bv, d), oi = __shfl_xor_sync(KV_FULL, bi, d);
        k5_take(bv, bi, ov, oi);
    }
    if (lane == 0) { sh_v[w] = bv; sh_i[w] = bi; }
    __syncthreads();
    if (tid == 0) {
        for (int k = 1; k < K5_THREADS / 32; ++k) k5_take(bv, bi, sh_v[k], sh_i[k]);
        if (prior) k5_take(bv, bi, prior[0], prior[1]);
        best_out[0] = bv;
        best_out[1] = bi;
        *ticket = 0;
    }
}

// Accept the best move if it strictly improves the current TEL (Section 5.2's rule), applying it
// to the base order in place.  One thread block; state = {cur_tel, accepted flag, iterations}.
__global__ void k5_accept_move(int* __restrict__ order, int n, const i64* __restrict__ best,
                               i64* __restrict__ cur_tel, int* __restrict__ accepted,
                               int* __restrict__ scratch /* [n] */, int sampled, u64 seed, int iteration) {
    __shared__ int sh_do;
    __shared__ Move mv;
    if (threadIdx.x == 0) {
        bool improve = best[1] != INT64_MAX && best[0] < *cur_tel;
        if (improve) {
            mv = sampled ? kv_sample_move(n, seed, iteration, best[1]) : kv_decode_move(n, best[1]);
            if ((unsigned)mv.i >= (unsigned)n || (unsigned)mv.j >= (unsigned)n) improve = false;   // not a move of this list
        }
        if (improve) *cur_tel = best[0];
        sh_do = improve ? 1 : 0;
        *accepted = improve ? 1 : 0;
    }
    __syncthreads();
    if (!sh_do) return;
    const Move m = mv;
    if (m.type == 0) {
        if (threadIdx.x == 0) { int x = order[m.i]; order[m.i] = order[m.j]; order[m.j] = x; }
        return;
    }
    // insert: build the moved range in scratch, then copy it back
    const int lo = min(m.i, m.j), hi = max(m.i, m.j);
    for (int q = lo + threadIdx.x; q <= hi; q += blockDim.x) scratch[q] = order[kv_map_pos(m, q)];
    __syncthreads();
    for (int q = lo + threadIdx.x; q <= hi; q += blockDim.x) order[q] = scratch[q];
}
