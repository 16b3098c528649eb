// K2b -- Phase 1 of Sorted-F with Algorithm 3 (Local Swap Search, Section 5.2 / the supplement to Section 5) as the
// batch solver, all batches in one launch of one CTA (the batches depend on each other: each one
// is built from what the previous ones left).
//
// Algorithm 3 on the remaining requests, sorted by ascending s+o (ties: lower index):
//   first fit  -- in that order a request is taken iff it still fits; because the sizes ascend,
//                 the result is the longest prefix whose sum(s+o) <= M;
//   improvement -- walk r_out over X (insertion order, a swapped-in request keeps the place of the
//                 one it replaces) and r_in over the requests outside X (sorted order); the first
//                 pair with  mem + (s+o)_in - (s+o)_out <= M  and  F(X') < F(X)  is swapped and the
//                 walk starts over; |X| never changes, so F drops iff o_in < o_out (with Section 7's
//                 prefill weight alpha = a_num / a_den: iff a_num s_in + a_den o_in is smaller).
// The pair walk is not executed cell by cell.  For one r_out the admissible r_in are the outside
// requests among the first ub positions (sizes ascend: (s+o)_in <= cap is a prefix), and the first
// of them with o_in < o_out is the first position where the running minimum of o over outside
// requests drops below o_out; so one min-scan per step plus two binary searches per member of X
// find, for every r_out at once, whether it has a partner, the lowest such member wins (that is
// the pair the printed loops reach first), and one thread looks up its partner.
#pragma once

#include "common.cuh"

#define K2L_THREADS 1024

__device__ __forceinline__ int k2l_warp_incl_sum(int v, int lane) {
    for (int d = 1; d < 32; d <<= 1) { const int y = __shfl_up_sync(KV_FULL, v, d); if (lane >= d) v += y; }
    return v;
}
__device__ __forceinline__ i64 k2l_warp_incl_sum64(i64 v, int lane) {
    for (int d = 1; d < 32; d <<= 1) { const i64 y = __shfl_up_sync(KV_FULL, v, d); if (lane >= d) v += y; }
    return v;
}
__device__ __forceinline__ int k2l_warp_incl_min(int v, int lane) {
    for (int d = 1; d < 32; d <<= 1) { const int y = __shfl_up_sync(KV_FULL, v, d); if (lane >= d) v = min(v, y); }
    return v;
}

// first index in [0, len) with a[idx] > key (a ascending)
__device__ __forceinline__ int k2l_upper_bound(const int* a, int len, i64 key) {
    int lo = 0, hi = len;
    while (lo < hi) { const int mid = (lo + hi) >> 1; if ((i64)a[mid] <= key) lo = mid + 1; else hi = mid; }
    return lo;
}
// first index in [0, len) with a[idx] < thr (a non-increasing); len if none
__device__ __forceinline__ int k2l_first_below(const int* a, int len, int thr) {
    int lo = 0, hi = len;
    while (lo < hi) { const int mid = (lo + hi) >> 1; if (a[mid] < thr) hi = mid; else lo = mid + 1; }
    return lo;
}

struct K2lShared {
    i64 sh64[33];
    int sh32[33];
    int pick[2];
    i64 mem;
};

// One batch of Algorithm 3 out of the entries of sorted_ids[0 .. n) (request ids by ascending
// (s+o, index)) whose `removed` flag is clear.  Called by all K2L_THREADS threads of a CTA; the
// scratch arrays hold n ints each and may live in shared or global memory.  Writes the batch in X's
// walking order to out[0 .. k0), sets the members' removed flags and returns k0 (the same value
// in every thread).
__device__ int k2l_batch(const int* s, const int* o, const int* sorted_ids, int n, i64 M, int a_num, int a_den,
                         int* removed, int* rem, int* remT, int* remO, int* inX, int* pm, int* xpos,
                         int* out, int* status, K2lShared& sh) {
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    // (a) remaining requests in sorted order -> rem / remT / remO
    int m = 0;
    for (int base = 0; base < n; base += K2L_THREADS) {
        const int i = base + tid;
        const int f = (i < n && !removed[i]) ? 1 : 0;
        const int incl = k2l_warp_incl_sum(f, lane);
        if (lane == 31) sh.sh32[w] = incl;
        __syncthreads();
        int before = 0, total = 0;
        for (int k = 0; k < 32; ++k) { const int v = sh.sh32[k]; if (k < w) before += v; total += v; }
        if (f) {
            const int p = m + before + incl - 1;
            const int id = sorted_ids[i];
            rem[p] = i; remT[p] = s[id] + o[id]; remO[p] = a_num * s[id] + a_den * o[id];   // weight: o when alpha = 0
        }
        m += total;
        __syncthreads();
    }
    // (b) first fit = longest prefix with sum(s+o) <= M
    int k0 = 0;
    i64 run = 0;
    for (int base = 0; base < m; base += K2L_THREADS) {
        const int p = base + tid;
        const i64 v = p < m ? (i64)remT[p] : 0;
        const i64 incl = k2l_warp_incl_sum64(v, lane);
        if (lane == 31) sh.sh64[w] = incl;
        __syncthreads();
        i64 before = 0, total = 0;
        for (int k = 0; k < 32; ++k) { const i64 x = sh.sh64[k]; if (k < w) before += x; total += x; }
        const i64 pre = run + before + incl;
        const int ok = (p < m && pre <= M) ? 1 : 0;
        const int cnt = __syncthreads_count(ok);
        if (ok && (p + 1 == m || p + 1 == base + cnt)) sh.mem = pre;      // last request taken so far
        k0 += cnt;
        run += total;
        __syncthreads();
        if (cnt < min(K2L_THREADS, m - base)) break;
    }
    i64 mem = sh.mem;
    for (int p = tid; p < m; p += K2L_THREADS) { inX[p] = p < k0 ? 1 : 0; if (p < k0) xpos[p] = p; }
    __syncthreads();
    // (c) improving swaps; every swap lowers sum(o) over X by at least 1
    const i64 step_cap = ((i64)k0 << 30) + 16;          // sum(o) over X <= k0 * 2^30
    for (i64 step = 0;; ++step) {
        int run_min = INT_MAX;
        for (int base = 0; base < m; base += K2L_THREADS) {
            const int p = base + tid;
            const int v = (p < m && !inX[p]) ? remO[p] : INT_MAX;
            const int incl = k2l_warp_incl_min(v, lane);
            if (lane == 31) sh.sh32[w] = incl;
            __syncthreads();
            int before = run_min, total = run_min;
            for (int k = 0; k < 32; ++k) { const int x = sh.sh32[k]; if (k < w) before = min(before, x); total = min(total, x); }
            if (p < m) pm[p] = min(before, incl);
            run_min = total;
            __syncthreads();
        }
        int mine = INT_MAX;
        for (int k = tid; k < k0; k += K2L_THREADS) {
            const int pos = xpos[k];
            const int ub = k2l_upper_bound(remT, m, M - mem + remT[pos]);
            if (ub > 0 && pm[ub - 1] < remO[pos]) { mine = k; break; }
        }
        mine = kv_warp_min(mine);
        if (lane == 0) sh.sh32[w] = mine;
        __syncthreads();
        if (tid == 0) {
            int kstar = INT_MAX;
            for (int k = 0; k < 32; ++k) kstar = min(kstar, sh.sh32[k]);
            sh.pick[0] = kstar;
            if (kstar != INT_MAX) {
                const int pos = xpos[kstar];
                const int ub = k2l_upper_bound(remT, m, M - mem + remT[pos]);
                const int j = k2l_first_below(pm, ub, remO[pos]);
                inX[pos] = 0; inX[j] = 1; xpos[kstar] = j;
                sh.mem = mem + remT[j] - remT[pos];
            }
        }
        __syncthreads();
        if (sh.pick[0] == INT_MAX) break;
        mem = sh.mem;
        if (step > kv_loop_cap(step_cap)) { if (tid == 0) atomicExch(status, KV_DEV_LOOP_CAP); break; }
        __syncthreads();
    }
    // (d) hand the batch out and retire its requests
    for (int k = tid; k < k0; k += K2L_THREADS) {
        const int si = rem[xpos[k]];
        out[k] = sorted_ids[si];
        removed[si] = 1;
    }
    __syncthreads();
    return k0;
}

// sorted_ids: request ids by ascending (s+o, index).  Scratch arrays hold n ints each.
// order_out receives every batch in X's walking order (the caller sorts each batch by (o, index)).
__global__ void __launch_bounds__(K2L_THREADS)
k2_local_swap(const int* __restrict__ s, const int* __restrict__ o, const int* __restrict__ sorted_ids,
              int n, i64 M, int a_num, int a_den, int* removed, int* rem, int* remT, int* remO, int* inX, int* pm, int* xpos,
              int* __restrict__ order_out, int* __restrict__ batch_off, int* __restrict__ num_batches,
              int* status) {
    __shared__ K2lShared sh;
    const int tid = threadIdx.x;
    for (int i = tid; i < n; i += K2L_THREADS) removed[i] = 0;
    if (tid == 0) batch_off[0] = 0;
    __syncthreads();
    int done = 0, nb = 0;
    while (done < n) {
        const int k0 = k2l_batch(s, o, sorted_ids, n, M, a_num, a_den, removed, rem, remT, remO, inX, pm, xpos,
                                 order_out + done, status, sh);
        done += k0;
        ++nb;
        if (tid == 0) batch_off[nb] = done;
        __syncthreads();
    }
    if (tid == 0) *num_batches = nb;
}
