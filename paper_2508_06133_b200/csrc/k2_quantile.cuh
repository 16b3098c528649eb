// K2d -- Algorithm 4 (Quantile Greedy Selection, Section 5.3) as the Phase-1 solver.
//
// One batch out of the remaining requests, which are kept as a list `rem` in ascending (o, index)
// -- the order the algorithm sorts by first; taking a batch out keeps the list sorted, so it is
// sorted once.  Per batch, the host issues
//   k2q_begin        sampling keys  mix(seed ^ mix(batch * 2^32 + id))  per list position
//   K1 sort          positions by key: the first m = max(1, floor(nr/2)) are the sample
//   k2q_sample_keys  s+o and o of the sample members, as two segments
//   K1 sort          both segments: Q_p and Q_o are the elements at position floor(3 (m-1) / 10)
//   k2q_pass1        first fit over the list under both thresholds (one CTA)
//   k2q_ratio_keys   o/(s+o) of the positions not yet chosen as a fixed-point key
//   K1 sort          positions by that key (stable: equal ratios keep the list order)
//   k2q_pass2_emit   first fit over the sorted positions, then the batch (already in ascending
//                    (o, index), being a sub-list of rem) and the compacted remaining list
// and reads the batch size back.
//
// The ratio key floor(o * 2^F / (s+o)) orders the requests exactly as the rationals do when
// 2^F exceeds the product of any two denominators: two different ratios differ by at least
// 1 / ((s_a+o_a)(s_b+o_b)) > 2^-F, so their keys differ; equal ratios give equal keys.
//
// First fit is sequential by definition (whether a request is admitted depends on the memory the
// earlier ones took).  Here a CTA takes 1024 list positions at a time: requests that cannot fit
// even alone in what is left are dropped (the free memory only shrinks, so they would be refused
// at their turn anyway), an inclusive scan over the sizes of the others finds the first one that
// no longer fits after its predecessors; everything before it is admitted, it is refused, and the
// walk goes on right after it.  Every turn either finishes a tile or admits at least one request.
#pragma once

#include "common.cuh"

#define K2Q_THREADS 1024
#define K2Q_CHOSEN_KEY (1ull << 63)

// layout of the small device state (ints)
#define K2Q_COUNT 0        // size of the batch just selected
#define K2Q_MEM_LO 2       // memory used after pass 1 (low / high word)
#define K2Q_MEM_HI 3
#define K2Q_SEG1 4         // {0, nr}
#define K2Q_SEG2 6         // {0, m, 2m}
#define K2Q_SMALL_INTS 16

__global__ void k2q_begin(const int* __restrict__ rem, int nr, u64 seed, int batch,
                          u64* __restrict__ keys, int* __restrict__ vals, int* __restrict__ chosen,
                          int* __restrict__ small) {
    const int a = blockIdx.x * blockDim.x + threadIdx.x;
    if (a == 0) {
        const int m = nr / 2 > 1 ? nr / 2 : 1;
        small[K2Q_SEG1] = 0; small[K2Q_SEG1 + 1] = nr;
        small[K2Q_SEG2] = 0; small[K2Q_SEG2 + 1] = m; small[K2Q_SEG2 + 2] = 2 * m;
    }
    if (a >= nr) return;
    const int id = rem[a];
    keys[a] = kv_mix64(seed ^ kv_mix64(((u64)(unsigned)batch << 32) + (u64)id));
    vals[a] = a;
    chosen[a] = 0;
}

__global__ void k2q_sample_keys(const int* __restrict__ rem, const int* __restrict__ by_key, int m,
                                const int* __restrict__ s, const int* __restrict__ o, u64* __restrict__ keys) {
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= m) return;
    const int id = rem[by_key[r]];
    keys[r] = (u64)(s[id] + o[id]);
    keys[m + r] = (u64)o[id];
}

__global__ void k2q_ratio_keys(const int* __restrict__ rem, int nr, const int* __restrict__ s, const int* __restrict__ o,
                               const int* __restrict__ chosen, int F, u64* __restrict__ keys, int* __restrict__ vals) {
    const int a = blockIdx.x * blockDim.x + threadIdx.x;
    if (a >= nr) return;
    const int id = rem[a];
    keys[a] = chosen[a] ? K2Q_CHOSEN_KEY : (((u64)o[id] << F) / (u64)(s[id] + o[id]));
    vals[a] = a;
}

struct K2qShared {
    i64 warp_tot[32];
    i64 sum;
    int first;
    int iwarp[32];
};

// First fit over list[0 .. cnt) (list == nullptr: the positions 0 .. cnt-1 themselves).  elig(a, T, o)
// says whether position a may be admitted at all.  Returns the memory in use afterwards; sets
// chosen[a] = 1 for every admitted position.  Called by all K2Q_THREADS threads.
template <typename Elig>
__device__ i64 k2q_first_fit(const int* __restrict__ list, int cnt, const int* __restrict__ rem,
                             const int* __restrict__ s, const int* __restrict__ o, i64 M, i64 mem,
                             int* __restrict__ chosen, Elig elig, K2qShared& sh) {
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    int pos = 0;
    while (pos < cnt) {                                   // pos grows by at least one per turn
        const i64 slack = M - mem;
        if (slack < 2) break;                             // every request has s + o >= 2
        if (tid == 0) sh.first = K2Q_THREADS;
        const int idx = pos + tid;
        int a = -1;
        i64 T = 0;
        if (idx < cnt) {
            a = list ? list[idx] : idx;
            const int id = rem[a];
            const int oi = o[id];
            const i64 Ti = (i64)s[id] + oi;
            if (Ti <= slack && elig(a, Ti, oi)) T = Ti;
        }
        i64 incl = T;
        for (int d = 1; d < 32; d <<= 1) {
            const i64 y = __shfl_up_sync(KV_FULL, incl, d);
            if (lane >= d) incl += y;
        }
        if (lane == 31) sh.warp_tot[w] = incl;
        __syncthreads();
        for (int k = 0; k < w; ++k) incl += sh.warp_tot[k];
        if (T > 0 && incl > slack) atomicMin(&sh.first, tid);
        __syncthreads();
        const int f = sh.first;
        if (T > 0 && tid < f) chosen[a] = 1;
        if (f < K2Q_THREADS ? tid == f : tid == K2Q_THREADS - 1) sh.sum = f < K2Q_THREADS ? incl - T : incl;
        __syncthreads();
        mem += sh.sum;
        pos += f < K2Q_THREADS ? f + 1 : K2Q_THREADS;
    }
    return mem;
}

__global__ void __launch_bounds__(K2Q_THREADS)
k2q_pass1(const int* __restrict__ rem, int nr, int m, const int* __restrict__ s, const int* __restrict__ o, i64 M,
          const u64* __restrict__ sorted_sample /* s+o at [0,m), o at [m,2m) */, int* __restrict__ chosen,
          int* __restrict__ small) {
    __shared__ K2qShared sh;
    const int q = (int)((3ll * (m - 1)) / 10);
    const i64 Qp = (i64)sorted_sample[q], Qo = (i64)sorted_sample[m + q];
    const i64 mem = k2q_first_fit(nullptr, nr, rem, s, o, M, 0,
                                  chosen, [=](int, i64 T, int oi) { return T <= Qp && (i64)oi <= Qo; }, sh);
    if (threadIdx.x == 0) {
        small[K2Q_MEM_LO] = (int)(mem & 0xffffffffll);
        small[K2Q_MEM_HI] = (int)(mem >> 32);
    }
}

// Pass 2, then hand the batch out.  by_ratio: the list positions in ascending ratio (positions
// chosen in pass 1 sort to the end and are not eligible).  The batch is appended to order_out at
// `done`, batch_off[nb + 1] is set, rem_next receives the positions not chosen, in list order.
__global__ void __launch_bounds__(K2Q_THREADS)
k2q_pass2_emit(const int* __restrict__ rem, int* __restrict__ rem_next, int nr, const int* __restrict__ s,
               const int* __restrict__ o, i64 M, const int* __restrict__ by_ratio, int* __restrict__ chosen,
               int* __restrict__ small, int* __restrict__ order_out, int done, int* __restrict__ batch_off, int nb) {
    __shared__ K2qShared sh;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const i64 mem0 = ((i64)small[K2Q_MEM_HI] << 32) | (i64)(unsigned)small[K2Q_MEM_LO];
    k2q_first_fit(by_ratio, nr, rem, s, o, M, mem0, chosen,
                  [=](int a, i64, int) { return chosen[a] == 0; }, sh);
    __syncthreads();                                      // chosen[] of this CTA is complete
    int taken = 0;                                        // chosen positions before this tile
    for (int base = 0; base < nr; base += K2Q_THREADS) {
        const int a = base + tid;
        const int flag = (a < nr) ? chosen[a] : 0;
        int incl = flag;
        for (int d = 1; d < 32; d <<= 1) {
            const int y = __shfl_up_sync(KV_FULL, incl, d);
            if (lane >= d) incl += y;
        }
        if (lane == 31) sh.iwarp[w] = incl;
        __syncthreads();
        int before = 0, total = 0;
        for (int k = 0; k < 32; ++k) { const int c = sh.iwarp[k]; if (k < w) before += c; total += c; }
        const int rank = taken + before + incl - flag;    // chosen positions before a
        if (a < nr) {
            if (flag) order_out[done + rank] = rem[a];
            else rem_next[a - rank] = rem[a];
        }
        taken += total;
        __syncthreads();
    }
    if (tid == 0) {
        small[K2Q_COUNT] = taken;
        batch_off[nb + 1] = done + taken;
    }
}
