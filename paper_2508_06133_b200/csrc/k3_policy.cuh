// K3 -- policy sweep: many independent instances, each list-scheduled (Algorithm 1 Phase 2) under the
// order policies of Section 2.3 / Section 7 (index order, shortest decode first, smallest s+o first)
// and under Sorted-F with prefix-F batch selection, one warp per (instance, policy) pair.
#pragma once

#include "common.cuh"
#include "k2_fmetric.cuh"
#include "sim.cuh"
#include "sim_reg.cuh"
#include "sim_hyb.cuh"

// ------------------------------------------------------------------------------------------------
// Policy sweep: one warp per (instance, policy) pair, up to K3P_MAX_WARPS pairs of one instance per
// CTA.  Dynamic shared memory: int s[n], o[n] once per CTA; per warp the simulator's ring
// (SIM::ring_cells(L) ints), PT P[n+2], O[n+2] (PT = int32 when n * M < 2^31, else int64), int
// boff[n+2], a 256-bin histogram, and 16-bit: three id buffers [n] and batch numbers [n].  Orders are built by
// a single-warp radix sort (k3_warp_radix_sort) on the fields of the policy's key.
// ------------------------------------------------------------------------------------------------
// One pass of a stable least-significant-digit radix sort run by a single warp on shared memory:
// the m ids of `in` are written to `out` in ascending order of digit(id), an 8-bit value; ids with
// equal digits keep their order.  `hist` is 256 ints of shared memory.  Counting uses shared atomics
// (a sum does not depend on the order of its terms); in the scatter every chunk of 32 ids is ranked
// with a match-any vote (lanes with the same digit form a group whose lowest lane books the group's
// bins), so the result does not depend on timing.
template <class IT, class DIGIT>
__device__ __forceinline__ void k3_warp_radix_pass(const IT* in, IT* out, int m, int* hist, int lane, DIGIT digit) {
    for (int b = lane; b < 256; b += 32) hist[b] = 0;
    __syncwarp();
    const unsigned lt = (1u << lane) - 1u;
    for (int e = lane; e < m; e += 32) atomicAdd(&hist[KV_IDX(digit(in[e]), 256, 901)], 1);   // count (order-free)
    __syncwarp();
    {                                                                // exclusive scan of the 256 bins, 8 per lane
        int v[8], sum = 0;
#pragma unroll
        for (int k = 0; k < 8; ++k) { v[k] = hist[8 * lane + k]; sum += v[k]; }
        int incl = sum;
        for (int dlt = 1; dlt < 32; dlt <<= 1) {
            const int y = __shfl_up_sync(KV_FULL, incl, dlt);
            if (lane >= dlt) incl += y;
        }
        int run = incl - sum;
#pragma unroll
        for (int k = 0; k < 8; ++k) { hist[8 * lane + k] = run; run += v[k]; }
    }
    __syncwarp();
    for (int base = 0; base < m; base += 32) {                       // scatter
        const int e = base + lane;
        const int id = e < m ? in[e] : 0;
        const int d = e < m ? digit(id) : 256 + lane;
        const unsigned peers = __match_any_sync(KV_FULL, d);
        int pos = 0;
        if (e < m) pos = (int)KV_IDX(hist[KV_IDX(d, 256, 902)] + __popc(peers & lt), m, 903);
        __syncwarp();
        if (e < m) {
            out[pos] = (IT)id;
            if ((peers & lt) == 0) hist[d] += __popc(peers);
        }
        __syncwarp();
    }
}

// The m ids of `a` stably re-ordered by ascending field(id) (`bytes` 8-bit digits, least significant
// first).  a and b are two id buffers of m ints; returns the one that holds the result.
template <class IT, class FIELD>
__device__ __forceinline__ IT* k3_warp_radix_sort(IT* a, IT* b, int m, int* hist, int lane, FIELD field, int bytes) {
    for (int k = 0; k < bytes; ++k) {
        k3_warp_radix_pass(a, b, m, hist, lane, [&](int id) { return (field(id) >> (8 * k)) & 255; });
        IT* x = a; a = b; b = x;
    }
    return a;
}

__host__ __device__ __forceinline__ int k3_bytes_of(unsigned v) { int b = 1; while (v >> (8 * b) && b < 4) ++b; return b; }

typedef unsigned short k3_id_t;                     // request ids and list positions of the policy kernel (n < 65,536)

#define K3P_MAX_WARPS 4                             // instance-policy pairs per CTA of the policy kernel

// Single-warp forms of K2's prefix sums and batch selection (k2_fmetric.cuh has the block-wide ones):
// P[0] = O[0] = 0, P[q+1] = P[q] + s+o, O[q+1] = O[q] + o over the list `ids`; then the batch
// boundaries by the F-metric rule (smallest F = sum(o)/k^2 over the prefixes that fit M, ties to the
// larger batch).  Sums are computed in PT, which the caller has checked to be wide enough.
template <typename PT, typename IT>
__device__ __forceinline__ void k3_warp_prefix_sums(const int* s, const int* o, const IT* ids, int n, PT* P, PT* O, int lane) {
    PT ct = 0, co = 0;                              // totals of the chunks before this one (same in every lane)
    if (lane == 0) { P[0] = 0; O[0] = 0; }
    for (int base = 0; base < n; base += 32) {
        const int q = base + lane;
        PT it = 0, io = 0;
        if (q < n) { const int id = ids[q]; it = (PT)s[id] + (PT)o[id]; io = (PT)o[id]; }
        for (int d = 1; d < 32; d <<= 1) {
            const PT yt = __shfl_up_sync(KV_FULL, it, d), yo = __shfl_up_sync(KV_FULL, io, d);
            if (lane >= d) { it += yt; io += yo; }
        }
        if (q < n) { P[q + 1] = ct + it; O[q + 1] = co + io; }
        ct += __shfl_sync(KV_FULL, it, 31);
        co += __shfl_sync(KV_FULL, io, 31);
    }
    __syncwarp();
}

template <typename PT>
__device__ __forceinline__ int k3_warp_select_batches(const PT* P, const PT* O, int n, i64 M, int* batch_off, int lane) {
    int a = 0, nb = 0;
    if (lane == 0) batch_off[0] = 0;
    while (a < n) {
        int lo_k = 1, hi_k = n - a;                 // k_max by binary search on P (every lane does the same search)
        const i64 Pa = (i64)P[a], Oa = (i64)O[a];
        while (lo_k < hi_k) {
            const int mid = (lo_k + hi_k + 1) >> 1;
            if ((i64)P[a + mid] - Pa <= M) lo_k = mid; else hi_k = mid - 1;
        }
        const int kmax = lo_k;                      // >= 1 because every request fits on its own
        u64 bs = 0, bk = 0;
        for (int k = 1 + lane; k <= kmax; k += 32) {
            const u64 sum = (u64)((i64)O[a + k] - Oa);
            if (k2_f_better(sum, (u64)k, bs, bk)) { bs = sum; bk = (u64)k; }
        }
        for (int d = 16; d >= 1; d >>= 1) {
            const u64 os = __shfl_xor_sync(KV_FULL, bs, d), ok = __shfl_xor_sync(KV_FULL, bk, d);
            if (k2_f_better(os, ok, bs, bk)) { bs = os; bk = ok; }
        }
        a += (int)bk;
        ++nb;
        if (lane == 0) batch_off[KV_IDX(nb, n + 1, 907)] = a;
    }
    __syncwarp();
    return nb;
}

// Bytes of shared memory one warp of the policy kernel needs besides the instance's (s, o):
// the simulator's ring, P and O, the batch offsets, the radix histogram and four 16-bit id arrays.
__host__ __device__ inline size_t k3_policy_warp_bytes(int n, int ring_cells, int pt_bytes) {
    const size_t b = (size_t)ring_cells * 4 + (size_t)(n + 2) * 2 * pt_bytes + (size_t)(n + 2) * 4 + 256 * 4 + (size_t)n * 8;
    return (b + 15) & ~(size_t)15;
}

// grid = B * groups CTAs of W = blockDim.x / 32 warps; CTA (b, g) evaluates instance b under
// policies[g * W .. g * W + W - 1], one warp each; (s, o) of the instance are staged once per CTA.
template <class SIM, typename PT>
__global__ void __launch_bounds__(32 * K3P_MAX_WARPS)
k3_eval_policy(const int* __restrict__ s_all, const int* __restrict__ o_all, int n, int L, int M, int omax,
               const int* __restrict__ policies, int num_policies, int groups,
               i64* __restrict__ tel_out, int* __restrict__ starts_out, int* status) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, W = blockDim.x >> 5;
    const int b = blockIdx.x / groups, kpol = (blockIdx.x % groups) * W + warp;
    int* s = (int*)smem_raw;
    int* o = s + n;
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        s[i] = s_all[(size_t)b * n + i];
        o[i] = o_all[(size_t)b * n + i];
    }
    __syncthreads();
    if (kpol >= num_policies) return;               // a last group that is not full
    const int policy = policies[kpol];
    unsigned char* mine = smem_raw + (((size_t)n * 8 + 15) & ~(size_t)15) +
                          (size_t)warp * k3_policy_warp_bytes(n, SIM::ring_cells(L), (int)sizeof(PT));
    int* ring = (int*)mine;                           // first: 16-byte aligned for the vector loads
    PT* P = (PT*)(ring + SIM::ring_cells(L));         // a multiple of 4 ints: 8-byte aligned
    PT* O = P + (n + 2);
    int* boff = (int*)(O + (n + 2));                  // n + 2 batch offsets
    int* hist = boff + n + 2;                         // 256 bins of the radix passes
    k3_id_t* bufa = (k3_id_t*)(hist + 256);
    k3_id_t* bufb = bufa + n;
    k3_id_t* byo = bufb + n;                          // ids by ascending (o, id) (Sorted-F keeps them for its second sort)
    k3_id_t* bat = byo + n;                           // batch number of every request (Sorted-F)

    for (int i = lane; i < n; i += 32) bufa[i] = (k3_id_t)i;
    __syncwarp();
    const int o_bytes = k3_bytes_of((unsigned)omax), t_bytes = k3_bytes_of((unsigned)M);
    auto f_o = [&](int id) { return o[id]; };
    auto f_t = [&](int id) { return s[id] + o[id]; };
    k3_id_t* ord = bufa;                              // FCFS: the identity order
    // every sort is a chain of stable passes from the identity order, so ties end in ascending id
    if (policy == SCHED_POLICY_SOF) {
        ord = k3_warp_radix_sort(bufa, bufb, n, hist, lane, f_o, o_bytes);
    } else if (policy == SCHED_POLICY_TOTAL_SIZE) {
        ord = k3_warp_radix_sort(bufa, bufb, n, hist, lane, f_t, t_bytes);
    } else if (policy == SCHED_POLICY_SORTED_F) {
        // ascending (s+o, o, id) = the (o, id) order re-sorted stably by s+o; F-metric batch boundaries;
        // then every batch by ascending (o, id) = the (o, id) order re-sorted stably by batch number
        ord = k3_warp_radix_sort(bufa, bufb, n, hist, lane, f_o, o_bytes);
        for (int i = lane; i < n; i += 32) byo[i] = ord[i];
        __syncwarp();
        k3_id_t* other = ord == bufa ? bufb : bufa;
        ord = k3_warp_radix_sort(ord, other, n, hist, lane, f_t, t_bytes);
        k3_warp_prefix_sums(s, o, ord, n, P, O, lane);
        const int nb = k3_warp_select_batches(P, O, n, (i64)M, boff, lane);
        for (int bi = 0; bi < nb; ++bi)
            for (int q = boff[bi] + lane; q < boff[bi + 1]; q += 32) bat[KV_IDX(ord[KV_IDX(q, n, 904)], n, 905)] = bi;
        __syncwarp();
        auto f_b = [&](int id) { return bat[id]; };
        ord = k3_warp_radix_sort(byo, ord == bufa ? bufb : bufa, n, hist, lane, f_b, k3_bytes_of((unsigned)nb));
    }
    SIM sim;
    sim.attach(ring, L);
    sim.reset(lane);
    int* starts = starts_out ? starts_out + ((size_t)b * num_policies + kpol) * n : nullptr;
    for (int q = 0; q < n; ++q) {
        const int id = (int)KV_IDX(ord[q], n, 906);
        const int pstart = sim.admit(s[id], o[id], M, lane, status);
        if (starts && lane == 0) starts[id] = pstart;
    }
    if (lane == 0) tel_out[(size_t)b * num_policies + kpol] = sim.total();
}

