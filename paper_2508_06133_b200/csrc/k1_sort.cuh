// K1 -- segmented LSD radix sort of (64-bit key, int32 value) pairs, one CTA per segment
// (CTAs stride over the segments when there are more segments than CTAs).
//
// Used for the request orderings the method needs: ascending (s+o, o, index) over the whole
// backlog (the order Algorithm 3 starts from), ascending (o, index) inside every selected batch
// (Algorithm 1, Phase 1: "sort requests in X* in nondecreasing order of o_i"), and the order
// policies.  Keys are built so that they are unique (the request index is part of the key or the
// input is in index order), hence the result does not depend on anything but the keys.
//
// A pass handles one 8-bit digit: a shared-memory histogram, an exclusive scan over the 256 bins,
// then tiles of 256 elements in order; inside a tile, __match_any_sync groups the lanes of a warp
// by digit, the per-warp counts are turned into offsets by one thread per digit, and every
// element is scattered to  bin offset + elements of its digit in earlier tiles/warps + its rank
// among equal digits in its warp  -- which keeps each pass stable.  Digits whose byte is zero in
// `byte_mask` are skipped (the host knows how many bits the keys use).
#pragma once

#include "common.cuh"

#define K1_THREADS 256
#define K1_WARPS (K1_THREADS / 32)

__global__ void __launch_bounds__(K1_THREADS)
k1_radix_sort_segments(u64* __restrict__ keys_a, int* __restrict__ vals_a,
                       u64* __restrict__ keys_b, int* __restrict__ vals_b,
                       const int* __restrict__ seg_off, const int* __restrict__ num_segments_ptr,
                       int num_segments, unsigned byte_mask) {
    __shared__ int hist[256];
    __shared__ int digit_off[256];
    __shared__ int warp_cnt[K1_WARPS][256];
    __shared__ int warp_tot[K1_WARPS];

    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    if (num_segments_ptr) num_segments = *num_segments_ptr;     // count produced on the device
    for (int seg = blockIdx.x; seg < num_segments; seg += gridDim.x) {
    const int lo = seg_off[seg], hi = seg_off[seg + 1];
    const int m = hi - lo;
    if (m <= 1) continue;
    u64* ksrc = keys_a; int* vsrc = vals_a;
    u64* kdst = keys_b; int* vdst = vals_b;

    for (int byte = 0; byte < 8; ++byte) {
        if (!((byte_mask >> byte) & 1u)) continue;
        const int shift = byte * 8;
        hist[tid] = 0;
        __syncthreads();
        for (int i = lo + tid; i < hi; i += K1_THREADS)
            atomicAdd(&hist[(int)((ksrc[i] >> shift) & 0xff)], 1);
        __syncthreads();
        // exclusive scan of the 256 bins: warp scans, then the 8 warp totals
        {
            int v = hist[tid], incl = v;
            for (int d = 1; d < 32; d <<= 1) {
                int y = __shfl_up_sync(KV_FULL, incl, d);
                if (lane >= d) incl += y;
            }
            if (lane == 31) warp_tot[w] = incl;
            __syncthreads();
            int base = 0;
            for (int k = 0; k < w; ++k) base += warp_tot[k];
            digit_off[tid] = base + incl - v;
        }
        __syncthreads();
        for (int tile = 0; tile < m; tile += K1_THREADS) {
            const int i = lo + tile + tid;
            const bool valid = i < hi;
            u64 key = 0; int val = 0; int d = 256;
            if (valid) { key = ksrc[i]; val = vsrc[i]; d = (int)((key >> shift) & 0xff); }
            for (int k = 0; k < K1_WARPS; ++k) warp_cnt[k][tid] = 0;
            __syncthreads();
            const unsigned peers = __match_any_sync(KV_FULL, d);
            const int rank = __popc(peers & ((1u << lane) - 1u));
            if (valid && rank == 0) warp_cnt[w][d] = __popc(peers);
            __syncthreads();
            {
                int acc = digit_off[tid];
                for (int k = 0; k < K1_WARPS; ++k) {
                    int c = warp_cnt[k][tid];
                    warp_cnt[k][tid] = acc;
                    acc += c;
                }
                digit_off[tid] = acc;
            }
            __syncthreads();
            if (valid) {
                const int dst = lo + (int)KV_IDX(warp_cnt[w][d] + rank, hi - lo, 701);
                kdst[dst] = key;
                vdst[dst] = val;
            }
            __syncthreads();
        }
        u64* tk = ksrc; ksrc = kdst; kdst = tk;
        int* tv = vsrc; vsrc = vdst; vdst = tv;
    }
    if (ksrc != keys_a) {                      // odd number of passes: bring the result home
        for (int i = lo + tid; i < hi; i += K1_THREADS) { keys_a[i] = ksrc[i]; vals_a[i] = vsrc[i]; }
    }
    __syncthreads();
    }   // segments
}

// Keys for the whole-backlog sort: (s+o) in the high word, o in the low word; values = request ids
// in index order, so equal keys keep ascending index.
__global__ void k1_keys_total_size(const int* __restrict__ s, const int* __restrict__ o, int n,
                                   u64* __restrict__ keys, int* __restrict__ vals, int policy) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    u64 T = (u64)(s[i] + o[i]), O = (u64)o[i];
    u64 k;
    if (policy == SCHED_POLICY_SOF) k = O << 32;
    else if (policy == SCHED_POLICY_TOTAL_SIZE) k = T << 32;
    else if (policy == SCHED_POLICY_FCFS) k = 0;
    else k = (T << 32) | O;
    keys[i] = k;
    vals[i] = i;
}

// Keys for the per-batch sort: (o, request id) of the request at every position of `order`.
__global__ void k1_keys_output_then_id(const int* __restrict__ o, const int* __restrict__ order, int n,
                                       u64* __restrict__ keys, int* __restrict__ vals) {
    int q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= n) return;
    int id = order[q];
    keys[q] = ((u64)o[id] << 32) | (u64)(unsigned)id;
    vals[q] = id;
}

// Keys for checking explicit start times: (start, request id) per candidate; also writes the
// segment offsets c * n, c = 0 .. count.
__global__ void k1_keys_start_then_id(const int* __restrict__ starts, int n, long long total,
                                      u64* __restrict__ keys, int* __restrict__ vals,
                                      int* __restrict__ seg_off, int count) {
    long long k = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (k <= count) seg_off[k] = (int)(k * n);
    if (k >= total) return;
    const int id = (int)(k % n);
    keys[k] = ((u64)(unsigned)starts[k] << 32) | (u64)(unsigned)id;
    vals[k] = id;
}
