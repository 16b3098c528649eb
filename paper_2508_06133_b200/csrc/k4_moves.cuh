// K4 -- neighbourhood generation: move index -> (type, i, j), and the launch order of a sweep.
//
// A candidate of a sweep is a move (swap or insert of list positions, the paper's improving-swap
// idea of Section 5.2 applied to the ordered list I') relative to the base order.  The move itself
// is never materialised as a permutation: the simulator maps positions through kv_map_pos().  What
// this file adds is the order in which candidates are handed to warps: a candidate only has to be
// simulated from its first moved position, so its cost is the length of the list suffix behind that
// position.  The 32 warps of a CTA run one candidate each and the CTA lasts as long as its longest
// one; candidates are therefore bucketed by first moved position (counting sort: histogram, scan,
// scatter) so that neighbours in launch order have (almost) equal suffix lengths and the longest
// candidates are launched first.  The order inside a bucket is arbitrary; results are written per
// candidate index, so they do not depend on it.
#pragma once

#include "common.cuh"

struct MoveSource {          // where candidate c's move comes from
    int mode;                // 0: codes[c]; 1: code = first + c; 2: sampled move m = first + c
    const i64* codes;
    i64 first;
    u64 seed;
    int iteration;
};

__device__ __forceinline__ Move k4_move_of(const MoveSource& src, int n, i64 c) {
    if (src.mode == 0) return kv_decode_move(n, src.codes[c]);
    if (src.mode == 1) return kv_decode_move(n, src.first + c);
    return kv_sample_move(n, src.seed, src.iteration, src.first + c);
}

__global__ void k4_first_pos_histogram(MoveSource src, int n, i64 count, int* __restrict__ bins,
                                       int* __restrict__ first_pos) {
    const i64 c = (i64)blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= count) return;
    const Move m = k4_move_of(src, n, c);
    int fp = min(m.i, m.j);
    if (fp < 0 || fp >= n) fp = n - 1;               // invalid code: the evaluator rejects it, any bucket will do
    first_pos[c] = fp;
    atomicAdd(&bins[KV_IDX(fp, n, 501)], 1);
}

// exclusive scan of bins[0..n) in place (one CTA; n is at most a few hundred thousand)
__global__ void __launch_bounds__(1024) k4_scan_bins(int* __restrict__ bins, int n) {
    __shared__ int warp_tot[32];
    __shared__ int carry;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    if (tid == 0) carry = 0;
    __syncthreads();
    for (int base = 0; base < n; base += 1024) {
        const int i = base + tid;
        const int v = i < n ? bins[i] : 0;
        int incl = v;
        for (int d = 1; d < 32; d <<= 1) {
            const int y = __shfl_up_sync(KV_FULL, incl, d);
            if (lane >= d) incl += y;
        }
        if (lane == 31) warp_tot[w] = incl;
        __syncthreads();
        int before = carry;
        for (int k = 0; k < w; ++k) before += warp_tot[k];
        if (i < n) bins[i] = before + incl - v;
        __syncthreads();
        if (tid == 1023) carry = before + incl;
        __syncthreads();
    }
}

__global__ void k4_scatter_by_first_pos(const int* __restrict__ first_pos, int n, i64 count, int* __restrict__ bins,
                                        int* __restrict__ launch_order) {
    const i64 c = (i64)blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= count) return;
    const int slot = atomicAdd(&bins[KV_IDX(first_pos[c], n, 502)], 1);
    launch_order[KV_IDX(slot, count, 503)] = (int)c;
}
