// K2c -- Algorithm 2 (exact dynamic programme, Section 5.1 / the supplement to Section 5) as the Phase-1 solver.
//
//   dp[k][m] = min { sum of o over X : |X| = k, sum of (s+o) over X = m },   m <= M,
// built by taking the remaining requests one at a time (ascending index); a cell is overwritten only
// by a strictly smaller value, as in the printed listing.  The listing walks k downwards in place so
// that a request is used at most once; here every request is one launch that reads the previous
// table and writes the next one (same values: row k+1 only ever reads row k as it was before the
// request).  Instead of the listing's path sets, one bit per (request, k, m) records whether that
// request overwrote the cell; walking the requests backwards from the chosen cell reproduces exactly
// the set the listing's path[k][m] would hold.  The batch is the cell with the smallest
// F = dp[k][m] / k^2 (compared exactly as dp_a * k_b^2 < dp_b * k_a^2), ties to the larger k
// (Section 3), then to the smaller m.
#pragma once

#include "common.cuh"

#define K2D_INF 0x7fffffff

__global__ void k2d_init(int* __restrict__ dp, i64 cells) {
    const i64 i = (i64)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < cells) dp[i] = i == 0 ? 0 : K2D_INF;
}

// One request, the a-th of the remaining list (size mi = s+o, output oi).  Thread = 32 consecutive
// m of one row k.
// took: bit (k * words + w) * 32 + b of this request's slab.
__global__ void k2d_step(const int* __restrict__ old_dp, int* __restrict__ new_dp, unsigned* __restrict__ took,
                         int rows, int W /* M + 1 */, int words, const int* __restrict__ s, const int* __restrict__ o,
                         const int* __restrict__ rem, int a) {
    const i64 t = (i64)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= (i64)rows * words) return;
    const int id = rem[a];
    const int oi = o[id], mi = s[id] + oi;
    const int k = (int)(t / words), w = (int)(t % words);
    unsigned bits = 0;
    for (int b = 0; b < 32; ++b) {
        const int m = w * 32 + b;
        if (m >= W) break;
        const int cur = old_dp[(i64)k * W + m];
        int nv = cur;
        if (k >= 1 && m >= mi) {
            const int src = old_dp[(i64)(k - 1) * W + (m - mi)];
            if (src != K2D_INF && src + oi < cur) { nv = src + oi; bits |= 1u << b; }
        }
        new_dp[(i64)k * W + m] = nv;
    }
    took[t] = bits;
}

// best cell by (F ascending, k descending, m ascending); one CTA.  out = {k, m, value}.
__device__ __forceinline__ bool k2d_better(int va, int ka, int ma, int vb, int kb, int mb) {
    if (kb == 0) return ka != 0;
    if (ka == 0) return false;
    const i64 l = (i64)va * kb * kb, r = (i64)vb * ka * ka;
    if (l != r) return l < r;
    if (ka != kb) return ka > kb;
    return ma < mb;
}

__global__ void __launch_bounds__(1024) k2d_select(const int* __restrict__ dp, int rows, int W, int* __restrict__ out) {
    __shared__ int sv[32], sk[32], sm[32];
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    int bv = 0, bk = 0, bm = 0;
    const i64 cells = (i64)rows * W;
    for (i64 i = (i64)W + tid; i < cells; i += 1024) {          // rows k >= 1
        const int v = dp[i];
        if (v == K2D_INF) continue;
        const int k = (int)(i / W), m = (int)(i % W);
        if (k2d_better(v, k, m, bv, bk, bm)) { bv = v; bk = k; bm = m; }
    }
    for (int d = 16; d >= 1; d >>= 1) {
        const int ov = __shfl_xor_sync(KV_FULL, bv, d), ok = __shfl_xor_sync(KV_FULL, bk, d), om = __shfl_xor_sync(KV_FULL, bm, d);
        if (k2d_better(ov, ok, om, bv, bk, bm)) { bv = ov; bk = ok; bm = om; }
    }
    if (lane == 0) { sv[w] = bv; sk[w] = bk; sm[w] = bm; }
    __syncthreads();
    if (tid == 0) {
        for (int x = 1; x < 32; ++x) if (k2d_better(sv[x], sk[x], sm[x], bv, bk, bm)) { bv = sv[x]; bk = sk[x]; bm = sm[x]; }
        out[0] = bk; out[1] = bm; out[2] = bv;
    }
}

// Walk the requests backwards from the chosen cell, hand the batch out (ascending index; the caller
// sorts each batch by (o, index)) and compact the remaining list.  One CTA of 128 threads; nr <= 128.
__global__ void __launch_bounds__(128)
k2d_apply(const int* __restrict__ s, const int* __restrict__ o, const unsigned* __restrict__ took, int W, int words,
          int rows, const int* __restrict__ pick, int* __restrict__ rem, int* __restrict__ nr_io,
          int* __restrict__ order_out, int* __restrict__ batch_off, int* __restrict__ nb_io, int* __restrict__ done_io) {
    __shared__ int chosen[128];
    __shared__ int ids[128];
    const int tid = threadIdx.x;
    const int nr = *nr_io;
    if (tid < nr) { ids[tid] = rem[tid]; chosen[tid] = 0; }
    __syncthreads();
    if (tid == 0) {
        int k = pick[0], m = pick[1];
        for (int a = nr - 1; a >= 0 && k > 0; --a) {
            const i64 slab = (i64)a * rows * words;
            const unsigned bits = took[slab + (i64)k * words + (m >> 5)];
            if ((bits >> (m & 31)) & 1u) {
                chosen[a] = 1;
                k -= 1;
                m -= s[ids[a]] + o[ids[a]];
            }
        }
        int done = *done_io, left = 0;
        for (int a = 0; a < nr; ++a) {
            if (chosen[a]) order_out[done++] = ids[a];
            else rem[left++] = ids[a];
        }
        const int nb = *nb_io + 1;
        batch_off[nb] = done;
        *nb_io = nb; *done_io = done; *nr_io = left;
    }
}
