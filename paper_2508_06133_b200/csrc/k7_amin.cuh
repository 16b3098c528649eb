// K7 -- Sorted-F + A_min, Phase 2 (Section 5.5 "Handling Prediction Uncertainty via Adaptive Output
// Length Refinement"; Algorithm 5, the supplement to Section 5): the executor when only a lower bound l_i <= o_i of
// every decode length is known.  Many independent scenarios (a backlog, its list and one vector of
// lower bounds each), one CTA per scenario.
//
// Every request carries a running estimate e_i (initially l_i).  Iteration t = 1, 2, ...:
//   1. requests that have run their o_i rounds leave; every other running request is about to run
//      round number t - p_i, so e_i <- max(e_i, t - p_i);
//   2. the head of the pending queue (list order) starts, p = t - 1, iff the memory PROJECTED from
//      the estimates stays within M in every round >= t with it; the first refusal ends the round's
//      admissions (Algorithm 1, Phase 2, on the estimates);
//   3. while the projection exceeds M, the running request with the smallest estimate (ties: lower
//      request index) is evicted: it loses its progress, keeps its estimate and goes back to its
//      place in the list;
//   4. the round runs.
//
// How the kernel avoids touching every running request in every round.
//   occ[tau] is the projected memory of round tau: request j contributes s_j + (tau - p_j) for
//   tau in [p_j + 1, p_j + e_j].  A request whose estimate e (fixed at its admission) is below its
//   true length o is OVERDUE in rounds p+e+1 .. p+o: there its estimate is t - p, i.e. step 1 extends
//   its projection by exactly the current round.  The overdue requests are kept as two aggregates,
//   cnt = how many and A = sum of (s_j - p_j), so step 1 is occ[t] += A + cnt * t; a request joins the
//   aggregates at p+e+1 and leaves them at p+o+1 through per-round event cells (dc, dA) written when
//   it is admitted (and taken back if it is evicted).  A is kept modulo 2^32: the sum A + cnt * t is
//   a memory amount and fits, its two terms need not.  The estimate of a running request is never
//   stored: it is max(e at admission, t - p).
//   The projection is within M in every round >= t at the end of an iteration, so only step 1 can
//   break it, and only in round t: "the projection exceeds M" is occ[t] > M.
//   While the head of the queue is refused nothing is admitted and occ only grows, so the bound on
//   its wait that the window test gives (a cell over budget by x at offset r needs min(x, r+1) more
//   rounds) stays valid until the next eviction.  Rounds in which nothing can happen (no overflow;
//   head still bound to wait, or not even its first round fits) are walked by one warp, 32 rounds
//   per step (the running aggregates of a round are prefix sums of the event cells).
#pragma once

#include "common.cuh"

#define K7_THREADS 256
#define K7_MAX_N 4096
#define K7_MAX_O 8192
#define K7_ID_BITS 20

struct AminParams {
    int n_max;
    const int* n_each;           // [B]
    const int* s;                // [B, n_max] by request id
    const int* lower;
    const int* o;
    const int* order;            // [B, n_max] the list: request ids; or one row shared by all (order_stride 0)
    size_t order_stride;
    int M;
    int L;                       // ring length, a power of two >= the longest decode + 2
    int* start_out;              // [B, n_max] by request id
    i64* tel_out;                // [B] sum of (p + o)
    i64* evict_out;              // [B] evictions
    i64* peak_out;               // [B] largest memory actually in use in a round
    int* status;
};

enum { K7_ACT_WORK = 0, K7_ACT_DONE = 1, K7_ACT_CAP = 2 };

struct K7Ctl {
    int t, remaining, peak, act;
    unsigned cnt, A;
};

__device__ __forceinline__ int k7_block_max(int v, int* red) {
    const int tid = threadIdx.x;
    v = kv_warp_max(v);
    if ((tid & 31) == 0) red[tid >> 5] = v;
    __syncthreads();
    int r = red[0];
#pragma unroll
    for (int k = 1; k < K7_THREADS / 32; ++k) r = max(r, red[k]);
    __syncthreads();
    return r;
}
__device__ __forceinline__ int k7_block_min(int v, int* red) {
    const int tid = threadIdx.x;
    v = kv_warp_min(v);
    if ((tid & 31) == 0) red[tid >> 5] = v;
    __syncthreads();
    int r = red[0];
#pragma unroll
    for (int k = 1; k < K7_THREADS / 32; ++k) r = min(r, red[k]);
    __syncthreads();
    return r;
}
__device__ __forceinline__ u64 k7_block_min64(u64 v, u64* red) {
    const int tid = threadIdx.x;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) { const u64 w = __shfl_xor_sync(KV_FULL, v, d); v = w < v ? w : v; }
    if ((tid & 31) == 0) red[tid >> 5] = v;
    __syncthreads();
    u64 r = red[0];
#pragma unroll
    for (int k = 1; k < K7_THREADS / 32; ++k) r = red[k] < r ? red[k] : r;
    __syncthreads();
    return r;
}

__global__ void __launch_bounds__(K7_THREADS) k7_amin(const AminParams P) {
    extern __shared__ __align__(16) unsigned char k7_smem[];
    __shared__ K7Ctl ctl;
    __shared__ int red[K7_THREADS / 32];
    __shared__ u64 red64[K7_THREADS / 32];
    __shared__ u64 acc;
    const int tid = threadIdx.x;
    const int b = blockIdx.x;
    const int n = P.n_each[b];
    const int nm = P.n_max;
    // per list position: prefill, true length, estimate while pending, start (-1: pending), request id
    int* ps = reinterpret_cast<int*>(k7_smem);
    int* po = ps + nm;
    int* pe = po + nm;
    int* pp = pe + nm;
    int* pid = pp + nm;
    int* occ = pid + nm;                                          // projected memory per round
    int* dc = occ + P.L;                                          // change of cnt at the start of a round
    unsigned* dA = reinterpret_cast<unsigned*>(dc + P.L);         // change of A
    int* fin = reinterpret_cast<int*>(dA + P.L);                  // requests that leave at the start of a round

    const size_t base = (size_t)b * nm;
    const int* ord = P.order + (size_t)b * P.order_stride;
    if (tid == 0) acc = 0;
    __syncthreads();
    {
        u64 part = 0;
        bool bad = false;
        for (int q = tid; q < n; q += K7_THREADS) {
            const int id = ord[q];
            if (id < 0 || id >= n) { bad = true; continue; }      // never read outside the row
            ps[q] = P.s[base + id]; po[q] = P.o[base + id]; pe[q] = P.lower[base + id];
            pp[q] = -1; pid[q] = id;
            part += (u64)po[q];
        }
        for (int k = tid; k < P.L; k += K7_THREADS) { occ[k] = 0; dc[k] = 0; dA[k] = 0u; fin[k] = 0; }
        if (part) atomicAdd(&acc, part);
        if (__syncthreads_or(bad ? 1 : 0)) {
            if (tid == 0) atomicExch(P.status, KV_DEV_LOOP_CAP);
            return;
        }
    }
    const i64 sum_o = (i64)acc;
    __syncthreads();
    i64 round_cap = 16 + sum_o * (i64)(n + 1);
    if (round_cap > (1ll << 30)) round_cap = 1ll << 30;           // t stays a 32-bit round index
    const i64 turn_cap = round_cap;

    const int mask = P.L - 1;
    const int M = P.M;
    int t = 1, remaining = n, peak = 0;
    unsigned cnt = 0, A = 0;
    int head = 0, frontier = 0, npe = 0;     // first pending position; first never-started one; pending ones below it
    int t_ok = 1;                            // the head cannot start in an iteration before this one
    i64 evictions = 0;
    bool failed = false;

    for (i64 turn = 0;; ++turn) {
        if (turn > turn_cap) { failed = true; break; }
        if (tid < 32) {
            // rounds in which nothing can be decided (step 1 only), 32 at a time: lane l takes round
            // t + l.  A round reads only its own cells and the running (cnt, A, remaining), which are
            // prefix sums of the event cells, so the 32 rounds are evaluated together and the walk
            // stops at the first lane whose round needs the whole CTA (or ends the run).
            const int lane = tid;
            int act = K7_ACT_WORK;
            const int head_s = head < n ? ps[head] : 0;
            for (;;) {
                const int tau = t + lane;
                const int k = tau & mask;
                int cs = dc[k];
                unsigned as = dA[k];
                int fs = fin[k];
                const int oc = occ[k];
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const int c2 = __shfl_up_sync(KV_FULL, cs, d);
                    const unsigned a2 = __shfl_up_sync(KV_FULL, as, d);
                    const int f2 = __shfl_up_sync(KV_FULL, fs, d);
                    if (lane >= d) { cs += c2; as += a2; fs += f2; }
                }
                const unsigned cnt_l = cnt + (unsigned)cs, A_l = A + as;
                const int rem_l = remaining - fs;
                const int u = oc + (int)(A_l + cnt_l * (unsigned)tau);
                const bool done = rem_l == 0;
                // the head's first round is the current one: if it does not fit there, the window
                // test cannot succeed in this iteration and the CTA need not be woken for it
                const bool work = u > M || (head < n && tau >= t_ok && u + head_s + 1 <= M);
                const bool cap = (i64)tau >= round_cap;
                const unsigned stops = __ballot_sync(KV_FULL, done || work || cap);
                const int first = stops ? __ffs(stops) - 1 : 32;
                if (lane <= first) { dc[k] = 0; dA[k] = 0u; fin[k] = 0; }          // events consumed
                if (lane < first) occ[k] = 0;                                        // a round that is over
                else if (lane == first) occ[k] = u;
                peak = max(peak, kv_warp_max(lane < first ? u : 0));
                const int src = first < 32 ? first : 31;
                cnt = __shfl_sync(KV_FULL, cnt_l, src);
                A = __shfl_sync(KV_FULL, A_l, src);
                remaining = __shfl_sync(KV_FULL, rem_l, src);
                if (first < 32) {
                    t += first;
                    const int why = done ? K7_ACT_DONE : (work ? K7_ACT_WORK : K7_ACT_CAP);
                    act = __shfl_sync(KV_FULL, why, first);
                    break;
                }
                t += 32;
            }
            if (lane == 0) { ctl.t = t; ctl.remaining = remaining; ctl.peak = peak; ctl.act = act; ctl.cnt = cnt; ctl.A = A; }
        }
        __syncthreads();
        t = ctl.t; remaining = ctl.remaining; peak = ctl.peak; cnt = ctl.cnt; A = ctl.A;
        const int act = ctl.act;
        __syncthreads();
        if (act == K7_ACT_DONE) break;
        if (act == K7_ACT_CAP) { failed = true; break; }

        // ---- step 2: admissions of iteration t
        if (head < n && t >= t_ok) {
            for (;;) {
                const int q = head;
                const int s = ps[q], o = po[q], e = pe[q];
                int need = INT_MIN;
                for (int x = tid; x < e; x += K7_THREADS) {
                    const int over = occ[(t + x) & mask] + s + 1 + x - M;
                    need = max(need, min(over, x + 1));
                }
                need = k7_block_max(need, red);
                if (need > 0) { t_ok = t + need; break; }
                for (int x = tid; x < e; x += K7_THREADS) occ[(t + x) & mask] += s + 1 + x;
                if (tid == 0) {
                    pp[q] = t - 1;
                    if (e < o) {                                   // overdue in rounds t+e .. t+o-1
                        const unsigned v = (unsigned)(s - (t - 1));
                        dc[(t + e) & mask] += 1; dA[(t + e) & mask] += v;
                        dc[(t + o) & mask] -= 1; dA[(t + o) & mask] -= v;
                    }
                    fin[(t + o) & mask] += 1;
                }
                if (q == frontier) ++frontier; else --npe;
                if (npe == 0) {
                    head = frontier;
                    __syncthreads();
                } else {                                           // an evicted request further down the list
                    int first = INT_MAX;
                    for (int k = q + 1 + tid; k < frontier; k += K7_THREADS)
                        if (pp[k] < 0) { first = k; break; }
                    head = k7_block_min(first, red);
                    if (head == INT_MAX) { failed = true; break; }
                }
                if (head >= n) break;
            }
            if (failed) break;
        }
        __syncthreads();

        // ---- step 3: ordered eviction while round t is over budget
        while (occ[t & mask] > M) {
            u64 best = ~0ull;
            for (int q = tid; q < frontier; q += K7_THREADS) {
                const int p = pp[q];
                if (p >= 0 && t <= p + po[q]) {
                    const int est = max(pe[q], t - p);
                    const u64 key = ((u64)(unsigned)est << (2 * K7_ID_BITS)) | ((u64)(unsigned)pid[q] << K7_ID_BITS) | (u64)(unsigned)q;
                    best = key < best ? key : best;
                }
            }
            best = k7_block_min64(best, red64);
            if (best == ~0ull) { failed = true; break; }
            const int q = (int)(best & ((1u << K7_ID_BITS) - 1));
            const int est = (int)(best >> (2 * K7_ID_BITS));
            const int p = pp[q], s = ps[q], o = po[q], e0 = pe[q];
            const int cells = p + est - t + 1;                     // what is left of its projection
            for (int x = tid; x < cells; x += K7_THREADS) occ[(t + x) & mask] -= s + (t + x - p);
            const unsigned v = (unsigned)(s - p);
            const bool overdue = e0 < o && t >= p + e0 + 1;
            if (overdue) { cnt -= 1u; A -= v; }
            __syncthreads();
            if (tid == 0) {
                if (e0 < o) {
                    if (!overdue) { dc[(p + e0 + 1) & mask] -= 1; dA[(p + e0 + 1) & mask] -= v; }
                    dc[(p + o + 1) & mask] += 1; dA[(p + o + 1) & mask] += v;
                }
                fin[(p + o + 1) & mask] -= 1;
                pe[q] = est;
                pp[q] = -1;
            }
            ++evictions; ++npe;
            head = min(head, q);
            t_ok = t + 1;
            __syncthreads();
        }
        if (failed) break;

        // ---- step 4: the round runs
        const int used = occ[t & mask];
        __syncthreads();
        peak = max(peak, used);
        if (tid == 0) occ[t & mask] = 0;
        ++t;
    }
    if (failed) {
        if (tid == 0) atomicExch(P.status, KV_DEV_LOOP_CAP);
        return;
    }
    if (tid == 0) acc = 0;
    __syncthreads();
    u64 part = 0;
    for (int q = tid; q < n; q += K7_THREADS) {
        P.start_out[base + KV_IDX(pid[q], n, 1101)] = pp[q];
        part += (u64)((i64)pp[q] + po[q]);
    }
    if (part) atomicAdd(&acc, part);
    __syncthreads();
    if (tid == 0) { P.tel_out[b] = (i64)acc; P.evict_out[b] = evictions; P.peak_out[b] = peak; }
}
