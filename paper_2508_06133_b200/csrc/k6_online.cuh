// K6 -- online arrivals (Section 6.2 "Heuristics under Online Arrival"; Section 7, "Experiment under
// Online Poisson Arrivals"): many independent arrival streams, one CTA each, one policy per launch.
//
// Model.  Request i arrives at the integer time a_i >= 0 (non-decreasing in i) and may start at any
// p_i >= a_i: it is first seen by iteration a_i + 1.  In iteration t the policy orders the pending
// requests and the executor admits the longest prefix of that order that fits the live memory
// profile (Algorithm 1, Phase 2: stop at the first request that does not fit).
//   FCFS            arrival order;
//   SOF             ascending (o, index), recomputed every iteration;
//   Sorted-F-Online a cached priority list: arrivals go to its tail; it is planned again when it has
//                   never been planned, `period` iterations after the last plan, when it had run
//                   empty, or when the arrivals since the last plan reach half of the backlog at
//                   that plan.  A plan sorts the pending requests by ascending (s+o, index), orders
//                   the first `lookahead` of them by Sorted-F with Algorithm 3 (batch after batch,
//                   every batch by ascending (o, index)) and lets the others follow in sorted order.
//
// The iterations are not walked one by one.  Nothing changes between two iterations unless a
// request arrives, a plan is due, or the head of the list starts; while the head is refused, the
// window test yields the same lower bound on the wait as in the offline simulator (a cell over
// budget by e at offset r needs min(e, r+1) more rounds), so the loop jumps to the earliest of:
// that bound, the next arrival, the next due plan.
//
// Memory profile: a ring of L >= o_max rounds in shared memory, cell (tau mod L) = tokens in use in
// round tau for tau in [t, t + L); rounds that are over are cleared when t moves.
#pragma once

#include "common.cuh"
#include "k2_local_swap.cuh"

#define K6_THREADS K2L_THREADS
#define K6_MAX_N 2048            // requests per stream
#define K6_MAX_LOOKAHEAD 1024
#define K6_MAX_O 8192
#define K6_IDX_BITS 12           // (o << 12) | index fits 32 bits for o <= 2^14, index < 2^12

struct OnlineParams {
    int n_max;
    const int* n_each;           // [B]
    const int* a;                // [B, n_max]
    const int* s;
    const int* o;
    int M;
    int policy, period, lookahead;
    int L;                       // ring length, a power of two >= the longest decode
    int npow2;                   // power of two >= n_max
    int* start_out;              // [B, n_max]
    i64* latency_out;            // [B]  sum of (p + o - a)
    int* status;
};

struct K6Shared {
    K2lShared ls;
    int red[32];
};

__device__ __forceinline__ int k6_block_max(int v, int* red) {
    const int tid = threadIdx.x;
    v = kv_warp_max(v);
    if ((tid & 31) == 0) red[tid >> 5] = v;
    __syncthreads();
    int r = red[0];
    for (int k = 1; k < K6_THREADS / 32; ++k) r = max(r, red[k]);
    __syncthreads();
    return r;
}
__device__ __forceinline__ int k6_block_min(int v, int* red) {
    const int tid = threadIdx.x;
    v = kv_warp_min(v);
    if ((tid & 31) == 0) red[tid >> 5] = v;
    __syncthreads();
    int r = red[0];
    for (int k = 1; k < K6_THREADS / 32; ++k) r = min(r, red[k]);
    __syncthreads();
    return r;
}

// ascending bitonic sort of keys[0 .. len), len a power of two, by all threads of the CTA
__device__ void k6_bitonic_sort(u64* keys, int len) {
    const int tid = threadIdx.x;
    for (int size = 2; size <= len; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            for (int k = tid; k < (len >> 1); k += K6_THREADS) {
                const int lo = ((k / stride) * (stride << 1)) + (k % stride);
                const int hi = lo + stride;
                const bool up = ((lo & size) == 0);
                const u64 x = keys[lo], y = keys[hi];
                if ((x > y) == up) { keys[lo] = y; keys[hi] = x; }
            }
            __syncthreads();
        }
    }
}

// Smallest wait (in iterations) that the window of (s, o) at iteration t asks for; <= 0: it fits.
__device__ __forceinline__ int k6_window_need(const int* ring, int mask, int t, int s, int o, int M, int* red) {
    int need = INT_MIN;
    for (int x = threadIdx.x; x < o; x += K6_THREADS) {
        const int e = ring[(t + x) & mask] + s + 1 + x - M;
        need = max(need, min(e, x + 1));
    }
    return k6_block_max(need, red);
}

__global__ void __launch_bounds__(K6_THREADS) k6_online(const OnlineParams P) {
    extern __shared__ __align__(16) unsigned char k6_smem[];
    __shared__ K6Shared sh;
    const int tid = threadIdx.x;
    const int b = blockIdx.x;
    const int n = P.n_each[b];
    const int W = P.lookahead;
    // dynamic shared memory: sort keys first (8-byte aligned), then the int arrays
    u64* keys = reinterpret_cast<u64*>(k6_smem);
    int* sa = reinterpret_cast<int*>(keys + P.npow2);
    int* ss = sa + P.n_max;
    int* so = ss + P.n_max;
    int* ring = so + P.n_max;
    int* C = ring + P.L;                 // Sorted-F-Online: the cached list; SOF: started flags
    int* C2 = C + P.n_max;
    int* win = C2 + P.n_max;             // 9 arrays of `lookahead` ints for Algorithm 3
    int* removed = win + W;
    int* rem = removed + W;
    int* remT = rem + W;
    int* remO = remT + W;
    int* inX = remO + W;
    int* pm = inX + W;
    int* xpos = pm + W;
    int* bout = xpos + W;

    const size_t base = (size_t)b * P.n_max;
    i64 horizon = 2;
    for (int i = tid; i < n; i += K6_THREADS) {
        sa[i] = P.a[base + i]; ss[i] = P.s[base + i]; so[i] = P.o[base + i];
        C[i] = 0;
    }
    for (int k = tid; k < P.L; k += K6_THREADS) ring[k] = 0;
    __syncthreads();
    for (int i = 0; i < n; ++i) horizon += so[i];      // same in every thread
    horizon += sa[n - 1];
    const i64 turn_cap = 4 * (horizon + n) + 64;       // every turn is an arrival, a plan or a wait that ends

    const int mask = P.L - 1;
    const int M = P.M;
    int t = 1, nvis = 0, remaining = n;
    int fcfs_next = 0;                                  // FCFS: next request in arrival order
    int ch = 0, ce = 0;                                 // Sorted-F-Online: pending = C[ch .. ce)
    bool computed = false;
    int t_last = 0, backlog_last = 0, new_since = 0;
    bool changed = true;                                // pending set differs from the one last planned
    i64 latency = 0;

    for (i64 turn = 0; remaining > 0; ++turn) {
        if (turn > kv_loop_cap(turn_cap)) { if (tid == 0) atomicExch(P.status, KV_DEV_LOOP_CAP); break; }
        // arrivals seen by iteration t
        const int old = nvis;
        while (nvis < n && sa[nvis] <= t - 1) ++nvis;
        const int newly = nvis - old;
        if (P.policy == SCHED_POLICY_SORTED_F) {
            const bool was_empty = (ce == ch);
            for (int k = tid; k < newly; k += K6_THREADS) C[ce + k] = old + k;
            ce += newly;
            new_since += newly;
            __syncthreads();
            if (newly > 0) changed = true;
            const bool due = ce > ch && (!computed || t - t_last >= P.period || was_empty || 2 * new_since >= backlog_last);
            if (due && !changed) {
                // same pending set as at the last plan (no arrival, no start since): the plan is a
                // function of that set alone, so it would come out as the list already is
                t_last = t;
            } else if (due) {
                // ---- plan: pending by ascending (s+o, index)
                const int m = ce - ch;
                int len = 2;
                while (len < m) len <<= 1;
                for (int k = tid; k < len; k += K6_THREADS) {
                    u64 key = ~0ull;
                    if (k < m) { const int id = C[ch + k]; key = ((u64)(unsigned)(ss[id] + so[id]) << 32) | (u64)(unsigned)id; }
                    keys[k] = key;
                }
                __syncthreads();
                k6_bitonic_sort(keys, len);
                const int wn = m < W ? m : W;
                for (int k = tid; k < wn; k += K6_THREADS) { win[k] = (int)(keys[k] & 0xffffffffu); removed[k] = 0; }
                __syncthreads();
                int done = 0;
                while (done < wn) {                     // every batch places at least one request
                    const int k0 = k2l_batch(ss, so, win, wn, (i64)M, 0, 1, removed, rem, remT, remO, inX, pm, xpos,
                                             bout, P.status, sh.ls);
                    if (k0 < 1) { if (tid == 0) atomicExch(P.status, KV_DEV_LOOP_CAP); done = wn; break; }
                    // the batch by ascending (o, index): rank of every member among the members
                    for (int k = tid; k < k0; k += K6_THREADS) {
                        const int id = bout[k];
                        const int key = (so[id] << K6_IDX_BITS) | id;
                        int rank = 0;
                        for (int j = 0; j < k0; ++j) { const int jd = bout[j]; rank += (((so[jd] << K6_IDX_BITS) | jd) < key) ? 1 : 0; }
                        C2[done + rank] = id;
                    }
                    done += k0;
                    __syncthreads();
                }
                for (int k = wn + tid; k < m; k += K6_THREADS) C2[k] = (int)(keys[k] & 0xffffffffu);
                __syncthreads();
                for (int k = tid; k < m; k += K6_THREADS) C[k] = C2[k];
                __syncthreads();
                ch = 0; ce = m;
                computed = true; t_last = t; backlog_last = m; new_since = 0;
                changed = false;
            }
        }
        // ---- admission: the longest prefix of the list that fits
        int r = -1, need = 0;
        for (;;) {
            if (P.policy == SCHED_POLICY_FCFS) {
                r = fcfs_next < nvis ? fcfs_next : -1;
            } else if (P.policy == SCHED_POLICY_SOF) {
                int best = INT_MAX;
                for (int i = tid; i < nvis; i += K6_THREADS)
                    if (!C[i]) best = min(best, (so[i] << K6_IDX_BITS) | i);
                best = k6_block_min(best, sh.red);
                r = best == INT_MAX ? -1 : (best & ((1 << K6_IDX_BITS) - 1));
            } else {
                r = ch < ce ? C[ch] : -1;
            }
            if (r < 0) break;
            const int s = ss[r], o = so[r];
            need = k6_window_need(ring, mask, t, s, o, M, sh.red);
            if (need > 0) break;
            for (int x = tid; x < o; x += K6_THREADS) ring[(t + x) & mask] += s + 1 + x;
            if (tid == 0) P.start_out[base + KV_IDX(r, n, 1001)] = t - 1;
            latency += (i64)(t - 1) + o - sa[r];
            --remaining;
            if (P.policy == SCHED_POLICY_FCFS) ++fcfs_next;
            else if (P.policy == SCHED_POLICY_SOF) { if (tid == 0) C[r] = 1; }
            else { ++ch; changed = true; }
            __syncthreads();
        }
        if (remaining == 0) break;
        // ---- the next iteration at which anything can change
        i64 t_next;
        if (r < 0) {
            t_next = (i64)sa[nvis] + 1;                 // nothing pending: wait for the next arrival
        } else {
            t_next = (i64)t + need;
            if (nvis < n) t_next = min(t_next, (i64)sa[nvis] + 1);
            if (P.policy == SCHED_POLICY_SORTED_F) t_next = min(t_next, (i64)t_last + P.period);
        }
        const int d = (int)(t_next - t);
        for (int k = tid; k < min(d, P.L); k += K6_THREADS) ring[(t + k) & mask] = 0;
        t = (int)t_next;
        __syncthreads();
    }
    if (tid == 0) P.latency_out[b] = latency;
}
