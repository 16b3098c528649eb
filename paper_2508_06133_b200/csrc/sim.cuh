// Warp-level schedule simulator: Phase 2 of Algorithm 1 (Appendix C) for one ordered list.
//
// One warp owns one candidate.  Its state is the per-round occupancy of the requests admitted so
// far, U[x] for rounds x >= t (x is 0-based: x = tau - 1 for the paper's round tau), kept in a ring
// of L int32 cells in shared memory, plus three scalars: t (the round index the next request may
// start at; a request starting at p = t is resident in cells t .. t+o-1), hz (all cells >= hz are
// zero) and the TEL accumulated so far.
//
// Admission of a request (s, o): it fits at start p iff U[x] + s + 1 + (x - p) <= M for every
// x in [p, p+o) -- the batch memory constraint of Section 2.1 in every round it is resident, which
// is what Algorithm 1's completion-time checks amount to because the occupancy of a fixed set of
// running requests only grows between completions.  Starts never go backwards along the list (a
// request that does not fit blocks everything behind it), so the start is the smallest p >= t
// that fits.  Nothing is admitted while the head is blocked, hence the timeline is constant during
// the search and p can be found by skipping: a violating cell x with excess e = v - M > 0 rules
// out every advance smaller than min(e, x - p + 1) (either the ramp has dropped by e or the window
// has moved past x); cells already checked stay fine when p grows, so only the cells that enter
// the window on the right are looked at again.
//
// Invariant: every cell of a round < t is zero, so a ring slot is clean when it is reused.
#pragma once

#include "common.cuh"

struct SimState {
    int t;       // next admissible start (0-based round index)
    int tr;      // t mod L
    int hz;      // cells of rounds >= hz are zero
    i64 tel;     // sum of completion times so far
};

__device__ __forceinline__ int kv_wrap(int idx, int L) {   // idx < 3L
    if (idx >= L) idx -= L;
    if (idx >= L) idx -= L;
    return idx;
}

// Admit one request; returns its start time.  All 32 lanes call this with identical arguments.
// The search loop is bounded: the advance can never exceed hz - t <= omax.
__device__ __forceinline__ int sim_admit(int* __restrict__ ring, int L, int M, SimState& st,
                                         int s, int o, int lane, int* status) {
    const int t = st.t, tr = st.tr;
    const int live = st.hz - t;          // cells at r >= live are zero
    int delta = 0, lo = 0, hi = o;
    for (int guard = 0;; ++guard) {
        int need = 0;
        const int hi_c = hi < live ? hi : live;
        for (int r = lo + lane; r < hi_c; r += 32) {
            int rel = r - delta;                         // offset inside the window starting at t+delta
            if (rel >= 0) {
                int e = ring[kv_wrap(tr + r, L)] + s + 1 + rel - M;
                if (e > 0) need = max(need, min(e, rel + 1));
            }
        }
        need = kv_warp_max(need);
        if (need == 0) break;
        delta += need;
        lo = hi;
        hi = o + delta;
        if (guard > L) { if (lane == 0) atomicExch(status, KV_DEV_LOOP_CAP); break; }
    }
    // rounds t .. t+delta-1 are over: clear their cells, then add the ramp s+1 .. s+o
    for (int r = lane; r < delta; r += 32) ring[kv_wrap(tr + r, L)] = 0;
    __syncwarp();
    for (int r = lane; r < o; r += 32) ring[kv_wrap(tr + delta + r, L)] += s + 1 + r;
    __syncwarp();
    const int p = t + delta;
    st.t = p;
    st.tr = kv_wrap(tr + delta, L);
    st.hz = max(st.hz, p + o);
    st.tel += p + o;
    return p;
}

__device__ __forceinline__ void sim_reset(int* ring, int L, SimState& st, int lane) {
    for (int r = lane; r < L; r += 32) ring[r] = 0;
    __syncwarp();
    st.t = 0; st.tr = 0; st.hz = 0; st.tel = 0;
}
