// Warp-level schedule simulator: Phase 2 of Algorithm 1 (Appendix C) for one ordered list.
//
// One warp owns one candidate.  Its state is the per-round occupancy of the requests admitted so
// far, kept for the rounds x >= t (x is 0-based: x = tau - 1 for the paper's round tau) in a ring
// of L int32 cells in shared memory, plus three scalars: t (the round index the next request may
// start at; a request starting at p = t is resident in cells t .. t+o-1), hz (no admitted request
// is resident in a round >= hz) and the TEL accumulated so far.
//
// Cell encoding.  The ring does not hold the occupancy U[x] itself but V[x] = U[x] + x.  A request
// (s, o) that starts at p uses s + 1 + (x - p) tokens in round x (Section 2.1: token j needs s + j),
// so with V the test loses its per-cell term:
//     fits at p   <=>   U[x] + s + 1 + (x - p) <= M  for x in [p, p+o)
//                 <=>   max_{x in [p, p+o)} V[x]  <=  M - s - 1 + p            (one max-scan)
//     admit at p  :     V[x] += s + 1 + (x - p)      for x in [p, p+o)          (ramp add)
// A cell that no request occupies holds its own round index x; when round x is over its slot is
// handed to round x + L by writing x + L.  (V < 2^31 because M < 2^30 and sum(o) + max(o) < 2^30.)
//
// Admission rule.  The request fits iff the batch memory constraint of Section 2.1 holds in every
// round it is resident -- what Algorithm 1's completion-time checks amount to, because the
// occupancy of a fixed set of running requests only grows between completions.  Starts never go
// backwards along the list (a request that does not fit blocks everything behind it), so the start
// is the smallest p >= t that fits.  Nothing is admitted while the head is blocked, hence the
// timeline is constant during the search and p is found by skipping: a violating cell with excess
// e > 0 at offset r from the window start rules out every advance smaller than min(e, r + 1)
// (either the ramp has dropped by e or the window has moved past the cell); cells already checked
// stay fine when p grows, so only the cells that enter the window on the right are looked at again.
//
// Two code shapes with identical results:
//   sim_admit<NIT>, NIT >= 1: the window (<= 128*NIT - 6 cells) is loaded once with 16-byte shared
//     loads into registers, checked, and written back -- one read and one write per cell;
//   sim_admit<0>: any window length, cells are re-read by the write pass.
#pragma once

#include "common.cuh"

struct SimState {
    int t;       // next admissible start (0-based round index)
    int tr;      // t mod L
    int hz;      // no admitted request is resident in a round >= hz
    i64 tel;     // sum of completion times so far
};

__device__ __forceinline__ int kv_wrap(int idx, int L) {   // idx < 3L
    if (idx >= L) idx -= L;
    if (idx >= L) idx -= L;
    return idx;
}

__device__ __forceinline__ int kv_wrap1(int idx, int L) {  // idx < 2L
    return idx >= L ? idx - L : idx;
}

__device__ __forceinline__ void sim_reset(int* ring, int L, SimState& st, int lane) {
    for (int r = lane; r < L; r += 32) ring[r] = r;        // empty cells hold their round index
    __syncwarp();
    st.t = 0; st.tr = 0; st.hz = 0; st.tel = 0;
}

// ---- slow part of an admission whose first test failed: finish the search for the start, release
//      the rounds that are over and add the ramp to the cells beyond the old window.
//      `delta` is the advance already implied by the cells of [t, t+o).  Returns the final advance.
__device__ __forceinline__ int sim_search_beyond(int* __restrict__ ring, int L, int t, int tr, int live,
                                                 int o, int kadm, int delta, int lane, int* status) {
    int lo = o, hi = o + delta;
    for (int guard = 0;; ++guard) {
        int nd = 0;
        const int hi_c = hi < live ? hi : live;              // cells at r >= live are empty: never in the way
        for (int r = lo + lane; r < hi_c; r += 32) {
            const int rel = r - delta;
            if (rel >= 0) {
                const int e = ring[kv_wrap1(tr + r, L)] + kadm - delta;
                if (e > 0) nd = max(nd, min(e, rel + 1));
            }
        }
        nd = kv_warp_max(nd);
        if (nd == 0) break;
        delta += nd;
        lo = hi;
        hi = o + delta;
        if (guard > L) { if (lane == 0) atomicExch(status, KV_DEV_LOOP_CAP); break; }
    }
    return delta;
}

__device__ __forceinline__ void sim_finish_beyond(int* __restrict__ ring, int L, int t, int tr,
                                                  int o, int kw, int delta, int lane) {
    // cells r in [o, o+delta): rounds < t+delta are over, the others join the new window
    for (int r = o + lane; r < delta; r += 32) ring[kv_wrap(tr + r, L)] = t + L + r;
    __syncwarp();
    const int from = o > delta ? o : delta;
    for (int r = from + lane; r < o + delta; r += 32) ring[kv_wrap(tr + r, L)] += kw + r - delta;
}

// Admit one request; returns its start time.  All 32 lanes call this with identical arguments.
template <int NIT>
__device__ __forceinline__ int sim_admit(int* __restrict__ ring, int L, int M, SimState& st,
                                         int s, int o, int lane, int* status) {
    const int t = st.t, tr = st.tr;
    const int m = tr & 3, ar = tr - m;               // L is a multiple of 4: t and tr agree mod 4
    const int span = m + o;                          // cells from the aligned start to the window end
    const int nit = (span + 127) >> 7;               // 16-byte groups: 32 lanes x 4 cells per round
    const int kadm = s + 1 - M - t;                  // V + kadm > 0  <=>  the cell is over budget
    const int kw = s + 1;                            // ramp value at the window start
    const int g4l = lane << 2;
    int delta = 0;

    if (NIT > 0) {
        int4 buf[NIT > 0 ? NIT : 1];
        int vmax = -1;
#pragma unroll
        for (int it = 0; it < NIT; ++it) {
            if (it >= nit) break;
            const int g4 = g4l + (it << 7);
            int4 v = make_int4(-1, -1, -1, -1);
            if (g4 < span) v = *reinterpret_cast<const int4*>(ring + kv_wrap1(ar + g4, L));
            buf[it] = v;
            const int lim = span - g4;               // cells c >= lim are past the window end
            const int mm = it == 0 ? m - g4 : 0;     // cells c < mm are before the window start
            if (it == 0) { if (0 < mm) v.x = -1; if (1 < mm) v.y = -1; if (2 < mm) v.z = -1; }
            if (it == nit - 1) { if (lim < 4) { v.w = -1; if (lim < 3) v.z = -1; if (lim < 2) v.y = -1; if (lim < 1) v.x = -1; } }
            vmax = max(max(vmax, max(v.x, v.y)), max(v.z, v.w));
        }
        vmax = kv_warp_max(vmax);
        if (vmax + kadm > 0) {
            // blocked: advance implied by the cells of the window
            int need = 0;
#pragma unroll
            for (int it = 0; it < NIT; ++it) {
                if (it >= nit) break;
                const int r0 = g4l + (it << 7) - m;
                const int4 v = buf[it];
                if ((unsigned)(r0 + 0) < (unsigned)o) need = max(need, min(v.x + kadm, r0 + 1));
                if ((unsigned)(r0 + 1) < (unsigned)o) need = max(need, min(v.y + kadm, r0 + 2));
                if ((unsigned)(r0 + 2) < (unsigned)o) need = max(need, min(v.z + kadm, r0 + 3));
                if ((unsigned)(r0 + 3) < (unsigned)o) need = max(need, min(v.w + kadm, r0 + 4));
            }
            delta = kv_warp_max(need);
            delta = sim_search_beyond(ring, L, t, tr, st.hz - t, o, kadm, delta, lane, status);
            const int kwd = kw - delta, dead = t + L;
#pragma unroll
            for (int it = 0; it < NIT; ++it) {
                if (it >= nit) break;
                const int g4 = g4l + (it << 7), r0 = g4 - m;
                if (g4 < span) {
                    int4 v = buf[it];
                    if ((unsigned)(r0 + 0) < (unsigned)o) v.x = r0 + 0 >= delta ? v.x + kwd + r0 + 0 : dead + r0 + 0;
                    if ((unsigned)(r0 + 1) < (unsigned)o) v.y = r0 + 1 >= delta ? v.y + kwd + r0 + 1 : dead + r0 + 1;
                    if ((unsigned)(r0 + 2) < (unsigned)o) v.z = r0 + 2 >= delta ? v.z + kwd + r0 + 2 : dead + r0 + 2;
                    if ((unsigned)(r0 + 3) < (unsigned)o) v.w = r0 + 3 >= delta ? v.w + kwd + r0 + 3 : dead + r0 + 3;
                    *reinterpret_cast<int4*>(ring + kv_wrap1(ar + g4, L)) = v;
                }
            }
            __syncwarp();
            sim_finish_beyond(ring, L, t, tr, o, kw, delta, lane);
        } else {
#pragma unroll
            for (int it = 0; it < NIT; ++it) {
                if (it >= nit) break;
                const int g4 = g4l + (it << 7);
                if (g4 < span) {
                    int4 v = buf[it];
                    const int lim = span - g4;
                    const int mm = it == 0 ? m - g4 : 0;
                    const int kr = kw + g4 - m;      // ramp value of this group's first cell
                    int ax = kr, ay = kr + 1, az = kr + 2, aw = kr + 3;
                    if (it == 0) { if (0 < mm) ax = 0; if (1 < mm) ay = 0; if (2 < mm) az = 0; }
                    if (it == nit - 1) { if (lim < 4) { aw = 0; if (lim < 3) az = 0; if (lim < 2) ay = 0; } }
                    v.x += ax; v.y += ay; v.z += az; v.w += aw;
                    *reinterpret_cast<int4*>(ring + kv_wrap1(ar + g4, L)) = v;
                }
            }
        }
    } else {
        // streamed form: same arithmetic, cells re-read instead of cached
        int vmax = -1;
        for (int r = lane; r < o; r += 32) vmax = max(vmax, ring[kv_wrap1(tr + r, L)]);
        vmax = kv_warp_max(vmax);
        if (vmax + kadm > 0) {
            int need = 0;
            for (int r = lane; r < o; r += 32) need = max(need, min(ring[kv_wrap1(tr + r, L)] + kadm, r + 1));
            delta = kv_warp_max(need);
            delta = sim_search_beyond(ring, L, t, tr, st.hz - t, o, kadm, delta, lane, status);
            for (int r = lane; r < o; r += 32) {
                const int idx = kv_wrap1(tr + r, L);
                ring[idx] = r >= delta ? ring[idx] + kw + r - delta : t + L + r;
            }
            __syncwarp();
            sim_finish_beyond(ring, L, t, tr, o, kw, delta, lane);
        } else {
            for (int r = lane; r < o; r += 32) ring[kv_wrap1(tr + r, L)] += kw + r;
        }
    }
    __syncwarp();
    const int p = t + delta;
    st.t = p;
    st.tr = kv_wrap(tr + delta, L);
    st.hz = max(st.hz, p + o);
    st.tel += p + o;
    return p;
}

// Number of 128-cell rounds a handle's longest window needs (0: use the streamed form).
static inline int sim_pick_nit(int omax) {
    const int need = (omax + 3 + 127) / 128;          // span <= 3 + omax
    const int sizes[] = {1, 2, 3, 5, 9};
    for (int k = 0; k < 5; ++k) if (need <= sizes[k]) return sizes[k];
    return 0;
}
