// Warp-level schedule simulator: Phase 2 of Algorithm 1 (the supplement to Section 3) for one ordered list.
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
//   cached (NIT >= 1, windows of at most 32*NIT full 16-byte groups): the window is loaded once
//     with 16-byte shared loads into registers, checked, and written back -- one read and one
//     write per cell;
//   streamed (longer windows, or NIT = 0): any window length, cells are re-read by the write pass.
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
    return (int)KV_IDX(idx, L, 301);
}

__device__ __forceinline__ int kv_wrap1(int idx, int L) {  // idx < 2L
    return (int)KV_IDX(idx >= L ? idx - L : idx, L, 302);
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
        if (guard > kv_loop_cap(L)) { if (lane == 0) atomicExch(status, KV_DEV_LOOP_CAP); break; }
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
//
// Register-cached form: the window [t, t+o) is split at 16-byte boundaries of the ring into a head
// (0..3 cells, lanes 0..2), a body of full 4-cell groups (group g of round `it` belongs to lane
// g - 32*it; no masks needed) and a tail (0..3 cells, lanes 4..6).
template <int NIT>
__device__ __forceinline__ int sim_admit(int* __restrict__ ring, int L, int M, SimState& st,
                                         int s, int o, int lane, int* status) {
    const int t = st.t, tr = st.tr;
    const int kadm = s + 1 - M - t;                  // V + kadm > 0  <=>  the cell is over budget
    const int kw = s + 1;                            // ramp value at the window start
    int delta = 0;

    const int h = (4 - (tr & 3)) & 3;                // L is a multiple of 4: t and tr agree mod 4
    const int hc = o < h ? o : h;                    // head cells
    const int nbody = (o - hc) >> 2;                 // full groups
    if (NIT > 0 && nbody <= 32 * NIT) {
        const int tc = (o - hc) & 3;                 // tail cells
        const int nit = (nbody + 31) >> 5;
        const int ab = kv_wrap1(tr + hc, L);         // ring index of the first body cell (16-byte aligned)
        // scalar cell of this lane: head cell `lane` or tail cell `lane - 4`
        int sr = -1;
        if (lane < hc) sr = lane;
        else if ((unsigned)(lane - 4) < (unsigned)tc) sr = hc + (nbody << 2) + lane - 4;
        int sidx = 0, sv = -1;
        if (sr >= 0) { sidx = kv_wrap1(tr + sr, L); sv = ring[sidx]; }
        int4 buf[NIT > 0 ? NIT : 1];
        int vmax = sv;
#pragma unroll
        for (int it = 0; it < NIT; ++it) {
            if (it >= nit) break;
            const int g = lane + (it << 5);
            int4 v = make_int4(-1, -1, -1, -1);
            if (g < nbody) v = *reinterpret_cast<const int4*>(ring + kv_wrap1(ab + (g << 2), L));
            buf[it] = v;
            vmax = max(max(vmax, max(v.x, v.y)), max(v.z, v.w));
        }
        vmax = kv_warp_max(vmax);
        const int rl = hc + (lane << 2);             // window offset of this lane's group in round 0
        if (vmax + kadm <= 0) {
            if (sr >= 0) ring[sidx] = sv + kw + sr;
#pragma unroll
            for (int it = 0; it < NIT; ++it) {
                if (it >= nit) break;
                const int g = lane + (it << 5);
                if (g < nbody) {
                    int4 v = buf[it];
                    const int k0 = kw + rl + (it << 7);
                    v.x += k0; v.y += k0 + 1; v.z += k0 + 2; v.w += k0 + 3;
                    *reinterpret_cast<int4*>(ring + kv_wrap1(ab + (g << 2), L)) = v;
                }
            }
        } else {
            // blocked: advance implied by the cells of the window (empty filler cells hold -1)
            int need = 0;
            if (sr >= 0) need = min(sv + kadm, sr + 1);
#pragma unroll
            for (int it = 0; it < NIT; ++it) {
                if (it >= nit) break;
                const int4 v = buf[it];
                if (max(max(v.x, v.y), max(v.z, v.w)) + kadm > 0) {
                    const int r1 = rl + (it << 7) + 1;
                    need = max(need, max(max(min(v.x + kadm, r1), min(v.y + kadm, r1 + 1)),
                                         max(min(v.z + kadm, r1 + 2), min(v.w + kadm, r1 + 3))));
                }
            }
            delta = kv_warp_max(need);
            const int live = st.hz - t;
            if (o < live) delta = sim_search_beyond(ring, L, t, tr, live, o, kadm, delta, lane, status);
            const int kwd = kw - delta, dead = t + L;
            if (sr >= 0) ring[sidx] = sr >= delta ? sv + kwd + sr : dead + sr;
#pragma unroll
            for (int it = 0; it < NIT; ++it) {
                if (it >= nit) break;
                const int g = lane + (it << 5);
                if (g < nbody) {
                    int4 v = buf[it];
                    const int r0 = rl + (it << 7);
                    if (r0 >= delta) {
                        const int k0 = kwd + r0;
                        v.x += k0; v.y += k0 + 1; v.z += k0 + 2; v.w += k0 + 3;
                    } else {
                        v.x = dead + r0;                                              // r0 < delta
                        v.y = r0 + 1 >= delta ? v.y + kwd + r0 + 1 : dead + r0 + 1;
                        v.z = r0 + 2 >= delta ? v.z + kwd + r0 + 2 : dead + r0 + 2;
                        v.w = r0 + 3 >= delta ? v.w + kwd + r0 + 3 : dead + r0 + 3;
                    }
                    *reinterpret_cast<int4*>(ring + kv_wrap1(ab + (g << 2), L)) = v;
                }
            }
            __syncwarp();
            sim_finish_beyond(ring, L, t, tr, o, kw, delta, lane);
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

// The shared-memory simulator behind the interface the kernels use (see RegSim for the other one).
template <int NIT>
struct SmemSim {
    static constexpr bool kUsesSmem = true;
    __host__ __device__ static constexpr int ring_cells(int L) { return L; }   // shared-memory ints per warp
    static constexpr int kWarps = 24;                 // warps per CTA of the persistent kernels
    int* ring;
    int L;
    SimState st;

    __device__ __forceinline__ void attach(int* ring_, int L_) { ring = ring_; L = L_; }
    __device__ __forceinline__ void reset(int lane) { sim_reset(ring, L, st, lane); }
    __device__ __forceinline__ void load(const int* __restrict__ snap, const SnapHeader& h, int lane) {
        for (int r = lane; r < L; r += 32) ring[r] = snap[r];
        st.t = h.t; st.hz = h.hz; st.tr = h.t % L;
        st.tel = ((i64)h.tel_hi << 32) | (i64)(unsigned)h.tel_lo;
        __syncwarp();
    }
    __device__ __forceinline__ void store(int* __restrict__ snap, SnapHeader* hdr, int lane) const {
        for (int r = lane; r < L; r += 32) snap[r] = ring[r];
        if (lane == 0) {
            SnapHeader h; h.t = st.t; h.hz = st.hz;
            h.tel_lo = (int)(st.tel & 0xffffffffll); h.tel_hi = (int)(st.tel >> 32);
            *hdr = h;
        }
    }
    __device__ __forceinline__ int admit(int s, int o, int M, int lane, int* status) {
        return sim_admit<NIT>(ring, L, M, st, s, o, lane, status);
    }
    __device__ __forceinline__ i64 total() const { return st.tel; }
};

// Number of 128-cell rounds a handle's longest window needs (0: use the streamed form).
static inline int sim_pick_nit(int omax) {
    const int need = (omax / 4 + 31) / 32;            // full 4-cell groups of the longest window
    const int sizes[] = {1, 2, 4, 8};
    for (int k = 0; k < 4; ++k) if (need <= sizes[k]) return sizes[k];
    return 8;                                         // longer windows take the streamed form
}
