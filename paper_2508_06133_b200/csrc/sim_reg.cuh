// Register-resident schedule simulator: same admission rule and cell encoding as sim.cuh, but the
// occupancy timeline of a candidate lives in the registers of its warp.
//
// Layout.  The timeline covers L = 32 * NREG consecutive rounds starting at the 32-aligned round
// T0 = t & ~31.  Register R[c] of lane l holds the cell of round T0 + 32 c + l, as V = U + round
// index (an unoccupied cell holds its round index).  Whenever t crosses a multiple of 32 the
// registers are rotated by one (R[0], whose rounds are all over and already re-labelled for the
// rounds L later, becomes R[NREG-1]), so every access uses compile-time register numbers and the
// window of a request, rounds [t, t+o), is always R[0 .. nch-1] with nch = ceil((t%32 + o) / 32).
// NREG = ceil((31 + omax) / 32) registers are enough for the longest window.
//
// Admission of (s, o) at the earliest start p >= t (Algorithm 1, Phase 2):
//   1. vmax = max of V over the window (lanes outside the window masked);  fits  <=>
//      vmax + s + 1 - M - t <= 0;
//   2. if not, the advance implied by the window is  max over its cells of min(V + s+1-M-t, r+1),
//      r = offset in the window (see sim.cuh for why); the rounds that are over are re-labelled,
//      t moves, and step 1 is repeated at the new start (it also covers the cells that entered the
//      window on the right);
//   3. the ramp s+1+r is added to the window.
// No shared memory, no address arithmetic, no loads or stores: two integer instructions per cell
// chunk and admission in the common case.
#pragma once

#include "common.cuh"

// Runs BODY(c) for c = nch-1 down to 1 through a jump table (a switch that falls through), so that
// only the registers of the window are touched: the cases are entry points into straight-line
// code, which keeps the compiler from predicating all NREG bodies.
#define KV_RS_CASE(c, BODY) case (c) + 1: if constexpr ((c) < NREG) { BODY(c) } [[fallthrough]];
#define KV_RS_CHUNKS(nch, BODY)                                                                       \
    switch (nch) {                                                                                    \
        KV_RS_CASE(32, BODY) KV_RS_CASE(31, BODY) KV_RS_CASE(30, BODY) KV_RS_CASE(29, BODY)           \
        KV_RS_CASE(28, BODY) KV_RS_CASE(27, BODY) KV_RS_CASE(26, BODY) KV_RS_CASE(25, BODY)           \
        KV_RS_CASE(24, BODY) KV_RS_CASE(23, BODY) KV_RS_CASE(22, BODY) KV_RS_CASE(21, BODY)           \
        KV_RS_CASE(20, BODY) KV_RS_CASE(19, BODY) KV_RS_CASE(18, BODY) KV_RS_CASE(17, BODY)           \
        KV_RS_CASE(16, BODY) KV_RS_CASE(15, BODY) KV_RS_CASE(14, BODY) KV_RS_CASE(13, BODY)           \
        KV_RS_CASE(12, BODY) KV_RS_CASE(11, BODY) KV_RS_CASE(10, BODY) KV_RS_CASE(9, BODY)            \
        KV_RS_CASE(8, BODY) KV_RS_CASE(7, BODY) KV_RS_CASE(6, BODY) KV_RS_CASE(5, BODY)               \
        KV_RS_CASE(4, BODY) KV_RS_CASE(3, BODY) KV_RS_CASE(2, BODY) KV_RS_CASE(1, BODY)               \
        default: break;                                                                               \
    }

template <int NREG>
struct RegSim {
    static_assert(NREG >= 2 && NREG <= 33, "the chunk switch covers up to 33 registers");
    static constexpr int kCells = 32 * NREG;
    static constexpr bool kUsesSmem = false;
#ifndef KV_REG33_WARPS
#define KV_REG33_WARPS 16
#endif
    // warps per CTA of the persistent kernels, limited by the register file (64K / threads)
    static constexpr int kWarps = NREG > 17 ? KV_REG33_WARPS : (NREG > 9 ? 24 : 32);
    int R[NREG];
    int t;
    i64 tel;

    __device__ __forceinline__ void attach(int*, int) {}
    __device__ __forceinline__ i64 total() const { return tel; }

    __device__ __forceinline__ void reset(int lane) {
#pragma unroll
        for (int c = 0; c < NREG; ++c) R[c] = 32 * c + lane;
        t = 0; tel = 0;
    }

    // snapshot layout: kCells ints, R[c] of lane l at [32 c + l]
    __device__ __forceinline__ void load(const int* __restrict__ snap, const SnapHeader& h, int lane) {
#pragma unroll
        for (int c = 0; c < NREG; ++c) R[c] = snap[32 * c + lane];
        t = h.t;
        tel = ((i64)h.tel_hi << 32) | (i64)(unsigned)h.tel_lo;
    }

    __device__ __forceinline__ void store(int* __restrict__ snap, SnapHeader* hdr, int lane) const {
#pragma unroll
        for (int c = 0; c < NREG; ++c) snap[32 * c + lane] = R[c];
        if (lane == 0) {
            SnapHeader h; h.t = t; h.hz = 0;
            h.tel_lo = (int)(tel & 0xffffffffll); h.tel_hi = (int)(tel >> 32);
            *hdr = h;
        }
    }

    __device__ __forceinline__ void rotate() {
        const int first = R[0];
#pragma unroll
        for (int c = 0; c + 1 < NREG; ++c) R[c] = R[c + 1];
        R[NREG - 1] = first;
    }

    // Admit one request; returns its start.  All 32 lanes call this with identical (s, o).
    __device__ __forceinline__ int admit(int s, int o, int M, int lane, int* status) {
        int kadm = s + 1 - M - t;                      // V + kadm > 0  <=>  the cell is over budget
        for (int guard = 0;; ++guard) {
            const int tm = t & 31;
            const int rl = lane - tm;                  // window offset of this lane's cell of R[0]
            const int ol = o - rl;                     // cell of R[c] is inside the window iff 32 c < ol
            const int nch = (tm + o + 31) >> 5;
            const bool in0 = rl >= 0 && ol > 0;
            int vmax = in0 ? R[0] : -1;
#define KV_RS_MAX(c) vmax = max(vmax, 32 * (c) < ol ? R[c] : -1);
            KV_RS_CHUNKS(nch, KV_RS_MAX)
#undef KV_RS_MAX
            vmax = kv_warp_max(vmax);
            if (vmax + kadm <= 0) break;
            int need = in0 ? min(R[0] + kadm, rl + 1) : 0;
#define KV_RS_NEED(c) if (32 * (c) < ol) need = max(need, min(R[c] + kadm, rl + 1 + 32 * (c)));
            KV_RS_CHUNKS(nch, KV_RS_NEED)
#undef KV_RS_NEED
            int delta = kv_warp_max(need);             // >= 1: the worst cell alone asks for it
            kadm -= delta;
            // rounds t .. t+delta-1 are over: re-label their cells for the rounds L later
            while (delta > 0) {
                const int tm2 = t & 31;
                const int step = min(delta, 32 - tm2);
                if (lane >= tm2 && lane < tm2 + step) R[0] = t - tm2 + lane + kCells;
                t += step;
                delta -= step;
                if (tm2 + step == 32) rotate();
            }
            if (guard > kCells) { if (lane == 0) atomicExch(status, KV_DEV_LOOP_CAP); break; }
        }
        const int tm = t & 31;
        const int rl = lane - tm;
        const int ol = o - rl;
        const int nch = (tm + o + 31) >> 5;
        const int k0 = s + 1 + rl;                     // ramp value of this lane's cell of R[0]
        if (rl >= 0 && ol > 0) R[0] += k0;
#define KV_RS_ADD(c) if (32 * (c) < ol) R[c] += k0 + 32 * (c);
        KV_RS_CHUNKS(nch, KV_RS_ADD)
#undef KV_RS_ADD
        tel += t + o;
        return t;
    }
};

// Registers needed for the longest window of a handle (0: too long, use the shared-memory form).
static inline int sim_pick_nreg(int omax) {
    const int need = (31 + omax + 31) / 32;
    const int sizes[] = {2, 3, 5, 9, 17, 33};
    for (int k = 0; k < 6; ++k) if (need <= sizes[k]) return sizes[k];
    return 0;
}
