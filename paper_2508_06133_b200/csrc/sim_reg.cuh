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
// No shared memory, no address arithmetic, no loads or stores: two integer instructions per
// 32-cell chunk and admission in the common case.
#pragma once

#include "common.cuh"

// a + b issued as a multiply-add by one (the multiplier is read from constant memory so that it is
// not folded away): on B200 plain integer adds, max/min, compares and selects all go through the
// half-rate integer ALU pipe, multiply-adds through the FMA pipe, so moving the ramp adds there
// relieves the pipe that limits this kernel.
__constant__ int kv_const_one = 1;
__device__ __forceinline__ int kv_add_fma_pipe(int a, int b) {
#ifdef __CUDA_ARCH__
    int r;
    asm("mad.lo.s32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(kv_const_one), "r"(b));
    return r;
#else
    return a + b;
#endif
}

// The passes over the window are specialised on a bucket (KLO, KHI] of the chunk count nch, chosen
// by a short tree of warp-uniform branches: chunks 1 .. KLO-1 are certainly inside the window (one
// instruction each), chunks KLO .. KHI-1 are masked by lane, and no other register is touched.
// STMT(KLO, KHI) is expanded once per bucket.
#define KV_RS_BUCKETS(nch, STMT)                                                                        \
    if (nch <= 8) {                                                                                     \
        if (nch <= 4) { if (nch <= 2) { STMT(0, 2) } else { STMT(2, 4) } }                              \
        else { if (nch <= 6) { STMT(4, 6) } else { STMT(6, 8) } }                                       \
    } else if (nch <= 16) {                                                                             \
        if (nch <= 12) { if (nch <= 10) { STMT(8, 10) } else { STMT(10, 12) } } else { STMT(12, 16) }   \
    } else {                                                                                            \
        if (nch <= 24) { STMT(16, 24) } else { STMT(24, 33) }                                           \
    }

template <int NREG>
struct RegSim {
    static_assert(NREG >= 2 && NREG <= 33, "the bucket tree covers up to 33 registers");
    static constexpr int kCells = 32 * NREG;
    static constexpr bool kUsesSmem = false;
    __host__ __device__ static constexpr int ring_cells(int) { return 0; }   // shared-memory ints per warp
    // warps per CTA of the persistent kernels, limited by the register file (64K / threads)
#ifndef KV_REG33_WARPS
#define KV_REG33_WARPS 32
#endif
    static constexpr int kWarps = NREG > 17 ? KV_REG33_WARPS : 32;
    int R[NREG];
    int t;
    int tm, rl;              // t mod 32 and (lane - tm): window offset of this lane's cell of R[0]
    i64 tel;

    __device__ __forceinline__ void attach(int*, int) {}
    __device__ __forceinline__ i64 total() const { return tel; }

    __device__ __forceinline__ void reset(int lane) {
#pragma unroll
        for (int c = 0; c < NREG; ++c) R[c] = 32 * c + lane;
        t = 0; tel = 0; tm = 0; rl = lane;
    }

    // snapshot layout: kCells ints, R[c] of lane l at [32 c + l]
    __device__ __forceinline__ void load(const int* __restrict__ snap, const SnapHeader& h, int lane) {
#pragma unroll
        for (int c = 0; c < NREG; ++c) R[c] = snap[32 * c + lane];
        t = h.t;
        tm = t & 31; rl = lane - tm;
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

    // rl = window offset of this lane's cell of R[0]; the cell of R[c] is inside the window iff
    // 32 c < ol (and rl >= 0 for c = 0), with ol = o - rl.
    template <int KLO, int KHI>
    __device__ __forceinline__ int pass_max(int rl, int ol) const {
        int v = (rl >= 0 && ol > 0) ? R[0] : -1;
        constexpr int KI = KLO < KHI ? KLO : KHI;      // chunks 1 .. KI-1 need no mask
#pragma unroll
        for (int c = 1; c + 1 < KI; c += 2) v = __vimax3_s32(v, R[c], R[c + 1]);
        if constexpr (KI >= 2 && ((KI - 1) & 1)) v = max(v, R[KI - 1]);
#pragma unroll
        for (int c = (KI > 1 ? KI : 1); c < KHI; ++c) v = max(v, (32 * c < ol) ? R[c] : -1);
        return v;
    }
    template <int KLO, int KHI>
    __device__ __forceinline__ void pass_add(int rl, int ol, int k0) {
        if (rl >= 0 && ol > 0) R[0] = kv_add_fma_pipe(R[0], k0);
#pragma unroll
        for (int c = 1; c < KHI; ++c)
            if (c < KLO || 32 * c < ol) R[c] = kv_add_fma_pipe(R[c], k0 + 32 * c);
    }
    template <int KLO, int KHI>
    __device__ __forceinline__ int pass_need(int rl, int ol, int kadm) const {
        int need = (rl >= 0 && ol > 0) ? min(R[0] + kadm, rl + 1) : 0;
#pragma unroll
        for (int c = 1; c < KHI; ++c)
            if (c < KLO || 32 * c < ol) need = max(need, __viaddmin_s32(R[c], kadm, rl + 1 + 32 * c));
        return need;
    }

    // Rounds t .. t+delta-1 are over: their cells are re-labelled for the rounds L later and the
    // registers rotate once per 32-round boundary crossed.  The rotation sits behind a real branch
    // (it is rare; as predicated moves it would cost NREG instructions on every call).
    __device__ __forceinline__ void advance(int delta, int lane) {
        const int step = min(delta, 32 - tm);
        if (rl >= 0 && rl < step) R[0] = t + rl + kCells;
        t += step;
        delta -= step;
        if (tm + step == 32) {
            asm volatile("" ::: "memory");
            rotate();
            while (delta >= 32) { R[0] = t + lane + kCells; t += 32; delta -= 32; rotate(); }
            if (lane < delta) R[0] = t + lane + kCells;
            t += delta;
        }
        tm = t & 31;
        rl = lane - tm;
    }

    // Admit one request; returns its start.  All 32 lanes call this with identical (s, o).
    // Each turn of the loop is one bucket dispatch at the current t: test; if the request fits, add
    // its ramp and return; otherwise compute the advance the window asks for, move t, and try again
    // (the next test also covers the cells that entered the window on the right).
    __device__ __forceinline__ int admit(int s, int o, int M, int lane, int* status) {
        int kadm = s + 1 - M - t;                      // V + kadm > 0  <=>  the cell is over budget
        int delta = 0;
#define KV_RS_TRY(A, B)                                                            \
        {                                                                          \
            int vmax = pass_max<A, (B < NREG ? B : NREG)>(rl, ol);                 \
            vmax = kv_warp_max(vmax);                                              \
            if (vmax + kadm <= 0) {                                                \
                pass_add<A, (B < NREG ? B : NREG)>(rl, ol, s + 1 + rl);            \
                tel += t + o;                                                      \
                return t;                                                          \
            }                                                                      \
            delta = pass_need<A, (B < NREG ? B : NREG)>(rl, ol, kadm);             \
        }
        {   // common case: the request fits at t
            const int ol = o - rl, nch = (tm + o + 31) >> 5;
            KV_RS_BUCKETS(nch, KV_RS_TRY)
        }
        for (int guard = 0;; ++guard) {
            delta = kv_warp_max(delta);                // >= 1: the worst cell alone asks for it
            kadm -= delta;
            advance(delta, lane);
            const int ol = o - rl, nch = (tm + o + 31) >> 5;
            KV_RS_BUCKETS(nch, KV_RS_TRY)
            if (guard > kCells) { if (lane == 0) atomicExch(status, KV_DEV_LOOP_CAP); return t; }
        }
#undef KV_RS_TRY
    }
};

// Registers needed for the longest window of a handle (0: too long, use the shared-memory form).
static inline int sim_pick_nreg(int omax) {
    const int need = (31 + omax + 31) / 32;
    const int sizes[] = {2, 3, 5, 9, 17, 33};
    for (int k = 0; k < 6; ++k) if (need <= sizes[k]) return sizes[k];
    return 0;
}
