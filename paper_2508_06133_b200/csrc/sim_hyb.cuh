// Hybrid schedule simulator for decode lengths beyond what the register-resident simulator covers:
// the first 32 * 33 rounds of the timeline live in registers exactly as in sim_reg.cuh (same cell
// encoding V = U + round index, same rotation at every 32-round boundary), the rounds after them in
// a per-warp ring of FC chunks of 32 cells in shared memory ("far" part).  Lane l owns column l of
// every chunk, in registers and in the ring alike, so no lane ever reads another lane's cell and no
// warp synchronisation is needed around the shared-memory accesses.
//
// At a rotation the register that holds only finished rounds (already re-labelled for the rounds
// one whole span later) goes to the slot of the first far chunk, and that chunk's cells become the
// last register.  A request whose window ends inside the registers -- nch = ceil((t%32 + o)/32) <=
// 33, the common case: most decode lengths are short even when the longest is not -- never touches
// shared memory and costs what it costs in the register simulator; a longer window continues over
// the first nch - 33 far chunks with one shared load (test) or load + store (ramp add) per chunk.
//
// State size (snapshot layout): L = 32 * (33 + FC) ints, the registers first (R[c] of lane l at
// [32 c + l]), then the far chunks in timeline order.  FC is chosen by the host so that
// 32 * (33 + FC) >= 31 + the longest decode.
#pragma once

#include "common.cuh"
#include "sim_reg.cuh"

struct HybSim {
    static constexpr int NREG = 33;
    static constexpr bool kUsesSmem = true;
    static constexpr int kWarps = 24;                 // 33 timeline registers + the ring bookkeeping need more than 64 registers
    __host__ __device__ static constexpr int ring_cells(int L) { return L - 32 * NREG; }

    int R[NREG];
    int t;
    int tm, rl;              // t mod 32 and (lane - tm): window offset of this lane's cell of R[0]
    i64 tel;
    int* far;                // this lane's column of the far ring: far[32 * slot]
    int FC, fb;              // chunks in the far ring; slot of the first far chunk
    int span;                // 32 * (NREG + FC): rounds covered by the whole state

    __device__ __forceinline__ void attach(int* ring, int L) {
        far = ring + (threadIdx.x & 31);
        FC = (L >> 5) - NREG;
        span = L;
        fb = 0;
    }
    __device__ __forceinline__ i64 total() const { return tel; }
    __device__ __forceinline__ int slot_of(int k) const { const int x = fb + k; return (int)KV_IDX(x >= FC ? x - FC : x, FC, 201); }

    __device__ __forceinline__ void reset(int lane) {
#pragma unroll
        for (int c = 0; c < NREG; ++c) R[c] = 32 * c + lane;
        for (int k = 0; k < FC; ++k) far[32 * k] = 32 * (NREG + k) + lane;
        fb = 0; t = 0; tel = 0; tm = 0; rl = lane;
    }
    __device__ __forceinline__ void load(const int* __restrict__ snap, const SnapHeader& h, int lane) {
#pragma unroll
        for (int c = 0; c < NREG; ++c) R[c] = snap[KV_IDX(32 * c + lane, span, 202)];
        for (int k = 0; k < FC; ++k) far[32 * k] = snap[KV_IDX(32 * (NREG + k) + lane, span, 203)];
        fb = 0;
        t = h.t; tm = t & 31; rl = lane - tm;
        tel = ((i64)h.tel_hi << 32) | (i64)(unsigned)h.tel_lo;
    }
    __device__ __forceinline__ void store(int* __restrict__ snap, SnapHeader* hdr, int lane) const {
#pragma unroll
        for (int c = 0; c < NREG; ++c) snap[KV_IDX(32 * c + lane, span, 204)] = R[c];
        for (int k = 0; k < FC; ++k) snap[KV_IDX(32 * (NREG + k) + lane, span, 205)] = far[32 * slot_of(k)];
        if (lane == 0) {
            SnapHeader h; h.t = t; h.hz = 0;
            h.tel_lo = (int)(tel & 0xffffffffll); h.tel_hi = (int)(tel >> 32);
            *hdr = h;
        }
    }

    // R[0] (all its rounds over, cells already re-labelled one span ahead) becomes the last far
    // chunk; the first far chunk becomes the last register.
    __device__ __forceinline__ void rotate() {
        const int first = R[0];
#pragma unroll
        for (int c = 0; c + 1 < NREG; ++c) R[c] = R[c + 1];
        int* cell = far + 32 * KV_IDX(fb, FC, 206);
        R[NREG - 1] = *cell;
        *cell = first;
        fb = fb + 1 == FC ? 0 : fb + 1;
    }

    __device__ __forceinline__ void advance(int delta, int lane) {
        const int step = min(delta, 32 - tm);
        if ((unsigned)rl < (unsigned)step) R[0] = t + rl + span;
        t += step;
        delta -= step;
        if (tm + step == 32) {
            asm volatile("" ::: "memory");
            rotate();
            while (delta >= 32) { R[0] = t + lane + span; t += 32; delta -= 32; rotate(); }
            if (lane < delta) R[0] = t + lane + span;
            t += delta;
        }
        tm = t & 31;
        rl = lane - tm;
    }

    // ---- passes over a window that ends inside the registers (as in the register simulator)
    template <int KLO, int KHI>
    __device__ __forceinline__ int pass_max_from(int v, int ol) const {
        constexpr int KI = KLO < KHI ? KLO : KHI;
#pragma unroll
        for (int c = 1; c + 1 < KI; c += 2) v = __vimax3_s32(v, R[c], R[c + 1]);
        if constexpr (KI >= 2 && ((KI - 1) & 1)) v = max(v, R[KI - 1]);
#pragma unroll
        for (int c = (KI > 1 ? KI : 1); c < KHI; ++c) if (32 * c < ol) v = max(v, R[c]);
        return v;
    }
    template <int KLO, int KHI>
    __device__ __forceinline__ void pass_add(int rl, int ol, int k0) {
        if ((unsigned)rl < (unsigned)(ol + rl)) R[0] = R[0] + k0;     // 0 <= rl < o in one compare
#pragma unroll
        for (int c = 1; c < KHI; ++c)
            if (c < KLO || 32 * c < ol) R[c] = R[c] + (k0 + 32 * c);
    }
    // wait bound of every chunk behind the first, registers and far ring (rare path, see admit)
    __device__ __forceinline__ int need_behind(int ol, int kadm, int nfar) const {
        int need = 0;
#pragma unroll
        for (int c = 1; c < NREG; ++c)
            if (32 * c < ol) need = max(need, __viaddmin_s32(R[c], kadm, rl + 1 + 32 * c));
        for (int k = 0; k < nfar; ++k)
            if (32 * (NREG + k) < ol)
                need = max(need, __viaddmin_s32(far[32 * slot_of(k)], kadm, rl + 1 + 32 * (NREG + k)));
        return need;
    }

    // Admit one request; returns its start.  All 32 lanes call this with identical (s, o).  Same
    // turn structure as the register simulator: the first chunk alone decides whether the request
    // has to wait and for how long at least; otherwise the whole window is tested and, if it fits,
    // the ramp is added; a window that reaches beyond the registers continues over the far ring.
    __device__ __forceinline__ int admit(int s, int o, int M, int lane, int* status) {
        int kadm = s + 1 - M - t;                      // V + kadm > 0  <=>  the cell is over budget
        for (int guard = 0;; ++guard) {
            const int ol = o - rl;
            const int v0 = (unsigned)rl < (unsigned)o ? R[0] : -1;        // 0 <= rl < o: the cell is in the window
            int delta = kv_warp_max(__viaddmin_s32(v0, kadm, rl + 1));
            if (delta <= 0) {
                const int nch = (tm + o + 31) >> 5;
                if (nch <= NREG) {
#define KV_HS_TRY(A, B)                                                            \
                    if constexpr ((A) < NREG) {                                    \
                        int vmax = pass_max_from<A, (B < NREG ? B : NREG)>(v0, ol); \
                        vmax = kv_warp_max(vmax);                                  \
                        if (vmax + kadm <= 0) {                                    \
                            pass_add<A, (B < NREG ? B : NREG)>(rl, ol, s + 1 + rl); \
                            tel += t + o;                                          \
                            return t;                                              \
                        }                                                          \
                    }
                    KV_RS_BUCKETS_MIX(nch, KV_HS_TRY)
#undef KV_HS_TRY
                    delta = kv_warp_max(need_behind(ol, kadm, 0));
                } else {
                    // every register is inside the window (R[0] from this lane's offset on), then the
                    // first nfar far chunks; far chunk k holds window offsets rl + 32 (NREG + k)
                    const int nfar = nch - NREG;
                    int v = v0;
#pragma unroll
                    for (int c = 1; c + 1 < NREG; c += 2) v = __vimax3_s32(v, R[c], R[c + 1]);
                    for (int k = 0; k < nfar; ++k) {
                        const int x = far[32 * slot_of(k)];
                        v = max(v, (32 * (NREG + k) < ol) ? x : -1);
                    }
                    const int vmax = kv_warp_max(v);
                    if (vmax + kadm <= 0) {
                        const int k0 = s + 1 + rl;
                        if (rl >= 0) R[0] = R[0] + k0;
#pragma unroll
                        for (int c = 1; c < NREG; ++c) R[c] = R[c] + (k0 + 32 * c);
                        for (int k = 0; k < nfar; ++k) {
                            if (32 * (NREG + k) < ol) {
                                int* cell = far + 32 * slot_of(k);
                                *cell += k0 + 32 * (NREG + k);
                            }
                        }
                        tel += t + o;
                        return t;
                    }
                    delta = kv_warp_max(need_behind(ol, kadm, nfar));
                }
            }
            kadm -= delta;                             // >= 1: the worst cell alone asks for it
            advance(delta, lane);
            if (guard > kv_loop_cap(span)) { if (lane == 0) atomicExch(status, KV_DEV_LOOP_CAP); return t; }
        }
    }
};

// Far chunks needed beyond the 33 registers for the longest decode of a handle.
static inline int sim_pick_far_chunks(int omax) {
    const int chunks = (31 + omax + 31) / 32;
    return chunks > HybSim::NREG ? chunks - HybSim::NREG : 1;
}
