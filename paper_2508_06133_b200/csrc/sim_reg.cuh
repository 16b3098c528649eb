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
// Admission of (s, o) at the earliest start p >= t (Algorithm 1, Phase 2), one turn per candidate
// start:
//   1. first chunk only: a cell over budget by e = V + s+1-M-t > 0 at window offset r rules out
//      every advance below min(e, r+1) (see sim.cuh for why).  If the largest such bound over the
//      cells of R[0] is positive, the rounds that are over are re-labelled, t moves by it, and the
//      turn ends -- a request that waits nearly always waits for the rounds right in front of it;
//   2. otherwise vmax = max of V over the whole window (lanes outside it masked); the request fits
//      <=>  vmax + s+1-M-t <= 0, and then
//   3. the ramp s+1+r is added to the window.
//   (rare: no cell of the first chunk is over budget but a later one is -- the bound is then taken
//   over all chunks and t moves by it.)
// No shared memory, no address arithmetic, no loads or stores: one and a half integer instructions
// per 32-cell chunk and admission for the two window passes.
#pragma once

#include "common.cuh"

// The passes over the window are specialised on the chunk count nch by a tree of warp-uniform
// branches whose split points follow the chunk counts of the mixed chat/document backlogs (short
// windows, which are the most frequent, are reached first).  STMT(KLO, KHI) is expanded once per
// leaf and handles nch in (KLO, KHI]: chunks 1 .. KLO-1 are certainly inside the window (one
// instruction each per pass), chunks KLO .. KHI-1 are masked by lane, and no other register is
// touched.  KV_RS_BUCKETS_EXACT has one leaf per chunk count (a single masked chunk per pass);
// KV_RS_BUCKETS_MIX is exact up to 16 chunks and two chunk counts per leaf beyond.
#define KV_RS_BUCKETS_EXACT(nch, STMT) \
    if (nch <= 7) { \
      if (nch <= 4) { \
        if (nch <= 2) { \
          if (nch <= 1) { \
            STMT(0, 1) \
          } else { \
            STMT(1, 2) \
          } \
        } else { \
          if (nch <= 3) { \
            STMT(2, 3) \
          } else { \
            STMT(3, 4) \
          } \
        } \
      } else { \
        if (nch <= 5) { \
          STMT(4, 5) \
        } else { \
          if (nch <= 6) { \
            STMT(5, 6) \
          } else { \
            STMT(6, 7) \
          } \
        } \
      } \
    } else { \
      if (nch <= 12) { \
        if (nch <= 9) { \
          if (nch <= 8) { \
            STMT(7, 8) \
          } else { \
            STMT(8, 9) \
          } \
        } else { \
          if (nch <= 10) { \
            STMT(9, 10) \
          } else { \
            if (nch <= 11) { \
              STMT(10, 11) \
            } else { \
              STMT(11, 12) \
            } \
          } \
        } \
      } else { \
        if (nch <= 15) { \
          if (nch <= 13) { \
            STMT(12, 13) \
          } else { \
            if (nch <= 14) { \
              STMT(13, 14) \
            } else { \
              STMT(14, 15) \
            } \
          } \
        } else { \
          if (nch <= 18) { \
            if (nch <= 16) { \
              STMT(15, 16) \
            } else { \
              if (nch <= 17) { \
                STMT(16, 17) \
              } else { \
                STMT(17, 18) \
              } \
            } \
          } else { \
            if (nch <= 25) { \
              if (nch <= 21) { \
                if (nch <= 19) { \
                  STMT(18, 19) \
                } else { \
                  if (nch <= 20) { \
                    STMT(19, 20) \
                  } else { \
                    STMT(20, 21) \
                  } \
                } \
              } else { \
                if (nch <= 23) { \
                  if (nch <= 22) { \
                    STMT(21, 22) \
                  } else { \
                    STMT(22, 23) \
                  } \
                } else { \
                  if (nch <= 24) { \
                    STMT(23, 24) \
                  } else { \
                    STMT(24, 25) \
                  } \
                } \
              } \
            } else { \
              if (nch <= 32) { \
                if (nch <= 28) { \
                  if (nch <= 26) { \
                    STMT(25, 26) \
                  } else { \
                    if (nch <= 27) { \
                      STMT(26, 27) \
                    } else { \
                      STMT(27, 28) \
                    } \
                  } \
                } else { \
                  if (nch <= 31) { \
                    if (nch <= 29) { \
                      STMT(28, 29) \
                    } else { \
                      if (nch <= 30) { \
                        STMT(29, 30) \
                      } else { \
                        STMT(30, 31) \
                      } \
                    } \
                  } else { \
                    STMT(31, 32) \
                  } \
                } \
              } else { \
                STMT(32, 33) \
              } \
            } \
          } \
        } \
      } \
    }

#define KV_RS_BUCKETS_MIX(nch, STMT) \
    if (nch <= 7) { \
      if (nch <= 4) { \
        if (nch <= 2) { \
          if (nch <= 1) { \
            STMT(0, 1) \
          } else { \
            STMT(1, 2) \
          } \
        } else { \
          if (nch <= 3) { \
            STMT(2, 3) \
          } else { \
            STMT(3, 4) \
          } \
        } \
      } else { \
        if (nch <= 5) { \
          STMT(4, 5) \
        } else { \
          if (nch <= 6) { \
            STMT(5, 6) \
          } else { \
            STMT(6, 7) \
          } \
        } \
      } \
    } else { \
      if (nch <= 12) { \
        if (nch <= 9) { \
          if (nch <= 8) { \
            STMT(7, 8) \
          } else { \
            STMT(8, 9) \
          } \
        } else { \
          if (nch <= 10) { \
            STMT(9, 10) \
          } else { \
            if (nch <= 11) { \
              STMT(10, 11) \
            } else { \
              STMT(11, 12) \
            } \
          } \
        } \
      } else { \
        if (nch <= 15) { \
          if (nch <= 13) { \
            STMT(12, 13) \
          } else { \
            if (nch <= 14) { \
              STMT(13, 14) \
            } else { \
              STMT(14, 15) \
            } \
          } \
        } else { \
          if (nch <= 18) { \
            if (nch <= 16) { \
              STMT(15, 16) \
            } else { \
              STMT(16, 18) \
            } \
          } else { \
            if (nch <= 24) { \
              if (nch <= 20) { \
                STMT(18, 20) \
              } else { \
                if (nch <= 22) { \
                  STMT(20, 22) \
                } else { \
                  STMT(22, 24) \
                } \
              } \
            } else { \
              if (nch <= 32) { \
                if (nch <= 28) { \
                  if (nch <= 26) { \
                    STMT(24, 26) \
                  } else { \
                    STMT(26, 28) \
                  } \
                } else { \
                  if (nch <= 30) { \
                    STMT(28, 30) \
                  } else { \
                    STMT(30, 32) \
                  } \
                } \
              } else { \
                STMT(32, 33) \
              } \
            } \
          } \
        } \
      } \
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
        for (int c = 0; c < NREG; ++c) R[c] = snap[KV_IDX(32 * c + lane, kCells, 101)];
        t = h.t;
        tm = t & 31; rl = lane - tm;
        tel = ((i64)h.tel_hi << 32) | (i64)(unsigned)h.tel_lo;
    }

    __device__ __forceinline__ void store(int* __restrict__ snap, SnapHeader* hdr, int lane) const {
#pragma unroll
        for (int c = 0; c < NREG; ++c) snap[KV_IDX(32 * c + lane, kCells, 102)] = R[c];
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
    __device__ __forceinline__ void pass_add(int rl, int ol, int k0) {
        if ((unsigned)rl < (unsigned)(ol + rl)) R[0] = R[0] + k0;     // 0 <= rl < o in one compare
#pragma unroll
        for (int c = 1; c < KHI; ++c)
            if (c < KLO || 32 * c < ol) R[c] = R[c] + (k0 + 32 * c);
    }
    // Rounds t .. t+delta-1 are over: their cells are re-labelled for the rounds L later and the
    // registers rotate once per 32-round boundary crossed.  The rotation sits behind a real branch
    // (it is rare; as predicated moves it would cost NREG instructions on every call).
    __device__ __forceinline__ void advance(int delta, int lane) {
        const int step = min(delta, 32 - tm);
        if ((unsigned)rl < (unsigned)step) R[0] = t + rl + kCells;
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

    // rest of the window maximum, given the (masked) first chunk
    template <int KLO, int KHI>
    __device__ __forceinline__ int pass_max_from(int v, int ol) const {
        constexpr int KI = KLO < KHI ? KLO : KHI;      // chunks 1 .. KI-1 need no mask
#pragma unroll
        for (int c = 1; c + 1 < KI; c += 2) v = __vimax3_s32(v, R[c], R[c + 1]);
        if constexpr (KI >= 2 && ((KI - 1) & 1)) v = max(v, R[KI - 1]);
#pragma unroll
        for (int c = (KI > 1 ? KI : 1); c < KHI; ++c) if (32 * c < ol) v = max(v, R[c]);
        return v;
    }
    // wait bound of the chunks behind the first, every one masked (rare path, see admit)
    __device__ __forceinline__ int need_behind(int ol, int kadm) const {
        int need = 0;
#pragma unroll
        for (int c = 1; c < NREG; ++c)
            if (32 * c < ol) need = max(need, __viaddmin_s32(R[c], kadm, rl + 1 + 32 * c));
        return need;
    }

    // Admit one request; returns its start.  All 32 lanes call this with identical (s, o).
    //
    // A request that has to wait almost always waits because the rounds right in front of it are
    // full: the cells over budget sit at the left end of the window and the wait is the offset
    // behind the last of them, a few rounds.  Each turn therefore first looks at the first chunk(s)
    // alone: a cell over budget by e at window offset r rules out every advance below
    // min(e, r + 1) (the start has to move e rounds for the ramp to drop below the budget there, or
    // r + 1 rounds for the cell to leave the window).  If that bound is positive the request cannot
    // start at t; t moves by the bound -- a lower bound of the true wait, so no feasible start is
    // skipped -- and the turn is over without a pass over the whole window.  Otherwise one bucket
    // dispatch tests the whole window and, if it fits, adds the ramp.  The remaining case (the only
    // cells over budget lie behind the pre-tested chunks) takes the bound from all chunks.
    __device__ __forceinline__ int admit(int s, int o, int M, int lane, int* status) {
        int kadm = s + 1 - M - t;                      // V + kadm > 0  <=>  the cell is over budget
        for (int guard = 0;; ++guard) {
            const int ol = o - rl;
            const int v0 = (unsigned)rl < (unsigned)o ? R[0] : -1;        // 0 <= rl < o: the cell is in the window
            int need = __viaddmin_s32(v0, kadm, rl + 1);               // masked lanes: below zero
            int delta = kv_warp_max(need);
            if (delta <= 0) {
                const int nch = (tm + o + 31) >> 5;
#define KV_RS_TRY(A, B)                                                            \
                if constexpr ((A) < NREG) {                                        \
                    int vmax = pass_max_from<A, (B < NREG ? B : NREG)>(v0, ol);    \
                    vmax = kv_warp_max(vmax);                                      \
                    if (vmax + kadm <= 0) {                                        \
                        pass_add<A, (B < NREG ? B : NREG)>(rl, ol, s + 1 + rl);    \
                        tel += t + o;                                              \
                        return t;                                                  \
                    }                                                              \
                }
                KV_RS_BUCKETS_EXACT(nch, KV_RS_TRY)
#undef KV_RS_TRY
                delta = kv_warp_max(need_behind(ol, kadm));   // >= 1: the worst cell alone asks for it
            }
            kadm -= delta;
            advance(delta, lane);
            if (guard > kv_loop_cap(kCells)) { if (lane == 0) atomicExch(status, KV_DEV_LOOP_CAP); return t; }
        }
    }
};

// Registers needed for the longest window of a handle (0: too long, use the shared-memory form).
static inline int sim_pick_nreg(int omax) {
    const int need = (31 + omax + 31) / 32;
    const int sizes[] = {2, 3, 5, 9, 17, 33};
    for (int k = 0; k < 6; ++k) if (need <= sizes[k]) return sizes[k];
    return 0;
}
