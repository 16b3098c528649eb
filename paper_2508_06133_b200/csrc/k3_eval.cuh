// K3 (+K4) -- batched schedule evaluation kernels.
//
//   k3_gather_table   (s, o) of the request at every position of the base order.
//   k3_base_run       one warp list-schedules the base order and stores the simulator state in
//                     front of every `stride`-th position (snapshots) plus the start of every position.
//   k3_eval_moves     one warp per candidate; the candidate is a move applied to the base order
//                     (K4: index -> (type, i, j) -> position map, never materialised; launch order
//                     bucketed by first moved position); simulation resumes from the last snapshot
//                     at or before the first moved position.
//   k3_eval_orders    explicit permutations, simulated from t = 0.
//   (k3_policy.cuh)   k3_eval_policy: one warp per (instance, policy) pair: order construction,
//                     optional prefix-F batching, simulation -- all in shared memory.
//   k3_check_starts   explicit start times: occupancy by the integer program's memory row
//                     (Section 6.1), flag raised at the first round above M.
//
// The request table is staged into shared memory once per CTA with a bulk asynchronous copy
// (cp.async.bulk + mbarrier, no multicast) when it fits; otherwise it is read through L1/L2.
#pragma once

#include "common.cuh"
#include "k2_fmetric.cuh"
#include "k4_moves.cuh"
#include "sim.cuh"
#include "sim_reg.cuh"
#include "sim_hyb.cuh"

#define K3S_WARPS 16                       // warps per CTA of the start-time checker

// ------------------------------------------------------------------------------------------------
// Bulk copy global -> shared with a bounded wait.  bytes is a multiple of 16, both addresses are
// 16-byte aligned.  Returns false (in every thread) if the copy did not land within the cap; the
// caller must then leave without touching the destination.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned kv_smem_addr(const void* p) {
    return (unsigned)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ int kv_mbar_wait(unsigned bar, int max_spins) {
    for (int spin = 0; spin < max_spins; ++spin) {
        unsigned done;
        asm volatile(
            "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n selp.u32 %0, 1, 0, p;\n}\n"
            : "=r"(done) : "r"(bar) : "memory");
        if (done) return 1;
    }
    return 0;
}

__device__ bool kv_bulk_load(void* smem_dst, const void* gsrc, unsigned bytes, u64* mbar, int* sh_flag, int* status) {
    const unsigned bar = kv_smem_addr(mbar);
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
        const unsigned chunk = 32768;
        for (unsigned off = 0; off < bytes; off += chunk) {
            unsigned sz = bytes - off < chunk ? bytes - off : chunk;
            asm volatile(
                "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                ::"r"(kv_smem_addr((const char*)smem_dst + off)), "l"((const char*)gsrc + off), "r"(sz), "r"(bar)
                : "memory");
        }
        // bounded wait; if it runs out, flag the failure and give the copy one more bounded
        // chance to land so that the CTA does not exit with a transfer still in flight
        int ok = kv_mbar_wait(bar, 1 << 22);
        if (!ok) {
            atomicExch(status, KV_DEV_TMA_TIMEOUT);
            kv_mbar_wait(bar, 1 << 22);
        }
        *sh_flag = ok;
    }
    __syncthreads();
    return *sh_flag != 0;
}

// ------------------------------------------------------------------------------------------------
__global__ void k3_gather_table(const int2* __restrict__ tbl_id, const int* __restrict__ order, int n,
                                int2* __restrict__ tbl_base) {
    int q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q < n) tbl_base[q] = tbl_id[order[q]];
}

__global__ void k3_make_table(const int* __restrict__ s, const int* __restrict__ o, int total, int2* __restrict__ tbl) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < total) tbl[i] = make_int2(s[i], o[i]);
}

__global__ void k3_iota(int* a, int n) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) a[i] = i;
}

// ------------------------------------------------------------------------------------------------
// Base run: positions 0 .. n-1 of the base order; snapshot idx holds the state in front of
// position idx * stride.  One warp.  Dynamic shared memory: the simulator's ring, if it has one.
// ------------------------------------------------------------------------------------------------
template <class SIM>
__global__ void __launch_bounds__(32)
k3_base_run(const int2* __restrict__ tbl_base, int n, int L, int M, int stride, int snap_count,
            int* __restrict__ snap_ring, SnapHeader* __restrict__ snap_hdr,
            int* __restrict__ base_starts_pos, i64* __restrict__ base_tel, int* status) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int lane = threadIdx.x;
    SIM sim;
    sim.attach((int*)smem_raw, L);
    sim.reset(lane);
    for (int q0 = 0; q0 < n; q0 += 32) {
        const int qq = q0 + lane;
        int2 so = qq < n ? tbl_base[qq] : make_int2(1, 1);
        const int cnt = min(32, n - q0);
        for (int k = 0; k < cnt; ++k) {
            const int q = q0 + k;
            if (q % stride == 0) {
                const int idx = (int)KV_IDX(q / stride, snap_count, 401);
                sim.store(snap_ring + (size_t)idx * L, snap_hdr + idx, lane);
            }
            const int s = __shfl_sync(KV_FULL, so.x, k), o = __shfl_sync(KV_FULL, so.y, k);
            const int p = sim.admit(s, o, M, lane, status);
            if (lane == 0) base_starts_pos[q] = p;
        }
    }
    if (lane == 0) *base_tel = sim.total();
}

// ------------------------------------------------------------------------------------------------
// Moves.  mode 0: codes[c]; mode 1: code = first + c; mode 2: sampled move m = first + c.
// ------------------------------------------------------------------------------------------------
struct MoveEvalParams {
    int n, L, M, stride, snap_count;
    const int2* tbl_base;
    int table_in_smem;
    unsigned table_bytes;              // multiple of 16
    const int* snap_ring;
    const SnapHeader* snap_hdr;
    MoveSource src;
    i64 count;
    const int* launch_order;           // candidate index of every launch slot (K4)
    i64* tel_out;
    int tel_by_slot;                   // 1: tel_out is indexed by launch slot (full-sector writes; the arg-min maps
                                       // slots back through launch_order), 0: by candidate index
    int* starts_out;                   // nullable [count][n], by request id
    const int* base_order;
    const int* base_starts_pos;
    int* status;
};

// One warp per candidate, no loop over candidates (a persistent loop around the simulator costs
// ~15 % more instructions per admission with this compiler): warp w of CTA b takes launch slot
// 32 b + w, whose candidate K4 chose so that the warps of a CTA have nearly equal work.
template <class SIM, bool kStarts>
__global__ void __launch_bounds__(SIM::kWarps * 32, 1)
k3_eval_moves(const MoveEvalParams p) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ u64 mbar;
    __shared__ int sh_flag;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int2* tbl = p.tbl_base;
    size_t ring_off = 0;
    if (p.table_in_smem) {
        if (!kv_bulk_load(smem_raw, p.tbl_base, p.table_bytes, &mbar, &sh_flag, p.status)) return;
        tbl = (const int2*)smem_raw;
        ring_off = (p.table_bytes + 127) & ~(size_t)127;
    }
    const int n = p.n, L = p.L, M = p.M;
    const i64 slot = (i64)blockIdx.x * (blockDim.x >> 5) + warp;
    if (slot >= p.count) return;
    const i64 c = KV_IDX(p.launch_order[slot], p.count, 402);
    i64* tel_dst = p.tel_out + (p.tel_by_slot ? slot : c);
    SIM sim;
    sim.attach((int*)(smem_raw + ring_off) + (size_t)warp * SIM::ring_cells(L), L);
    const Move mv = k4_move_of(p.src, n, c);
    if ((unsigned)mv.i >= (unsigned)n || (unsigned)mv.j >= (unsigned)n) {      // code outside the neighbourhood
        if (lane == 0) *tel_dst = INT64_MAX;
        return;
    }
    const int first_pos = min(mv.i, mv.j);
    const int idx = (int)KV_IDX(first_pos / p.stride, p.snap_count, 403);
    const int q_start = idx * p.stride;
    // restore the base run's state in front of q_start
    sim.load(p.snap_ring + (size_t)idx * L, p.snap_hdr[idx], lane);
    int* starts = kStarts ? p.starts_out + (size_t)c * n : nullptr;
    if (kStarts)
        for (int q = lane; q < q_start; q += 32) starts[KV_IDX(p.base_order[q], n, 406)] = p.base_starts_pos[q];
    for (int q0 = q_start; q0 < n; q0 += 32) {
        const int qq = q0 + lane;
        int2 so = make_int2(1, 1);
        int id = 0;
        if (qq < n) {
            const int bp = (int)KV_IDX(kv_map_pos(mv, qq), n, 404);
            so = tbl[bp];
            if (kStarts) id = p.base_order[bp];
        }
        const int cnt = min(32, n - q0);
        for (int k = 0; k < cnt; ++k) {
            const int s = __shfl_sync(KV_FULL, so.x, k), o = __shfl_sync(KV_FULL, so.y, k);
            const int pstart = sim.admit(s, o, M, lane, p.status);
            if (kStarts && lane == k) starts[KV_IDX(id, n, 405)] = pstart;
        }
    }
    if (lane == 0) *tel_dst = sim.total();
}

// ------------------------------------------------------------------------------------------------
// Explicit orders: orders[c][q] = request id at position q.
// ------------------------------------------------------------------------------------------------
struct OrderEvalParams {
    int n, L, M;
    const int2* tbl_id;
    int table_in_smem;
    unsigned table_bytes;
    const int* orders;
    i64 count;
    i64* tel_out;
    int* starts_out;
    int* status;
};

template <class SIM, bool kStarts>
__global__ void __launch_bounds__(SIM::kWarps * 32, 1)
k3_eval_orders(const OrderEvalParams p) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ u64 mbar;
    __shared__ int sh_flag;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int2* tbl = p.tbl_id;
    size_t ring_off = 0;
    if (p.table_in_smem) {
        if (!kv_bulk_load(smem_raw, p.tbl_id, p.table_bytes, &mbar, &sh_flag, p.status)) return;
        tbl = (const int2*)smem_raw;
        ring_off = (p.table_bytes + 127) & ~(size_t)127;
    }
    const int n = p.n, L = p.L, M = p.M;
    const i64 c = (i64)blockIdx.x * (blockDim.x >> 5) + warp;      // every order has the same length
    if (c >= p.count) return;
    SIM sim;
    sim.attach((int*)(smem_raw + ring_off) + (size_t)warp * SIM::ring_cells(L), L);
    const int* ord = p.orders + (size_t)c * n;
    int* starts = kStarts ? p.starts_out + (size_t)c * n : nullptr;
    sim.reset(lane);
    int bad = 0;
    for (int q0 = 0; q0 < n; q0 += 32) {
        const int qq = q0 + lane;
        int2 so = make_int2(1, 1);
        int id = 0;
        if (qq < n) { id = ord[qq]; if ((unsigned)id >= (unsigned)n) { id = 0; bad = 1; } so = tbl[id]; }
        if (__any_sync(KV_FULL, bad)) {                                       // an id outside 0..n-1
            if (lane == 0) p.tel_out[c] = INT64_MAX;
            return;
        }
        const int cnt = min(32, n - q0);
        for (int k = 0; k < cnt; ++k) {
            const int s = __shfl_sync(KV_FULL, so.x, k), o = __shfl_sync(KV_FULL, so.y, k);
            const int pstart = sim.admit(s, o, M, lane, p.status);
            if (kStarts && lane == k) starts[id] = pstart;
        }
    }
    if (lane == 0) p.tel_out[c] = sim.total();
}

// ------------------------------------------------------------------------------------------------
// Explicit start times p[c][i].  One warp per candidate.  Requests are visited in ascending start
// order (ids sorted by K1 beforehand: sorted_ids[c][k]); the ring then only has to cover omax
// rounds ahead of the current start.  feasible[c] = 0 as soon as a cell exceeds M (the remaining
// requests are still summed into the TEL but no longer placed).
// ------------------------------------------------------------------------------------------------
struct StartsEvalParams {
    int n, L, M;
    const int2* tbl_id;
    const int* starts;        // [count][n]
    const int* sorted_ids;    // [count][n] ids by ascending (start, id)
    i64 count;
    i64* tel_out;
    unsigned char* feasible_out;
    unsigned int* counter;
};

__global__ void __launch_bounds__(K3S_WARPS * 32, 1)
k3_check_starts(const StartsEvalParams p) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int* ring = (int*)smem_raw + (size_t)warp * p.L;
    const int n = p.n, L = p.L, M = p.M;
    for (;;) {
        unsigned c32 = 0;
        if (lane == 0) c32 = atomicAdd(p.counter, 1u);
        const i64 c = (i64)__shfl_sync(KV_FULL, c32, 0);
        if (c >= p.count) break;
        const int* st_c = p.starts + (size_t)c * n;
        const int* ids = p.sorted_ids + (size_t)c * n;
        for (int r = lane; r < L; r += 32) ring[r] = 0;
        __syncwarp();
        int t = 0, tr = 0;
        i64 tel = 0;
        bool ok = true;
        for (int q0 = 0; q0 < n; q0 += 32) {
            const int qq = q0 + lane;
            int2 so = make_int2(1, 1);
            int pi = 0;
            if (qq < n) { const int id = ids[qq]; so = p.tbl_id[id]; pi = st_c[id]; }
            const int cnt = min(32, n - q0);
            for (int k = 0; k < cnt; ++k) {
                const int s = __shfl_sync(KV_FULL, so.x, k), o = __shfl_sync(KV_FULL, so.y, k);
                const int pk = __shfl_sync(KV_FULL, pi, k);
                tel += (i64)pk + o;
                if (!ok) continue;
                // advance the ring to round pk: cells of rounds t .. pk-1 are finished
                const int adv = pk - t;
                if (adv < 0) { ok = false; continue; }                       // starts not ascending: unsorted or negative input
                if (adv >= L) { for (int r = lane; r < L; r += 32) ring[r] = 0; }
                else for (int r = lane; r < adv; r += 32) ring[kv_wrap(tr + r, L)] = 0;
                __syncwarp();
                tr = adv >= L ? 0 : kv_wrap(tr + adv, L);
                t = pk;
                int over = 0;
                for (int r = lane; r < o; r += 32) {
                    const int idx = kv_wrap(tr + r, L);
                    const int v = ring[idx] + s + 1 + r;
                    ring[idx] = v;
                    over |= v > M;
                }
                __syncwarp();
                if (__any_sync(KV_FULL, over)) ok = false;
            }
        }
        if (lane == 0) {
            p.tel_out[c] = tel;
            if (p.feasible_out) p.feasible_out[c] = ok ? 1 : 0;
        }
    }
}
