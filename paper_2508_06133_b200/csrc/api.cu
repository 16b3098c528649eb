// Host side of the kvsched C-ABI (see include/kvsched.h for the contract of every entry point).
// All scheduling arithmetic runs in the kernels of k1_sort / k2_fmetric / k3_eval / k5_argmin; this
// file validates arguments, owns device memory and enqueues launches.  There is no CPU fallback.
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>
#include <new>
#include <unordered_map>
#include <vector>

#include "common.cuh"
#include "k1_sort.cuh"
#include "k2_fmetric.cuh"
#include "k2_local_swap.cuh"
#include "k2_dp.cuh"
#include "k2_quantile.cuh"
#include "k3_eval.cuh"
#include "k3_policy.cuh"
#include "k5_argmin.cuh"
#include "k6_online.cuh"
#include "k7_amin.cuh"

thread_local char g_last_cuda_error[256] = "";

int kv_cuda_fail(cudaError_t e, const char* what) {
    snprintf(g_last_cuda_error, sizeof(g_last_cuda_error), "%s: %s", what, cudaGetErrorString(e));
    return e == cudaErrorMemoryAllocation ? SCHED_E_NOMEM : SCHED_E_CUDA;
}

namespace {

const i64 kSweepChunk = 1ll << 22;          // candidates per launch inside a sweep
const size_t kSnapBudget = 512ull << 20;    // bytes of snapshot memory before striding kicks in

// Runs CALL(SIM) with SIM = the simulator class of the handle: the register-resident one when the
// longest window fits 33 registers per lane, else the hybrid one (registers + a shared-memory ring
// for the far rounds); the all-shared-memory one on request (KVSCHED_SIM=smem).
#define KV_DISPATCH_SIM(h, CALL)                               \
    if ((h)->hyb) {                                             \
        CALL(HybSim);                                           \
    } else if ((h)->nreg > 0) {                                      \
        switch ((h)->nreg) {                                    \
            case 2: CALL(RegSim<2>); break;                     \
            case 3: CALL(RegSim<3>); break;                     \
            case 5: CALL(RegSim<5>); break;                     \
            case 9: CALL(RegSim<9>); break;                     \
            case 17: CALL(RegSim<17>); break;                   \
            default: CALL(RegSim<33>); break;                   \
        }                                                       \
    } else {                                                    \
        switch ((h)->nit) {                                     \
            case 1: CALL(SmemSim<1>); break;                    \
            case 2: CALL(SmemSim<2>); break;                    \
            case 4: CALL(SmemSim<4>); break;                    \
            case 8: CALL(SmemSim<8>); break;                    \
            default: CALL(SmemSim<0>); break;                   \
        }                                                       \
    }

int bits_of(u64 v) { int b = 0; while (v) { ++b; v >>= 1; } return b; }

// byte mask for a 64-bit key whose low word uses lo_bits and high word hi_bits
unsigned key_byte_mask(int lo_bits, int hi_bits) {
    unsigned m = 0;
    for (int b = 0; b < (lo_bits + 7) / 8; ++b) m |= 1u << b;
    for (int b = 0; b < (hi_bits + 7) / 8; ++b) m |= 1u << (4 + b);
    return m;
}

// ------------------------------------------------------------------------------------------------
// Device-memory cache.  Creating and destroying a handle allocates and frees a few hundred MB (base
// run snapshots, staging, per-candidate scratch); cudaFree of such blocks was seen to take from 2 ms
// to more than half a second on a busy machine.  Blocks of at least 1 MiB therefore go back to a
// process-wide per-device free list (at most KVSCHED_POOL_MB MiB in total, default 1024, 0 turns the
// cache off) and are handed out again to later requests of similar size.  kv_free() waits for the
// device first, exactly as cudaFree does, so a cached block is never still in use.
// sched_release_cached_memory() returns everything to the driver.
// ------------------------------------------------------------------------------------------------
struct PoolBlock { void* p; size_t bytes; int device; };
std::mutex g_pool_mu;
std::vector<PoolBlock> g_pool_free;
std::unordered_map<void*, PoolBlock> g_pool_live;
size_t g_pool_cached = 0;
const size_t kPoolMinBlock = 1ull << 20;

size_t pool_cap_bytes() {
    static const size_t cap = [] {
        const char* e = getenv("KVSCHED_POOL_MB");
        const long long mb = e ? atoll(e) : 1024;
        return (size_t)(mb < 0 ? 0 : mb) << 20;
    }();
    return cap;
}

void pool_trim_locked(int device) {             // device < 0: every device
    for (size_t k = 0; k < g_pool_free.size();) {
        if (device < 0 || g_pool_free[k].device == device) {
            cudaFree(g_pool_free[k].p);
            g_pool_cached -= g_pool_free[k].bytes;
            g_pool_free[k] = g_pool_free.back();
            g_pool_free.pop_back();
        } else {
            ++k;
        }
    }
}

cudaError_t kv_malloc(void** out, size_t bytes) {
    *out = nullptr;
    if (bytes < kPoolMinBlock || pool_cap_bytes() == 0) return cudaMalloc(out, bytes);
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const size_t want = (bytes + (kPoolMinBlock - 1)) & ~(kPoolMinBlock - 1);
    std::lock_guard<std::mutex> lock(g_pool_mu);
    int best = -1;
    for (size_t k = 0; k < g_pool_free.size(); ++k) {
        const PoolBlock& b = g_pool_free[k];
        if (b.device == dev && b.bytes >= want && b.bytes <= 2 * want && (best < 0 || b.bytes < g_pool_free[best].bytes))
            best = (int)k;
    }
    if (best >= 0) {
        const PoolBlock b = g_pool_free[best];
        g_pool_free[best] = g_pool_free.back();
        g_pool_free.pop_back();
        g_pool_cached -= b.bytes;
        g_pool_live[b.p] = b;
        *out = b.p;
        return cudaSuccess;
    }
    e = cudaMalloc(out, want);
    if (e == cudaErrorMemoryAllocation) {       // give the cached blocks back and try once more
        cudaGetLastError();
        pool_trim_locked(dev);
        e = cudaMalloc(out, want);
    }
    if (e == cudaSuccess) g_pool_live[*out] = PoolBlock{*out, want, dev};
    return e;
}

void kv_free(void* p) {
    if (!p) return;
    std::unique_lock<std::mutex> lock(g_pool_mu);
    auto it = g_pool_live.find(p);
    if (it == g_pool_live.end()) { lock.unlock(); cudaFree(p); return; }
    const PoolBlock b = it->second;
    g_pool_live.erase(it);
    if (g_pool_cached + b.bytes > pool_cap_bytes()) { lock.unlock(); cudaFree(p); return; }
    lock.unlock();
    int prev = -1;
    cudaGetDevice(&prev);
    if (prev != b.device) cudaSetDevice(b.device);
    cudaDeviceSynchronize();                    // what cudaFree would have waited for
    if (prev != b.device && prev >= 0) cudaSetDevice(prev);
    lock.lock();
    g_pool_free.push_back(b);
    g_pool_cached += b.bytes;
}

template <typename T>
int dev_alloc(T** p, size_t count) {
    *p = nullptr;
    if (count == 0) count = 1;
    KV_CUDA(kv_malloc((void**)p, count * sizeof(T)));
    return SCHED_OK;
}

int ensure_stage(sched_ctx* h, size_t bytes) {
    if (h->stage_cap >= bytes) return SCHED_OK;
    if (h->d_stage) { kv_free(h->d_stage); h->d_stage = nullptr; h->stage_cap = 0; }
    KV_CUDA(kv_malloc((void**)&h->d_stage, bytes));
    h->stage_cap = bytes;
    return SCHED_OK;
}

int ensure_tel(sched_ctx* h, i64 count) {
    if (h->tel_cap >= count) return SCHED_OK;
    if (h->d_tel) { kv_free(h->d_tel); h->d_tel = nullptr; h->tel_cap = 0; }
    KV_TRY(dev_alloc(&h->d_tel, (size_t)count + 2));
    h->tel_cap = count;
    return SCHED_OK;
}

struct DeviceGuard {
    int prev;
    bool ok;
    explicit DeviceGuard(int dev) : prev(-1), ok(false) {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = (prev == dev) || cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard() { if (ok && prev >= 0) cudaSetDevice(prev); }
};

#define KV_ENTER(h)                                                  \
    if (!(h)) return SCHED_E_INVAL;                                  \
    DeviceGuard guard__((h)->device);                                \
    if (!guard__.ok) return kv_cuda_fail(cudaGetLastError(), "cudaSetDevice")

int check_launch(sched_ctx* h) {
    h->launches += 1;
    KV_CUDA(cudaGetLastError());
    return SCHED_OK;
}

int validate_instance(i64 total, const int32_t* s, const int32_t* o, i64 M) {
    for (i64 i = 0; i < total; ++i) {
        if (s[i] < 1 || o[i] < 1) return SCHED_E_INVAL;
        if ((i64)s[i] + (i64)o[i] > M) return SCHED_E_INVAL;
    }
    return SCHED_OK;
}

void free_ctx(sched_ctx* h) {
    if (!h) return;
    void* ptrs[] = {h->d_s, h->d_o, h->d_tbl_id, h->d_tbl_base, h->d_order, h->d_snap_ring, h->d_snap_hdr,
                    h->d_base_tel, h->d_counter, h->d_status, h->d_tel, h->d_best, h->d_partials, h->d_ticket,
                    h->d_keys_a, h->d_keys_b, h->d_vals_a, h->d_vals_b, h->d_prefP, h->d_prefO,
                    h->d_batch_off, h->d_num_batches, h->d_seg_off, h->d_stage, h->d_base_starts,
                    h->d_state, h->d_sort, h->d_k4, h->d_ls};
    for (void* p : ptrs) if (p) kv_free(p);
    if (h->h_pinned) cudaFreeHost(h->h_pinned);
    if (h->ev_k3_begin) cudaEventDestroy(h->ev_k3_begin);
    if (h->ev_k3_end) cudaEventDestroy(h->ev_k3_end);
    if (h->own_stream) cudaStreamDestroy(h->own_stream);
    delete h;
}

int k3_warps(const sched_ctx* h) {
    int w = 0;
#define GETW(SIM) w = SIM::kWarps
    KV_DISPATCH_SIM(h, GETW);
#undef GETW
    if (h->ring_cells > 0) {                  // one ring per warp has to fit in shared memory
        const int fit = (int)(((size_t)h->smem_optin - 2048) / ((size_t)h->ring_cells * sizeof(int)));
        if (fit < w) w = fit;
    }
    return w;
}

size_t k3_smem_bytes(const sched_ctx* h, bool* table_in_smem, unsigned* table_bytes) {
    const size_t rings = (size_t)k3_warps(h) * h->ring_cells * sizeof(int);
    const unsigned tb = (unsigned)(((size_t)h->n * sizeof(int2) + 15) & ~(size_t)15);
    const size_t with_table = ((size_t)tb + 127) / 128 * 128 + rings;
    if (with_table <= (size_t)h->smem_optin - 2048) {
        *table_in_smem = true; *table_bytes = tb; return with_table;
    }
    *table_in_smem = false; *table_bytes = tb; return rings;
}

int create_common(sched_ctx** out, int B, int n, const int32_t* s, const int32_t* o, i64 M) {
    if (!out) return SCHED_E_INVAL;
    *out = nullptr;
    if (B < 1 || n < 1 || !s || !o || M < 1) return SCHED_E_INVAL;
    if (M >= (1ll << 30)) return SCHED_E_UNSUPPORTED;
    const i64 total = (i64)B * n;
    KV_TRY(validate_instance(total, s, o, M));
    int omax = 0; i64 sum_max = 0;
    for (int b = 0; b < B; ++b) {
        i64 sum = 0;
        for (int i = 0; i < n; ++i) { int v = o[(i64)b * n + i]; sum += v; if (v > omax) omax = v; }
        if (sum > sum_max) sum_max = sum;
    }
    if (sum_max + omax >= (1ll << 30)) return SCHED_E_UNSUPPORTED;

    sched_ctx* h = new (std::nothrow) sched_ctx();
    if (!h) return SCHED_E_NOMEM;
    memset(h, 0, sizeof(*h));
    int rc = SCHED_OK;
    do {
        if (cudaGetDevice(&h->device) != cudaSuccess) { rc = kv_cuda_fail(cudaGetLastError(), "cudaGetDevice"); break; }
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, h->device) != cudaSuccess) { rc = kv_cuda_fail(cudaGetLastError(), "cudaGetDeviceProperties"); break; }
        h->sm_count = prop.multiProcessorCount;
        h->smem_optin = (int)prop.sharedMemPerBlockOptin;
        h->B = B; h->n = n; h->M = M; h->omax = omax; h->sum_o_max = sum_max;
        h->g_num = 0; h->g_den = 1;
        h->nreg = sim_pick_nreg(omax);
        h->hyb = h->nreg == 0;
        if (const char* kind = getenv("KVSCHED_SIM")) {             // testing knob: "smem" / "hybrid" force that simulator
            if (strcmp(kind, "smem") == 0) { h->nreg = 0; h->hyb = false; }
            if (strcmp(kind, "hybrid") == 0) { h->nreg = 0; h->hyb = true; }
        }
        h->nit = sim_pick_nit(omax);
        if (const char* cap = getenv("KVSCHED_MAX_NIT")) {          // tuning knob: windows beyond the cap stream
            const int c = atoi(cap);
            if (c == 0 || c == 1 || c == 2 || c == 4 || c == 8) h->nit = c < h->nit ? c : h->nit;
        }
        // cells per simulator state: registers x 32 lanes, or a ring whose length is a multiple of
        // 32 cells (a wrapped 16-byte access then keeps its bank)
        h->L = h->hyb ? 32 * (HybSim::NREG + sim_pick_far_chunks(omax)) : h->nreg > 0 ? 32 * h->nreg : (omax + 8 + 31) & ~31;
        h->ring_cells = h->hyb ? HybSim::ring_cells(h->L) : h->nreg > 0 ? 0 : h->L;
        if (k3_warps(h) < 1) { rc = SCHED_E_UNSUPPORTED; break; }
        if (cudaStreamCreateWithFlags(&h->own_stream, cudaStreamNonBlocking) != cudaSuccess) { rc = kv_cuda_fail(cudaGetLastError(), "cudaStreamCreate"); break; }
        h->stream = h->own_stream;
        if (cudaEventCreate(&h->ev_k3_begin) != cudaSuccess || cudaEventCreate(&h->ev_k3_end) != cudaSuccess) { rc = kv_cuda_fail(cudaGetLastError(), "cudaEventCreate"); break; }
#define A(call) if ((rc = (call)) != SCHED_OK) break
        A(dev_alloc(&h->d_s, total)); A(dev_alloc(&h->d_o, total));
        A(dev_alloc(&h->d_tbl_id, total + 2));
        A(dev_alloc(&h->d_counter, 4)); A(dev_alloc(&h->d_status, 1));
        A(dev_alloc(&h->d_best, 2)); A(dev_alloc(&h->d_partials, 2 * 4096)); A(dev_alloc(&h->d_ticket, 1));
        A(dev_alloc(&h->d_state, 4));
        if (cudaMallocHost(&h->h_pinned, 64) != cudaSuccess) { rc = kv_cuda_fail(cudaGetLastError(), "cudaMallocHost"); break; }
        if (B == 1) {
            A(dev_alloc(&h->d_tbl_base, n + 2)); A(dev_alloc(&h->d_order, n));
            A(dev_alloc(&h->d_base_starts, n)); A(dev_alloc(&h->d_base_tel, 1));
            A(dev_alloc(&h->d_keys_a, n)); A(dev_alloc(&h->d_keys_b, n));
            A(dev_alloc(&h->d_vals_a, n)); A(dev_alloc(&h->d_vals_b, n));
            A(dev_alloc(&h->d_prefP, n + 1)); A(dev_alloc(&h->d_prefO, n + 1));
            A(dev_alloc(&h->d_batch_off, n + 1)); A(dev_alloc(&h->d_num_batches, 1)); A(dev_alloc(&h->d_seg_off, 2));
            size_t per = (size_t)h->L * sizeof(int);
            i64 stride = (i64)(((size_t)n * per + kSnapBudget - 1) / kSnapBudget);
            if (stride < 1) stride = 1;
            h->snap_stride = (int)stride;
            h->snap_count = (n + h->snap_stride - 1) / h->snap_stride;
            A(dev_alloc(&h->d_snap_ring, (size_t)h->snap_count * h->L));
            A(dev_alloc(&h->d_snap_hdr, h->snap_count));
        }
#undef A
        cudaStream_t st = h->stream;
#define C(call) if ((call) != cudaSuccess) { rc = kv_cuda_fail(cudaGetLastError(), #call); break; }
        C(cudaMemcpyAsync(h->d_s, s, total * sizeof(int), cudaMemcpyHostToDevice, st));
        C(cudaMemcpyAsync(h->d_o, o, total * sizeof(int), cudaMemcpyHostToDevice, st));
        C(cudaMemsetAsync(h->d_tbl_id, 0, (total + 2) * sizeof(int2), st));
        C(cudaMemsetAsync(h->d_status, 0, sizeof(int), st));
        C(cudaMemsetAsync(h->d_ticket, 0, sizeof(unsigned), st));
        C(cudaMemsetAsync(h->d_counter, 0, 4 * sizeof(unsigned), st));
        k3_make_table<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(h->d_s, h->d_o, (int)total, h->d_tbl_id);
        if ((rc = check_launch(h)) != SCHED_OK) break;
        if (B == 1) {
            C(cudaMemsetAsync(h->d_tbl_base, 0, (n + 2) * sizeof(int2), st));
            k3_iota<<<(n + 255) / 256, 256, 0, st>>>(h->d_order, n);
            if ((rc = check_launch(h)) != SCHED_OK) break;
            int seg[2] = {0, n};
            C(cudaMemcpyAsync(h->d_seg_off, seg, sizeof(seg), cudaMemcpyHostToDevice, st));
        }
        // opt in to large dynamic shared memory once
        {
            const int dyn = h->smem_optin - 2048;
            cudaError_t e1 = cudaSuccess, e2 = cudaSuccess, e3 = cudaSuccess, e4 = cudaSuccess;
#define SETATTR(N)                                                                                         \
            e1 = cudaFuncSetAttribute(k3_eval_moves<N, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn);  \
            if (e1 == cudaSuccess) e1 = cudaFuncSetAttribute(k3_eval_moves<N, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn);  \
            e2 = cudaFuncSetAttribute(k3_eval_orders<N, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn); \
            if (e2 == cudaSuccess) e2 = cudaFuncSetAttribute(k3_eval_orders<N, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn); \
            e3 = cudaFuncSetAttribute(k3_eval_policy<N, int>, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn - 2048); \
            if (e3 == cudaSuccess) e3 = cudaFuncSetAttribute(k3_eval_policy<N, i64>, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn - 2048); \
            e4 = cudaFuncSetAttribute(k3_base_run<N>, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn)
            KV_DISPATCH_SIM(h, SETATTR);
#undef SETATTR
            if (e1 != cudaSuccess || e2 != cudaSuccess || e3 != cudaSuccess || e4 != cudaSuccess) {
                rc = kv_cuda_fail(cudaGetLastError(), "cudaFuncSetAttribute(MaxDynamicSharedMemorySize)"); break;
            }
        }
        C(cudaFuncSetAttribute(k3_check_starts, cudaFuncAttributeMaxDynamicSharedMemorySize, h->smem_optin - 2048));
        C(cudaStreamSynchronize(st));       // s, o may be pageable host memory owned by the caller
#undef C
    } while (0);
    if (rc != SCHED_OK) { free_ctx(h); return rc; }
    *out = h;
    return SCHED_OK;
}

// Base order -> position-ordered table, snapshots, base TEL.
int ensure_base(sched_ctx* h) {
    if (h->base_ready) return SCHED_OK;
    const int n = h->n;
    k3_gather_table<<<(n + 255) / 256, 256, 0, h->stream>>>(h->d_tbl_id, h->d_order, n, h->d_tbl_base);
    KV_TRY(check_launch(h));
#define RUN(N) k3_base_run<N><<<1, 32, (size_t)h->ring_cells * sizeof(int), h->stream>>>(                  \
        h->d_tbl_base, n, h->L, (int)h->M, h->snap_stride, h->snap_count, h->d_snap_ring, h->d_snap_hdr, \
        h->d_base_starts, h->d_base_tel, h->d_status)
    KV_DISPATCH_SIM(h, RUN);
#undef RUN
    KV_TRY(check_launch(h));
    h->base_ready = true;
    return SCHED_OK;
}

// one warp per candidate: CTAs needed for `count` candidates
unsigned k3_grid(const sched_ctx* h, i64 count) {
    const int w = k3_warps(h);
    const i64 ctas = (count + w - 1) / w;
    return (unsigned)(ctas < 1 ? 1 : ctas);
}

// K4: launch order of `count` candidates, bucketed by first moved position (longest suffix first)
int order_candidates(sched_ctx* h, const MoveSource& src, i64 count) {
    const size_t need = ((size_t)h->n + 1 + 2 * (size_t)count) * sizeof(int) + 256;
    if (h->k4_cap < need) {
        if (h->d_k4) { kv_free(h->d_k4); h->d_k4 = nullptr; h->k4_cap = 0; }
        KV_CUDA(kv_malloc((void**)&h->d_k4, need));
        h->k4_cap = need;
    }
    int* bins = (int*)h->d_k4;
    int* first_pos = bins + h->n + 1;
    int* launch_order = first_pos + count;
    KV_CUDA(cudaMemsetAsync(bins, 0, ((size_t)h->n + 1) * sizeof(int), h->stream));
    const unsigned blocks = (unsigned)((count + 255) / 256);
    k4_first_pos_histogram<<<blocks, 256, 0, h->stream>>>(src, h->n, count, bins, first_pos);
    KV_TRY(check_launch(h));
    k4_scan_bins<<<1, 1024, 0, h->stream>>>(bins, h->n);
    KV_TRY(check_launch(h));
    k4_scatter_by_first_pos<<<blocks, 256, 0, h->stream>>>(first_pos, h->n, count, bins, launch_order);
    KV_TRY(check_launch(h));
    return SCHED_OK;
}

// by_slot: TELs are left in launch-slot order (h->d_k4's launch_order maps a slot to its candidate
// until the next call); the sweeps that only need the arg-min use it, see launch_argmin.
int launch_moves(sched_ctx* h, int mode, const i64* codes, i64 first, u64 seed, int iteration,
                 i64 count, i64* tel_out, int* starts_out, bool by_slot = false) {
    if (count <= 0) return SCHED_OK;
    if (count >= (1ll << 31)) return SCHED_E_UNSUPPORTED;
    KV_TRY(ensure_base(h));
    MoveEvalParams p;
    memset(&p, 0, sizeof(p));
    bool in_smem; unsigned tb;
    const size_t smem = k3_smem_bytes(h, &in_smem, &tb);
    p.n = h->n; p.L = h->L; p.M = (int)h->M; p.stride = h->snap_stride;
    p.tbl_base = h->d_tbl_base; p.table_in_smem = in_smem ? 1 : 0; p.table_bytes = tb;
    p.snap_ring = h->d_snap_ring; p.snap_hdr = h->d_snap_hdr; p.snap_count = h->snap_count;
    p.src.mode = mode; p.src.codes = codes; p.src.first = first; p.src.seed = seed; p.src.iteration = iteration;
    p.count = count; p.tel_out = tel_out; p.tel_by_slot = by_slot ? 1 : 0; p.starts_out = starts_out;
    p.base_order = h->d_order; p.base_starts_pos = h->d_base_starts;
    p.status = h->d_status;
    KV_TRY(order_candidates(h, p.src, count));
    p.launch_order = (const int*)h->d_k4 + h->n + 1 + count;
    KV_CUDA(cudaEventRecord(h->ev_k3_begin, h->stream));
#define RUN(N)                                                                                    \
    if (starts_out) k3_eval_moves<N, true><<<k3_grid(h, count), k3_warps(h) * 32, smem, h->stream>>>(p);  \
    else k3_eval_moves<N, false><<<k3_grid(h, count), k3_warps(h) * 32, smem, h->stream>>>(p)
    KV_DISPATCH_SIM(h, RUN);
#undef RUN
    KV_TRY(check_launch(h));
    KV_CUDA(cudaEventRecord(h->ev_k3_end, h->stream));
    h->ev_valid = true;
    h->evaluations += count;
    return SCHED_OK;
}

const int* last_launch_order(const sched_ctx* h, i64 count) { return (const int*)h->d_k4 + h->n + 1 + count; }

int launch_argmin(sched_ctx* h, const i64* tel, i64 count, i64 index_base, const i64* prior, i64* best_out,
                  const int* index_map = nullptr) {
    i64 blocks = (count / 2 + K5_THREADS - 1) / K5_THREADS;
    if (blocks < 1) blocks = 1;
    if (blocks > 4 * h->sm_count) blocks = 4 * h->sm_count;
    if (blocks > 4096) blocks = 4096;
    k5_argmin<<<(unsigned)blocks, K5_THREADS, 0, h->stream>>>(tel, count, index_base, index_map, prior, h->d_partials, h->d_ticket, best_out);
    return check_launch(h);
}

i64 neighbourhood_size(int n, int nb, i64 samples) {
    const i64 nsw = (i64)n * (n - 1) / 2;
    return nb == SCHED_NBHD_SWAP ? nsw : nb == SCHED_NBHD_SWAP_INSERT ? nsw + (i64)n * (n - 1) : samples;
}

// Checked build only: the word in which KV_IDX records the first index that left its array.  Reads
// it after the device is idle, clears it, and turns a recorded index into SCHED_E_INTERNAL with the
// site and value in sched_last_cuda_error().
int read_checked_word() {
#ifdef KVSCHED_CHECKED
    unsigned long long w = 0ull;
    KV_CUDA(cudaDeviceSynchronize());
    KV_CUDA(cudaMemcpyFromSymbol(&w, kv_checked_word, sizeof(w)));
    if (w != 0ull) {
        const unsigned long long zero = 0ull;
        cudaMemcpyToSymbol(kv_checked_word, &zero, sizeof(zero));
        long long idx = (long long)(w & 0xffffffffffull);
        if (idx & (1ll << 39)) idx -= (1ll << 40);
        snprintf(g_last_cuda_error, sizeof(g_last_cuda_error), "checked build: index %lld outside its array at site %d",
                 idx, (int)(w >> 40));
        return SCHED_E_INTERNAL;
    }
#endif
    return SCHED_OK;
}

int read_status(sched_ctx* h) {
    int* hp = (int*)h->h_pinned;
    KV_CUDA(cudaMemcpyAsync(hp, h->d_status, sizeof(int), cudaMemcpyDeviceToHost, h->stream));
    KV_CUDA(cudaStreamSynchronize(h->stream));
    if (*hp != KV_DEV_OK) {
        cudaMemsetAsync(h->d_status, 0, sizeof(int), h->stream);
        return SCHED_E_INTERNAL;
    }
    return read_checked_word();
}

#ifdef KVSCHED_CHECKED
__global__ void kv_check_index_probe(long long idx, long long limit, int* sink) {
    *sink = (int)KV_IDX(idx, limit, 9999);
}
#endif

bool is_permutation(const int32_t* a, int n, std::vector<unsigned char>& seen) {
    seen.assign(n, 0);
    for (int q = 0; q < n; ++q) {
        int v = a[q];
        if (v < 0 || v >= n || seen[v]) return false;
        seen[v] = 1;
    }
    return true;
}

}  // namespace

extern "C" {

int sched_init(sched_handle* out, int32_t n, const int32_t* s, const int32_t* o, int64_t M) {
    return create_common(out, 1, n, s, o, M);
}

int sched_init_batch(sched_handle* out, int32_t B, int32_t n_each, const int32_t* s, const int32_t* o, int64_t M) {
    if (n_each > 1024) return SCHED_E_UNSUPPORTED;
    int rc = create_common(out, B, n_each, s, o, M);
    if (rc == SCHED_OK) (*out)->batch_handle = true;
    return rc;
}

int sched_set_stream(sched_handle h, void* cuda_stream) {
    KV_ENTER(h);
    KV_CUDA(cudaStreamSynchronize(h->stream));
    h->stream = cuda_stream ? (cudaStream_t)cuda_stream : h->own_stream;
    return SCHED_OK;
}

int sched_sync(sched_handle h) {
    KV_ENTER(h);
    return read_status(h);
}

int sched_set_prefill_weight(sched_handle h, int32_t alpha_num, int32_t alpha_den) {
    if (!h) return SCHED_E_INVAL;
    if (alpha_num < 0 || alpha_den < 1 || alpha_num > (1 << 20) || alpha_den > (1 << 20)) return SCHED_E_INVAL;
    h->g_num = alpha_num; h->g_den = alpha_den;
    return SCHED_OK;
}

int sched_set_base_order(sched_handle h, const int32_t* order) {
    KV_ENTER(h);
    if (h->batch_handle || !order) return SCHED_E_INVAL;
    std::vector<unsigned char> seen;
    if (!is_permutation(order, h->n, seen)) return SCHED_E_NOT_PERMUTATION;
    KV_CUDA(cudaMemcpyAsync(h->d_order, order, (size_t)h->n * sizeof(int), cudaMemcpyHostToDevice, h->stream));
    KV_CUDA(cudaStreamSynchronize(h->stream));
    h->base_ready = false;
    return SCHED_OK;
}

int sched_get_base_order(sched_handle h, int32_t* order_out) {
    KV_ENTER(h);
    if (h->batch_handle || !order_out) return SCHED_E_INVAL;
    KV_CUDA(cudaMemcpyAsync(order_out, h->d_order, (size_t)h->n * sizeof(int), cudaMemcpyDeviceToHost, h->stream));
    KV_CUDA(cudaStreamSynchronize(h->stream));
    return SCHED_OK;
}

int sched_eval_batch_dev(sched_handle h, int kind, int64_t count, const void* candidates,
                         int64_t* tel_out, uint8_t* feasible_out, int32_t* starts_out) {
    KV_ENTER(h);
    if (count < 0 || !tel_out || (count > 0 && !candidates)) return SCHED_E_INVAL;
    if (count == 0) return SCHED_OK;
    if (count >= (1ll << 31)) return SCHED_E_UNSUPPORTED;
    const int n = h->n;
    if (kind == SCHED_CAND_POLICY) {
        if (n >= 65536) return SCHED_E_UNSUPPORTED;                    // ids are 16-bit inside the kernel
        const bool narrow = (i64)n * h->M < (1ll << 31);               // prefix sums of s+o fit 32 bits
        const size_t shared_so = ((size_t)n * 8 + 15) & ~(size_t)15;
        const size_t per_warp = k3_policy_warp_bytes(n, h->ring_cells, narrow ? 4 : 8);
        const size_t room = (size_t)h->smem_optin - 4096;
        if (shared_so + per_warp > room) return SCHED_E_UNSUPPORTED;
        int W = (int)((room - shared_so) / per_warp);                  // pairs of one instance per CTA
        if (W > K3P_MAX_WARPS) W = K3P_MAX_WARPS;
        if ((i64)W > count) W = (int)count;
        const int groups = (int)((count + W - 1) / W);
        const size_t smem = shared_so + (size_t)W * per_warp;
        const i64 ctas = (i64)h->B * groups;
        if (ctas >= (1ll << 31)) return SCHED_E_UNSUPPORTED;
#define RUN(N)                                                                                                       \
        if (narrow) k3_eval_policy<N, int><<<(unsigned)ctas, 32 * W, smem, h->stream>>>(h->d_s, h->d_o, n, h->L, (int)h->M, h->omax, \
                                                                  (const int*)candidates, (int)count, groups, \
                                                                  (i64*)tel_out, starts_out, h->d_status);   \
        else k3_eval_policy<N, i64><<<(unsigned)ctas, 32 * W, smem, h->stream>>>(h->d_s, h->d_o, n, h->L, (int)h->M, h->omax, \
                                                                  (const int*)candidates, (int)count, groups, \
                                                                  (i64*)tel_out, starts_out, h->d_status)
        KV_CUDA(cudaEventRecord(h->ev_k3_begin, h->stream));
        KV_DISPATCH_SIM(h, RUN);
#undef RUN
        KV_TRY(check_launch(h));
        KV_CUDA(cudaEventRecord(h->ev_k3_end, h->stream));
        h->ev_valid = true;
        h->evaluations += (i64)h->B * count;
        if (feasible_out) KV_CUDA(cudaMemsetAsync(feasible_out, 1, (size_t)((i64)h->B * count), h->stream));
        return SCHED_OK;
    }
    if (h->batch_handle) return SCHED_E_INVAL;
    if (kind == SCHED_CAND_MOVE) {
        KV_TRY(launch_moves(h, 0, (const i64*)candidates, 0, 0, 0, count, (i64*)tel_out, starts_out));
        if (feasible_out) KV_CUDA(cudaMemsetAsync(feasible_out, 1, (size_t)count, h->stream));
        return SCHED_OK;
    }
    if (kind == SCHED_CAND_ORDER) {
        OrderEvalParams p;
        memset(&p, 0, sizeof(p));
        bool in_smem; unsigned tb;
        const size_t smem = k3_smem_bytes(h, &in_smem, &tb);
        p.n = n; p.L = h->L; p.M = (int)h->M; p.tbl_id = h->d_tbl_id;
        p.table_in_smem = in_smem ? 1 : 0; p.table_bytes = tb;
        p.orders = (const int*)candidates; p.count = count; p.tel_out = (i64*)tel_out; p.starts_out = starts_out;
        p.status = h->d_status;
        KV_CUDA(cudaEventRecord(h->ev_k3_begin, h->stream));
#define RUN(N)                                                                                     \
        if (starts_out) k3_eval_orders<N, true><<<k3_grid(h, count), k3_warps(h) * 32, smem, h->stream>>>(p);  \
        else k3_eval_orders<N, false><<<k3_grid(h, count), k3_warps(h) * 32, smem, h->stream>>>(p)
        KV_DISPATCH_SIM(h, RUN);
#undef RUN
        KV_TRY(check_launch(h));
        KV_CUDA(cudaEventRecord(h->ev_k3_end, h->stream));
        h->ev_valid = true;
        h->evaluations += count;
        if (feasible_out) KV_CUDA(cudaMemsetAsync(feasible_out, 1, (size_t)count, h->stream));
        return SCHED_OK;
    }
    if (kind == SCHED_CAND_START_TIMES) {
        if (starts_out) return SCHED_E_INVAL;
        const i64 total = count * n;
        if (total >= (1ll << 31)) return SCHED_E_UNSUPPORTED;
        // ids of every candidate by ascending (start, id): K1 with one segment per candidate
        const size_t need = (size_t)total * (2 * sizeof(u64) + 2 * sizeof(int)) + (size_t)(count + 1) * sizeof(int) + 64;
        if (h->sort_cap < need) {
            if (h->d_sort) { kv_free(h->d_sort); h->d_sort = nullptr; h->sort_cap = 0; }
            KV_CUDA(kv_malloc((void**)&h->d_sort, need));
            h->sort_cap = need;
        }
        u64* ka = (u64*)h->d_sort; u64* kb = ka + total;
        int* va = (int*)(kb + total); int* vb = va + total; int* seg = vb + total;
        k1_keys_start_then_id<<<(unsigned)((total + 255) / 256), 256, 0, h->stream>>>((const int*)candidates, n, total, ka, va, seg, (int)count);
        KV_TRY(check_launch(h));
        const unsigned mask = key_byte_mask(bits_of((u64)n), 31);
        k1_radix_sort_segments<<<(unsigned)(count < 65535 ? count : 65535), K1_THREADS, 0, h->stream>>>(ka, va, kb, vb, seg, nullptr, (int)count, mask);
        KV_TRY(check_launch(h));
        StartsEvalParams p;
        memset(&p, 0, sizeof(p));
        p.n = n; p.L = (h->omax + 8 + 31) & ~31; p.M = (int)h->M; p.tbl_id = h->d_tbl_id;
        p.starts = (const int*)candidates; p.sorted_ids = va; p.count = count;
        p.tel_out = (i64*)tel_out; p.feasible_out = feasible_out; p.counter = h->d_counter;
        KV_CUDA(cudaMemsetAsync(h->d_counter, 0, sizeof(unsigned), h->stream));
        int sw = (int)(((size_t)h->smem_optin - 2048) / ((size_t)p.L * sizeof(int)));
        if (sw > K3S_WARPS) sw = K3S_WARPS;
        if (sw < 1) return SCHED_E_UNSUPPORTED;
        const i64 sctas = (count + sw - 1) / sw;
        k3_check_starts<<<(unsigned)(sctas < h->sm_count ? sctas : h->sm_count), sw * 32,
                          (size_t)sw * p.L * sizeof(int), h->stream>>>(p);
        KV_TRY(check_launch(h));
        h->evaluations += count;
        return SCHED_OK;
    }
    return SCHED_E_INVAL;
}

int sched_eval_batch(sched_handle h, int kind, int64_t count, const void* candidates,
                     int64_t* tel_out, uint8_t* feasible_out, int32_t* starts_out) {
    KV_ENTER(h);
    if (count < 0 || !tel_out || (count > 0 && !candidates)) return SCHED_E_INVAL;
    if (count == 0) return SCHED_OK;
    const int n = h->n;
    size_t cand_bytes = 0; i64 outs = count;
    if (kind == SCHED_CAND_ORDER) {
        if (h->batch_handle) return SCHED_E_INVAL;
        std::vector<unsigned char> seen;
        for (i64 c = 0; c < count; ++c)
            if (!is_permutation((const int32_t*)candidates + c * n, n, seen)) return SCHED_E_NOT_PERMUTATION;
        cand_bytes = (size_t)count * n * sizeof(int);
    } else if (kind == SCHED_CAND_MOVE) {
        if (h->batch_handle || n < 2) return SCHED_E_INVAL;
        const i64 total = neighbourhood_size(n, SCHED_NBHD_SWAP_INSERT, 0);
        for (i64 c = 0; c < count; ++c) {
            i64 code = ((const i64*)candidates)[c];
            if (code < 0 || code >= total) return SCHED_E_INVAL;
        }
        cand_bytes = (size_t)count * sizeof(i64);
    } else if (kind == SCHED_CAND_START_TIMES) {
        if (h->batch_handle || starts_out) return SCHED_E_INVAL;
        for (i64 k = 0; k < count * n; ++k) {
            int v = ((const int32_t*)candidates)[k];
            if (v < 0 || v >= (1 << 30)) return SCHED_E_INVAL;
        }
        cand_bytes = (size_t)count * n * sizeof(int);
    } else if (kind == SCHED_CAND_POLICY) {
        for (i64 c = 0; c < count; ++c) {
            int v = ((const int32_t*)candidates)[c];
            if (v < SCHED_POLICY_FCFS || v > SCHED_POLICY_SORTED_F) return SCHED_E_INVAL;
        }
        cand_bytes = (size_t)count * sizeof(int);
        outs = (i64)h->B * count;
    } else {
        return SCHED_E_INVAL;
    }
    // staging layout: candidates | tel | feasible | starts
    const size_t off_tel = (cand_bytes + 255) & ~(size_t)255;
    const size_t off_feas = off_tel + (((size_t)outs * sizeof(i64) + 255) & ~(size_t)255);
    const size_t off_starts = off_feas + (((size_t)outs + 255) & ~(size_t)255);
    const size_t starts_bytes = starts_out ? (size_t)outs * n * sizeof(int) : 0;
    KV_TRY(ensure_stage(h, off_starts + starts_bytes + 256));
    char* base = (char*)h->d_stage;
    KV_CUDA(cudaMemcpyAsync(base, candidates, cand_bytes, cudaMemcpyHostToDevice, h->stream));
    int rc = sched_eval_batch_dev(h, kind, count, base, (int64_t*)(base + off_tel),
                                  feasible_out ? (uint8_t*)(base + off_feas) : nullptr,
                                  starts_out ? (int32_t*)(base + off_starts) : nullptr);
    if (rc != SCHED_OK) { cudaStreamSynchronize(h->stream); return rc; }
    KV_CUDA(cudaMemcpyAsync(tel_out, base + off_tel, (size_t)outs * sizeof(i64), cudaMemcpyDeviceToHost, h->stream));
    if (feasible_out) KV_CUDA(cudaMemcpyAsync(feasible_out, base + off_feas, (size_t)outs, cudaMemcpyDeviceToHost, h->stream));
    if (starts_out) KV_CUDA(cudaMemcpyAsync(starts_out, base + off_starts, starts_bytes, cudaMemcpyDeviceToHost, h->stream));
    return read_status(h);
}

int sched_sweep_dev(sched_handle h, int sampled, uint64_t seed, int32_t iteration,
                    int64_t first_code, int64_t count, int64_t* tel_out, int64_t* best_out) {
    KV_ENTER(h);
    if (h->batch_handle || h->n < 2 || count <= 0 || first_code < 0 || !best_out) return SCHED_E_INVAL;
    if (!sampled && first_code + count > neighbourhood_size(h->n, SCHED_NBHD_SWAP_INSERT, 0)) return SCHED_E_INVAL;
    if (((uintptr_t)tel_out & 7) || ((uintptr_t)best_out & 7)) return SCHED_E_INVAL;
    i64* tel = (i64*)tel_out;
    for (i64 done = 0; done < count; done += kSweepChunk) {
        const i64 c = count - done < kSweepChunk ? count - done : kSweepChunk;
        i64* dst;
        if (tel) dst = tel + done;
        else { KV_TRY(ensure_tel(h, c)); dst = h->d_tel; }
        const bool by_slot = tel == nullptr;       // nobody reads the scratch TELs by candidate index
        KV_TRY(launch_moves(h, sampled ? 2 : 1, nullptr, first_code + done, seed, iteration, c, dst, nullptr, by_slot));
        KV_TRY(launch_argmin(h, dst, c, first_code + done, done ? (const i64*)best_out : nullptr, (i64*)best_out,
                             by_slot ? last_launch_order(h, c) : nullptr));
    }
    return SCHED_OK;
}

static int phase1_dp(sched_handle h);
static int phase1_quantile(sched_handle h, u64 seed);

static int sorted_f_common_dev(sched_handle h, int solver, int32_t* order_out, int32_t* batch_offsets_out,
                               int32_t* num_batches_out, int64_t* tel_out, u64 seed = 0) {
    KV_ENTER(h);
    if (h->batch_handle) return SCHED_E_INVAL;
    const int n = h->n;
    cudaStream_t st = h->stream;
    if (solver == 0) {
        // S1: ascending (s+o, o, index)
        k1_keys_total_size<<<(n + 255) / 256, 256, 0, st>>>(h->d_s, h->d_o, n, h->d_keys_a, h->d_vals_a, SCHED_POLICY_SORTED_F);
        KV_TRY(check_launch(h));
        k1_radix_sort_segments<<<1, K1_THREADS, 0, st>>>(h->d_keys_a, h->d_vals_a, h->d_keys_b, h->d_vals_b, h->d_seg_off, nullptr, 1,
                                                          key_byte_mask(bits_of((u64)h->omax), bits_of((u64)h->M)));
        KV_TRY(check_launch(h));
        // S2: prefix sums + F-metric batch boundaries
        k2_prefix_f<<<1, 1024, 0, st>>>(h->d_s, h->d_o, h->d_vals_a, n, h->M, h->d_prefP, h->d_prefO, h->d_batch_off, h->d_num_batches,
                                        (i64)h->g_num, (i64)h->g_den);
        KV_TRY(check_launch(h));
    } else if (solver == 2) {
        KV_TRY(phase1_dp(h));
    } else if (solver == 3) {
        KV_TRY(phase1_quantile(h, seed));
    } else {
        // Algorithm 3: ascending (s+o, index), then first fit + improving swaps, batch after batch
        if (!h->d_ls) KV_TRY(dev_alloc(&h->d_ls, 7 * (size_t)n + 32));
        k1_keys_total_size<<<(n + 255) / 256, 256, 0, st>>>(h->d_s, h->d_o, n, h->d_keys_a, h->d_vals_a, SCHED_POLICY_TOTAL_SIZE);
        KV_TRY(check_launch(h));
        k1_radix_sort_segments<<<1, K1_THREADS, 0, st>>>(h->d_keys_a, h->d_vals_a, h->d_keys_b, h->d_vals_b, h->d_seg_off, nullptr, 1,
                                                          key_byte_mask(0, bits_of((u64)h->M)));
        KV_TRY(check_launch(h));
        int* ls = h->d_ls;
        if ((i64)h->g_num * h->M + (i64)h->g_den * h->omax >= (1ll << 31)) return SCHED_E_UNSUPPORTED;   // 32-bit weights
        k2_local_swap<<<1, K2L_THREADS, 0, st>>>(h->d_s, h->d_o, h->d_vals_a, n, h->M, h->g_num, h->g_den, ls, ls + n, ls + 2 * (size_t)n,
                                                 ls + 3 * (size_t)n, ls + 4 * (size_t)n, ls + 5 * (size_t)n, ls + 6 * (size_t)n,
                                                 h->d_vals_b, h->d_batch_off, h->d_num_batches, h->d_status);
        KV_TRY(check_launch(h));
        KV_CUDA(cudaMemcpyAsync(h->d_vals_a, h->d_vals_b, (size_t)n * sizeof(int), cudaMemcpyDeviceToDevice, st));
    }
    // each batch by ascending (o, index)
    k1_keys_output_then_id<<<(n + 255) / 256, 256, 0, st>>>(h->d_o, h->d_vals_a, n, h->d_keys_a, h->d_vals_a);
    KV_TRY(check_launch(h));
    int grid = n < 4 * h->sm_count ? n : 4 * h->sm_count;
    k1_radix_sort_segments<<<grid, K1_THREADS, 0, st>>>(h->d_keys_a, h->d_vals_a, h->d_keys_b, h->d_vals_b, h->d_batch_off, h->d_num_batches, 0,
                                                         key_byte_mask(bits_of((u64)n), bits_of((u64)h->omax)));
    KV_TRY(check_launch(h));
    KV_CUDA(cudaMemcpyAsync(h->d_order, h->d_vals_a, (size_t)n * sizeof(int), cudaMemcpyDeviceToDevice, st));
    h->base_ready = false;
    KV_TRY(ensure_base(h));
    if (order_out) KV_CUDA(cudaMemcpyAsync(order_out, h->d_order, (size_t)n * sizeof(int), cudaMemcpyDeviceToDevice, st));
    if (batch_offsets_out) KV_CUDA(cudaMemcpyAsync(batch_offsets_out, h->d_batch_off, (size_t)(n + 1) * sizeof(int), cudaMemcpyDeviceToDevice, st));
    if (num_batches_out) KV_CUDA(cudaMemcpyAsync(num_batches_out, h->d_num_batches, sizeof(int), cudaMemcpyDeviceToDevice, st));
    if (tel_out) KV_CUDA(cudaMemcpyAsync(tel_out, h->d_base_tel, sizeof(i64), cudaMemcpyDeviceToDevice, st));
    return SCHED_OK;
}

static int sorted_f_common_host(sched_handle h, int solver, int32_t* order_out, int32_t* batch_offsets_out,
                                int32_t* num_batches_out, int64_t* tel_out, u64 seed = 0) {
    KV_ENTER(h);
    KV_TRY(sorted_f_common_dev(h, solver, nullptr, nullptr, nullptr, nullptr, seed));
    const int n = h->n;
    cudaStream_t st = h->stream;
    int nb = 0;
    KV_CUDA(cudaMemcpyAsync(&nb, h->d_num_batches, sizeof(int), cudaMemcpyDeviceToHost, st));
    if (order_out) KV_CUDA(cudaMemcpyAsync(order_out, h->d_order, (size_t)n * sizeof(int), cudaMemcpyDeviceToHost, st));
    if (tel_out) KV_CUDA(cudaMemcpyAsync(tel_out, h->d_base_tel, sizeof(i64), cudaMemcpyDeviceToHost, st));
    KV_CUDA(cudaStreamSynchronize(st));
    if (num_batches_out) *num_batches_out = nb;
    if (batch_offsets_out) {
        KV_CUDA(cudaMemcpyAsync(batch_offsets_out, h->d_batch_off, (size_t)(nb + 1) * sizeof(int), cudaMemcpyDeviceToHost, st));
    }
    return read_status(h);
}

// Algorithm 2 batch after batch; leaves the batches (members in ascending index) in d_vals_a and the
// boundaries in d_batch_off / d_num_batches.  Synchronises once per batch (n <= 128 batches).
static int phase1_dp(sched_handle h) {
    const int n = h->n;
    if (n > 128) return SCHED_E_UNSUPPORTED;
    const int W = (int)h->M + 1, words = (W + 31) / 32;
    const i64 cells_max = (i64)(n + 1) * W;
    if (cells_max > (1ll << 26)) return SCHED_E_UNSUPPORTED;
    cudaStream_t st = h->stream;
    int *dpA = nullptr, *dpB = nullptr, *small = nullptr;
    unsigned* took = nullptr;
    int rc = SCHED_OK;
    do {
        if ((rc = dev_alloc(&dpA, (size_t)cells_max)) != SCHED_OK) break;
        if ((rc = dev_alloc(&dpB, (size_t)cells_max)) != SCHED_OK) break;
        if ((rc = dev_alloc(&took, (size_t)n * (n + 1) * words)) != SCHED_OK) break;
        if ((rc = dev_alloc(&small, 8)) != SCHED_OK) break;            // {pick k, m, v, -, nr, nb, done, -}
        int init[8] = {0, 0, 0, 0, n, 0, 0, 0};
        int zero = 0;
#define DP_CUDA(call) if ((call) != cudaSuccess) { rc = kv_cuda_fail(cudaGetLastError(), #call); break; }
        DP_CUDA(cudaMemcpyAsync(small, init, sizeof(init), cudaMemcpyHostToDevice, st));
        DP_CUDA(cudaMemcpyAsync(h->d_batch_off, &zero, sizeof(int), cudaMemcpyHostToDevice, st));
        k3_iota<<<(n + 255) / 256, 256, 0, st>>>(h->d_vals_b, n);       // remaining list, ascending index
        if ((rc = check_launch(h)) != SCHED_OK) break;
        int nr = n;
        int* hp = (int*)h->h_pinned;
        while (nr > 0 && rc == SCHED_OK) {
            const int rows = nr + 1;
            const i64 cells = (i64)rows * W;
            k2d_init<<<(unsigned)((cells + 255) / 256), 256, 0, st>>>(dpA, cells);
            if ((rc = check_launch(h)) != SCHED_OK) break;
            int *cur = dpA, *nxt = dpB;
            const i64 threads = (i64)rows * words;
            for (int a = 0; a < nr; ++a) {
                k2d_step<<<(unsigned)((threads + 127) / 128), 128, 0, st>>>(cur, nxt, took + (size_t)a * rows * words, rows, W, words,
                                                                             h->d_s, h->d_o, h->d_vals_b, a);
                if ((rc = check_launch(h)) != SCHED_OK) break;
                int* tmp = cur; cur = nxt; nxt = tmp;
            }
            if (rc != SCHED_OK) break;
            k2d_select<<<1, 1024, 0, st>>>(cur, rows, W, small);
            if ((rc = check_launch(h)) != SCHED_OK) break;
            k2d_apply<<<1, 128, 0, st>>>(h->d_s, h->d_o, took, W, words, rows, small, h->d_vals_b, small + 4,
                                         h->d_vals_a, h->d_batch_off, small + 5, small + 6);
            if ((rc = check_launch(h)) != SCHED_OK) break;
            DP_CUDA(cudaMemcpyAsync(hp, small + 4, sizeof(int), cudaMemcpyDeviceToHost, st));
            DP_CUDA(cudaStreamSynchronize(st));
            if (*hp >= nr) { rc = SCHED_E_INTERNAL; break; }            // every batch places at least one request
            nr = *hp;
        }
        if (rc != SCHED_OK) break;
        DP_CUDA(cudaMemcpyAsync(h->d_num_batches, small + 5, sizeof(int), cudaMemcpyDeviceToDevice, st));
        DP_CUDA(cudaStreamSynchronize(st));
#undef DP_CUDA
    } while (0);
    cudaStreamSynchronize(st);
    if (dpA) kv_free(dpA);
    if (dpB) kv_free(dpB);
    if (took) kv_free(took);
    if (small) kv_free(small);
    return rc;
}

// Algorithm 4 batch after batch; leaves the batches (members in ascending (o, index)) in d_vals_a and
// the boundaries in d_batch_off / d_num_batches.  Reads the batch size back once per batch.
static int phase1_quantile(sched_handle h, u64 seed) {
    const int n = h->n;
    cudaStream_t st = h->stream;
    // fixed-point ratio key: 2^F must exceed the product of two sizes s+o <= M, and o * 2^F must fit
    const int F = 2 * bits_of((u64)h->M);
    if (F + bits_of((u64)h->omax) > 63) return SCHED_E_UNSUPPORTED;
    if (!h->d_ls) KV_TRY(dev_alloc(&h->d_ls, 7 * (size_t)n + 32));
    int* rem = h->d_ls;
    int* rem_next = rem + n;
    int* chosen = rem + 2 * (size_t)n;
    int* va = rem + 3 * (size_t)n;
    int* vb = rem + 4 * (size_t)n;
    int* small = rem + 5 * (size_t)n + (n & 1);            // even offset: nothing here needs more
    u64 *ka = h->d_keys_a, *kb = h->d_keys_b;
    const int blocks = (n + 255) / 256;
    // the remaining list: everything, ascending (o, index)
    k1_keys_total_size<<<blocks, 256, 0, st>>>(h->d_s, h->d_o, n, ka, rem, SCHED_POLICY_SOF);
    KV_TRY(check_launch(h));
    k1_radix_sort_segments<<<1, K1_THREADS, 0, st>>>(ka, rem, kb, rem_next, h->d_seg_off, nullptr, 1,
                                                      key_byte_mask(0, bits_of((u64)h->omax)));
    KV_TRY(check_launch(h));
    int zero = 0;
    KV_CUDA(cudaMemcpyAsync(h->d_batch_off, &zero, sizeof(int), cudaMemcpyHostToDevice, st));
    const unsigned mask_size = key_byte_mask(bits_of((u64)h->M), 0);
    const unsigned mask_ratio = key_byte_mask(F + 1 < 32 ? F + 1 : 32, F + 1 > 32 ? F + 1 - 32 : 0) | 0x80u;
    int nr = n, nb = 0, done = 0;
    int* hp = (int*)h->h_pinned;
    while (nr > 0) {
        const int m = nr / 2 > 1 ? nr / 2 : 1;
        const int g = (nr + 255) / 256;
        k2q_begin<<<g, 256, 0, st>>>(rem, nr, seed, nb, ka, va, chosen, small);
        KV_TRY(check_launch(h));
        k1_radix_sort_segments<<<1, K1_THREADS, 0, st>>>(ka, va, kb, vb, small + K2Q_SEG1, nullptr, 1, 0xffu);
        KV_TRY(check_launch(h));
        k2q_sample_keys<<<(m + 255) / 256, 256, 0, st>>>(rem, va, m, h->d_s, h->d_o, ka);
        KV_TRY(check_launch(h));
        k1_radix_sort_segments<<<2, K1_THREADS, 0, st>>>(ka, va, kb, vb, small + K2Q_SEG2, nullptr, 2, mask_size);
        KV_TRY(check_launch(h));
        k2q_pass1<<<1, K2Q_THREADS, 0, st>>>(rem, nr, m, h->d_s, h->d_o, h->M, ka, chosen, small);
        KV_TRY(check_launch(h));
        k2q_ratio_keys<<<g, 256, 0, st>>>(rem, nr, h->d_s, h->d_o, chosen, F, ka, va);
        KV_TRY(check_launch(h));
        k1_radix_sort_segments<<<1, K1_THREADS, 0, st>>>(ka, va, kb, vb, small + K2Q_SEG1, nullptr, 1, mask_ratio);
        KV_TRY(check_launch(h));
        k2q_pass2_emit<<<1, K2Q_THREADS, 0, st>>>(rem, rem_next, nr, h->d_s, h->d_o, h->M, va, chosen, small,
                                                  h->d_vals_a, done, h->d_batch_off, nb);
        KV_TRY(check_launch(h));
        KV_CUDA(cudaMemcpyAsync(hp, small + K2Q_COUNT, sizeof(int), cudaMemcpyDeviceToHost, st));
        KV_CUDA(cudaStreamSynchronize(st));
        const int took = *hp;
        if (took < 1 || took > nr) return SCHED_E_INTERNAL;      // every batch places at least one request
        nr -= took; done += took; ++nb;
        int* tmp = rem; rem = rem_next; rem_next = tmp;
    }
    KV_CUDA(cudaMemcpyAsync(h->d_num_batches, &nb, sizeof(int), cudaMemcpyHostToDevice, st));
    KV_CUDA(cudaStreamSynchronize(st));                          // nb lives on this stack frame
    return SCHED_OK;
}

int sched_sorted_f_dev(sched_handle h, int32_t* order_out, int32_t* batch_offsets_out,
                       int32_t* num_batches_out, int64_t* tel_out) {
    return sorted_f_common_dev(h, 0, order_out, batch_offsets_out, num_batches_out, tel_out);
}

int sched_sorted_f_local_swap_dev(sched_handle h, int32_t* order_out, int32_t* batch_offsets_out,
                                  int32_t* num_batches_out, int64_t* tel_out) {
    return sorted_f_common_dev(h, 1, order_out, batch_offsets_out, num_batches_out, tel_out);
}

int sched_sorted_f_local_swap(sched_handle h, int32_t* order_out, int32_t* batch_offsets_out,
                              int32_t* num_batches_out, int64_t* tel_out) {
    return sorted_f_common_host(h, 1, order_out, batch_offsets_out, num_batches_out, tel_out);
}

int sched_sorted_f_dp(sched_handle h, int32_t* order_out, int32_t* batch_offsets_out,
                      int32_t* num_batches_out, int64_t* tel_out) {
    return sorted_f_common_host(h, 2, order_out, batch_offsets_out, num_batches_out, tel_out);
}

int sched_sorted_f_quantile(sched_handle h, uint64_t seed, int32_t* order_out, int32_t* batch_offsets_out,
                            int32_t* num_batches_out, int64_t* tel_out) {
    return sorted_f_common_host(h, 3, order_out, batch_offsets_out, num_batches_out, tel_out, (u64)seed);
}

int sched_sorted_f(sched_handle h, int32_t* order_out, int32_t* batch_offsets_out,
                   int32_t* num_batches_out, int64_t* tel_out) {
    return sorted_f_common_host(h, 0, order_out, batch_offsets_out, num_batches_out, tel_out);
}

int sched_local_search(sched_handle h, int neighbourhood, int32_t iters, uint64_t seed,
                       int64_t samples_per_iter, int32_t* order_inout, int64_t* tel_out,
                       int32_t* iters_done_out, int64_t* trace_out) {
    KV_ENTER(h);
    if (h->batch_handle || iters < 0) return SCHED_E_INVAL;
    if (neighbourhood < SCHED_NBHD_SWAP || neighbourhood > SCHED_NBHD_SAMPLED) return SCHED_E_INVAL;
    if (neighbourhood == SCHED_NBHD_SAMPLED && samples_per_iter < 1) return SCHED_E_INVAL;
    const int n = h->n;
    if (order_inout) KV_TRY(sched_set_base_order(h, order_inout));
    cudaStream_t st = h->stream;
    const int sampled = neighbourhood == SCHED_NBHD_SAMPLED ? 1 : 0;
    const i64 total = n >= 2 ? neighbourhood_size(n, neighbourhood, samples_per_iter) : 0;
    KV_TRY(ensure_base(h));
    i64* d_cur = (i64*)h->d_state;               // {current TEL, accepted flag}
    int* d_acc = (int*)(d_cur + 1);
    KV_CUDA(cudaMemcpyAsync(d_cur, h->d_base_tel, sizeof(i64), cudaMemcpyDeviceToDevice, st));
    i64* hp = (i64*)h->h_pinned;                 // {best TEL, best code, accepted, base TEL}
    int it = 0;
    i64 cur_tel = 0;
    KV_CUDA(cudaMemcpyAsync(&hp[3], h->d_base_tel, sizeof(i64), cudaMemcpyDeviceToHost, st));
    KV_CUDA(cudaStreamSynchronize(st));
    cur_tel = hp[3];
    for (; it < iters && total > 0; ++it) {
        KV_TRY(ensure_tel(h, total < kSweepChunk ? total : kSweepChunk));
        for (i64 done = 0; done < total; done += kSweepChunk) {
            const i64 c = total - done < kSweepChunk ? total - done : kSweepChunk;
            KV_TRY(launch_moves(h, sampled ? 2 : 1, nullptr, done, seed, it, c, h->d_tel, nullptr, true));
            KV_TRY(launch_argmin(h, h->d_tel, c, done, done ? h->d_best : nullptr, h->d_best, last_launch_order(h, c)));
        }
        k5_accept_move<<<1, 256, 0, st>>>(h->d_order, n, h->d_best, d_cur, d_acc, h->d_vals_b, sampled, seed, it);
        KV_TRY(check_launch(h));
        KV_CUDA(cudaMemcpyAsync(&hp[0], h->d_best, 2 * sizeof(i64), cudaMemcpyDeviceToHost, st));
        KV_CUDA(cudaMemcpyAsync(&hp[2], d_acc, sizeof(int), cudaMemcpyDeviceToHost, st));
        KV_CUDA(cudaStreamSynchronize(st));
        if (trace_out) { trace_out[2 * it] = hp[1]; trace_out[2 * it + 1] = hp[0]; }
        const bool accepted = *(int*)&hp[2] != 0;
        if (accepted) {
            cur_tel = hp[0];
            h->base_ready = false;
            KV_TRY(ensure_base(h));
            // the re-simulated base order must reproduce the TEL that won the sweep
            KV_CUDA(cudaMemcpyAsync(&hp[3], h->d_base_tel, sizeof(i64), cudaMemcpyDeviceToHost, st));
            KV_CUDA(cudaStreamSynchronize(st));
            if (hp[3] != cur_tel) return SCHED_E_INTERNAL;
        } else if (!sampled) {
            ++it;
            break;
        }
    }
    if (order_inout) KV_CUDA(cudaMemcpyAsync(order_inout, h->d_order, (size_t)n * sizeof(int), cudaMemcpyDeviceToHost, st));
    if (tel_out) *tel_out = cur_tel;
    if (iters_done_out) *iters_done_out = it;
    return read_status(h);
}

int sched_accept_move(sched_handle h, int64_t best_tel, int64_t best_index, int sampled, uint64_t seed,
                      int32_t iteration, int32_t* accepted_out, int64_t* tel_out) {
    KV_ENTER(h);
    if (h->batch_handle || h->n < 2 || best_index < 0 || iteration < 0) return SCHED_E_INVAL;
    const int n = h->n;
    if (!sampled && best_index >= neighbourhood_size(n, SCHED_NBHD_SWAP_INSERT, 0)) return SCHED_E_INVAL;
    cudaStream_t st = h->stream;
    KV_TRY(ensure_base(h));
    i64* d_cur = (i64*)h->d_state;               // {current TEL, accepted flag}
    int* d_acc = (int*)(d_cur + 1);
    i64* hp = (i64*)h->h_pinned;                 // {best TEL, best index, accepted, base TEL}
    hp[0] = best_tel; hp[1] = best_index;
    KV_CUDA(cudaMemcpyAsync(h->d_best, hp, 2 * sizeof(i64), cudaMemcpyHostToDevice, st));
    KV_CUDA(cudaMemcpyAsync(d_cur, h->d_base_tel, sizeof(i64), cudaMemcpyDeviceToDevice, st));
    k5_accept_move<<<1, 256, 0, st>>>(h->d_order, n, h->d_best, d_cur, d_acc, h->d_vals_b, sampled ? 1 : 0, seed, iteration);
    KV_TRY(check_launch(h));
    KV_CUDA(cudaMemcpyAsync(&hp[2], d_acc, sizeof(int), cudaMemcpyDeviceToHost, st));
    KV_CUDA(cudaStreamSynchronize(st));
    const bool accepted = *(int*)&hp[2] != 0;
    if (accepted) {
        h->base_ready = false;
        KV_TRY(ensure_base(h));
    }
    KV_CUDA(cudaMemcpyAsync(&hp[3], h->d_base_tel, sizeof(i64), cudaMemcpyDeviceToHost, st));
    KV_CUDA(cudaStreamSynchronize(st));
    // the re-simulated order must reproduce the TEL that the caller's sweep reported for this move
    if (accepted && hp[3] != best_tel) return SCHED_E_INTERNAL;
    if (accepted_out) *accepted_out = accepted ? 1 : 0;
    if (tel_out) *tel_out = hp[3];
    return read_status(h);
}

int sched_last_eval_kernel_ms(sched_handle h, float* ms_out) {
    KV_ENTER(h);
    if (!ms_out || !h->ev_valid) return SCHED_E_INVAL;
    KV_CUDA(cudaEventSynchronize(h->ev_k3_end));
    KV_CUDA(cudaEventElapsedTime(ms_out, h->ev_k3_begin, h->ev_k3_end));
    return SCHED_OK;
}

int sched_online_simulate(int32_t B, int32_t n_max, const int32_t* n_each, const int32_t* arrival,
                          const int32_t* s, const int32_t* o, int64_t M, int32_t policy, int32_t period,
                          int32_t lookahead, int32_t* start_out, int64_t* latency_out, float* kernel_ms_out) {
    if (B < 1 || n_max < 1 || n_max > K6_MAX_N || !n_each || !arrival || !s || !o || !start_out || !latency_out)
        return SCHED_E_INVAL;
    if (policy != SCHED_POLICY_FCFS && policy != SCHED_POLICY_SOF && policy != SCHED_POLICY_SORTED_F) return SCHED_E_INVAL;
    if (period < 1 || lookahead < 1 || M < 2) return SCHED_E_INVAL;
    if (M >= (1ll << 30) || lookahead > K6_MAX_LOOKAHEAD) return SCHED_E_UNSUPPORTED;
    int omax = 1;
    for (int b = 0; b < B; ++b) {
        const int n = n_each[b];
        if (n < 1 || n > n_max) return SCHED_E_INVAL;
        const size_t base = (size_t)b * n_max;
        i64 sum_o = 0;
        for (int i = 0; i < n; ++i) {
            const int ai = arrival[base + i], si = s[base + i], oi = o[base + i];
            if (ai < 0 || si < 1 || oi < 1 || (i64)si + oi > M) return SCHED_E_INVAL;
            if (i > 0 && ai < arrival[base + i - 1]) return SCHED_E_INVAL;
            if (ai >= (1 << 29)) return SCHED_E_UNSUPPORTED;
            omax = oi > omax ? oi : omax;
            sum_o += oi;
        }
        if (sum_o >= (1ll << 29)) return SCHED_E_UNSUPPORTED;
    }
    if (omax > K6_MAX_O) return SCHED_E_UNSUPPORTED;
    OnlineParams P;
    memset(&P, 0, sizeof(P));
    P.n_max = n_max; P.M = (int)M; P.policy = policy; P.period = period; P.lookahead = lookahead;
    P.L = 32; while (P.L < omax) P.L <<= 1;
    P.npow2 = 2; while (P.npow2 < n_max) P.npow2 <<= 1;
    const size_t smem = sizeof(u64) * (size_t)P.npow2 + sizeof(int) * ((size_t)5 * n_max + P.L + (size_t)9 * lookahead);
    int dev = 0, optin = 0;
    KV_CUDA(cudaGetDevice(&dev));
    KV_CUDA(cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    if (smem + 4096 > (size_t)optin) return SCHED_E_UNSUPPORTED;
    KV_CUDA(cudaFuncSetAttribute(k6_online, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));

    const size_t cells = (size_t)B * n_max;
    int *d_n = nullptr, *d_a = nullptr, *d_s = nullptr, *d_o = nullptr, *d_start = nullptr, *d_status = nullptr;
    i64* d_lat = nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    int rc = SCHED_OK;
    do {
#define ON_CUDA(call) if ((call) != cudaSuccess) { rc = kv_cuda_fail(cudaGetLastError(), #call); break; }
        if ((rc = dev_alloc(&d_n, (size_t)B)) != SCHED_OK) break;
        if ((rc = dev_alloc(&d_a, cells)) != SCHED_OK) break;
        if ((rc = dev_alloc(&d_s, cells)) != SCHED_OK) break;
        if ((rc = dev_alloc(&d_o, cells)) != SCHED_OK) break;
        if ((rc = dev_alloc(&d_start, cells)) != SCHED_OK) break;
        if ((rc = dev_alloc(&d_lat, (size_t)B)) != SCHED_OK) break;
        if ((rc = dev_alloc(&d_status, 1)) != SCHED_OK) break;
        ON_CUDA(cudaEventCreate(&e0));
        ON_CUDA(cudaEventCreate(&e1));
        ON_CUDA(cudaMemcpy(d_n, n_each, sizeof(int) * (size_t)B, cudaMemcpyHostToDevice));
        ON_CUDA(cudaMemcpy(d_a, arrival, sizeof(int) * cells, cudaMemcpyHostToDevice));
        ON_CUDA(cudaMemcpy(d_s, s, sizeof(int) * cells, cudaMemcpyHostToDevice));
        ON_CUDA(cudaMemcpy(d_o, o, sizeof(int) * cells, cudaMemcpyHostToDevice));
        ON_CUDA(cudaMemset(d_start, 0xff, sizeof(int) * cells));          // -1 where there is no request
        ON_CUDA(cudaMemset(d_status, 0, sizeof(int)));
        P.n_each = d_n; P.a = d_a; P.s = d_s; P.o = d_o; P.start_out = d_start; P.latency_out = d_lat; P.status = d_status;
        ON_CUDA(cudaEventRecord(e0, 0));
        k6_online<<<B, K6_THREADS, smem, 0>>>(P);
        ON_CUDA(cudaGetLastError());
        ON_CUDA(cudaEventRecord(e1, 0));
        ON_CUDA(cudaDeviceSynchronize());
        int status = 0;
        ON_CUDA(cudaMemcpy(&status, d_status, sizeof(int), cudaMemcpyDeviceToHost));
        if (status != 0) { rc = SCHED_E_INTERNAL; break; }
        if ((rc = read_checked_word()) != SCHED_OK) break;
        ON_CUDA(cudaMemcpy(start_out, d_start, sizeof(int) * cells, cudaMemcpyDeviceToHost));
        ON_CUDA(cudaMemcpy(latency_out, d_lat, sizeof(i64) * (size_t)B, cudaMemcpyDeviceToHost));
        if (kernel_ms_out) ON_CUDA(cudaEventElapsedTime(kernel_ms_out, e0, e1));
#undef ON_CUDA
    } while (0);
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    int* frees[] = {d_n, d_a, d_s, d_o, d_start, d_status};
    for (int* ptr : frees) if (ptr) kv_free(ptr);
    if (d_lat) kv_free(d_lat);
    return rc;
}

// Shared by the two A_min entry points: validates the scenarios on the host, stages them, runs k7_amin.
// order_host: [B, n_max] host lists, or NULL when order_dev (one device row of n_max entries) is given.
static int amin_run(int32_t B, int32_t n_max, const int32_t* n_each, const int32_t* s, const int32_t* lower,
                    const int32_t* o, int64_t M, const int32_t* order_host, const int32_t* order_dev,
                    int32_t* start_out, int64_t* tel_out, int64_t* evictions_out, int64_t* peak_out,
                    float* kernel_ms_out) {
    if (B < 1 || n_max < 1 || !n_each || !s || !lower || !o || (!order_host && !order_dev) || !start_out || !tel_out)
        return SCHED_E_INVAL;
    if (M < 2) return SCHED_E_INVAL;
    if (n_max > K7_MAX_N || M >= (1ll << 30)) return SCHED_E_UNSUPPORTED;
    int omax = 1;
    std::vector<unsigned char> seen;
    for (int b = 0; b < B; ++b) {
        const int n = n_each[b];
        if (n < 1 || n > n_max) return SCHED_E_INVAL;
        const size_t base = (size_t)b * n_max;
        for (int i = 0; i < n; ++i) {
            const int si = s[base + i], oi = o[base + i], li = lower[base + i];
            if (si < 1 || oi < 1 || li < 1 || li > oi || (i64)si + oi > M) return SCHED_E_INVAL;
            omax = oi > omax ? oi : omax;
        }
        if (order_host) {
            seen.assign((size_t)n, 0);
            for (int q = 0; q < n; ++q) {
                const int id = order_host[base + q];
                if (id < 0 || id >= n || seen[id]) return SCHED_E_NOT_PERMUTATION;
                seen[id] = 1;
            }
        }
    }
    if (omax > K7_MAX_O) return SCHED_E_UNSUPPORTED;
    AminParams P;
    memset(&P, 0, sizeof(P));
    P.n_max = n_max; P.M = (int)M;
    P.L = 32; while (P.L < omax + 2) P.L <<= 1;
    const size_t smem = sizeof(int) * ((size_t)5 * n_max + (size_t)4 * P.L);
    int dev = 0, optin = 0;
    KV_CUDA(cudaGetDevice(&dev));
    KV_CUDA(cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    if (smem + 1024 > (size_t)optin) return SCHED_E_UNSUPPORTED;
    KV_CUDA(cudaFuncSetAttribute(k7_amin, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));

    const size_t cells = (size_t)B * n_max;
    int *d_n = nullptr, *d_s = nullptr, *d_l = nullptr, *d_o = nullptr, *d_ord = nullptr, *d_start = nullptr, *d_status = nullptr;
    i64* d_res = nullptr;                                   // tel | evictions | peak, B each
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    int rc = SCHED_OK;
    do {
#define AM_CUDA(call) if ((call) != cudaSuccess) { rc = kv_cuda_fail(cudaGetLastError(), #call); break; }
        if ((rc = dev_alloc(&d_n, (size_t)B)) != SCHED_OK) break;
        if ((rc = dev_alloc(&d_s, cells)) != SCHED_OK) break;
        if ((rc = dev_alloc(&d_l, cells)) != SCHED_OK) break;
        if ((rc = dev_alloc(&d_o, cells)) != SCHED_OK) break;
        if (order_host && (rc = dev_alloc(&d_ord, cells)) != SCHED_OK) break;
        if ((rc = dev_alloc(&d_start, cells)) != SCHED_OK) break;
        if ((rc = dev_alloc(&d_res, (size_t)3 * B)) != SCHED_OK) break;
        if ((rc = dev_alloc(&d_status, 1)) != SCHED_OK) break;
        AM_CUDA(cudaEventCreate(&e0));
        AM_CUDA(cudaEventCreate(&e1));
        AM_CUDA(cudaMemcpy(d_n, n_each, sizeof(int) * (size_t)B, cudaMemcpyHostToDevice));
        AM_CUDA(cudaMemcpy(d_s, s, sizeof(int) * cells, cudaMemcpyHostToDevice));
        AM_CUDA(cudaMemcpy(d_l, lower, sizeof(int) * cells, cudaMemcpyHostToDevice));
        AM_CUDA(cudaMemcpy(d_o, o, sizeof(int) * cells, cudaMemcpyHostToDevice));
        if (order_host) AM_CUDA(cudaMemcpy(d_ord, order_host, sizeof(int) * cells, cudaMemcpyHostToDevice));
        AM_CUDA(cudaMemset(d_start, 0xff, sizeof(int) * cells));           // -1 where a row has no request
        AM_CUDA(cudaMemset(d_status, 0, sizeof(int)));
        P.n_each = d_n; P.s = d_s; P.lower = d_l; P.o = d_o;
        P.order = order_host ? d_ord : order_dev;
        P.order_stride = order_host ? (size_t)n_max : 0;
        P.start_out = d_start; P.tel_out = d_res; P.evict_out = d_res + B; P.peak_out = d_res + 2 * (size_t)B;
        P.status = d_status;
        AM_CUDA(cudaEventRecord(e0, 0));
        k7_amin<<<B, K7_THREADS, smem, 0>>>(P);
        AM_CUDA(cudaGetLastError());
        AM_CUDA(cudaEventRecord(e1, 0));
        AM_CUDA(cudaDeviceSynchronize());
        int status = 0;
        AM_CUDA(cudaMemcpy(&status, d_status, sizeof(int), cudaMemcpyDeviceToHost));
        if (status != 0) { rc = SCHED_E_INTERNAL; break; }
        if ((rc = read_checked_word()) != SCHED_OK) break;
        AM_CUDA(cudaMemcpy(start_out, d_start, sizeof(int) * cells, cudaMemcpyDeviceToHost));
        AM_CUDA(cudaMemcpy(tel_out, d_res, sizeof(i64) * (size_t)B, cudaMemcpyDeviceToHost));
        if (evictions_out) AM_CUDA(cudaMemcpy(evictions_out, d_res + B, sizeof(i64) * (size_t)B, cudaMemcpyDeviceToHost));
        if (peak_out) AM_CUDA(cudaMemcpy(peak_out, d_res + 2 * (size_t)B, sizeof(i64) * (size_t)B, cudaMemcpyDeviceToHost));
        if (kernel_ms_out) AM_CUDA(cudaEventElapsedTime(kernel_ms_out, e0, e1));
#undef AM_CUDA
    } while (0);
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    int* frees[] = {d_n, d_s, d_l, d_o, d_ord, d_start, d_status};
    for (int* ptr : frees) if (ptr) kv_free(ptr);
    if (d_res) kv_free(d_res);
    return rc;
}

int sched_amin_simulate(int32_t B, int32_t n_max, const int32_t* n_each, const int32_t* s, const int32_t* lower,
                        const int32_t* o, int64_t M, const int32_t* order, int32_t* start_out, int64_t* tel_out,
                        int64_t* evictions_out, int64_t* peak_out, float* kernel_ms_out) {
    if (!order) return SCHED_E_INVAL;
    return amin_run(B, n_max, n_each, s, lower, o, M, order, nullptr, start_out, tel_out, evictions_out, peak_out,
                    kernel_ms_out);
}

int sched_sorted_f_amin(int32_t n, const int32_t* s, const int32_t* lower, const int32_t* o, int64_t M,
                        int32_t phase1, int32_t* order_out, int32_t* start_out, int64_t* tel_out,
                        int64_t* evictions_out, int64_t* peak_out) {
    if (n < 1 || !s || !lower || !o || !start_out || !tel_out) return SCHED_E_INVAL;
    if (phase1 != 0 && phase1 != 1) return SCHED_E_INVAL;
    for (int i = 0; i < n; ++i)
        if (s[i] < 1 || o[i] < 1 || lower[i] < 1 || lower[i] > o[i] || (i64)s[i] + o[i] > M) return SCHED_E_INVAL;
    // Phase 1 sees the lower bounds in place of the decode lengths
    sched_handle h = nullptr;
    KV_TRY(sched_init(&h, n, s, lower, M));
    int rc = sorted_f_common_dev(h, phase1, nullptr, nullptr, nullptr, nullptr);
    if (rc == SCHED_OK) rc = sched_sync(h);
    if (rc == SCHED_OK && order_out &&
        cudaMemcpy(order_out, h->d_order, sizeof(int) * (size_t)n, cudaMemcpyDeviceToHost) != cudaSuccess)
        rc = kv_cuda_fail(cudaGetLastError(), "cudaMemcpy(order_out)");
    if (rc == SCHED_OK)
        rc = amin_run(1, n, &n, s, lower, o, M, nullptr, h->d_order, start_out, tel_out, evictions_out, peak_out, nullptr);
    sched_destroy(h);
    return rc;
}

int sched_build_flags(void) {
#ifdef KVSCHED_CHECKED
    return SCHED_BUILD_CHECKED;
#else
    return 0;
#endif
}

int sched_debug_check_index(int64_t index, int64_t limit) {
#ifdef KVSCHED_CHECKED
    int* sink = nullptr;
    KV_CUDA(cudaMalloc((void**)&sink, sizeof(int)));
    kv_check_index_probe<<<1, 1>>>((long long)index, (long long)limit, sink);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    cudaFree(sink);
    if (e != cudaSuccess) return kv_cuda_fail(e, "kv_check_index_probe");
    return read_checked_word();
#else
    (void)index; (void)limit;
    return SCHED_E_UNSUPPORTED;
#endif
}

int sched_debug_set_loop_cap(int32_t cap) {
    const int v = cap < 0 ? 0x7fffffff : cap;
    KV_CUDA(cudaDeviceSynchronize());           // no kernel of this device may see the value change under it
    KV_CUDA(cudaMemcpyToSymbol(kv_test_loop_cap, &v, sizeof(int)));
    KV_CUDA(cudaDeviceSynchronize());
    return SCHED_OK;
}

int sched_release_cached_memory(void) {
    std::lock_guard<std::mutex> lock(g_pool_mu);
    pool_trim_locked(-1);
    return SCHED_OK;
}

int sched_stats(sched_handle h, int64_t* kernel_launches_out, int64_t* evaluations_out) {
    if (!h) return SCHED_E_INVAL;
    if (kernel_launches_out) *kernel_launches_out = h->launches;
    if (evaluations_out) *evaluations_out = h->evaluations;
    return SCHED_OK;
}

int sched_destroy(sched_handle h) {
    if (!h) return SCHED_E_INVAL;
    DeviceGuard guard(h->device);
    cudaStreamSynchronize(h->stream);
    free_ctx(h);
    return SCHED_OK;
}

const char* sched_strerror(int code) {
    switch (code) {
        case SCHED_OK: return "ok";
        case SCHED_E_INVAL: return "invalid argument";
        case SCHED_E_NOT_PERMUTATION: return "candidate is not a permutation of 0..n-1";
        case SCHED_E_CUDA: return "CUDA runtime error";
        case SCHED_E_NOMEM: return "out of memory";
        case SCHED_E_INTERNAL: return "a bounded device loop hit its cap, or the checked build caught an index outside its array";
        case SCHED_E_UNSUPPORTED: return "size not supported by this build";
        default: return "unknown error code";
    }
}

const char* sched_last_cuda_error(void) { return g_last_cuda_error; }

}  // extern "C"
