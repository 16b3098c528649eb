// sched_argmin_static_dev -- the arg-min reduction over a TEL array for callers that may not
// allocate device memory.
//
// Who needs this: code that runs where cudaMalloc is off limits -- a serving process whose memory
// pool has already claimed the whole GPU, a plug-in that was handed a fixed set of buffers by its
// host application, or a latency-critical loop that must not hit the allocator's implicit
// device-wide synchronisation.  Such a caller already holds the per-candidate TELs (for example
// from sched_sweep_dev's tel_out) and only wants the best (TEL, index) pair.  The ordinary path
// keeps its per-block partial results and its ticket counter in memory the handle cudaMalloc'd;
// here they live in a fixed array that is part of the library image, so nothing is allocated,
// freed or resized by this call -- not by the CUDA runtime and not by any other library.
//
// Cost of that choice: every GPU that loads the library carries the array (16 KiB + 256 bytes)
// until the process exits, all calls on one device share it, and it still holds whatever the
// previous call left there.  The ticket counter is therefore cleared on the stream before every
// launch, and two calls whose kernels could run at the same time on one device (different
// streams, different host threads) would overwrite each other's partial results: callers must
// order them.
#include <stdio.h>

#include <mutex>

#include "common.cuh"

#define KS_THREADS 256
#define KS_MAX_BLOCKS 1024
#define KS_MAX_DEVICES 64
#define KS_MAX_COUNT (1ll << 26)          // documented limit of the entry point (candidates per call)

// [0 .. 2*KS_MAX_BLOCKS) : per-block (TEL, index) partials;  [2*KS_MAX_BLOCKS] : ticket counter
// (stored in a 64-bit slot, only its low 32 bits are used); padded to a multiple of 256 bytes.
static __device__ __align__(256) i64 g_argmin_scratch[2 * KS_MAX_BLOCKS + 32];

namespace {

__device__ __forceinline__ void ks_take(i64& bv, i64& bi, i64 v, i64 i) {
    if (v < bv || (v == bv && i < bi)) { bv = v; bi = i; }
}

// Same reduction as the handle-based arg-min: smallest TEL, lowest index among equals; the last
// block to finish folds the partials.  `scratch` is the device address of g_argmin_scratch.
__global__ void __launch_bounds__(KS_THREADS)
ks_argmin(const i64* __restrict__ tel, i64 count, i64 index_base, i64* __restrict__ scratch, i64* __restrict__ best_out) {
    __shared__ i64 sh_v[KS_THREADS / 32], sh_i[KS_THREADS / 32];
    __shared__ bool is_last;
    i64* partials = scratch;
    unsigned int* ticket = reinterpret_cast<unsigned int*>(scratch + 2 * KS_MAX_BLOCKS);
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    i64 bv = INT64_MAX, bi = INT64_MAX;
    for (i64 k = (i64)blockIdx.x * KS_THREADS + tid; k < count; k += (i64)gridDim.x * KS_THREADS)
        ks_take(bv, bi, tel[k], index_base + k);
    for (int d = 16; d >= 1; d >>= 1) {
        const i64 ov = __shfl_xor_sync(KV_FULL, bv, d), oi = __shfl_xor_sync(KV_FULL, bi, d);
        ks_take(bv, bi, ov, oi);
    }
    if (lane == 0) { sh_v[w] = bv; sh_i[w] = bi; }
    __syncthreads();
    if (tid == 0) {
        for (int k = 1; k < KS_THREADS / 32; ++k) ks_take(bv, bi, sh_v[k], sh_i[k]);
        partials[2 * blockIdx.x] = bv;
        partials[2 * blockIdx.x + 1] = bi;
        __threadfence();
        is_last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    bv = INT64_MAX; bi = INT64_MAX;
    const volatile i64* pp = partials;
    for (int k = tid; k < (int)gridDim.x; k += KS_THREADS) ks_take(bv, bi, pp[2 * k], pp[2 * k + 1]);
    for (int d = 16; d >= 1; d >>= 1) {
        const i64 ov = __shfl_xor_sync(KV_FULL, bv, d), oi = __shfl_xor_sync(KV_FULL, bi, d);
        ks_take(bv, bi, ov, oi);
    }
    if (lane == 0) { sh_v[w] = bv; sh_i[w] = bi; }
    __syncthreads();
    if (tid == 0) {
        for (int k = 1; k < KS_THREADS / 32; ++k) ks_take(bv, bi, sh_v[k], sh_i[k]);
        best_out[0] = bv;
        best_out[1] = bi;
    }
}

std::mutex g_setup_mutex;
i64* g_scratch_addr[KS_MAX_DEVICES];     // device address of g_argmin_scratch, per device ordinal

// In host code `g_argmin_scratch` is only a handle for the runtime, not an address a kernel could
// use; the real device address is looked up once per device, with that device current.
int scratch_address(i64** out) {
    int dev = -1;
    KV_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= KS_MAX_DEVICES) return SCHED_E_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[dev]) {
        i64* p = nullptr;
        KV_CUDA(cudaGetSymbolAddress((void**)&p, g_argmin_scratch));
        if (!p) return SCHED_E_CUDA;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return SCHED_OK;
}

}  // namespace

extern "C" int sched_argmin_static_dev(const int64_t* tel, int64_t count, int64_t index_base,
                                       int64_t* best_out, void* cuda_stream) {
    if (!tel || !best_out || count < 1 || index_base < 0) return SCHED_E_INVAL;
    if (count > KS_MAX_COUNT) {
        snprintf(g_last_cuda_error, sizeof(g_last_cuda_error),
                 "sched_argmin_static_dev: count %lld exceeds the fixed limit of %lld candidates",
                 (long long)count, (long long)KS_MAX_COUNT);
        return SCHED_E_UNSUPPORTED;
    }
    i64* scratch = nullptr;
    KV_TRY(scratch_address(&scratch));
    cudaStream_t st = (cudaStream_t)cuda_stream;
    i64 blocks = (count + KS_THREADS - 1) / KS_THREADS;
    if (blocks > KS_MAX_BLOCKS) blocks = KS_MAX_BLOCKS;
    // the array keeps the previous call's contents: the ticket has to start at zero
    KV_CUDA(cudaMemsetAsync(scratch + 2 * KS_MAX_BLOCKS, 0, sizeof(i64), st));
    ks_argmin<<<(unsigned)blocks, KS_THREADS, 0, st>>>((const i64*)tel, count, index_base, scratch, (i64*)best_out);
    KV_CUDA(cudaGetLastError());
    return SCHED_OK;
}
