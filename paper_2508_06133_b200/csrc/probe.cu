// Peak-rate probes for the roofline of the schedule simulator (measurement support; the paper has no
// counterpart).  Each probe is a kernel of independent, irreducible dependency chains that keeps one
// execution resource of every SM busy; the host times it with CUDA events and reports lane
// operations (32 per warp instruction) or bytes per second at whatever clock the device runs.
//
//   0  int32 add            a += b; b += a                       (integer ALU pipe)
//   1  int32 add + max      a += b; b = max(b, a)                (integer ALU pipe, two opcodes)
//   2  int32 multiply-add   a = a * k + b; b = b * k + a         (FMA pipe)
//   3  two-pipe mix         one multiply-add, one 3-input max, one add per step: one operation on
//                           the FMA pipe for two on the integer ALU pipe
//   4  shared-memory loads  16 bytes per thread and access, conflict-free
//   5  shared-memory stores 16 bytes per thread and access, conflict-free
//   6  int32 max + xor      a = max(a, b); b ^= a                (integer ALU pipe only: the compiler may
//                           split plain adds between the ALU and the FMA pipe, never a maximum or a
//                           logic operation)
//
// Chains of the form (a, b) -> (a + b, a + 2b) cannot be strength-reduced, and eight of them per
// thread hide the pipe latency; every result is folded into one word that is stored when a runtime
// flag is set, so nothing is dead code.
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/kvsched.h"

namespace {

constexpr int kChains = 8;         // independent chains per thread
constexpr int kUnroll = 16;        // steps per chain and loop iteration
constexpr int kThreads = 512;
constexpr int kCtasPerSm = 4;

template <int KIND>
__global__ void __launch_bounds__(kThreads) probe_alu(int iters, int seed, int mul, int* sink, int store) {
    int a[kChains], b[kChains];
#pragma unroll
    for (int c = 0; c < kChains; ++c) { a[c] = seed + threadIdx.x + c; b[c] = seed * 3 + c + blockIdx.x; }
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
#pragma unroll
            for (int c = 0; c < kChains; ++c) {
                if (KIND == 0) { a[c] += b[c]; b[c] += a[c]; }
                if (KIND == 1) { a[c] += b[c]; b[c] = max(b[c], a[c]); }
                if (KIND == 2) { a[c] = a[c] * mul + b[c]; b[c] = b[c] * mul + a[c]; }
                if (KIND == 6) { a[c] = max(a[c], b[c]); b[c] ^= a[c]; }
                if (KIND == 3) {
                    a[c] = a[c] * mul + b[c];                                   // FMA pipe
                    b[c] = __vimax3_s32(b[c], a[c], a[(c + 1) % kChains]);      // integer ALU pipe
                    a[c] += b[c];                                               // either pipe
                }
            }
        }
    }
    int acc = 0;
#pragma unroll
    for (int c = 0; c < kChains; ++c) acc ^= a[c] ^ b[c];
    if (store) sink[blockIdx.x * blockDim.x + threadIdx.x] = acc;
}

__global__ void __launch_bounds__(kThreads) probe_smem_ld(int iters, int seed, int* sink, int store) {
    __shared__ int4 buf[kThreads * 2];
    buf[threadIdx.x] = make_int4(seed, threadIdx.x, 2, 3);
    buf[threadIdx.x + kThreads] = make_int4(seed, threadIdx.x, 5, 7);
    __syncthreads();
    const unsigned base = (unsigned)__cvta_generic_to_shared(buf + threadIdx.x);
    int acc = seed;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            int4 v;
            asm volatile("ld.volatile.shared.v4.s32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                         : "r"(base + ((u & 1) ? (unsigned)(kThreads * sizeof(int4)) : 0u)) : "memory");
            if ((u & 3) == 3) acc ^= v.x;                 // one integer operation per four loads keeps the ALU out of the way
        }
    }
    if (store) sink[blockIdx.x * blockDim.x + threadIdx.x] = acc;
}

__global__ void __launch_bounds__(kThreads) probe_smem_st(int iters, int seed, int* sink, int store) {
    __shared__ int4 buf[kThreads * 2];
    const unsigned base = (unsigned)__cvta_generic_to_shared(buf + threadIdx.x);
    const int x = seed + threadIdx.x;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            asm volatile("st.shared.v4.s32 [%0], {%1, %2, %3, %4};"
                         :: "r"(base + ((u & 1) ? (unsigned)(kThreads * sizeof(int4)) : 0u)), "r"(x), "r"(it), "r"(seed), "r"(x)
                         : "memory");
        }
    }
    __syncthreads();
    const int4 v = buf[threadIdx.x];
    if (store) sink[blockIdx.x * blockDim.x + threadIdx.x] = v.x ^ v.y ^ v.z ^ v.w;
}

}  // namespace

extern "C" int sched_probe_peaks(double* out, int32_t n_out, int32_t repeats, void* cuda_stream) {
    if (!out || n_out < SCHED_PROBE_COUNT || repeats < 1 || repeats > 64) return SCHED_E_INVAL;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return SCHED_E_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return SCHED_E_CUDA;
    const int grid = sms * kCtasPerSm;
    int* sink = nullptr;
    if (cudaMalloc((void**)&sink, (size_t)grid * kThreads * sizeof(int)) != cudaSuccess) { cudaGetLastError(); return SCHED_E_NOMEM; }
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    int rc = SCHED_OK;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) rc = SCHED_E_CUDA;
    const int iters = 256;
    // per thread: instructions (kinds 0-2: two per chain step, kind 3: three) or bytes (16 per access)
    const double per_thread[SCHED_PROBE_COUNT] = {
        2.0 * kChains * kUnroll * iters, 2.0 * kChains * kUnroll * iters, 2.0 * kChains * kUnroll * iters,
        3.0 * kChains * kUnroll * iters, 16.0 * kUnroll * iters * 8, 16.0 * kUnroll * iters * 8,
        2.0 * kChains * kUnroll * iters};
    for (int k = 0; k < SCHED_PROBE_COUNT && rc == SCHED_OK; ++k) {
        double best = 0.0;
        for (int r = 0; r <= repeats && rc == SCHED_OK; ++r) {           // r = 0 warms up
            if (cudaEventRecord(e0, st) != cudaSuccess) { rc = SCHED_E_CUDA; break; }
            switch (k) {
                case 0: probe_alu<0><<<grid, kThreads, 0, st>>>(iters, 12345 + r, 3, sink, 0); break;
                case 1: probe_alu<1><<<grid, kThreads, 0, st>>>(iters, 12345 + r, 3, sink, 0); break;
                case 2: probe_alu<2><<<grid, kThreads, 0, st>>>(iters, 12345 + r, 3, sink, 0); break;
                case 3: probe_alu<3><<<grid, kThreads, 0, st>>>(iters, 12345 + r, 3, sink, 0); break;
                case 4: probe_smem_ld<<<grid, kThreads, 0, st>>>(iters * 8, 12345 + r, sink, 0); break;
                case 5: probe_smem_st<<<grid, kThreads, 0, st>>>(iters * 8, 12345 + r, sink, 0); break;
                default: probe_alu<6><<<grid, kThreads, 0, st>>>(iters, 12345 + r, 3, sink, 0); break;
            }
            if (cudaGetLastError() != cudaSuccess || cudaEventRecord(e1, st) != cudaSuccess ||
                cudaEventSynchronize(e1) != cudaSuccess) { rc = SCHED_E_CUDA; break; }
            float ms = 0.f;
            if (cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess) { rc = SCHED_E_CUDA; break; }
            if (r > 0 && ms > 0.f) {
                const double rate = per_thread[k] * (double)grid * kThreads / (ms * 1e-3);
                if (rate > best) best = rate;
            }
        }
        out[k] = best;
    }
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    cudaFree(sink);
    return rc;
}
