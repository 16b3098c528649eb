// Shared declarations of the kvsched GPU library: handle layout, error helpers, small device
// utilities.  Everything here is integer arithmetic; nothing is shared with the CPU checker.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/kvsched.h"

typedef long long i64;
typedef unsigned long long u64;

#define KV_WARP 32
#define KV_FULL 0xffffffffu

// Device-side status word (ctx->d_status[0]); non-zero means a bounded loop gave up.
enum { KV_DEV_OK = 0, KV_DEV_LOOP_CAP = 1, KV_DEV_TMA_TIMEOUT = 2 };

struct SnapHeader {          // simulator state in front of one list position (16 bytes)
    int t;                   // current round index (number of completed rounds = next start time)
    int hz;                  // first round after which the timeline is all zero
    int tel_lo, tel_hi;      // TEL of the positions before this one
};

struct sched_ctx {
    int device;
    cudaStream_t stream, own_stream;
    int B, n;                // instances, requests per instance
    i64 M;
    int omax;                // largest decode length over all instances
    int L;                   // cells per simulator state (32 * nreg; 32 * (33 + far chunks); or a ring of a multiple of 32 cells >= omax + 8)
    int nreg;                // > 0: register-resident simulator with this many registers per lane
    int nit;                 // shared-memory simulator: 128-cell rounds cached in registers (0: streamed)
    bool hyb;                // hybrid simulator: 33 registers per lane + a shared-memory ring for the rounds after them
    int ring_cells;          // shared-memory ints one simulator needs (0 for the register simulator)
    i64 sum_o_max;           // largest sum of o over instances (bounds every start time)
    int sm_count;
    int smem_optin;          // max dynamic shared memory per block (bytes)

    int *d_s, *d_o;          // [B*n]
    int2* d_tbl_id;          // (s, o) by request id [B*n]
    int2* d_tbl_base;        // (s, o) by base position [n]
    int* d_order;            // base order [n]
    bool base_ready;         // d_tbl_base + snapshots match d_order
    bool batch_handle;       // created by sched_init_batch
    int* d_base_starts;      // start of every position of the base order [n]
    i64* d_state;            // local-search state {current TEL, accepted flag}
    void* h_pinned;          // 64 bytes of pinned host memory for small read-backs
    void* d_sort;            // grow-only scratch for sorting explicit start times
    size_t sort_cap;
    int g_num, g_den;        // prefill weight alpha = g_num / g_den of the batch metric (0/1: the F-metric)
    int* d_ls;               // scratch of the Local Swap Search kernel: 7 arrays of n ints (lazy)
    void* d_k4;              // grow-only scratch of the launch ordering: bins[n+1], first_pos[count], order[count]
    size_t k4_cap;

    // snapshots of the base run
    int snap_stride, snap_count;
    int* d_snap_ring;        // [snap_count][L]
    SnapHeader* d_snap_hdr;  // [snap_count]
    i64* d_base_tel;         // [1]

    // scratch
    unsigned int* d_counter; // work counter(s)
    int* d_status;           // [1] device status
    i64* d_tel;              // [tel_cap] per-candidate TEL scratch
    i64 tel_cap;
    i64* d_best;             // [2] (TEL, index) + partials
    i64* d_partials;         // [2 * max_blocks]
    unsigned int* d_ticket;  // [1]

    // sort / F-metric scratch (single-instance handles)
    u64 *d_keys_a, *d_keys_b;
    int *d_vals_a, *d_vals_b;
    i64 *d_prefP, *d_prefO;  // [n+1]
    int* d_batch_off;        // [n+1]
    int* d_num_batches;      // [1]
    int* d_seg_off;          // [2] offsets {0, n} for whole-array sorts

    // staging for the host-pointer entry points
    void* d_stage;
    size_t stage_cap;

    i64 launches, evaluations;
    cudaEvent_t ev_k3_begin, ev_k3_end;   // around the most recent simulation-kernel launch
    bool ev_valid;
};

extern thread_local char g_last_cuda_error[256];
int kv_cuda_fail(cudaError_t e, const char* what);

#define KV_CUDA(expr)                                                        \
    do {                                                                     \
        cudaError_t e__ = (expr);                                            \
        if (e__ != cudaSuccess) return kv_cuda_fail(e__, #expr);             \
    } while (0)

#define KV_TRY(expr)                                                         \
    do {                                                                     \
        int rc__ = (expr);                                                   \
        if (rc__ != SCHED_OK) return rc__;                                   \
    } while (0)

// ------------------------------------------------------------------------------------ device utils
__device__ __forceinline__ int kv_lane() { return threadIdx.x & 31; }

__device__ __forceinline__ int kv_warp_max(int v) { return __reduce_max_sync(KV_FULL, v); }
__device__ __forceinline__ int kv_warp_min(int v) { return __reduce_min_sync(KV_FULL, v); }

// Checked build (-DKVSCHED_CHECKED, libkvsched_checked.so): every index that a kernel derives from
// data or from its own arithmetic goes through KV_IDX(index, limit, site) before it is used.  In a
// checked build an index outside 0 .. limit-1 is recorded (site number and value, first one wins)
// in a device word that the host reads with the status word, and element 0 is accessed instead, so
// nothing ever leaves its array; the host call then returns SCHED_E_INTERNAL.  In the normal build
// KV_IDX is the index itself.  (The memory checker of the toolkit is not always available; this is
// the library's own stand-in, run over the small parity cases.)
#ifdef KVSCHED_CHECKED
__device__ unsigned long long kv_checked_word = 0ull;      // 0, or (site << 40) | (index & 0xffffffffff)
__device__ __forceinline__ long long kv_checked_index(long long idx, long long limit, int site) {
    if (idx >= 0 && idx < limit) return idx;
    atomicCAS(&kv_checked_word, 0ull, ((unsigned long long)site << 40) | ((unsigned long long)idx & 0xffffffffffull));
    return 0;
}
#define KV_IDX(idx, limit, site) kv_checked_index((long long)(idx), (long long)(limit), (site))
#else
#define KV_IDX(idx, limit, site) (idx)
#endif

// Every device loop whose trip count depends on data carries a cap (its natural bound by
// construction); a loop that reaches it records KV_DEV_LOOP_CAP in the status word and leaves, and
// the host call returns SCHED_E_INTERNAL.  kv_test_loop_cap lowers every cap at once so that a test
// can watch that path work (sched_debug_set_loop_cap); INT_MAX leaves the natural bounds alone.
__constant__ int kv_test_loop_cap = 0x7fffffff;
__device__ __forceinline__ int kv_loop_cap(int natural) { return min(natural, kv_test_loop_cap); }
__device__ __forceinline__ i64 kv_loop_cap(i64 natural) { return natural < (i64)kv_test_loop_cap ? natural : (i64)kv_test_loop_cap; }

// splitmix64 step, used by the sampled neighbourhood (published generator by Steele, Lea, Flood).
__host__ __device__ __forceinline__ u64 kv_mix64(u64 z) {
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

struct Move { int type, i, j; };     // type 0 = swap (i < j), 1 = insert i -> j, -1 = identity

// Move code -> (type, i, j).  Swaps are numbered row by row: row i holds n-1-i codes and starts at
// i*(2n-i-1)/2.  The row is first guessed from a square root and then corrected with exact integer
// comparisons, so the result does not depend on floating-point rounding.  A code outside
// 0 .. n(n-1)/2 + n(n-1) - 1 (compared in 64 bits, before any narrowing) decodes to {-1, -1, -1}.
__host__ __device__ __forceinline__ Move kv_decode_move(int n, i64 code) {
    Move m;
    i64 nsw = (i64)n * (n - 1) / 2;
    if (code < 0 || code >= 3 * nsw) {              // outside the neighbourhood: no move (callers reject i, j < 0)
        m.type = -1; m.i = -1; m.j = -1;
        return m;
    }
    if (code < nsw) {
        double b = 2.0 * n - 1.0;
        i64 i = (i64)((b - sqrt(b * b - 8.0 * (double)code)) * 0.5);
        if (i < 0) i = 0;
        if (i > n - 2) i = n - 2;
        while (i > 0 && i * (2 * (i64)n - i - 1) / 2 > code) --i;
        while ((i + 1) * (2 * (i64)n - (i + 1) - 1) / 2 <= code) ++i;
        m.type = 0; m.i = (int)i; m.j = (int)(i + 1 + (code - i * (2 * (i64)n - i - 1) / 2));
    } else {
        i64 c = code - nsw;
        int i = (int)(c / (n - 1)), r = (int)(c % (n - 1));
        m.type = 1; m.i = i; m.j = r < i ? r : r + 1;
    }
    return m;
}

__host__ __device__ __forceinline__ Move kv_sample_move(int n, u64 seed, int it, i64 mcount) {
    u64 h1 = kv_mix64(seed ^ kv_mix64(((u64)(uint32_t)it << 32) + (u64)mcount));
    u64 h2 = kv_mix64(h1);
    Move m;
    m.type = (int)(h1 & 1);
    m.i = (int)((h1 >> 1) % (u64)n);
    m.j = (int)(((u64)m.i + 1 + h2 % (u64)(n - 1)) % (u64)n);
    if (m.type == 0 && m.i > m.j) { int x = m.i; m.i = m.j; m.j = x; }
    return m;
}

// Position q of the moved order -> position in the base order.
__host__ __device__ __forceinline__ int kv_map_pos(const Move& m, int q) {
    if (m.type == 0) return q == m.i ? m.j : (q == m.j ? m.i : q);
    if (m.type == 1) {
        if (m.i < m.j) return (q < m.i || q > m.j) ? q : (q == m.j ? m.i : q + 1);
        return (q < m.j || q > m.i) ? q : (q == m.j ? m.i : q - 1);
    }
    return q;
}
