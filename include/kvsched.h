/* kvsched -- batched evaluation of KV-cache-constrained request schedules on one GPU (sm_100a).
 *
 * Problem (paper, Section 2.1-2.2): n requests, all present at t = 0; request i has a prefill
 * length s_i and a decode length o_i; a single worker holds at most M tokens of KV cache.  A request
 * that starts at p_i >= 0 is resident in rounds p_i+1 .. p_i+o_i, uses s_i + (tau - p_i) tokens in
 * round tau, and completes at c_i = p_i + o_i (integer program of Section 6.1).  A schedule is
 * feasible iff the total usage never exceeds M; its cost is the total end-to-end latency
 * TEL = sum_i c_i, in rounds.
 *
 * An ORDER (a permutation of the requests) is turned into start times by Phase 2 of Algorithm 1
 * (the supplement to Section 3): every round, finished requests leave, then pending requests are admitted in list
 * order for as long as the memory of all running requests stays within M at every future round;
 * the first request that does not fit ends that round's admissions.
 *
 * Conventions of this interface
 *   - Every function returns SCHED_OK (0) or a negative SCHED_E_* code; nothing throws, and no GPU
 *     trap is ever used to report an error.  sched_strerror() names a code.
 *   - "host" pointers are ordinary CPU memory; "device" pointers are memory of the handle's GPU.
 *     The plain entry points take host pointers, copy in/out, and return when results are in the
 *     caller's buffers.  The *_dev entry points take device pointers, enqueue on the handle's
 *     stream and return without synchronising (sched_sync() waits).
 *   - The caller owns every buffer it passes.  The handle owns device copies of (s, o), the base
 *     order and all scratch memory; sched_destroy() frees them.
 *   - Device blocks of 1 MiB and more that the library frees (a destroyed handle's snapshots and
 *     scratch, outgrown staging buffers) are kept in a process-wide per-device cache -- at most
 *     KVSCHED_POOL_MB MiB in total (environment variable, default 1024, 0 disables the cache) -- and
 *     reused by later calls; sched_release_cached_memory() returns them to the driver.
 *   - A handle is tied to the CUDA device that was current in sched_init(); calls on one handle
 *     must not overlap in time.
 *   - Arrays are dense, row-major, int32 unless stated; TELs are int64.
 */
#ifndef KVSCHED_H
#define KVSCHED_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sched_ctx* sched_handle;

enum {
    SCHED_OK = 0,
    SCHED_E_INVAL = -1,            /* bad argument: n <= 0, s_i < 1, o_i < 1, M < 1, s_i + o_i > M, ... */
    SCHED_E_NOT_PERMUTATION = -2,  /* an ORDER candidate (or order_inout) is not a permutation of 0..n-1 */
    SCHED_E_CUDA = -3,             /* a CUDA runtime call failed (sched_last_cuda_error() has the text) */
    SCHED_E_NOMEM = -4,            /* host or device allocation failed */
    SCHED_E_INTERNAL = -5,         /* a bounded device loop hit its cap (or, in the checked build, an index
                                      left its array); results are not valid */
    SCHED_E_UNSUPPORTED = -6       /* sizes beyond what this build handles (see each call) */
};

/* What one candidate of sched_eval_batch() is. */
enum {
    SCHED_CAND_ORDER = 0,        /* int32[count][n]: a permutation; list-scheduled, always feasible     */
    SCHED_CAND_MOVE = 1,         /* int64[count]: move codes relative to the handle's base order         */
    SCHED_CAND_START_TIMES = 2,  /* int32[count][n]: explicit starts p_i; checked against the budget     */
    SCHED_CAND_POLICY = 3        /* int32[count]: SCHED_POLICY_* ids; each instance x each policy        */
};

/* Order policies (Section 2.3, the supplement to Section 2, Section 7). Ties always go to the lower request index. */
enum {
    SCHED_POLICY_FCFS = 0,        /* index order                                                         */
    SCHED_POLICY_SOF = 1,         /* shortest output first (MC-SF): ascending o                          */
    SCHED_POLICY_TOTAL_SIZE = 2,  /* smallest s+o first (MC-SF_2)                                        */
    SCHED_POLICY_SORTED_F = 3     /* Sorted-F with prefix-F batch selection, see sched_sorted_f()        */
};

/* Local-search neighbourhoods over positions of the base order.
 * Move codes: swap(i,j), 0 <= i < j < n, in lexicographic order, codes 0 .. n(n-1)/2 - 1; then
 * insert(i -> j), i != j (take the request at position i out and put it back so that it sits at
 * position j), code n(n-1)/2 + i*(n-1) + (j < i ? j : j-1). */
enum {
    SCHED_NBHD_SWAP = 0,         /* all n(n-1)/2 swaps                                                   */
    SCHED_NBHD_SWAP_INSERT = 1,  /* all swaps, then all n(n-1) inserts                                   */
    SCHED_NBHD_SAMPLED = 2       /* samples_per_iter moves per iteration from a counter-based hash       */
};

/* Create a handle for one instance (paper, Section 2.1: n, (s_i, o_i), M).
 *   s, o : host int32[n], copied.  Requires n >= 1, s_i >= 1, o_i >= 1, M >= 1 and s_i + o_i <= M
 *          (the paper's standing assumption; otherwise Algorithm 1 would never admit the request),
 *          else SCHED_E_INVAL.  SCHED_E_UNSUPPORTED if sum(o_i) + max(o_i) >= 2^30 or M >= 2^30.
 *   The base order starts as the identity. */
int sched_init(sched_handle* out, int32_t n, const int32_t* s, const int32_t* o, int64_t M);

/* Create a handle for B independent instances of n_each requests each (policy sweeps).
 *   s, o : host int32[B][n_each].  Same checks as sched_init for every instance.
 *   Only sched_eval_batch(SCHED_CAND_POLICY) is available on such a handle. n_each <= 1024. */
int sched_init_batch(sched_handle* out, int32_t B, int32_t n_each, const int32_t* s, const int32_t* o, int64_t M);

/* Use an existing CUDA stream (a cudaStream_t passed as void*) for all work of this handle.
 * NULL selects the handle's own stream again. */
int sched_set_stream(sched_handle h, void* cuda_stream);

/* Wait for everything enqueued on the handle's stream; reports device-side status
 * (SCHED_E_INTERNAL if any bounded loop gave up since the last call). */
int sched_sync(sched_handle h);

/* Prefill weight of the batch metric (Section 7, "Robustness to prefill weighting"):
 * G(X) = sum (alpha * s_i + o_i) / |X|^2 with alpha = alpha_num / alpha_den; alpha = 0 (the default,
 * 0/1) is the F-metric.  Applies to the following sched_sorted_f() and sched_sorted_f_local_swap()
 * calls of this handle (in Algorithm 3 a swap then improves iff alpha*s_in + o_in < alpha*s_out +
 * o_out); the exact DP and the POLICY candidates keep F.  Compared exactly on integer weights.
 * SCHED_E_INVAL unless 0 <= alpha_num <= 2^20 and 1 <= alpha_den <= 2^20. */
int sched_set_prefill_weight(sched_handle h, int32_t alpha_num, int32_t alpha_den);

/* Base order used by SCHED_CAND_MOVE candidates and by sched_local_search(). host int32[n]. */
int sched_set_base_order(sched_handle h, const int32_t* order);
int sched_get_base_order(sched_handle h, int32_t* order_out);

/* Evaluate `count` candidates at once (Algorithm 1 Phase 2 for ORDER / MOVE / POLICY; the memory
 * row and objective of the integer program, Section 6.1, for START_TIMES).
 *   candidates   : layout per `kind`, see SCHED_CAND_*.
 *   tel_out      : int64[count] (POLICY: int64[B][count]).  START_TIMES: sum(p_i + o_i), also when
 *                  infeasible.
 *   feasible_out : uint8[count], nullable.  1 unless a START_TIMES candidate exceeds M in some round
 *                  (ORDER / MOVE / POLICY candidates are feasible by construction).
 *   starts_out   : nullable; int32[count][n] start time p_i of every request i, indexed by request
 *                  id (ORDER, MOVE, and POLICY with layout [B][count][n_each]).
 * Host-pointer form: validates ORDER candidates (SCHED_E_NOT_PERMUTATION), MOVE codes and policy
 * ids (SCHED_E_INVAL) and negative start times (SCHED_E_INVAL) before any launch.
 * POLICY builds every order inside the kernel (one warp per instance-policy pair, all of an
 * instance's arrays in shared memory): SCHED_E_UNSUPPORTED when the instance does not fit there
 * (about n > 8,000 requests on a single-instance handle; batch handles are limited to 1,024). */
int sched_eval_batch(sched_handle h, int kind, int64_t count, const void* candidates,
                     int64_t* tel_out, uint8_t* feasible_out, int32_t* starts_out);

/* Same, device pointers, asynchronous on the handle's stream.  Candidates are not validated on the
 * host; a MOVE code outside the neighbourhood or an ORDER entry outside 0..n-1 yields
 * tel_out = INT64_MAX for that candidate (duplicate ids in an ORDER are not detected), a negative
 * start time yields feasible_out = 0. */
int sched_eval_batch_dev(sched_handle h, int kind, int64_t count, const void* candidates,
                         int64_t* tel_out, uint8_t* feasible_out, int32_t* starts_out);

/* Evaluate the contiguous move-code range [first_code, first_code + count) (SWAP_INSERT coding)
 * against the base order, or -- if sampled != 0 -- the sampled moves m = first_code .. first_code +
 * count - 1 of iteration `iteration` under `seed`; then reduce to the best (TEL, index) pair.
 *   tel_out  : device int64[count], nullable (per-candidate TELs are still reduced if NULL); any
 *              8-byte aligned address will do (e.g. a slice of a larger array).
 *   best_out : device int64[2] = {min TEL, lowest index (code or m) attaining it}.
 * Asynchronous on the handle's stream.  This is one neighbourhood sweep of sched_local_search().
 * SCHED_E_INVAL (nothing is launched): batch handle, n < 2, count <= 0, a range that leaves the
 * neighbourhood, best_out NULL, or tel_out / best_out not 8-byte aligned. */
int sched_sweep_dev(sched_handle h, int sampled, uint64_t seed, int32_t iteration,
                    int64_t first_code, int64_t count, int64_t* tel_out, int64_t* best_out);

/* Sorted-F (Algorithm 1 Phase 1 + Phase 2) with prefix-F batch selection: requests are sorted by
 * (s+o, o, index) ascending -- the order Algorithm 3 starts from; from the current offset a, with
 * k_max the longest prefix of the remaining requests whose sum(s+o) <= M, the batch is the prefix
 * of length k* = argmin_{1<=k<=k_max} (sum of o over the prefix) / k^2, ties to the larger k
 * (Section 3: minimise F, prefer the larger batch; compared exactly in integers); the batch is
 * sorted by (o, index) and appended.  The resulting order becomes the handle's base order.
 *   order_out         : host int32[n], nullable.
 *   batch_offsets_out : host int32[n+1], nullable; entries 0..num_batches are filled.
 *   num_batches_out, tel_out : nullable. */
int sched_sorted_f(sched_handle h, int32_t* order_out, int32_t* batch_offsets_out,
                   int32_t* num_batches_out, int64_t* tel_out);

/* Same, results left on the device; asynchronous.  order_out int32[n], batch_offsets_out
 * int32[n+1], num_batches_out int32[1], tel_out int64[1]; each nullable. */
int sched_sorted_f_dev(sched_handle h, int32_t* order_out, int32_t* batch_offsets_out,
                       int32_t* num_batches_out, int64_t* tel_out);

/* Sorted-F with Algorithm 3 (Local Swap Search, Section 5.2 and the supplement to Section 5) as the Phase-1 solver --
 * the variant the paper's experiments use at n = 2000.  Repeat on the requests not yet placed:
 * sort by ascending s+o (ties: lower index); first-fit fill up to sum(s+o) <= M; then, walking
 * r_out over the batch (insertion order; a swapped-in request takes the replaced one's place) and
 * r_in over the outside requests (sorted order), swap the first pair that keeps sum(s+o) <= M and
 * lowers F (same batch size, so iff o_in < o_out) and start the walk over, until no pair
 * qualifies; sort the batch by (o, index) and append it.  Outputs and side effects as
 * sched_sorted_f(): the order becomes the handle's base order.  Single-instance handles only. */
int sched_sorted_f_local_swap(sched_handle h, int32_t* order_out, int32_t* batch_offsets_out,
                              int32_t* num_batches_out, int64_t* tel_out);

/* Same, results left on the device; asynchronous (see sched_sorted_f_dev). */
int sched_sorted_f_local_swap_dev(sched_handle h, int32_t* order_out, int32_t* batch_offsets_out,
                                  int32_t* num_batches_out, int64_t* tel_out);

/* Sorted-F with Algorithm 4 (Quantile Greedy Selection, Section 5.3 and the supplement to Section 5) as the Phase-1
 * solver: repeat on the requests not yet placed { walk them in ascending (o, index); draw a sample
 * of max(1, floor(m/2)) of the m requests; Q_p, Q_o = 0.3-quantiles of s+o and of o over the sample;
 * pass 1 admits, in walking order, every request with s+o <= Q_p, o <= Q_o that still fits in M;
 * pass 2 walks the others in ascending o/(s+o) and admits every one that still fits; sort the batch
 * by (o, index); append }.  What the listing leaves open is fixed as follows.  Sample: request id of
 * batch number b (0-based) gets the key mix(seed ^ mix(b * 2^32 + id)), mix = one splitmix64 step;
 * the sample is the requests with the smallest keys (equal keys in walking order).  Quantile: the
 * element at 0-based position floor(3 (size-1) / 10) of the ascending values.  Ratios are compared
 * exactly; equal ratios keep the walking order.
 * SCHED_E_UNSUPPORTED when 2*bits(M) + bits(max o) > 63 (the exact ratio key would not fit 64 bits).
 * Host pointers; synchronises once per batch; outputs and side effects as sched_sorted_f(). */
int sched_sorted_f_quantile(sched_handle h, uint64_t seed, int32_t* order_out, int32_t* batch_offsets_out,
                            int32_t* num_batches_out, int64_t* tel_out);

/* Sorted-F with Algorithm 2 (exact dynamic programme, Section 5.1 and the supplement to Section 5) as the Phase-1
 * solver: repeat on the requests not yet placed { dp[k][m] = min sum of o over k-subsets whose
 * sum(s+o) is exactly m <= M, requests taken in ascending index, a cell replaced only by a strictly
 * smaller value; the batch is the cell minimising dp/k^2, ties to the larger k (Section 3), then the
 * smaller m, and its members are the listing's path set; sort it by (o, index); append }.
 * Meant for small instances (the paper recommends n <= 100): SCHED_E_UNSUPPORTED if n > 128 or
 * (n+1)*(M+1) > 2^26.  Host pointers; outputs and side effects as sched_sorted_f(). */
int sched_sorted_f_dp(sched_handle h, int32_t* order_out, int32_t* batch_offsets_out,
                      int32_t* num_batches_out, int64_t* tel_out);

/* Order-level local search from order_inout (NULL: from the handle's base order).  Each iteration
 * evaluates the whole neighbourhood with Algorithm 1 Phase 2, takes the best (TEL, code) pair --
 * lowest code among equal TELs -- and accepts it iff its TEL is strictly below the current one
 * (Section 5.2's improving-swap rule applied to list positions).  SWAP / SWAP_INSERT stop at the
 * first iteration without an improving move (that iteration is counted); SAMPLED always runs
 * `iters` iterations, drawing move m of iteration it from h1 = mix(seed ^ mix(it * 2^32 + m)),
 * h2 = mix(h1) (mix = splitmix64 step): type = h1 & 1, i = (h1 >> 1) mod n,
 * j = (i + 1 + h2 mod (n-1)) mod n, a swap normalised to i < j.
 *   order_inout    : host int32[n], nullable; receives the final order.
 *   tel_out        : final TEL.  iters_done_out: iterations executed.  Both nullable.
 *   trace_out      : nullable host int64[iters][2]: per iteration {best code, best TEL}.
 * The final order becomes the handle's base order, so a run can be resumed by calling again. */
int sched_local_search(sched_handle h, int neighbourhood, int32_t iters, uint64_t seed,
                       int64_t samples_per_iter, int32_t* order_inout, int64_t* tel_out,
                       int32_t* iters_done_out, int64_t* trace_out);

/* One acceptance step of the order-level local search for callers that run the neighbourhood sweep
 * themselves, e.g. split over several GPUs: every GPU sweeps its share of the move indices with
 * sched_sweep_dev(), the (TEL, index) pairs are reduced to the smallest one (ties: lower index) and
 * every GPU then makes this call with the same pair, so that all base orders stay identical.
 * The move is accepted iff best_tel is strictly below the TEL of the current base order (Section 5.2's
 * improving rule); it is then applied to the base order on the device and the base run with its
 * snapshots is rebuilt.
 *   best_tel, best_index : the winning pair; best_index is a move code (sampled = 0, SWAP_INSERT
 *                          coding) or the sample number m of iteration `iteration` under `seed`.
 *   accepted_out         : 1 if the move was applied, else 0; nullable.
 *   tel_out              : TEL of the base order after the call; nullable.
 * Synchronises the handle's stream.  SCHED_E_INVAL: batch handle, n < 2, index outside the
 * neighbourhood.  SCHED_E_INTERNAL: the applied move does not reproduce best_tel (the pair did not
 * come from a sweep of this base order). */
int sched_accept_move(sched_handle h, int64_t best_tel, int64_t best_index, int sampled, uint64_t seed,
                      int32_t iteration, int32_t* accepted_out, int64_t* tel_out);

/* Device time, in milliseconds, of the most recent schedule-simulation kernel launch of this handle
 * (the move / order evaluator), measured with CUDA events recorded on the handle's stream around
 * that launch.  Waits for the launch to finish.  SCHED_E_INVAL if there was none. */
int sched_last_eval_kernel_ms(sched_handle h, float* ms_out);

/* Arg-min over a TEL array without any allocation (the paper has no counterpart; this exists for
 * callers that are not allowed to allocate device memory: a serving process whose memory pool
 * already owns the whole GPU, a plug-in that works inside buffers it was given, a latency-critical
 * loop that must stay clear of the allocator's device-wide synchronisation).  No handle is needed.
 *   tel        : device int64[count], e.g. the tel_out of sched_sweep_dev.
 *   count      : 1 .. 2^26 candidates; larger counts are refused with SCHED_E_UNSUPPORTED (and a
 *                message in sched_last_cuda_error()), smaller or NULL arguments with SCHED_E_INVAL.
 *   index_base : added to the position of the winner (first move code / sample index of `tel`).
 *   best_out   : device int64[2] = {min TEL, lowest index attaining it}; same result as the
 *                best_out of sched_sweep_dev on the same TELs.
 *   cuda_stream: cudaStream_t (as void*) to enqueue on, NULL for the default stream; asynchronous.
 * Works on the CUDA device that is current in the calling thread.  Its partial results and ticket
 * counter live in a 16.25 KiB array inside the library image, present on every GPU that loads the
 * library until the process exits; this call never calls cudaMalloc/cudaFree or any allocating
 * routine.  The first call on each device looks up that array's device address (make that first
 * call before starting any stream capture).  All calls on a device share the array and it keeps the
 * previous call's contents (the counter is cleared on the stream before each launch), so two calls
 * whose kernels may overlap on one GPU race: order them on one stream or with events. */
int sched_argmin_static_dev(const int64_t* tel, int64_t count, int64_t index_base,
                            int64_t* best_out, void* cuda_stream);

/* Online arrivals (Section 6.2, "Heuristics under Online Arrival"; Section 7's Poisson experiment):
 * B independent arrival streams simulated to completion under one policy, one CTA per stream.
 * Stream b has n_each[b] <= n_max requests in row b of the [B, n_max] arrays arrival / s / o (row
 * entries past n_each[b] are ignored).  Request i arrives at the integer time arrival[i] >= 0
 * (non-decreasing within a row), may start at any p >= arrival[i] (it is first seen by iteration
 * arrival[i] + 1) and then occupies rounds p+1 .. p+o exactly as in the offline model.  In every
 * iteration the policy orders the pending requests and the longest prefix of that order that fits
 * the live memory profile is admitted (Algorithm 1, Phase 2).
 *   SCHED_POLICY_FCFS      arrival order.
 *   SCHED_POLICY_SOF       ascending (o, index), recomputed every iteration.
 *   SCHED_POLICY_SORTED_F  Sorted-F-Online: a cached priority list; arrivals are appended to it; it is
 *       planned again when it has never been planned, `period` iterations after the last plan, when
 *       it had run empty, or when the arrivals since the last plan reach half of the backlog size at
 *       that plan.  A plan sorts the pending requests by ascending (s+o, index), orders the first
 *       `lookahead` of them by Sorted-F with Algorithm 3 (every batch by ascending (o, index)) and
 *       appends the others in sorted order.  The paper uses period = 10, lookahead = 300.
 * start_out [B, n_max] receives the start times (-1 where a row has no request), latency_out [B] the
 * sum of (p + o - arrival) per stream; kernel_ms_out (nullable) the device time of the simulation.
 * All pointers are host memory; the call allocates and frees its own device buffers and
 * synchronises the device.  SCHED_E_INVAL: bad sizes, policy, period or lookahead < 1, a request with
 * s < 1, o < 1 or s+o > M, decreasing arrivals.  SCHED_E_UNSUPPORTED: n_max > 2048, lookahead > 1024,
 * o > 8192, M >= 2^30, arrival >= 2^29, or a stream whose decode lengths sum to 2^29 or more. */
int sched_online_simulate(int32_t B, int32_t n_max, const int32_t* n_each, const int32_t* arrival,
                          const int32_t* s, const int32_t* o, int64_t M, int32_t policy, int32_t period,
                          int32_t lookahead, int32_t* start_out, int64_t* latency_out, float* kernel_ms_out);

/* Sorted-F + A_min, Phase 2 (Section 5.5, "Handling Prediction Uncertainty via Adaptive Output Length
 * Refinement"; Algorithm 5 in the supplement to Section 5): B independent scenarios executed to completion when only a
 * lower bound lower[i] <= o[i] of every decode length is known to the scheduler, one CTA per scenario.
 * Scenario b has n_each[b] <= n_max requests in row b of the [B, n_max] arrays s / lower / o / order
 * (entries past n_each[b] are ignored); order is the list to execute, a permutation of 0..n_each[b]-1
 * (for the paper's method: Phase 1 run on the lower bounds).  Every request carries a running
 * estimate, initially lower[i].  Iteration t = 1, 2, ...: (1) requests that have run o[i] rounds
 * leave, every other running request's estimate becomes max(estimate, t - p_i); (2) pending requests
 * are admitted in list order, p = t - 1, for as long as the memory projected from the estimates stays
 * within M in every future round, stopping at the first that does not fit; (3) while the projection
 * exceeds M the running request with the smallest estimate (ties: lower request index) is evicted --
 * it loses its progress, keeps its estimate and returns to its place in the list; (4) the round runs.
 * o[i] is used only to see that a request has finished.  With lower = o this is Algorithm 1's Phase 2.
 *   start_out     : [B, n_max] final start time of every request, by request id (-1 where a row has
 *                   no request).
 *   tel_out       : [B] sum of (p_i + o_i).
 *   evictions_out : [B] number of evictions, nullable.   peak_out : [B] largest memory actually in use
 *                   in any round (never above M), nullable.   kernel_ms_out : device time, nullable.
 * All pointers are host memory; the call allocates and frees its own device buffers and synchronises
 * the device.  SCHED_E_INVAL: bad sizes, s < 1, lower < 1, lower > o, s + o > M;
 * SCHED_E_NOT_PERMUTATION: a row of order is not a permutation; SCHED_E_UNSUPPORTED: n_max > 4096,
 * o > 8192, M >= 2^30, or rows too large for the shared memory of one CTA (20 n_max + 16 L bytes,
 * L = the power of two >= max o + 2); SCHED_E_INTERNAL: a scenario did not finish within
 * 16 + (n+1) sum(o) rounds (capped at 2^30). */
int sched_amin_simulate(int32_t B, int32_t n_max, const int32_t* n_each, const int32_t* s, const int32_t* lower,
                        const int32_t* o, int64_t M, const int32_t* order, int32_t* start_out, int64_t* tel_out,
                        int64_t* evictions_out, int64_t* peak_out, float* kernel_ms_out);

/* Sorted-F + A_min end to end for one backlog (Algorithm 5): Phase 1 of Sorted-F on (s, lower) --
 * phase1 = 0: prefix-F batch selection as in sched_sorted_f(); 1: Algorithm 3 as in
 * sched_sorted_f_local_swap() -- then the executor of sched_amin_simulate() on the resulting list.
 *   order_out : host int32[n], nullable, the Phase-1 list.  Other outputs as above with B = 1.
 * Host pointers; creates and destroys a handle internally.  Errors as sched_init() and
 * sched_amin_simulate(). */
int sched_sorted_f_amin(int32_t n, const int32_t* s, const int32_t* lower, const int32_t* o, int64_t M,
                        int32_t phase1, int32_t* order_out, int32_t* start_out, int64_t* tel_out,
                        int64_t* evictions_out, int64_t* peak_out);

/* Peak rates of the execution resources that bound the schedule simulator, measured on the current
 * CUDA device by short probe kernels (measurement support for rooflines; the paper has no
 * counterpart).  Each probe keeps every SM busy with independent dependency chains of one kind of
 * work and is timed with CUDA events on `cuda_stream` (cudaStream_t as void*, NULL: default stream);
 * the best of `repeats` (1..64) timed launches after one warm-up launch is reported, in lane
 * operations per second (32 per warp instruction) or bytes per second, at whatever clock the device
 * runs while probed:
 *   out[SCHED_PROBE_INT_ADD]      32-bit integer adds
 *   out[SCHED_PROBE_INT_ADD_MAX]  adds and maxima alternating
 *   out[SCHED_PROBE_INT_MAD]      32-bit integer multiply-adds
 *   out[SCHED_PROBE_SIM_MIX]      a two-pipe mix: multiply-add, 3-input max, add in turn
 *   out[SCHED_PROBE_SMEM_LOAD]    shared-memory loads, 16 bytes per thread and access
 *   out[SCHED_PROBE_SMEM_STORE]   shared-memory stores, 16 bytes per thread and access
 *   out[SCHED_PROBE_INT_ALU]      maxima and exclusive-ors alternating: work that only the integer
 *                                 ALU pipe executes (the compiler may spread plain adds over the
 *                                 ALU and the multiply-add pipe, never these)
 *   out : host double[n_out], n_out >= SCHED_PROBE_COUNT.
 * Synchronous; allocates and frees a few MB of device memory; about 50 ms on one GPU.
 * SCHED_E_INVAL: NULL out, n_out too small, repeats out of range. */
enum {
    SCHED_PROBE_INT_ADD = 0,
    SCHED_PROBE_INT_ADD_MAX = 1,
    SCHED_PROBE_INT_MAD = 2,
    SCHED_PROBE_SIM_MIX = 3,
    SCHED_PROBE_SMEM_LOAD = 4,
    SCHED_PROBE_SMEM_STORE = 5,
    SCHED_PROBE_INT_ALU = 6,
    SCHED_PROBE_COUNT = 7
};
int sched_probe_peaks(double* out, int32_t n_out, int32_t repeats, void* cuda_stream);

/* Which build this library is: 0, or SCHED_BUILD_CHECKED for the checked build
 * (libkvsched_checked.so, compiled with -DKVSCHED_CHECKED), in which every index a kernel derives
 * from data or from its own arithmetic is range-checked before use.  An index outside its array is
 * recorded, element 0 is accessed in its place -- no access ever leaves an array, nothing traps --
 * and the host call that next reads the device status returns SCHED_E_INTERNAL with the site
 * number and the index in sched_last_cuda_error().  The checked build is several times slower; it
 * is the library's own memory checker, meant to be run over small cases. */
#define SCHED_BUILD_CHECKED 1
int sched_build_flags(void);

/* Test support for the checked build: passes `index` through the same range check against
 * 0 .. limit-1 inside a one-thread kernel and reports as any other call would: SCHED_OK if it was in
 * range, SCHED_E_INTERNAL (cleared afterwards) if not.  SCHED_E_UNSUPPORTED in the normal build.
 * Nothing is accessed out of range in either case. */
int sched_debug_check_index(int64_t index, int64_t limit);

/* Test support (the paper has no counterpart): every device loop of this library whose trip count
 * depends on the data is bounded by a cap that it can never reach on valid input; a loop that does
 * reach its cap records that in a status word and returns, the kernel ends normally, and the host
 * call that reads the status (the host-pointer entry points, sched_sync, sched_local_search,
 * sched_accept_move) returns SCHED_E_INTERNAL and clears it.  This call lowers every such cap on the
 * current CUDA device to `cap` iterations so that a test can make one run out (cap = 0: the first
 * request that has to wait gives up); a negative cap restores the natural bounds.  Results computed
 * while a lowered cap is in force are meaningless.  Synchronises the device; not for concurrent use
 * with running kernels of this library. */
int sched_debug_set_loop_cap(int32_t cap);

/* Give every cached device block (see "Conventions" above) back to the driver.  Always SCHED_OK. */
int sched_release_cached_memory(void);

/* Counters since sched_init: kernels launched by this handle, candidates evaluated. */
int sched_stats(sched_handle h, int64_t* kernel_launches_out, int64_t* evaluations_out);

int sched_destroy(sched_handle h);

const char* sched_strerror(int code);
/* Text of the last CUDA error seen by this library on the calling thread ("" if none). */
const char* sched_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* KVSCHED_H */
