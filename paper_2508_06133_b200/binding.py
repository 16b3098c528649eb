"""Thin ctypes binding of the kvsched C-ABI (``include/kvsched.h``): argument marshalling only.

Every step of the path runs in the CUDA library; this module allocates nothing but numpy / torch
buffers for inputs and outputs and raises ``SchedError`` on any non-zero return code.  There is no
CPU fallback: if ``libkvsched.so`` is missing, importing the library fails with instructions.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# KVSCHED_CHECKED=1 selects the checked build of the library (every kernel index range-checked)
CHECKED = os.environ.get("KVSCHED_CHECKED") == "1"
LIB_PATH = os.path.join(_HERE, "libkvsched_checked.so" if CHECKED else "libkvsched.so")
BUILD_CHECKED = 1

OK, E_INVAL, E_NOT_PERMUTATION, E_CUDA, E_NOMEM, E_INTERNAL, E_UNSUPPORTED = 0, -1, -2, -3, -4, -5, -6
CAND_ORDER, CAND_MOVE, CAND_START_TIMES, CAND_POLICY = 0, 1, 2, 3
POLICY_FCFS, POLICY_SOF, POLICY_TOTAL_SIZE, POLICY_SORTED_F = 0, 1, 2, 3
NBHD_SWAP, NBHD_SWAP_INSERT, NBHD_SAMPLED = 0, 1, 2

EXPORTS = [
    "sched_init", "sched_init_batch", "sched_set_stream", "sched_sync", "sched_set_prefill_weight", "sched_set_base_order",
    "sched_get_base_order", "sched_eval_batch", "sched_eval_batch_dev", "sched_sweep_dev",
    "sched_sorted_f", "sched_sorted_f_dev", "sched_sorted_f_local_swap", "sched_sorted_f_local_swap_dev", "sched_sorted_f_dp", "sched_sorted_f_quantile", "sched_online_simulate", "sched_amin_simulate", "sched_sorted_f_amin", "sched_local_search", "sched_accept_move", "sched_last_eval_kernel_ms", "sched_argmin_static_dev", "sched_probe_peaks", "sched_build_flags", "sched_debug_check_index", "sched_debug_set_loop_cap", "sched_release_cached_memory", "sched_stats", "sched_destroy",
    "sched_strerror", "sched_last_cuda_error",
]

_lib = None


class SchedError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        l = load()
        msg = l.sched_strerror(code).decode()
        cuda = l.sched_last_cuda_error().decode()
        super().__init__("%s failed: %s (%d)%s" % (where, msg, code, (" [" + cuda + "]") if cuda and code == E_CUDA else ""))


def load():
    """Load libkvsched.so (after torch, so that both share one CUDA runtime)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError("%s is not built: run `python -m paper_2508_06133_b200.build` "
                          "(needs nvcc; there is no CPU fallback)" % os.path.basename(LIB_PATH))
    try:
        import torch  # noqa: F401  (loads libcudart)
    except Exception:  # pragma: no cover
        pass
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, u64 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64
    lib.sched_init.argtypes = [C.POINTER(vp), i32, vp, vp, i64]
    lib.sched_init_batch.argtypes = [C.POINTER(vp), i32, i32, vp, vp, i64]
    lib.sched_set_stream.argtypes = [vp, vp]
    lib.sched_sync.argtypes = [vp]
    lib.sched_set_base_order.argtypes = [vp, vp]
    lib.sched_set_prefill_weight.argtypes = [vp, i32, i32]
    lib.sched_get_base_order.argtypes = [vp, vp]
    lib.sched_eval_batch.argtypes = [vp, C.c_int, i64, vp, vp, vp, vp]
    lib.sched_eval_batch_dev.argtypes = [vp, C.c_int, i64, vp, vp, vp, vp]
    lib.sched_sweep_dev.argtypes = [vp, C.c_int, u64, i32, i64, i64, vp, vp]
    lib.sched_sorted_f.argtypes = [vp, vp, vp, vp, vp]
    lib.sched_sorted_f_dev.argtypes = [vp, vp, vp, vp, vp]
    lib.sched_sorted_f_local_swap.argtypes = [vp, vp, vp, vp, vp]
    lib.sched_sorted_f_local_swap_dev.argtypes = [vp, vp, vp, vp, vp]
    lib.sched_sorted_f_dp.argtypes = [vp, vp, vp, vp, vp]
    lib.sched_sorted_f_quantile.argtypes = [vp, C.c_uint64, vp, vp, vp, vp]
    lib.sched_online_simulate.argtypes = [i32, i32, vp, vp, vp, vp, i64, i32, i32, i32, vp, vp, vp]
    lib.sched_amin_simulate.argtypes = [i32, i32, vp, vp, vp, vp, i64, vp, vp, vp, vp, vp, vp]
    lib.sched_sorted_f_amin.argtypes = [i32, vp, vp, vp, i64, i32, vp, vp, vp, vp, vp]
    lib.sched_local_search.argtypes = [vp, C.c_int, i32, u64, i64, vp, vp, vp, vp]
    lib.sched_accept_move.argtypes = [vp, i64, i64, C.c_int, u64, i32, vp, vp]
    lib.sched_release_cached_memory.argtypes = []
    lib.sched_stats.argtypes = [vp, vp, vp]
    lib.sched_last_eval_kernel_ms.argtypes = [vp, vp]
    lib.sched_argmin_static_dev.argtypes = [vp, i64, i64, vp, vp]
    lib.sched_probe_peaks.argtypes = [vp, i32, i32, vp]
    lib.sched_debug_set_loop_cap.argtypes = [i32]
    lib.sched_build_flags.argtypes = []
    lib.sched_debug_check_index.argtypes = [i64, i64]
    lib.sched_destroy.argtypes = [vp]
    lib.sched_strerror.argtypes = [C.c_int]
    lib.sched_strerror.restype = C.c_char_p
    lib.sched_last_cuda_error.argtypes = []
    lib.sched_last_cuda_error.restype = C.c_char_p
    for name in EXPORTS:
        if name not in ("sched_strerror", "sched_last_cuda_error"):
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


def _np_ptr(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


def _dev_ptr(t):
    """Device pointer of a contiguous CUDA torch tensor (or None)."""
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous()
    return C.c_void_p(t.data_ptr())


def _check(rc, where):
    if rc != OK:
        raise SchedError(rc, where)


class Scheduler:
    """One handle of the C library.  Methods mirror the C entry points one to one."""

    def __init__(self, s, o, M, *, batch=None):
        lib = load()
        s = np.ascontiguousarray(s, dtype=np.int32)
        o = np.ascontiguousarray(o, dtype=np.int32)
        self._h = C.c_void_p()
        self.M = int(M)
        if batch is None:
            self.B, self.n = 1, int(s.shape[0])
            rc = lib.sched_init(C.byref(self._h), self.n, _np_ptr(s), _np_ptr(o), self.M)
            where = "sched_init"
        else:
            self.B, self.n = int(s.shape[0]), int(s.shape[1])
            rc = lib.sched_init_batch(C.byref(self._h), self.B, self.n, _np_ptr(s), _np_ptr(o), self.M)
            where = "sched_init_batch"
        if rc != OK:
            self._h = None
            raise SchedError(rc, where)

    @classmethod
    def batch(cls, s, o, M):
        return cls(s, o, M, batch=True)

    # ---- lifetime
    def close(self):
        if getattr(self, "_h", None):
            load().sched_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    # ---- plumbing
    def set_stream(self, stream=None):
        """``stream``: a torch.cuda.Stream (or None for the handle's own stream)."""
        ptr = C.c_void_p(stream.cuda_stream) if stream is not None else None
        _check(load().sched_set_stream(self._h, ptr), "sched_set_stream")

    def sync(self):
        _check(load().sched_sync(self._h), "sched_sync")

    def stats(self):
        a, b = C.c_int64(0), C.c_int64(0)
        _check(load().sched_stats(self._h, C.byref(a), C.byref(b)), "sched_stats")
        return a.value, b.value

    def last_eval_kernel_ms(self):
        ms = C.c_float(0)
        _check(load().sched_last_eval_kernel_ms(self._h, C.byref(ms)), "sched_last_eval_kernel_ms")
        return ms.value

    def set_prefill_weight(self, alpha_num, alpha_den=1):
        """Batch metric G = sum(alpha*s + o)/k^2 with alpha = alpha_num/alpha_den (0: the F-metric)."""
        _check(load().sched_set_prefill_weight(self._h, alpha_num, alpha_den), "sched_set_prefill_weight")

    def set_base_order(self, order):
        order = np.ascontiguousarray(order, dtype=np.int32)
        if order.shape != (self.n,):
            raise SchedError(E_INVAL, "sched_set_base_order")
        _check(load().sched_set_base_order(self._h, _np_ptr(order)), "sched_set_base_order")

    def get_base_order(self):
        out = np.empty(self.n, dtype=np.int32)
        _check(load().sched_get_base_order(self._h, _np_ptr(out)), "sched_get_base_order")
        return out

    # ---- sched_eval_batch (host buffers)
    def eval_batch(self, kind, candidates, *, want_feasible=False, want_starts=False):
        """Returns (tel, feasible or None, starts or None) as numpy arrays."""
        if kind in (CAND_ORDER, CAND_START_TIMES):
            cand = np.ascontiguousarray(candidates, dtype=np.int32).reshape(-1, self.n)
            count, outs = cand.shape[0], cand.shape[0]
        elif kind == CAND_MOVE:
            cand = np.ascontiguousarray(candidates, dtype=np.int64).reshape(-1)
            count, outs = cand.shape[0], cand.shape[0]
        else:
            cand = np.ascontiguousarray(candidates, dtype=np.int32).reshape(-1)
            count, outs = cand.shape[0], cand.shape[0] * self.B
        tel = np.empty(outs, dtype=np.int64)
        feas = np.empty(outs, dtype=np.uint8) if want_feasible else None
        starts = np.empty((outs, self.n), dtype=np.int32) if want_starts else None
        _check(load().sched_eval_batch(self._h, kind, count, _np_ptr(cand), _np_ptr(tel), _np_ptr(feas), _np_ptr(starts)),
               "sched_eval_batch")
        if kind == CAND_POLICY:
            tel = tel.reshape(self.B, count)
            feas = feas.reshape(self.B, count) if feas is not None else None
            starts = starts.reshape(self.B, count, self.n) if starts is not None else None
        return tel, feas, starts

    # ---- device-pointer forms (torch CUDA tensors); asynchronous
    def eval_batch_dev(self, kind, count, candidates, tel_out, feasible_out=None, starts_out=None):
        _check(load().sched_eval_batch_dev(self._h, kind, count, _dev_ptr(candidates), _dev_ptr(tel_out),
                                           _dev_ptr(feasible_out), _dev_ptr(starts_out)), "sched_eval_batch_dev")

    def sweep_dev(self, count, best_out, *, first_code=0, sampled=False, seed=0, iteration=0, tel_out=None):
        _check(load().sched_sweep_dev(self._h, 1 if sampled else 0, seed, iteration, first_code, count,
                                      _dev_ptr(tel_out), _dev_ptr(best_out)), "sched_sweep_dev")

    def sorted_f_dev(self, order_out=None, batch_offsets_out=None, num_batches_out=None, tel_out=None):
        _check(load().sched_sorted_f_dev(self._h, _dev_ptr(order_out), _dev_ptr(batch_offsets_out),
                                         _dev_ptr(num_batches_out), _dev_ptr(tel_out)), "sched_sorted_f_dev")

    # ---- sched_sorted_f / sched_local_search (host buffers)
    def sorted_f(self):
        """Returns (order, batch_offsets[0..num_batches], TEL)."""
        order = np.empty(self.n, dtype=np.int32)
        offs = np.zeros(self.n + 1, dtype=np.int32)
        nb, tel = C.c_int32(0), C.c_int64(0)
        _check(load().sched_sorted_f(self._h, _np_ptr(order), _np_ptr(offs), C.byref(nb), C.byref(tel)), "sched_sorted_f")
        return order, offs[:nb.value + 1].copy(), tel.value

    def sorted_f_local_swap(self):
        """Sorted-F with Algorithm 3 as Phase-1 solver.  Returns (order, batch_offsets, TEL)."""
        order = np.empty(self.n, dtype=np.int32)
        offs = np.zeros(self.n + 1, dtype=np.int32)
        nb, tel = C.c_int32(0), C.c_int64(0)
        _check(load().sched_sorted_f_local_swap(self._h, _np_ptr(order), _np_ptr(offs), C.byref(nb), C.byref(tel)),
               "sched_sorted_f_local_swap")
        return order, offs[:nb.value + 1].copy(), tel.value

    def sorted_f_dp(self):
        """Sorted-F with the exact dynamic programme (Algorithm 2) as Phase-1 solver; small n only.
        Returns (order, batch_offsets, TEL)."""
        order = np.empty(self.n, dtype=np.int32)
        offs = np.zeros(self.n + 1, dtype=np.int32)
        nb, tel = C.c_int32(0), C.c_int64(0)
        _check(load().sched_sorted_f_dp(self._h, _np_ptr(order), _np_ptr(offs), C.byref(nb), C.byref(tel)),
               "sched_sorted_f_dp")
        return order, offs[:nb.value + 1].copy(), tel.value

    def sorted_f_quantile(self, seed=0):
        """Sorted-F with Quantile Greedy Selection (Algorithm 4) as Phase-1 solver.
        Returns (order, batch_offsets, TEL)."""
        order = np.empty(self.n, dtype=np.int32)
        offs = np.zeros(self.n + 1, dtype=np.int32)
        nb, tel = C.c_int32(0), C.c_int64(0)
        _check(load().sched_sorted_f_quantile(self._h, C.c_uint64(seed), _np_ptr(order), _np_ptr(offs), C.byref(nb), C.byref(tel)),
               "sched_sorted_f_quantile")
        return order, offs[:nb.value + 1].copy(), tel.value

    def sorted_f_local_swap_dev(self, order_out=None, batch_offsets_out=None, num_batches_out=None, tel_out=None):
        _check(load().sched_sorted_f_local_swap_dev(self._h, _dev_ptr(order_out), _dev_ptr(batch_offsets_out),
                                                    _dev_ptr(num_batches_out), _dev_ptr(tel_out)), "sched_sorted_f_local_swap_dev")

    def local_search(self, neighbourhood, iters, *, order=None, seed=0, samples_per_iter=0):
        """Returns (final order, TEL, iterations done, trace[(code, best TEL)])."""
        buf = None
        if order is not None:
            buf = np.ascontiguousarray(order, dtype=np.int32).copy()
            if buf.shape != (self.n,):
                raise SchedError(E_INVAL, "sched_local_search")
        trace = np.full((max(iters, 1), 2), -1, dtype=np.int64)
        tel, done = C.c_int64(0), C.c_int32(0)
        _check(load().sched_local_search(self._h, neighbourhood, iters, seed, samples_per_iter, _np_ptr(buf),
                                         C.byref(tel), C.byref(done), _np_ptr(trace)), "sched_local_search")
        final = buf if buf is not None else self.get_base_order()
        return final, tel.value, done.value, trace[:done.value].copy()

    def accept_move(self, best_tel, best_index, *, sampled=False, seed=0, iteration=0):
        """Apply the move iff it beats the base order's TEL (see sched_accept_move).
        Returns (accepted, TEL of the base order afterwards)."""
        acc, tel = C.c_int32(0), C.c_int64(0)
        _check(load().sched_accept_move(self._h, int(best_tel), int(best_index), 1 if sampled else 0, seed, iteration,
                                        C.byref(acc), C.byref(tel)), "sched_accept_move")
        return bool(acc.value), tel.value


def release_cached_memory():
    """Return the library's cached device blocks to the driver (sched_release_cached_memory)."""
    _check(load().sched_release_cached_memory(), "sched_release_cached_memory")


def build_flags():
    """0, or BUILD_CHECKED when the loaded library is the checked build (sched_build_flags)."""
    return load().sched_build_flags()


def debug_check_index(index, limit):
    """Checked build only: run ``index`` through the kernels' range check against 0..limit-1
    (sched_debug_check_index); raises SchedError(E_INTERNAL) if it is out of range."""
    _check(load().sched_debug_check_index(int(index), int(limit)), "sched_debug_check_index")


def debug_set_loop_cap(cap):
    """Lower (cap >= 0) or restore (cap < 0) the iteration caps of the library's device loops on the
    current device -- test support, see sched_debug_set_loop_cap."""
    _check(load().sched_debug_set_loop_cap(int(cap)), "sched_debug_set_loop_cap")


PROBE_NAMES = ("int_add", "int_add_max", "int_mad", "sim_mix", "smem_load", "smem_store", "int_alu")


def probe_peaks(repeats=5, stream=None):
    """Peak rates of the current CUDA device from the library's probe kernels (sched_probe_peaks):
    dict name -> lane operations per second (the four integer probes) or bytes per second (shared
    memory), measured now, at the clock the device runs at."""
    out = np.zeros(len(PROBE_NAMES), dtype=np.float64)
    ptr = C.c_void_p(stream.cuda_stream) if stream is not None else None
    _check(load().sched_probe_peaks(_np_ptr(out), len(out), int(repeats), ptr), "sched_probe_peaks")
    return dict(zip(PROBE_NAMES, out.tolist()))


def argmin_static_dev(tel, best_out, *, count=None, index_base=0, stream=None):
    """Best (TEL, index) of a device TEL tensor through ``sched_argmin_static_dev``: the variant of
    the arg-min that allocates nothing, for callers that may not touch the device allocator (its
    scratch is a fixed array inside the library).  ``tel``/``best_out`` are CUDA int64 tensors on the
    current device; asynchronous on ``stream`` (a torch.cuda.Stream) or the default stream.  Calls
    that could overlap on one GPU must be ordered by the caller: they share the scratch array."""
    n = int(tel.numel()) if count is None else int(count)
    ptr = C.c_void_p(stream.cuda_stream) if stream is not None else None
    _check(load().sched_argmin_static_dev(_dev_ptr(tel), n, index_base, _dev_ptr(best_out), ptr),
           "sched_argmin_static_dev")


def online_simulate(n_each, arrival, s, o, M, policy, period=10, lookahead=300):
    """B arrival streams under one online policy (rows of [B, n_max] arrays; see sched_online_simulate).
    Returns (start times [B, n_max], total latency per stream [B], kernel milliseconds)."""
    arrival = np.ascontiguousarray(arrival, dtype=np.int32)
    s = np.ascontiguousarray(s, dtype=np.int32)
    o = np.ascontiguousarray(o, dtype=np.int32)
    n_each = np.ascontiguousarray(n_each, dtype=np.int32)
    if arrival.ndim != 2 or s.shape != arrival.shape or o.shape != arrival.shape or n_each.shape != (arrival.shape[0],):
        raise ValueError("arrival, s, o must be [B, n_max] and n_each [B]")
    B, n_max = arrival.shape
    starts = np.empty((B, n_max), dtype=np.int32)
    lat = np.empty(B, dtype=np.int64)
    ms = C.c_float(0.0)
    _check(load().sched_online_simulate(B, n_max, _np_ptr(n_each), _np_ptr(arrival), _np_ptr(s), _np_ptr(o), int(M),
                                        int(policy), int(period), int(lookahead), _np_ptr(starts), _np_ptr(lat), C.byref(ms)),
           "sched_online_simulate")
    return starts, lat, ms.value


def amin_simulate(n_each, s, lower, o, M, order):
    """B scenarios of Sorted-F + A_min's executor (rows of [B, n_max] arrays; see sched_amin_simulate).
    Returns (start times [B, n_max], TEL [B], evictions [B], peak memory [B], kernel milliseconds)."""
    s = np.ascontiguousarray(s, dtype=np.int32)
    lower = np.ascontiguousarray(lower, dtype=np.int32)
    o = np.ascontiguousarray(o, dtype=np.int32)
    order = np.ascontiguousarray(order, dtype=np.int32)
    n_each = np.ascontiguousarray(n_each, dtype=np.int32)
    if s.ndim != 2 or lower.shape != s.shape or o.shape != s.shape or order.shape != s.shape or n_each.shape != (s.shape[0],):
        raise ValueError("s, lower, o, order must be [B, n_max] and n_each [B]")
    B, n_max = s.shape
    starts = np.empty((B, n_max), dtype=np.int32)
    tel = np.empty(B, dtype=np.int64)
    ev = np.empty(B, dtype=np.int64)
    peak = np.empty(B, dtype=np.int64)
    ms = C.c_float(0.0)
    _check(load().sched_amin_simulate(B, n_max, _np_ptr(n_each), _np_ptr(s), _np_ptr(lower), _np_ptr(o), int(M),
                                      _np_ptr(order), _np_ptr(starts), _np_ptr(tel), _np_ptr(ev), _np_ptr(peak),
                                      C.byref(ms)), "sched_amin_simulate")
    return starts, tel, ev, peak, ms.value


def sorted_f_amin(s, lower, o, M, phase1=0):
    """Sorted-F + A_min for one backlog: Phase 1 on the lower bounds (0: prefix-F, 1: Algorithm 3), then
    the adaptive executor.  Returns (order, start times, TEL, evictions, peak memory)."""
    s = np.ascontiguousarray(s, dtype=np.int32)
    lower = np.ascontiguousarray(lower, dtype=np.int32)
    o = np.ascontiguousarray(o, dtype=np.int32)
    if s.ndim != 1 or lower.shape != s.shape or o.shape != s.shape:
        raise ValueError("s, lower, o must be 1-D arrays of one length")
    n = s.shape[0]
    order = np.empty(n, dtype=np.int32)
    starts = np.empty(n, dtype=np.int32)
    tel, ev, peak = C.c_int64(0), C.c_int64(0), C.c_int64(0)
    _check(load().sched_sorted_f_amin(n, _np_ptr(s), _np_ptr(lower), _np_ptr(o), int(M), int(phase1), _np_ptr(order),
                                      _np_ptr(starts), C.byref(tel), C.byref(ev), C.byref(peak)), "sched_sorted_f_amin")
    return order, starts, tel.value, ev.value, peak.value
