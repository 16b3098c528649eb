"""ctypes front end of the CPU oracle (``oracle.cpp``) -- test infrastructure only.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this package; the
GPU library never does.  ``build()`` compiles ``oracle.cpp`` with g++ into ``liboracle.so`` next to
it; ``lib()`` builds on first use if the shared object is missing or older than the source.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle.cpp")
_SO = os.path.join(_HERE, "liboracle.so")
_lib = None

FCFS, SHORTEST_OUTPUT_FIRST, TOTAL_SIZE_FIRST = 0, 1, 2
SOF, SORTED_F = 1, 3                     # online policies: shortest decode first, Sorted-F-Online
ENUM_ALG1, ENUM_SUM, DP = 0, 1, 2
SWAP, SWAP_INSERT, SAMPLED = 0, 1, 2


def build(force: bool = False) -> str:
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + ".%d.tmp" % os.getpid()
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-pthread", "-shared", "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _SO)
    return _SO


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_bruteforce_opt.restype = C.c_longlong
        _lib.orc_bruteforce_best_order.restype = C.c_longlong
    return _lib


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def check_schedule(s, o, M, p):
    """Returns dict(feasible, tel, peak, first_bad_round, makespan) for explicit start times p."""
    s, o = _i32(s), _i32(o)
    p = np.ascontiguousarray(p, dtype=np.int64)
    out = [C.c_longlong(0) for _ in range(4)]
    rc = lib().orc_check_schedule(len(s), _p(s), _p(o), C.c_longlong(M), _p(p), *[C.byref(x) for x in out])
    return dict(feasible=rc == 1, rc=rc, tel=out[0].value, peak=out[1].value,
                first_bad_round=out[2].value, makespan=out[3].value)


def occupancy(s, o, p, length):
    s, o = _i32(s), _i32(o)
    p = np.ascontiguousarray(p, dtype=np.int64)
    U = np.zeros(length, dtype=np.int64)
    R = np.zeros(length, dtype=np.int64)
    lib().orc_occupancy(len(s), _p(s), _p(o), _p(p), C.c_longlong(length), _p(U), _p(R))
    return U, R


def _list(fn, s, o, M, order):
    s, o, order = _i32(s), _i32(o), _i32(order)
    p = np.zeros(len(s), dtype=np.int64)
    tel, mk = C.c_longlong(0), C.c_longlong(0)
    rc = fn(len(s), _p(s), _p(o), C.c_longlong(M), _p(order), _p(p), C.byref(tel), C.byref(mk))
    if rc != 0:
        raise ValueError("invalid instance (need s, o >= 1 and s + o <= M)")
    return p, tel.value, mk.value


def list_schedule_alg1(s, o, M, order):
    """Algorithm 1 Phase 2, literal.  Returns (starts p, TEL, makespan)."""
    return _list(lib().orc_list_schedule_alg1, s, o, M, order)


def list_schedule_rounds(s, o, M, order):
    """Same executor on the per-round occupancy array.  Returns (starts p, TEL, makespan)."""
    return _list(lib().orc_list_schedule_rounds, s, o, M, order)


def policy_order(s, o, policy):
    s, o = _i32(s), _i32(o)
    order = np.zeros(len(s), dtype=np.int32)
    lib().orc_policy_order(len(s), _p(s), _p(o), policy, _p(order))
    return order


def f_compare(sum_a, k_a, sum_b, k_b):
    return lib().orc_f_compare(C.c_longlong(sum_a), C.c_longlong(k_a), C.c_longlong(sum_b), C.c_longlong(k_b))


def _phase1(fn, ids, s, o, M, *extra):
    s, o, ids = _i32(s), _i32(o), _i32(ids)
    chosen = np.zeros(len(ids), dtype=np.int32)
    so, mem = C.c_longlong(0), C.c_longlong(0)
    c = fn(len(ids), _p(ids), _p(s), _p(o), C.c_longlong(M), *extra, _p(chosen), C.byref(so), C.byref(mem))
    if c < 0:
        raise ValueError("instance too large for this solver")
    return chosen[:c].copy(), so.value, mem.value


def phase1_enumerate(ids, s, o, M, reading):
    return _phase1(lib().orc_phase1_enumerate, ids, s, o, M, C.c_int(reading))


def phase1_dp(ids, s, o, M):
    return _phase1(lib().orc_phase1_dp, ids, s, o, M)


def sorted_f_exact(s, o, M, solver):
    s, o = _i32(s), _i32(o)
    n = len(s)
    order = np.zeros(n, dtype=np.int32)
    offs = np.zeros(n + 1, dtype=np.int32)
    nb = lib().orc_sorted_f_exact(n, _p(s), _p(o), C.c_longlong(M), solver, _p(order), _p(offs))
    if nb < 0:
        raise ValueError("exact Sorted-F failed")
    return order, offs[:nb + 1].copy()


def sorted_f_prefix(s, o, M):
    s, o = _i32(s), _i32(o)
    n = len(s)
    order = np.zeros(n, dtype=np.int32)
    offs = np.zeros(n + 1, dtype=np.int32)
    nb = lib().orc_sorted_f_prefix(n, _p(s), _p(o), C.c_longlong(M), _p(order), _p(offs))
    if nb < 0:
        raise ValueError("a request exceeds M")
    return order, offs[:nb + 1].copy()


def decode_move(n, code):
    t, i, j = C.c_int(0), C.c_int(0), C.c_int(0)
    if lib().orc_decode_move(n, C.c_longlong(code), C.byref(t), C.byref(i), C.byref(j)) != 0:
        raise ValueError("move code out of range")
    return t.value, i.value, j.value


def sample_move(n, seed, it, m):
    t, i, j = C.c_int(0), C.c_int(0), C.c_int(0)
    lib().orc_sample_move(n, C.c_ulonglong(seed), it, C.c_longlong(m), C.byref(t), C.byref(i), C.byref(j))
    return t.value, i.value, j.value


def apply_move(base, mtype, i, j):
    base = _i32(base)
    out = np.zeros_like(base)
    lib().orc_apply_move(len(base), _p(base), mtype, i, j, _p(out))
    return out


def eval_moves(s, o, M, base, types, mi, mj):
    s, o, base = _i32(s), _i32(o), _i32(base)
    types, mi, mj = _i32(types), _i32(mi), _i32(mj)
    tel = np.zeros(len(types), dtype=np.int64)
    rc = lib().orc_eval_moves(len(s), _p(s), _p(o), C.c_longlong(M), _p(base), C.c_longlong(len(types)),
                              _p(types), _p(mi), _p(mj), _p(tel))
    if rc != 0:
        raise ValueError("invalid instance")
    return tel


def eval_moves_threads(s, o, M, base, types, mi, mj, threads=1, literal=False):
    """``eval_moves`` with the candidates split over ``threads`` host threads (CPU-baseline timing);
    ``literal`` scores with Algorithm 1 Phase 2 as listed instead of the per-round form."""
    s, o, base = _i32(s), _i32(o), _i32(base)
    types, mi, mj = _i32(types), _i32(mi), _i32(mj)
    tel = np.zeros(len(types), dtype=np.int64)
    rc = lib().orc_eval_moves_threads(len(s), _p(s), _p(o), C.c_longlong(M), _p(base), C.c_longlong(len(types)),
                                      _p(types), _p(mi), _p(mj), _p(tel), int(threads), 1 if literal else 0)
    if rc != 0:
        raise ValueError("invalid instance")
    return tel


def local_search(s, o, M, neighbourhood, iters, order, seed=0, samples=0):
    """Returns (final order, TEL, iterations done, trace[(code, best TEL)] per iteration)."""
    s, o = _i32(s), _i32(o)
    order = _i32(order).copy()
    trace = np.full(2 * max(iters, 1), -1, dtype=np.int64)
    tel, done = C.c_longlong(0), C.c_int(0)
    rc = lib().orc_local_search(len(s), _p(s), _p(o), C.c_longlong(M), neighbourhood, iters,
                                C.c_ulonglong(seed), C.c_longlong(samples), _p(order),
                                C.byref(tel), C.byref(done), _p(trace))
    if rc != 0:
        raise ValueError("invalid instance")
    return order, tel.value, done.value, trace.reshape(-1, 2)[:done.value].copy()


def bruteforce_opt(s, o, M, upper_bound):
    """Optimum of the integer program strictly below ``upper_bound`` (or -1). Returns (TEL, p)."""
    s, o = _i32(s), _i32(o)
    p = np.zeros(len(s), dtype=np.int64)
    v = lib().orc_bruteforce_opt(len(s), _p(s), _p(o), C.c_longlong(M), C.c_longlong(upper_bound), _p(p))
    return v, p


def bruteforce_best_order(s, o, M):
    s, o = _i32(s), _i32(o)
    order = np.zeros(len(s), dtype=np.int32)
    v = lib().orc_bruteforce_best_order(len(s), _p(s), _p(o), C.c_longlong(M), _p(order))
    return v, order


def local_swap_batch(ids, s, o, M):
    """Algorithm 3 on the request set ``ids``.  Returns (X in walking order, accepted swaps)."""
    s, o, ids = _i32(s), _i32(o), _i32(ids)
    chosen = np.zeros(len(ids), dtype=np.int32)
    sw = C.c_longlong(0)
    c = lib().orc_local_swap_batch(len(ids), _p(ids), _p(s), _p(o), C.c_longlong(M), _p(chosen), C.byref(sw))
    if c < 0:
        raise ValueError("a request exceeds M")
    return chosen[:c].copy(), sw.value


def sorted_f_local_swap(s, o, M):
    """Sorted-F with Algorithm 3 as Phase-1 solver.  Returns (order, batch offsets, accepted swaps)."""
    s, o = _i32(s), _i32(o)
    n = len(s)
    order = np.zeros(n, dtype=np.int32)
    offs = np.zeros(n + 1, dtype=np.int32)
    sw = C.c_longlong(0)
    nb = lib().orc_sorted_f_local_swap(n, _p(s), _p(o), C.c_longlong(M), _p(order), _p(offs), C.byref(sw))
    if nb < 0:
        raise ValueError("a request exceeds M")
    return order, offs[:nb + 1].copy(), sw.value


def _sorted_g(fn, s, o, M, a_num, a_den):
    s, o = _i32(s), _i32(o)
    n = len(s)
    order = np.zeros(n, dtype=np.int32)
    offs = np.zeros(n + 1, dtype=np.int32)
    nb = fn(n, _p(s), _p(o), C.c_longlong(M), C.c_longlong(a_num), C.c_longlong(a_den), _p(order), _p(offs))
    if nb < 0:
        raise ValueError("bad weight or a request exceeds M")
    return order, offs[:nb + 1].copy()


def sorted_g_prefix(s, o, M, a_num, a_den):
    """Sorted-G (metric sum(alpha*s+o)/k^2, alpha = a_num/a_den) with prefix batch selection."""
    return _sorted_g(lib().orc_sorted_g_prefix, s, o, M, a_num, a_den)


def sorted_g_local_swap(s, o, M, a_num, a_den):
    """Sorted-G with Algorithm 3 as the batch solver."""
    return _sorted_g(lib().orc_sorted_g_local_swap, s, o, M, a_num, a_den)


def quantile_greedy_batch(ids, s, o, M, sample):
    """Algorithm 4 on the request set ``ids`` with the given sample.
    Returns (X in admission order, Q_p, Q_o)."""
    s, o, ids, sample = _i32(s), _i32(o), _i32(ids), _i32(sample)
    chosen = np.zeros(len(ids), dtype=np.int32)
    qp, qo = C.c_longlong(0), C.c_longlong(0)
    c = lib().orc_quantile_greedy_batch(len(ids), _p(ids), _p(s), _p(o), C.c_longlong(M), len(sample), _p(sample),
                                        _p(chosen), C.byref(qp), C.byref(qo))
    if c <= 0:
        raise ValueError("empty input, empty sample or a request that exceeds M")
    return chosen[:c].copy(), qp.value, qo.value


def quantile_sample(ids, o, seed, batch):
    """The reproducible 'random subset' of Algorithm 4 for batch number ``batch``."""
    o, ids = _i32(o), _i32(ids)
    out = np.zeros(max(1, len(ids)), dtype=np.int32)
    c = lib().orc_quantile_sample(len(ids), _p(ids), _p(o), C.c_uint64(seed), int(batch), _p(out))
    return out[:c].copy()


def sorted_f_quantile(s, o, M, seed):
    """Sorted-F with Algorithm 4 as Phase-1 solver.  Returns (order, batch offsets)."""
    s, o = _i32(s), _i32(o)
    n = len(s)
    order = np.zeros(n, dtype=np.int32)
    offs = np.zeros(n + 1, dtype=np.int32)
    nb = lib().orc_sorted_f_quantile(n, _p(s), _p(o), C.c_longlong(M), C.c_uint64(seed), _p(order), _p(offs))
    if nb < 0:
        raise ValueError("a request exceeds M")
    return order, offs[: nb + 1].copy()


def mix64(z):
    """One splitmix64 step from state ``z`` (the generator behind every sampled quantity)."""
    f = lib().orc_mix64
    f.restype = C.c_uint64
    return int(f(C.c_uint64(z & 0xFFFFFFFFFFFFFFFF)))


def online_schedule(a, s, o, M, policy, period=10, lookahead=300):
    """Online arrivals (FCFS, SOF recomputed every iteration, or Sorted-F-Online), iteration by
    iteration.  Returns (start times, total latency = sum of p + o - a)."""
    a, s, o = _i32(a), _i32(s), _i32(o)
    n = len(s)
    p = np.zeros(n, dtype=np.int64)
    tot = C.c_longlong(0)
    rc = lib().orc_online_schedule(n, _p(a), _p(s), _p(o), C.c_longlong(M), int(policy), int(period), int(lookahead),
                                   p.ctypes.data_as(C.c_void_p), C.byref(tot))
    if rc != 0:
        raise ValueError("invalid online instance or parameters (%d)" % rc)
    return p, tot.value


def amin_schedule(s, lower, o, M, order):
    """Phase 2 of Sorted-F + A_min (Algorithm 5) on the given list with lower bounds ``lower`` of the
    decode lengths.  Returns (final start times, TEL, evictions, peak memory actually used)."""
    s, lower, o, order = _i32(s), _i32(lower), _i32(o), _i32(order)
    n = len(s)
    p = np.zeros(n, dtype=np.int64)
    tel, ev, peak = C.c_longlong(0), C.c_longlong(0), C.c_longlong(0)
    rc = lib().orc_amin_schedule(n, _p(s), _p(lower), _p(o), C.c_longlong(M), _p(order),
                                 p.ctypes.data_as(C.c_void_p), C.byref(tel), C.byref(ev), C.byref(peak))
    if rc != 0:
        raise ValueError("invalid instance or iteration cap (%d)" % rc)
    return p, tel.value, ev.value, peak.value


def amin_schedule_rounds(s, lower, o, M, order):
    """Same executor on a per-round array of projected memory (O14'); same return values."""
    s, lower, o, order = _i32(s), _i32(lower), _i32(o), _i32(order)
    n = len(s)
    p = np.zeros(n, dtype=np.int64)
    tel, ev, peak = C.c_longlong(0), C.c_longlong(0), C.c_longlong(0)
    rc = lib().orc_amin_schedule_rounds(n, _p(s), _p(lower), _p(o), C.c_longlong(M), _p(order),
                                        p.ctypes.data_as(C.c_void_p), C.byref(tel), C.byref(ev), C.byref(peak))
    if rc != 0:
        raise ValueError("invalid instance or iteration cap (%d)" % rc)
    return p, tel.value, ev.value, peak.value
