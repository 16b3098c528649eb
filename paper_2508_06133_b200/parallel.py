"""Order-level local search with the neighbourhood sweep split over ranks (one process per GPU).

Every rank holds the same backlog and the same base order.  In every iteration rank r evaluates a
contiguous share of the move indices with the library's sweep (``sched_sweep_dev``), the ranks
agree on the smallest (TEL, index) pair with two all-reduce(min) operations of one int64 each --
first the TEL, then the lowest index among the ranks that attain it -- and every rank applies that
move with ``sched_accept_move``, so the base orders never diverge.  The result is the one
``sched_local_search`` gives on a single GPU: the same accepted moves, the same final order.

This module holds no scheduling arithmetic: the evaluation and the acceptance run in the CUDA
library, the exchange in ``torch.distributed`` (NCCL between GPUs; gloo in the CPU tests, where the
evaluator is a stand-in).
"""
from __future__ import annotations

import numpy as np

from . import binding as kv

I64_MAX = np.iinfo(np.int64).max


def neighbourhood_size(n: int, neighbourhood: int, samples_per_iter: int = 0) -> int:
    if n < 2:
        return 0
    if neighbourhood == kv.NBHD_SWAP:
        return n * (n - 1) // 2
    if neighbourhood == kv.NBHD_SWAP_INSERT:
        return n * (n - 1) // 2 + n * (n - 1)
    if neighbourhood == kv.NBHD_SAMPLED:
        return int(samples_per_iter)
    raise ValueError("unknown neighbourhood %r" % (neighbourhood,))


def shard(total: int, rank: int, world: int):
    """Contiguous share of the indices 0 .. total-1 for ``rank``: (first, count); shares differ by at
    most one index and cover the range exactly."""
    lo = total * rank // world
    hi = total * (rank + 1) // world
    return lo, hi - lo


class GpuEvaluator:
    """The two calls the search needs, on a ``binding.Scheduler`` handle."""

    def __init__(self, scheduler, device=None):
        import torch
        self.h = scheduler
        self.n = scheduler.n
        self.best = torch.zeros(2, dtype=torch.int64, device=device if device is not None else "cuda")

    def base_tel(self) -> int:
        return self.h.accept_move(I64_MAX, 0)[1]          # never accepted: reports the current TEL

    def sweep(self, first, count, sampled, seed, iteration):
        self.h.sweep_dev(count, self.best, first_code=first, sampled=sampled, seed=seed, iteration=iteration)
        self.h.sync()
        tel, idx = self.best.cpu().tolist()
        return int(tel), int(idx)

    def accept(self, tel, idx, sampled, seed, iteration):
        return self.h.accept_move(tel, idx, sampled=sampled, seed=seed, iteration=iteration)


class TorchComm:
    """all-reduce(min) of one int64 over a torch.distributed process group."""

    def __init__(self, group=None, device="cpu"):
        import torch.distributed as dist
        self.dist, self.group, self.device = dist, group, device
        self.rank = dist.get_rank(group)
        self.world = dist.get_world_size(group)

    def min(self, value: int) -> int:
        import torch
        t = torch.tensor([value], dtype=torch.int64, device=self.device)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MIN, group=self.group)
        return int(t.item())


class SingleRank:
    rank, world = 0, 1

    def min(self, value: int) -> int:
        return value


def sharded_iteration(evaluator, comm, total, sampled, seed, iteration):
    """One iteration of the search over ``total`` move indices: this rank sweeps its share, the ranks
    agree on the smallest (TEL, index) pair -- all-reduce(min) of the TEL, then of the lowest index
    among the ranks that attain it -- and every rank applies that pair through ``evaluator.accept``.
    Returns (accepted, TEL of the base order afterwards, winning index, winning TEL)."""
    first, count = shard(total, comm.rank, comm.world)
    tel, idx = evaluator.sweep(first, count, sampled, seed, iteration) if count > 0 else (I64_MAX, I64_MAX)
    best_tel = comm.min(tel)
    best_idx = comm.min(idx if tel == best_tel else I64_MAX)
    accepted, cur = evaluator.accept(best_tel, best_idx, sampled, seed, iteration)
    return accepted, cur, best_idx, best_tel


def sharded_local_search(evaluator, neighbourhood, iters, *, seed=0, samples_per_iter=0, comm=None):
    """Runs the search described in the module docstring.  ``evaluator`` has ``n``, ``base_tel()``,
    ``sweep(first, count, sampled, seed, iteration) -> (TEL, index)`` and
    ``accept(TEL, index, sampled, seed, iteration) -> (accepted, TEL)``; ``comm`` has ``rank``,
    ``world`` and ``min(int) -> int``.  Returns (TEL, iterations done, trace[(index, best TEL)]) --
    SWAP / SWAP_INSERT stop at the first iteration without an improving move (that iteration is
    counted), SAMPLED always runs ``iters`` iterations, as ``sched_local_search`` does."""
    comm = comm if comm is not None else SingleRank()
    sampled = neighbourhood == kv.NBHD_SAMPLED
    total = neighbourhood_size(evaluator.n, neighbourhood, samples_per_iter)
    cur = evaluator.base_tel()
    trace = []
    done = 0
    while done < iters and total > 0:
        accepted, cur, best_idx, best_tel = sharded_iteration(evaluator, comm, total, sampled, seed, done)
        trace.append((best_idx, best_tel))
        done += 1
        if not accepted and not sampled:
            break
    return cur, done, np.array(trace, dtype=np.int64).reshape(-1, 2)
