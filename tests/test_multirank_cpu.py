"""World-size-2 checks (gloo, CPU) of how the benchmark spreads one sampled neighbourhood over ranks
(disjoint contiguous sample slices, the same moves as a single rank would draw, the max-over-ranks
time reduction) and of the step it times under torchrun: one iteration of the sharded local search
with its all-reduce(min) exchange.  No GPU and no kernel is involved."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    count, n, seed, it = 1000, 500, 7, 3
    first, share = bench.rank_share(world * count, rank, world)
    ok_share = share == count
    ty, mi, mj = bench.sampled_move_positions(n, seed, it, first, count)
    mine = torch.from_numpy(np.stack([ty, mi, mj]))
    gathered = [torch.zeros_like(mine) for _ in range(world)]
    dist.all_gather(gathered, mine)
    whole = np.stack(bench.sampled_move_positions(n, seed, it, 0, world * count))
    ok = ok_share and bool((torch.cat(gathered, dim=1).numpy() == whole).all())
    firsts = [torch.zeros(1, dtype=torch.int64) for _ in range(world)]
    dist.all_gather(firsts, torch.tensor([first]))
    ok &= [int(f) for f in firsts] == [r * count for r in range(world)]
    slow = bench.max_over_ranks(10.0 + rank, dist, torch.device("cpu"))
    ok &= slow == 10.0 + world - 1
    out[rank] = ok
    dist.destroy_process_group()


def test_two_ranks_share_one_sampled_neighbourhood():
    world = 2
    port = 29500 + (os.getpid() % 2000)
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        assert dict(out) == {0: True, 1: True}


def test_sampled_positions_match_the_oracles_generator():
    import oracle as orc
    import bench
    n, seed, it = 97, 123456789, 5
    ty, mi, mj = bench.sampled_move_positions(n, seed, it, 40, 300)
    for k in range(300):
        t, i, j = orc.sample_move(n, seed, it, 40 + k)
        a, b = int(mi[k]), int(mj[k])
        if t == 0 and a > b:
            a, b = b, a
        assert (int(ty[k]), a, b) == (t, i, j)


# ---------------------------------------------------------------------------------------------
# The sharded local search (paper_2508_06133_b200/parallel.py) over two gloo ranks.  The evaluator
# is a stand-in that scores moves with the CPU oracle, so that what is checked here is the host
# logic: the shares, the two-step (TEL, index) reduction with its tie rule, the stop rule and that
# every rank applies the same move.  The expected result is the oracle's single-process search.
# ---------------------------------------------------------------------------------------------
class _OracleEvaluator:
    def __init__(self, s, o, M, order):
        import oracle as orc
        self.orc, self.s, self.o, self.M = orc, s, o, M
        self.order = np.array(order, dtype=np.int32)
        self.n = len(s)
        self.sweeps = []

    def base_tel(self):
        return self.orc.list_schedule_rounds(self.s, self.o, self.M, self.order)[1]

    def _move(self, idx, sampled, seed, it):
        return self.orc.sample_move(self.n, seed, it, idx) if sampled else self.orc.decode_move(self.n, idx)

    def sweep(self, first, count, sampled, seed, it):
        self.sweeps.append((first, count))
        mv = [self._move(first + k, sampled, seed, it) for k in range(count)]
        tels = self.orc.eval_moves(self.s, self.o, self.M, self.order, [m[0] for m in mv], [m[1] for m in mv], [m[2] for m in mv])
        k = int(np.argmin(tels))                                     # first minimum = lowest index
        return int(tels[k]), first + k

    def accept(self, tel, idx, sampled, seed, it):
        cur = self.base_tel()
        if tel < cur:
            self.order = self.orc.apply_move(self.order, *self._move(idx, sampled, seed, it))
            assert self.base_tel() == tel
            return True, tel
        return False, cur


def _search_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle as orc
    from paper_2508_06133_b200 import binding as kv, parallel as par
    rng = np.random.default_rng(5)
    n, M = 13, 60
    s = rng.integers(1, 25, n).astype(np.int32)
    o = rng.integers(1, 20, n).astype(np.int32)
    start = rng.permutation(n).astype(np.int32)
    ok = True
    for nbhd, iters, samples in ((kv.NBHD_SWAP, 50, 0), (kv.NBHD_SWAP_INSERT, 50, 0), (kv.NBHD_SAMPLED, 9, 37), (kv.NBHD_SAMPLED, 3, 1)):
        ev = _OracleEvaluator(s, o, M, start)
        tel, done, trace = par.sharded_local_search(ev, nbhd, iters, seed=11, samples_per_iter=samples,
                                                    comm=par.TorchComm(device="cpu"))
        r_order, r_tel, r_done, r_trace = orc.local_search(s, o, M, nbhd, iters, start, seed=11, samples=samples)
        ok &= tel == r_tel and done == r_done and (trace == r_trace).all() and (ev.order == r_order).all()
        total = par.neighbourhood_size(n, nbhd, samples)
        ok &= all(fc == par.shard(total, rank, world) for fc in ev.sweeps) or total < world
    # the step the benchmark times under torchrun: one iteration over a sampled neighbourhood split
    # over the ranks, exchange included; both ranks must end with the oracle's pair and order
    for samples, it in ((64, 0), (5, 1), (1, 2)):
        ev = _OracleEvaluator(s, o, M, start)
        accepted, cur, idx, tel = par.sharded_iteration(ev, par.TorchComm(device="cpu"), samples, True, 23, it)
        mv = [orc.sample_move(n, 23, it, m) for m in range(samples)]
        ref = orc.eval_moves(s, o, M, start, [m[0] for m in mv], [m[1] for m in mv], [m[2] for m in mv])
        k = int(np.argmin(ref))
        base_tel = orc.list_schedule_rounds(s, o, M, start)[1]
        ok &= (idx, tel) == (k, int(ref[k])) and accepted == (int(ref[k]) < base_tel)
        want = orc.apply_move(start, *mv[k]) if accepted else start
        ok &= (ev.order == want).all() and cur == min(base_tel, int(ref[k]))
    # shares: contiguous, disjoint, complete, also when there are fewer indices than ranks
    for total in (0, 1, 2, 7, 1000, 149985000):
        parts = [par.shard(total, r, 8) for r in range(8)]
        ok &= parts[0][0] == 0 and sum(c for _, c in parts) == total
        ok &= all(parts[k][0] + parts[k][1] == parts[k + 1][0] for k in range(7))
        ok &= max(c for _, c in parts) - min(c for _, c in parts) <= 1
    out[rank] = bool(ok)
    dist.destroy_process_group()


def test_two_ranks_run_one_local_search():
    world = 2
    port = 31500 + (os.getpid() % 2000)
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_search_worker, args=(world, port, out), nprocs=world, join=True)
        assert dict(out) == {0: True, 1: True}
