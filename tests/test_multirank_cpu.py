"""World-size-2 check (gloo, CPU) of how the benchmark spreads one sampled neighbourhood over ranks:
disjoint contiguous sample slices, the same moves as a single rank would draw, and the
max-over-ranks time reduction.  No GPU and no kernel is involved."""
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
    first = bench.rank_first_sample(rank, count)
    ty, mi, mj = bench.sampled_move_positions(n, seed, it, first, count)
    mine = torch.from_numpy(np.stack([ty, mi, mj]))
    gathered = [torch.zeros_like(mine) for _ in range(world)]
    dist.all_gather(gathered, mine)
    whole = np.stack(bench.sampled_move_positions(n, seed, it, 0, world * count))
    ok = bool((torch.cat(gathered, dim=1).numpy() == whole).all())
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
