"""CPU-side checks of the benchmark's support code: the reference arm prints one well-formed JSON line,
and the threaded form of the oracle's move evaluation (used only for the CPU-baseline timing) returns
exactly what the single-threaded routines return."""
import json
import os
import subprocess
import sys

import numpy as np

import oracle as orc
from paper_2508_06133_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_threaded_move_evaluation_equals_the_plain_one():
    inst = W.mixed_backlog(300, 11, 20000, name="threads")
    base, _ = orc.sorted_f_prefix(inst.s, inst.o, inst.M)
    n = inst.n
    total = n * (n - 1) // 2 + n * (n - 1)
    codes = (W.u64(9, 0, np.arange(97)) % np.uint64(total)).astype(np.int64)
    mv = [orc.decode_move(n, int(c)) for c in codes]
    ty, mi, mj = [m[0] for m in mv], [m[1] for m in mv], [m[2] for m in mv]
    ref = orc.eval_moves(inst.s, inst.o, inst.M, base, ty, mi, mj)
    for threads in (1, 2, 5, 200):
        assert (orc.eval_moves_threads(inst.s, inst.o, inst.M, base, ty, mi, mj, threads=threads) == ref).all()
    # Algorithm 1 Phase 2 as listed, on the moved orders one by one
    lit = orc.eval_moves_threads(inst.s, inst.o, inst.M, base, ty[:12], mi[:12], mj[:12], threads=3, literal=True)
    for k in range(12):
        cand = orc.apply_move(base, ty[k], mi[k], mj[k])
        assert lit[k] == orc.list_schedule_alg1(inst.s, inst.o, inst.M, cand)[1] == ref[k]


def test_reference_arm_prints_one_json_line():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "mixed_1k",
                        "--steps", "2", "--warmup", "1", "--ref-moves", "6"], capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "schedule_evals_per_sec" and d["unit"] == "evals/s"
    assert d["value"] > 0 and d["steps"] == 2 and d["warmup"] == 1 and d["higher_is_better"] is True
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1 and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": "evals/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["config"]["workload"] == "mixed_n1000" and d["config"]["moves_per_step"] == 6


def test_rank_shares_cover_a_step_exactly():
    import bench
    for total in (1, 7, 1 << 22):
        for world in (1, 2, 3, 8):
            parts = [bench.rank_share(total, r, world) for r in range(world)]
            assert parts[0][0] == 0 and sum(c for _, c in parts) == total
            assert all(parts[k][0] + parts[k][1] == parts[k + 1][0] for k in range(world - 1))
