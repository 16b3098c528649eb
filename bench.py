#!/usr/bin/env python
"""Throughput of batched schedule evaluation (headline backlog: n = 10,000, M = 262,144).

One step = one pass of the whole path on one batch: Sorted-F order construction (segmented radix
sort, F-metric batch selection, per-batch sort, base run with snapshots) followed by one sweep of
`--moves` sampled swap/insert moves (move generation fused into the simulator) and the arg-min
reduction.  `value` counts simulated candidate schedules per second with everything resident on
the device; `e2e` repeats the measurement through the host-pointer C-ABI calls, creating the
handle from host arrays and copying candidates in and TELs out inside the timed region.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--moves C] [--impl ours|reference]
                    [--workload mixed_10k|mixed_1k|paper_scale|heavy_100k|policy_sweep]

Under torchrun the `--moves` sampled moves of a step are ONE neighbourhood split over the ranks
(strong scaling): every rank rebuilds the Sorted-F order, sweeps its contiguous share, the ranks
agree on the best (TEL, index) pair with two all-reduce(min) of one int64 over NCCL, and every rank
applies that move to its base order.  Time is the max over ranks.

The roofline denominators are measured inside this run by the library's probe kernels
(`sched_probe_peaks`): `roofline.frac` is read against the measured rate of the integer ALU pipe (the
pipe every maximum, compare and select of the simulator has to go through); `roofline.frac_vs` gives
the same achieved figure against the other measured rates -- plain adds, which the compiler spreads
over two pipes, multiply-adds, a two-pipe mix -- and the instruction-issue limit.
"""
from __future__ import annotations

import argparse
import ctypes as C
import json
import os
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2508_06133_b200 import workloads as W  # noqa: E402

SM_COUNT = 148
INT_OPS_PER_CLK_PER_SM = 64              # fallback only: 32-bit integer adds per clock and SM when the probe cannot run
ISSUE_LANES_PER_CLK_PER_SM = 128         # 4 schedulers x 1 warp instruction (32 lanes) per clock
FALLBACK_HBM_GBS, FALLBACK_SM_MHZ = 6650.0, 1965.0
OPS_PER_CELL, BYTES_PER_CELL = 4.0, 8.0  # algorithmic cost of one timeline cell: 4 integer operations, 4 B read + 4 B written
# dram__bytes_read.sum + dram__bytes_write.sum of one simulator launch, from a one-pass ncu capture of
# this very launch (summary under profiles/); keyed by (workload, moves per launch) with a digest of
# the simulator's source files, so that it turns into null when the kernel changes
K3_TRAFFIC = {("mixed_n10000", 1 << 22): (61.21e6 + 10.59e6, "1e184f7ce88dd053")}
DEFAULT_MOVES = {"mixed_10k": 1 << 22, "mixed_1k": 499500, "paper_scale": 1 << 21, "heavy_100k": 1 << 18}


def simulator_digest() -> str:
    """Digest of the sources of the timed kernel (simulator + move evaluator)."""
    import hashlib
    hsh = hashlib.sha256()
    for name in ("sim_reg.cuh", "sim_hyb.cuh", "k3_eval.cuh", "k4_moves.cuh", "common.cuh"):
        with open(os.path.join(ROOT, "paper_2508_06133_b200", "csrc", name), "rb") as f:
            hsh.update(f.read())
    return hsh.hexdigest()[:16]


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p.get("hbm_gbs", FALLBACK_HBM_GBS)), float(p.get("sm_max_mhz", FALLBACK_SM_MHZ)), "measured"
    return FALLBACK_HBM_GBS, FALLBACK_SM_MHZ, "fallback"


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu, self.proc, self.path = gpu_index, None, "/tmp/kvsched_clocks_%d.csv" % os.getpid()

    def start(self):
        try:
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        sm, smax, reasons = [], [], set()
        for line in open(self.path):
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                smax.append(float(parts[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if sm:
            out["sm_mhz"] = float(np.median(sm))
            out["sm_max_mhz"] = float(max(smax))
            out["reasons"] = sorted(reasons)
        try:
            os.remove(self.path)
        except OSError:
            pass
        return out


def sampled_move_positions(n, seed, iteration, first, count):
    """(type, i, j) of the library's sampled moves, recomputed on the host for the work accounting
    and the CPU-baseline sample (same published splitmix64 construction as the header states)."""
    m = np.arange(first, first + count, dtype=np.uint64)
    with np.errstate(over="ignore"):
        def vmix(z):
            z = z + np.uint64(0x9E3779B97F4A7C15)
            z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
            z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
            return z ^ (z >> np.uint64(31))
        h1 = vmix(np.uint64(seed) ^ vmix((np.uint64(iteration) << np.uint64(32)) + m))
        h2 = vmix(h1)
    i = ((h1 >> np.uint64(1)) % np.uint64(n)).astype(np.int64)
    j = ((i.astype(np.uint64) + np.uint64(1) + h2 % np.uint64(n - 1)) % np.uint64(n)).astype(np.int64)
    return (h1 & np.uint64(1)).astype(np.int64), i, j


def rank_share(total: int, rank: int, world: int):
    """(first sample index, count) of `rank`'s contiguous share of one step's neighbourhood."""
    from paper_2508_06133_b200 import parallel as par
    return par.shard(total, rank, world)


def max_over_ranks(value: float, dist, device) -> float:
    """Slowest rank's figure (the time that counts for a job spread over ranks)."""
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def host_cores() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return max(1, os.cpu_count() or 1)


def run_reference(args, inst, rank):
    """The CPU oracle as it stands, timed on this machine's host cores on a bounded sample per step."""
    if rank != 0:
        return
    import oracle as orc
    cores = host_cores()
    base, _ = orc.sorted_f_prefix(inst.s, inst.o, inst.M)
    per_step = args.ref_moves if args.ref_moves > 0 else 16 * cores
    total = inst.n * (inst.n - 1) // 2 + inst.n * (inst.n - 1)

    def step(k):
        codes = (W.u64(1000 + k, 0, np.arange(per_step)) % np.uint64(total)).astype(np.int64)
        mv = [orc.decode_move(inst.n, int(c)) for c in codes]
        orc.sorted_f_prefix(inst.s, inst.o, inst.M)
        return orc.eval_moves_threads(inst.s, inst.o, inst.M, base, [m[0] for m in mv], [m[1] for m in mv],
                                      [m[2] for m in mv], threads=cores)
    for k in range(args.warmup):
        step(k)
    t0 = time.perf_counter()
    for k in range(args.steps):
        step(args.warmup + k)
    dt = time.perf_counter() - t0
    value = per_step * args.steps / dt
    sample = ("%d sampled swap/insert moves per step, oracle/oracle.cpp orc_eval_moves_threads (per-round form of "
              "Algorithm 1 Phase 2), candidates split over %d threads" % (per_step, cores))
    print(json.dumps({
        "impl": "reference", "metric": "schedule_evals_per_sec", "value": value, "unit": "evals/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
        "config": {"workload": inst.name, "n": inst.n, "M": inst.M, "sum_o": int(inst.o.sum()), "moves_per_step": per_step},
        "request_rounds_per_sec": value * float(inst.o.sum()),
        "cpu_baseline": {"value": value, "unit": "evals/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "evals/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def probe_rooflines(kv, stream, sm_mhz):
    """Measured peak rates (lane operations / bytes per second) from the library's probe kernels."""
    try:
        p = kv.probe_peaks(repeats=5, stream=stream)
        source = "measured in this run: sched_probe_peaks"
    except Exception as e:                                    # the probe is support code: fall back, say so
        p = {"int_add": SM_COUNT * INT_OPS_PER_CLK_PER_SM * sm_mhz * 1e6}
        source = "derived (probe failed: %s): %d SMs x %d int ops/clk/SM x sm_max_mhz" % (e, SM_COUNT, INT_OPS_PER_CLK_PER_SM)
    return p, source


def roofline_block(cells_per_launch, kern_s, probe, probe_source, sm_mhz_load, hbm_gbs, hbm_bytes, traffic, kernel, extra_ops=0.0):
    """`achieved` = algorithmic integer operations per launch / measured launch time, against the
    measured integer-add rate; the other measured rates and the issue limit beside it."""
    ops = OPS_PER_CELL * cells_per_launch + extra_ops
    ach = ops / kern_s                                           # integer operations per second
    # the pipe that bounds the simulator: maxima, compares, selects and masks execute only on the
    # integer ALU pipe (measured by the max/xor probe); plain adds alone can also use the
    # multiply-add pipe, which is what the int_add probe shows -- both fractions are reported
    peak_key = "int_alu" if probe.get("int_alu", 0) > 0 else "int_add"
    peak = probe[peak_key]
    frac_vs = {k: ach / v for k, v in probe.items() if k.startswith(("int_", "sim_")) and v > 0}
    issue_peak = SM_COUNT * ISSUE_LANES_PER_CLK_PER_SM * sm_mhz_load * 1e6
    frac_vs["issue_slots"] = ach / issue_peak
    rl = {"bound": "alu", "achieved": ach / 1e12, "peak": peak / 1e12, "unit": "Tint-op/s", "frac": ach / peak,
          "traffic": traffic, "kernel": kernel, "kernel_ms": kern_s * 1e3, "cells_per_launch": cells_per_launch,
          "ops_per_cell": OPS_PER_CELL,
          "peak_source": probe_source + (" int_alu: measured rate of the integer ALU pipe (max/xor chains, lane-ops/s); frac_vs.int_add is the same "
                                         "achieved figure against plain adds, which the compiler spreads over the ALU and the multiply-add pipe"
                                         if peak_key == "int_alu" else " int_add (lane-ops/s)"),
          "frac_vs": frac_vs,
          "probe_lane_ops_per_clk_per_sm": {k: v / (SM_COUNT * sm_mhz_load * 1e6) for k, v in probe.items()},
          "issue_peak_note": "derived: %d SMs x %d lanes/clk x %.0f MHz sampled under load" % (SM_COUNT, ISSUE_LANES_PER_CLK_PER_SM, sm_mhz_load),
          "hbm_bytes_per_launch": hbm_bytes, "hbm_frac": hbm_bytes / kern_s / 1e9 / hbm_gbs}
    if "smem_load" in probe and probe["smem_load"] > 0:
        smem_ach = BYTES_PER_CELL * cells_per_launch / kern_s
        smem_peak = 0.5 * (probe["smem_load"] + probe.get("smem_store", probe["smem_load"]))
        rl["smem"] = {"bound": "smem", "achieved": smem_ach / 1e9, "peak": smem_peak / 1e9, "unit": "GB/s",
                      "frac": smem_ach / smem_peak, "note": "4 B read + 4 B written per cell against the mean of the measured 16-byte load and store rates"}
    return rl


def cpu_baseline_legs(args, inst, base, ty, mi, mj, tel_check):
    """The oracle on a bounded sample of the step's own moves: per-round form on one thread and on all
    cores, and Algorithm 1 Phase 2 as listed (completion-time set tests) on a few candidates."""
    import oracle as orc
    cores = host_cores()
    budget = max(args.cpu_seconds, 0.5) / 3.0
    t0 = time.perf_counter()
    orc.eval_moves(inst.s, inst.o, inst.M, base, ty[:4], mi[:4], mj[:4])
    pilot = (time.perf_counter() - t0) / 4
    k1 = int(max(4, min(len(ty), budget / max(pilot, 1e-6))))
    t0 = time.perf_counter()
    ref1 = orc.eval_moves_threads(inst.s, inst.o, inst.M, base, ty[:k1], mi[:k1], mj[:k1], threads=1)
    dt1 = time.perf_counter() - t0
    kc = int(max(cores, min(len(ty), cores * budget / max(pilot, 1e-6))))
    t0 = time.perf_counter()
    refc = orc.eval_moves_threads(inst.s, inst.o, inst.M, base, ty[:kc], mi[:kc], mj[:kc], threads=cores)
    dtc = time.perf_counter() - t0
    assert (tel_check[:k1] == ref1).all() and (tel_check[:kc] == refc).all(), "GPU and oracle TELs differ on the CPU-baseline sample"
    out = {"value": kc / dtc, "unit": "evals/s", "cores": cores, "kind": "oracle",
           "sample": "first %d sampled moves of one step, oracle/oracle.cpp per-round form of Algorithm 1 Phase 2, candidates "
                     "split over %d threads; TELs equal the GPU's" % (kc, cores),
           "single_thread": {"value": k1 / dt1, "cores": 1, "sample": "first %d sampled moves, same routine, 1 thread" % k1}}
    if args.cpu_literal:
        kl = cores if inst.n <= 20000 else 0
        if kl:
            t0 = time.perf_counter()
            refl = orc.eval_moves_threads(inst.s, inst.o, inst.M, base, ty[:kl], mi[:kl], mj[:kl], threads=cores, literal=True)
            dtl = time.perf_counter() - t0
            assert (tel_check[:kl] == refl).all(), "GPU and the literal Algorithm 1 executor differ"
            out["literal_alg1"] = {"value": kl / dtl, "cores": cores, "per_thread_value": kl / dtl / cores,
                                   "sample": "first %d sampled moves, Algorithm 1 Phase 2 as listed (set tests at completion times), "
                                             "one candidate per thread; TELs equal the GPU's" % kl}
    return out


def bench_policy_sweep(args, rank, world, local_rank):
    """Configuration 3: 4,096 instances x 256 requests x 4 policies, one launch per step."""
    import torch
    from paper_2508_06133_b200 import binding as kv
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    s, o, M = W.policy_sweep()
    B, n = s.shape
    pols = torch.tensor([kv.POLICY_SORTED_F, kv.POLICY_FCFS, kv.POLICY_SOF, kv.POLICY_TOTAL_SIZE], dtype=torch.int32, device=dev)
    tel = torch.empty(B * 4, dtype=torch.int64, device=dev)
    stream = torch.cuda.Stream()
    h = kv.Scheduler.batch(s, o, M)
    h.set_stream(stream)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def step():
        flush.zero_()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        h.eval_batch_dev(kv.CAND_POLICY, 4, pols, tel)
        e1.record(stream)
        e1.synchronize()
        return e0.elapsed_time(e1), h.last_eval_kernel_ms()
    for _ in range(args.warmup):
        step()
    hbm_gbs, sm_max, _ = measured_peaks()
    probe, probe_source = probe_rooflines(kv, stream, sm_max)
    launches0, _ = h.stats()
    sampler = ClockSampler(local_rank)
    sampler.start()
    res = [step() for _ in range(args.steps)]
    torch.cuda.synchronize()
    time.sleep(0.3)
    clocks = sampler.stop()
    launches1, _ = h.stats()
    step_ms = [r[0] for r in res]
    kern_s = float(np.mean([r[1] for r in res])) * 1e-3
    pairs = B * 4
    value = pairs * args.steps / (sum(step_ms) * 1e-3)
    cells = 4.0 * float(o.astype(np.int64).sum())                   # every pair simulates its whole list
    # order construction: stable radix passes in shared memory (2 for shortest-decode-first, 2 for total-size-first,
    # 5 for Sorted-F at these sizes), each a count and a scatter visit of n ids, ~3 integer operations per visit
    sort_ops = 6.0 * B * 9 * n
    sm_load = clocks["sm_mhz"] or sm_max
    roofline = roofline_block(cells, kern_s, probe, probe_source, sm_load, hbm_gbs, 8.0 * B * n + 8.0 * pairs, None,
                              "k3_eval_policy", extra_ops=sort_ops)
    roofline["extra_ops_note"] = "order construction: 9 radix passes per instance x 2 visits x n ids x 3 integer operations"
    import oracle as orc
    got = tel.cpu().numpy().reshape(B, 4)
    cores = host_cores()
    t0 = time.perf_counter()
    nb = 0
    for b in range(0, B, max(1, B // 64)):
        refs = [orc.sorted_f_prefix(s[b], o[b], M)[0], orc.policy_order(s[b], o[b], orc.FCFS),
                orc.policy_order(s[b], o[b], orc.SHORTEST_OUTPUT_FIRST), orc.policy_order(s[b], o[b], orc.TOTAL_SIZE_FIRST)]
        assert got[b].tolist() == [orc.list_schedule_rounds(s[b], o[b], M, r)[1] for r in refs]
        nb += 4
    dt = time.perf_counter() - t0
    cpu = {"value": nb / dt, "unit": "evals/s", "cores": 1, "kind": "oracle",
           "sample": "%d of the %d instance-policy pairs, order construction + per-round executor, 1 thread (of %d cores); TELs equal the GPU's" % (nb, pairs, cores)}
    out = {"metric": "schedule_evals_per_sec", "value": value, "unit": "evals/s", "n_gpus": 1, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": float(np.mean(step_ms)), "ms_per_step_median": float(np.median(step_ms)),
           "ms_per_step_best": float(np.min(step_ms)), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
           "dtype": "int32", "data": "synthetic",
           "config": {"workload": "policy_sweep_4096x256x4", "instances": B, "n": n, "M": M, "policies": 4,
                      "l2": "flushed between steps (256 MiB write)"},
           "request_rounds_per_sec": value * float(o.sum()) / B,
           "roofline": roofline, "cpu_baseline": cpu, "e2e": None,
           "gpu_launches": int(launches1 - launches0), "clocks": clocks}
    print(json.dumps(out))
    h.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--moves", type=int, default=0, help="sampled moves of one step's neighbourhood (all ranks together); 0: the workload's default")
    ap.add_argument("--ref-moves", type=int, default=0, help="moves per step of the CPU reference arm (0: 16 per host core)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="mixed_10k", choices=["mixed_10k", "mixed_1k", "paper_scale", "heavy_100k", "policy_sweep"])
    ap.add_argument("--cpu-seconds", type=float, default=24.0, help="budget of the cpu_baseline legs (0: skip them)")
    ap.add_argument("--no-cpu-literal", dest="cpu_literal", action="store_false", help="skip the literal Algorithm 1 leg of the CPU baseline")
    ap.add_argument("--e2e-steps", type=int, default=3)
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.workload == "policy_sweep":
        if args.impl == "reference":
            if rank == 0:
                print(json.dumps({"impl": "reference", "unavailable": "the reference arm times the sweep workloads only"}))
            return
        if rank == 0:
            bench_policy_sweep(args, rank, world, local_rank)
        return
    inst = getattr(W, args.workload)()
    if args.impl == "reference":
        run_reference(args, inst, rank)
        return

    import torch
    import torch.distributed as dist
    from paper_2508_06133_b200 import binding as kv, parallel as par

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    # under torchrun (RANK set) the process group is used even with one rank, so that the very same
    # barrier / exchange / max-over-ranks path runs at every N
    multi = "RANK" in os.environ and "MASTER_ADDR" in os.environ
    if multi:
        dist.init_process_group("nccl", device_id=dev)

    n, sum_o = inst.n, int(inst.o.sum())
    total_moves = args.moves if args.moves > 0 else DEFAULT_MOVES[args.workload]
    first, count = rank_share(total_moves, rank, world)
    seed = 20250806
    stream = torch.cuda.Stream()
    h = kv.Scheduler(inst.s, inst.o, inst.M)
    h.set_stream(stream)
    best = torch.zeros(2, dtype=torch.int64, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)       # > 126 MB of L2
    evaluator = par.GpuEvaluator(h, device=dev) if multi else None
    comm = par.TorchComm(device=dev) if multi else None

    def step(k):
        """Whole path, device-resident; returns (step ms, simulator-kernel ms)."""
        flush.zero_()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        h.sorted_f_dev()
        if multi:
            # this rank's share of the neighbourhood, the 16-byte exchange, the same move on every rank
            par.sharded_iteration(evaluator, comm, total_moves, True, seed, k)
            kms = h.last_eval_kernel_ms()
        else:
            h.sweep_dev(count, best, sampled=True, seed=seed, iteration=k, first_code=first)
            kms = None
        e1.record(stream)
        e1.synchronize()
        return e0.elapsed_time(e1), (kms if kms is not None else h.last_eval_kernel_ms())

    for k in range(args.warmup):
        step(k)
    h.sync()
    hbm_gbs, sm_max, peak_kind = measured_peaks()
    probe, probe_source = probe_rooflines(kv, stream, sm_max)
    launches0, _ = h.stats()
    sampler = ClockSampler(local_rank)
    if multi:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    step_ms, kern_ms = [], []
    for k in range(args.steps):
        a, b = step(args.warmup + k)
        step_ms.append(a)
        kern_ms.append(b)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    if multi:
        dist.barrier()
    h.sync()
    launches1, _ = h.stats()
    total_ms = float(sum(step_ms))
    if multi:
        total_ms = max_over_ranks(total_ms, dist, dev)
    value = total_moves * args.steps / (total_ms * 1e-3)

    # ---- algorithmic work of the simulator launches: timeline cells that must be updated, i.e.
    #      the sum of o over the list positions from the first moved one to the end
    h.sorted_f_dev()
    h.sync()
    order = h.get_base_order()
    suffix_o = np.concatenate([np.cumsum(inst.o[order][::-1].astype(np.int64))[::-1], [0]])
    cells = []
    for k in range(args.steps):
        _, mi, mj = sampled_move_positions(n, seed, args.warmup + k, first, count)
        cells.append(int(suffix_o[np.minimum(mi, mj)].sum()))
    cells_per_launch = float(np.mean(cells))
    kern_s = float(np.mean(kern_ms)) * 1e-3
    state_cells = 32 * ((31 + int(inst.o.max()) + 31) // 32)
    hbm_bytes = 4.0 * n * state_cells + 8.0 * count + 4.0 * count + 8.0 * n   # snapshots read once, TELs out, launch order in, request table
    traffic = None
    known = K3_TRAFFIC.get((inst.name, count))
    if known is not None and known[1] == simulator_digest():
        traffic = known[0]
    sm_load = clocks["sm_mhz"] or sm_max
    roofline = roofline_block(cells_per_launch, kern_s, probe, probe_source, sm_load, hbm_gbs, hbm_bytes, traffic, "k3_eval_moves")
    # the survey's model-level figure: every evaluation counted as 4 * sum(o) operations, i.e. including the
    # list prefix that the snapshots of the base run make unnecessary -- a statement about the method, not
    # about how busy the SM is (that is `frac`, which counts only the cells actually re-simulated)
    roofline["model_level"] = {"ops_per_eval": OPS_PER_CELL * sum_o, "tera_ops_per_s": OPS_PER_CELL * sum_o * count / kern_s / 1e12,
                               "of_peak": OPS_PER_CELL * sum_o * count / kern_s / (roofline["peak"] * 1e12),
                               "note": "evals/s x 4 x sum(o) / peak; counts the prefix that snapshot reuse skips (cells re-simulated are %.0f %% of it)"
                                       % (100.0 * cells_per_launch / (float(sum_o) * count))}
    roofline["kernel_ms_median"] = float(np.median(kern_ms))
    roofline["kernel_ms_best"] = float(np.min(kern_ms))

    # ---- end to end through the host-pointer entry points (handle created from host arrays,
    #      candidates copied in, TELs copied out, all inside the timed region)
    total_codes = n * (n - 1) // 2 + n * (n - 1)
    s_pin = torch.from_numpy(inst.s.copy()).pin_memory()
    o_pin = torch.from_numpy(inst.o.copy()).pin_memory()
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    codes_pin = [torch.from_numpy((W.u64(seed + 1 + k + 100 * rank, 0, np.arange(count)) % np.uint64(total_codes)).astype(np.int64)).pin_memory()
                 for k in range(e2e_steps + 1)]
    tel_pin = torch.empty(count, dtype=torch.int64).pin_memory()

    def e2e_step(k):
        lib = kv.load()
        hh = kv.Scheduler(s_pin.numpy(), o_pin.numpy(), inst.M)
        hh.sorted_f()
        rc = lib.sched_eval_batch(hh._h, kv.CAND_MOVE, count, C.c_void_p(codes_pin[k].data_ptr()),
                                  C.c_void_p(tel_pin.data_ptr()), None, None)
        assert rc == 0, rc
        res = int(tel_pin.numpy().min())
        hh.close()
        return res
    e2e_step(e2e_steps)
    if multi:
        dist.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for k in range(e2e_steps):
        e2e_step(k)
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    if multi:
        dt = max_over_ranks(dt, dist, dev)
    e2e = {"value": world * count * e2e_steps / dt, "unit": "evals/s",
           "h2d_bytes_per_step": int(8 * n + 8 * count), "d2h_bytes_per_step": int(8 * count + 4 * n + 8),
           "steps": e2e_steps}

    # ---- CPU baseline: the oracle on a bounded sample of the same workload (rank 0, N = 1 only)
    cpu = None
    if rank == 0 and world == 1 and args.cpu_seconds > 0:
        import oracle as orc
        base, _ = orc.sorted_f_prefix(inst.s, inst.o, inst.M)
        assert (base == order).all(), "GPU and oracle disagree on the Sorted-F order"
        ty, mi, mj = sampled_move_positions(n, seed, args.warmup, 0, min(count, 1 << 14))
        swap = (ty == 0) & (mi > mj)
        mi2, mj2 = np.where(swap, mj, mi), np.where(swap, mi, mj)
        tel_dev = torch.empty(count, dtype=torch.int64, device=dev)
        h.sweep_dev(count, best, sampled=True, seed=seed, iteration=args.warmup, first_code=0, tel_out=tel_dev)
        h.sync()
        cpu = cpu_baseline_legs(args, inst, base, ty, mi2, mj2, tel_dev[:len(ty)].cpu().numpy())

    if rank == 0:
        out = {
            "metric": "schedule_evals_per_sec", "value": value, "unit": "evals/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_ms / args.steps,
            "ms_per_step_median": float(np.median(step_ms)), "ms_per_step_best": float(np.min(step_ms)),
            "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
            "config": {"workload": inst.name, "n": n, "M": inst.M, "sum_o": sum_o, "moves_per_step": total_moves,
                       "moves_per_step_per_gpu": count,
                       "neighbourhood": "sampled swap+insert moves of the Sorted-F order" +
                                        (", one neighbourhood split over the ranks, all-reduce(min) exchange and accepted move per step" if multi else ""),
                       "l2": "flushed between steps (256 MiB write)", "checksum": "%016x" % inst.checksum()},
            "request_rounds_per_sec": value * sum_o,
            "best_tel_last_step": int(best[0].item()) if not multi else int(evaluator.best[0].item()),
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e,
            "gpu_launches": int(launches1 - launches0), "clocks": clocks,
        }
        print(json.dumps(out))
    h.close()
    if multi:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
