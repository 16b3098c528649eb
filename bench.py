#!/usr/bin/env python
"""Throughput of batched schedule evaluation on the headline backlog (n = 10,000, M = 262,144).

One step = one pass of the whole path on one batch: Sorted-F order construction (segmented radix
sort, F-metric batch selection, per-batch sort, base run with snapshots) followed by one sweep of
`--moves` sampled swap/insert moves (move generation fused into the simulator) and the arg-min
reduction.  `value` counts simulated candidate schedules per second with everything resident on
the device; `e2e` repeats the measurement through the host-pointer C-ABI calls, creating the
handle from host arrays and copying candidates in and TELs out inside the timed region.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--moves C] [--impl ours|reference]

Under torchrun every rank evaluates its own slice of the sampled neighbourhood of the same backlog
(no data-path collective); time is the max over ranks, value the sum of evaluations over ranks.
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
SMEM_BYTES_PER_CLK_PER_SM = 128          # shared-memory bandwidth of one SM (probe: 126.6 with 16-byte loads)
INT_OPS_PER_CLK_PER_SM = 64              # 32-bit integer adds per clock and SM (probe: 63.7)
FALLBACK_HBM_GBS, FALLBACK_SM_MHZ = 6650.0, 1965.0
# dram__bytes_read.sum + dram__bytes_write.sum of one simulator launch, from a one-pass ncu capture of
# this very launch (summary under profiles/); keyed by (workload, moves per
# launch, simulator source files' digest) so that it turns into null when the kernel changes
K3_TRAFFIC = {("mixed_n10000", 1 << 22): (60.61e6 + 11.38e6, "21db94945fc6e5e0")}


def simulator_digest() -> str:
    """Digest of the sources of the timed kernel (simulator + move evaluator)."""
    import hashlib
    hsh = hashlib.sha256()
    for name in ("sim_reg.cuh", "k3_eval.cuh", "k4_moves.cuh", "common.cuh"):
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


def rank_first_sample(rank: int, count: int) -> int:
    """Ranks evaluate disjoint, contiguous slices of one sampled neighbourhood: rank r takes the
    sample indices [r * count, (r + 1) * count)."""
    return rank * count


def max_over_ranks(value: float, dist, device) -> float:
    """Slowest rank's figure (the time that counts for a job spread over ranks)."""
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def run_reference(args, inst, rank):
    """The CPU oracle as it stands, timed on this machine's host cores on a bounded sample per step."""
    if rank != 0:
        return
    import oracle as orc
    base, _ = orc.sorted_f_prefix(inst.s, inst.o, inst.M)
    per_step = args.ref_moves
    total = inst.n * (inst.n - 1) // 2 + inst.n * (inst.n - 1)

    def step(k):
        codes = (W.u64(1000 + k, 0, np.arange(per_step)) % np.uint64(total)).astype(np.int64)
        mv = [orc.decode_move(inst.n, int(c)) for c in codes]
        orc.sorted_f_prefix(inst.s, inst.o, inst.M)
        return orc.eval_moves(inst.s, inst.o, inst.M, base, [m[0] for m in mv], [m[1] for m in mv], [m[2] for m in mv])
    for k in range(args.warmup):
        step(k)
    t0 = time.perf_counter()
    for k in range(args.steps):
        step(args.warmup + k)
    dt = time.perf_counter() - t0
    value = per_step * args.steps / dt
    sample = "%d sampled swap/insert moves per step, single thread, oracle/oracle.cpp orc_eval_moves" % per_step
    print(json.dumps({
        "impl": "reference", "metric": "schedule_evals_per_sec", "value": value, "unit": "evals/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
        "config": {"workload": inst.name, "n": inst.n, "M": inst.M, "sum_o": int(inst.o.sum()), "moves_per_step": per_step},
        "request_rounds_per_sec": value * float(inst.o.sum()),
        "cpu_baseline": {"value": value, "unit": "evals/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "evals/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--moves", type=int, default=1 << 22, help="sampled moves evaluated per step and GPU")
    ap.add_argument("--ref-moves", type=int, default=96, help="moves per step of the CPU reference arm")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="mixed_10k", choices=["mixed_10k", "mixed_1k", "paper_scale", "heavy_100k"])
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="budget of the cpu_baseline leg")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    inst = getattr(W, args.workload)()
    if args.impl == "reference":
        run_reference(args, inst, rank)
        return

    import torch
    import torch.distributed as dist
    from paper_2508_06133_b200 import binding as kv

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    # under torchrun (RANK set) the process group is used even with one rank, so that the very same
    # barrier / max-over-ranks path runs at every N
    multi = "RANK" in os.environ and "MASTER_ADDR" in os.environ
    if multi:
        dist.init_process_group("nccl", device_id=dev)

    n, sum_o = inst.n, int(inst.o.sum())
    count = args.moves
    seed = 20250806
    stream = torch.cuda.Stream()
    h = kv.Scheduler(inst.s, inst.o, inst.M)
    h.set_stream(stream)
    best = torch.zeros(2, dtype=torch.int64, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)       # > 126 MB of L2

    def step(k):
        """Whole path, device-resident; returns (step ms, simulator-kernel ms)."""
        flush.zero_()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        h.sorted_f_dev()
        h.sweep_dev(count, best, sampled=True, seed=seed, iteration=k, first_code=rank_first_sample(rank, count))
        e1.record(stream)
        e1.synchronize()
        return e0.elapsed_time(e1), h.last_eval_kernel_ms()

    for k in range(args.warmup):
        step(k)
    h.sync()
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
    value = world * count * args.steps / (total_ms * 1e-3)

    # ---- algorithmic work of the simulator launches: timeline cells that must be updated, i.e.
    #      the sum of o over the list positions from the first moved one to the end
    order = h.get_base_order()
    suffix_o = np.concatenate([np.cumsum(inst.o[order][::-1].astype(np.int64))[::-1], [0]])
    cells = []
    for k in range(args.steps):
        _, mi, mj = sampled_move_positions(n, seed, args.warmup + k, rank_first_sample(rank, count), count)
        cells.append(int(suffix_o[np.minimum(mi, mj)].sum()))
    cells_per_launch = float(np.mean(cells))
    kern_s = float(np.mean(kern_ms)) * 1e-3
    hbm_gbs, sm_mhz, peak_kind = measured_peaks()
    smem_peak = SM_COUNT * SMEM_BYTES_PER_CLK_PER_SM * sm_mhz * 1e6 / 1e9          # GB/s
    alu_peak = SM_COUNT * INT_OPS_PER_CLK_PER_SM * sm_mhz * 1e6 / 1e12             # Tint-op/s
    smem_ach = 8.0 * cells_per_launch / kern_s / 1e9                               # read + write 4 B per cell
    alu_ach = 4.0 * cells_per_launch / kern_s / 1e12                               # 4 integer ops per cell
    roof_smem = {"bound": "smem", "achieved": smem_ach, "peak": smem_peak, "unit": "GB/s", "frac": smem_ach / smem_peak}
    roof_alu = {"bound": "alu", "achieved": alu_ach, "peak": alu_peak, "unit": "Tint-op/s", "frac": alu_ach / alu_peak}
    roofline = dict(roof_alu)
    ring_cells = (int(inst.o.max()) + 8 + 31) & ~31
    hbm_bytes = 4.0 * n * ring_cells + 8.0 * count + 4.0 * count + 8.0 * n   # snapshots read once, TELs out, launch order in, request table
    traffic = None
    known = K3_TRAFFIC.get((inst.name, count))
    if known is not None and known[1] == simulator_digest():
        traffic = known[0]
    roofline.update({"traffic": traffic, "kernel": "k3_eval_moves", "kernel_ms": kern_s * 1e3,
                     "cells_per_launch": cells_per_launch,
                     "peak_source": "derived: %d SMs x %d int ops/clk/SM x %s sm_max_mhz" % (SM_COUNT, INT_OPS_PER_CLK_PER_SM, peak_kind),
                     "hbm_bytes_per_launch": hbm_bytes, "hbm_frac": hbm_bytes / kern_s / 1e9 / hbm_gbs,
                     "smem": roof_smem})

    # ---- end to end through the host-pointer entry points (handle created from host arrays,
    #      candidates copied in, TELs copied out, all inside the timed region)
    total_codes = n * (n - 1) // 2 + n * (n - 1)
    s_pin = torch.from_numpy(inst.s.copy()).pin_memory()
    o_pin = torch.from_numpy(inst.o.copy()).pin_memory()
    e2e_steps = max(1, min(args.steps, 3))
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
    if rank == 0 and world == 1:
        import oracle as orc
        base, _ = orc.sorted_f_prefix(inst.s, inst.o, inst.M)
        assert (base == order).all(), "GPU and oracle disagree on the Sorted-F order"
        ty, mi, mj = sampled_move_positions(n, seed, args.warmup, 0, min(count, 4096))
        swap = (ty == 0) & (mi > mj)
        mi2, mj2 = np.where(swap, mj, mi), np.where(swap, mi, mj)
        t0 = time.perf_counter()
        orc.eval_moves(inst.s, inst.o, inst.M, base, ty[:4], mi2[:4], mj2[:4])
        pilot = (time.perf_counter() - t0) / 4
        k = int(max(8, min(len(ty), args.cpu_seconds / max(pilot, 1e-6))))
        t0 = time.perf_counter()
        ref = orc.eval_moves(inst.s, inst.o, inst.M, base, ty[:k], mi2[:k], mj2[:k])
        dt = time.perf_counter() - t0
        tel_dev = torch.empty(count, dtype=torch.int64, device=dev)
        h.sweep_dev(count, best, sampled=True, seed=seed, iteration=args.warmup, first_code=0, tel_out=tel_dev)
        h.sync()
        assert (tel_dev[:k].cpu().numpy() == ref).all(), "GPU and oracle TELs differ on the CPU-baseline sample"
        cpu = {"value": k / dt, "unit": "evals/s", "cores": 1, "kind": "oracle",
               "sample": "first %d sampled moves of one step (of %d), oracle/oracle.cpp orc_eval_moves, 1 thread; "
                         "TELs equal the GPU's" % (k, count)}

    if rank == 0:
        out = {
            "metric": "schedule_evals_per_sec", "value": value, "unit": "evals/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
            "config": {"workload": inst.name, "n": n, "M": inst.M, "sum_o": sum_o, "moves_per_step_per_gpu": count,
                       "neighbourhood": "sampled swap+insert moves of the Sorted-F order",
                       "l2": "flushed between steps (256 MiB write)", "checksum": "%016x" % inst.checksum()},
            "request_rounds_per_sec": value * sum_o,
            "best_tel_last_step": int(best[0].item()),
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e,
            "gpu_launches": int(launches1 - launches0), "clocks": clocks,
        }
        print(json.dumps(out))
    h.close()
    if multi:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
