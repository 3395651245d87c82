#!/usr/bin/env python
"""Benchmark of the broadcast-schedule generation on B200.

One "step" is one pass of the whole path over one workload: skips on the host,
then one launch that computes the receive and the send schedule of every rank
of p and writes both int32 tables to device memory.  Default workload: all
ranks of p = 2^27 - 1 (q = 27, 28 991 029 032 bytes of tables per step).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line (rank 0).  With N > 1 every rank runs an independent
replica of the workload (the path has no exchange step), timed as the maximum
over ranks.  `--impl reference` times the CPU oracle on a bounded sample of the
same workload on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "schedule_ranks_per_s"
UNIT = "ranks/s"
L2_BYTES = 126 * 2 ** 20


def workload_of(name: str):
    from paper_2407_18004_b200 import workloads
    table = {
        "p=2^27-1": workloads.P_LARGE,
        "p=2^20+1": workloads.P_MEDIUM,
        "p=1000": workloads.P_SMALL,
    }
    if name in table:
        return table[name]
    return int(name)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, copy read+write)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


def kernel_source_hash() -> str:
    """sha256 over the CUDA sources: a recorded DRAM-traffic figure is only quoted for the kernel it was taken on."""
    import glob
    import hashlib
    h = hashlib.sha256()
    for path in sorted(glob.glob(os.path.join(ROOT, "paper_2407_18004_b200", "csrc", "*"))):
        with open(path, "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def recorded_traffic(kernel: str, p: int):
    """dram read+write bytes per launch from profiles/dram_traffic.txt, or None when the sources changed since."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    if not os.path.exists(path):
        return None
    sha = kernel_source_hash()
    with open(path) as fh:
        for line in fh:
            parts = line.split()
            if len(parts) >= 5 and not line.startswith("#") and parts[0] == kernel and parts[1] == str(p) \
                    and parts[2] == sha:
                return int(parts[3]) + int(parts[4])
    return None


class ClockSampler:
    """nvidia-smi clock/throttle samples while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        inside = [l for (t, l) in self.lines if t0 <= t <= t1 + 0.05] or [l for (_, l) in self.lines]
        for line in inside:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); smax.append(float(parts[1])); power.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def time_oracle_sample(p: int, budget_ranks: int, mode: str = "broadcast"):
    """The oracle as it stands on a window of rows of the same workload (single thread)."""
    import oracle
    oracle.build()
    hi = min(budget_ranks, p)
    t0 = time.perf_counter()
    if mode == "allbroadcast":
        oracle.allbroadcast_schedule(p, p // 3, 0, hi)
    else:
        oracle.schedule_table(p, 0, 0, hi)
    dt = time.perf_counter() - t0
    full = (hi == p)
    what = "roots" if mode == "allbroadcast" else "ranks"
    sample = ("all %s of p=%d: receive rows by Algorithm 5, send rows gathered from them" % (what, p)) if full else (
        "%s [0,%d) of p=%d: receive row by Algorithm 5, send row by definition (q receive schedules per row)"
        % (what, hi, p))
    return hi / dt, dt, sample


def workload_label(mode: str, p: int, q: int) -> str:
    if mode == "allbroadcast":
        return ("Algorithm 7 tables of processor %d for all roots of p=%d (q=%d), recvblocks+sendblocks int32"
                % (p // 3, p, q))
    return "all ranks of p=%d (q=%d), root 0, recvblock+sendblock int32 tables" % (p, q)


def oracle_sample_size(p: int) -> int:
    # about 15 us per rank in window mode at q = 27 -> ~15-25 s
    q = max((p - 1).bit_length(), 1)
    return int(min(p, max(1024, 2 ** 20 * 27 * 28 // (q * (q + 1)))))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    p = workload_of(args.workload)
    q = max((p - 1).bit_length(), 0)
    per_step = max(oracle_sample_size(p) // max(args.steps + args.warmup, 1), 1024)
    per_step = min(per_step, p)
    import oracle
    oracle.build()
    def ref_step():
        if args.mode == "allbroadcast":
            oracle.allbroadcast_schedule(p, p // 3, 0, per_step)
        else:
            oracle.schedule_table(p, 0, 0, per_step)

    for _ in range(args.warmup):
        ref_step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        ref_step()
    dt = time.perf_counter() - t0
    value = per_step * args.steps / dt
    sample = ("each step: rows [0,%d) of the workload, receive row by Algorithm 5, send row by definition"
              % per_step)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32",
        "data": "synthetic",
        "config": {"workload": workload_label(args.mode, p, q), "sampled": True},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2407_18004_b200 as bs

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the schedule library has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    p = workload_of(args.workload)
    q = bs.bcast_q(p)
    table_bytes = 2 * p * q * 4
    recv = torch.empty((p, q), dtype=torch.int32, device="cuda")
    send = torch.empty((p, q), dtype=torch.int32, device="cuda")
    flush = None
    if table_bytes < 2 * L2_BYTES:
        flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()

    def step():
        bs.bcast_skips(p)
        if args.mode == "allbroadcast":
            bs.bcast_allbroadcast_schedule(p, p // 3, 0, p, recv, send, stream)
        else:
            bs.bcast_schedule(p, 0, 0, p, recv, send, stream)

    for _ in range(max(args.warmup, 3)):
        step()
        if flush is not None:
            flush.zero_()
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.15)
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    stops = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    barrier()
    t0 = time.time()
    for i in range(args.steps):
        if flush is not None:
            flush.zero_()
        starts[i].record(stream)
        step()
        stops[i].record(stream)
    barrier()
    t1 = time.time()
    clocks = sampler.stop(t0, t1)
    per_step_ms = [s.elapsed_time(e) for s, e in zip(starts, stops)]
    total_ms = sum(per_step_ms)
    if world > 1:
        t = torch.tensor([total_ms], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    ms_per_step = total_ms / args.steps
    value = world * p * args.steps / (total_ms * 1e-3)

    # ---------------- end to end: host output tables through bcast_schedule_host
    e2e = None
    if not args.no_e2e and args.mode == "broadcast":
        staging = torch.empty(512 * 2 ** 20, dtype=torch.uint8, device="cuda")
        try:
            hrecv = torch.empty((p, q), dtype=torch.int32, pin_memory=True)
            hsend = torch.empty((p, q), dtype=torch.int32, pin_memory=True)
        except RuntimeError as exc:
            hrecv = hsend = None
            e2e_err = str(exc).splitlines()[0]
        if hrecv is not None:
            bs.bcast_schedule_host(p, 0, 0, p, hrecv, hsend, staging, stream)
            torch.cuda.synchronize()
            e2e_steps = max(1, min(args.steps, args.e2e_steps))
            ev0 = torch.cuda.Event(enable_timing=True)
            ev1 = torch.cuda.Event(enable_timing=True)
            barrier()
            ev0.record(stream)
            for _ in range(e2e_steps):
                bs.bcast_skips(p)
                bs.bcast_schedule_host(p, 0, 0, p, hrecv, hsend, staging, stream)
            ev1.record(stream)
            barrier()
            e2e_ms = ev0.elapsed_time(ev1)
            if world > 1:
                t = torch.tensor([e2e_ms], dtype=torch.float64, device="cuda")
                dist.all_reduce(t, op=dist.ReduceOp.MAX)
                e2e_ms = float(t.item())
            e2e = {"value": world * p * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT,
                   "h2d_bytes_per_step": 0, "d2h_bytes_per_step": table_bytes, "steps": e2e_steps,
                   "ms_per_step": e2e_ms / e2e_steps,
                   "note": "bcast_schedule_host: tables land in pinned host memory; inputs are scalars"}
            del hrecv, hsend
        else:
            e2e = {"value": None, "unit": UNIT, "error": e2e_err}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    peak, peak_src = measured_peaks()
    kernel_ms = statistics.mean(per_step_ms)
    achieved = table_bytes / (kernel_ms * 1e-3) / 1e9
    traffic = recorded_traffic("schedule_table_kernel", p) if args.mode == "broadcast" else None

    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        v, dt, sample = time_oracle_sample(p, oracle_sample_size(p), args.mode)
        cpu_baseline = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample,
                        "seconds": dt, "host_cores_available": os.cpu_count()}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
        "config": {"workload": workload_label(args.mode, p, q),
                   "bytes_per_step": table_bytes, "replicas": world,
                   "l2": "tables larger than L2" if flush is None else "L2 flushed between steps"},
        "entries_per_s": value * 2 * q,
        "hbm_write_gbs": achieved * world,
        "ms_per_step_min": min(per_step_ms), "ms_per_step_median": statistics.median(per_step_ms),
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": traffic, "peak_source": peak_src,
                     "kernel": "schedule_table_kernel", "bytes_per_launch": table_bytes,
                     "frac_of_nominal_8TBs": achieved / 8000.0},
        "cpu_baseline": cpu_baseline,
        "e2e": e2e,
        "gpu_launches": args.steps,
        "clocks": clocks,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="p=2^27-1")
    ap.add_argument("--mode", default="broadcast", choices=["broadcast", "allbroadcast"],
                    help="broadcast: tables of all ranks for one root; allbroadcast: Algorithm 7's tables of one "
                         "processor for all roots (no host-table leg)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
