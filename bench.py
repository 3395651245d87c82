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

Other workloads of the same library, each with its own metric (`--mode`):
allbroadcast (Algorithm 7's tables), shifted (tables after Algorithm 1's
preamble), batch (2^24 independent queries), sweep (fused verification of every
p in [2, 65536]), simulate / reduce (Algorithm 1 and its reversal run by all
processors on device tables).
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
    return 6650.0, "fallback (6.65 TB/s: MEASURED_PEAKS.json is absent)"


KERNEL_SOURCES = {
    "schedule_table_kernel": ("schedule_core.cuh", "schedule_fast.cuh", "schedule_tile.cuh", "table_kernel.cuh",
                              "table_q_low.cu", "table_q_mid.cu", "table_q_high.cu", "table_q_top.cu", "bcast_sched.cu"),
    "schedule_batch_kernel": ("schedule_core.cuh", "schedule_fast.cuh", "schedule_tile.cuh", "bcast_sched.cu"),
    "verify_sweep_kernel": ("schedule_core.cuh", "schedule_fast.cuh", "schedule_tile.cuh", "bcast_sweep.cu"),
}


def kernel_source_hash(kernel: str) -> str:
    """sha256 over the CUDA sources a kernel is compiled from: a recorded counter is only quoted for the kernel it
    was taken on."""
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES[kernel]:
        with open(os.path.join(ROOT, "paper_2407_18004_b200", "csrc", name), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def recorded_counters(kernel: str, key: str):
    """A line `kernel key sha256-of-its-sources a b` of profiles/counters.txt as (a, b), or None when there is none for
    the sources as they are now (ncu counters of a small stand-in launch; see the file for what a and b are)."""
    path = os.path.join(ROOT, "profiles", "counters.txt")
    if not os.path.exists(path):
        return None
    sha = kernel_source_hash(kernel)
    with open(path) as fh:
        for line in fh:
            parts = line.split()
            if len(parts) >= 5 and not line.startswith("#") and parts[0] == kernel and parts[1] == key \
                    and parts[2] == sha:
                return float(parts[3]), float(parts[4])
    return None


def scaled_traffic(kernel: str, key: str, algorithmic_bytes: float):
    """DRAM bytes of one launch, scaled from the stand-in capture by the algorithmic bytes (a = DRAM bytes read +
    written by the stand-in launch, b = its algorithmic bytes; the traffic is all table rows, so it grows with them)."""
    rec = recorded_counters(kernel, key)
    return None if rec is None else rec[0] / rec[1] * algorithmic_bytes


def scaled_instructions(kernel: str, key: str, units: float):
    """Warp instructions of one launch, scaled from the stand-in capture by the units processed (a = warp
    instructions of the stand-in launch, b = its units)."""
    rec = recorded_counters(kernel, key)
    return None if rec is None else rec[0] / rec[1] * units


def max_over_ranks(ms: float, world: int, device: str = "cuda") -> float:
    """A time in ms as the maximum over all ranks of the job (replicas run side by side; the slowest counts)."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(units_per_rank, steps: int, world: int, total_ms: float) -> float:
    """Units all ranks processed in the timed steps per second of the slowest rank."""
    return world * units_per_rank * steps / (total_ms * 1e-3)


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


def time_oracle_sample(p: int, budget_ranks: int, mode: str = "broadcast", blocks: int = 0):
    """The oracle as it stands on a window of rows of the same workload (single thread)."""
    import oracle
    oracle.build()
    hi = min(budget_ranks, p)
    t0 = time.perf_counter()
    if mode == "allbroadcast":
        oracle.allbroadcast_schedule(p, p // 3, 0, hi)
    elif mode == "shifted":
        oracle.shifted_table(p, blocks, 0, 0, hi)
    else:
        oracle.schedule_table(p, 0, 0, hi)
    dt = time.perf_counter() - t0
    full = (hi == p)
    what = "roots" if mode == "allbroadcast" else "ranks"
    sample = ("all %s of p=%d: receive rows by Algorithm 5, send rows gathered from them" % (what, p)) if full else (
        "%s [0,%d) of p=%d: receive row by Algorithm 5, send row by definition (q receive schedules per row)"
        % (what, hi, p))
    return hi / dt, dt, sample


def workload_label(mode: str, p: int, q: int, blocks: int = 0) -> str:
    if mode == "shifted":
        return ("all ranks of p=%d (q=%d), root 0, tables with Algorithm 1's preamble for n=%d blocks applied"
                % (p, q, blocks))
    if mode == "allbroadcast":
        return ("Algorithm 7 tables of processor %d for all roots of p=%d (q=%d), recvblocks+sendblocks int32"
                % (p // 3, p, q))
    return "all ranks of p=%d (q=%d), root 0, recvblock+sendblock int32 tables" % (p, q)


def oracle_other_modes(p: int):
    """The oracle's other routes, timed beside the window mode (single thread, as it stands):
    receive rows alone on a window of the same p, and the all-ranks route (receive rows by Algorithm 5 for
    every rank, send rows gathered from them: one search per rank) on configuration 2 (p = 2^20 + 1) in full."""
    import oracle
    from paper_2407_18004_b200 import workloads
    rows = min(p, 2 ** 21)
    t0 = time.perf_counter()
    oracle.schedule_table(p, 0, 0, rows, want_send=False)
    dt_recv = time.perf_counter() - t0
    pm = workloads.P_MEDIUM
    t0 = time.perf_counter()
    oracle.schedule_table(pm, 0)
    dt_all = time.perf_counter() - t0
    return {
        "recv_rows_only": {"value": rows / dt_recv, "unit": "rows/s", "seconds": dt_recv,
                           "sample": "receive rows [0,%d) of p=%d by Algorithm 5 (one search per row)" % (rows, p)},
        "all_ranks_mode": {"value": pm / dt_all, "unit": UNIT, "seconds": dt_all,
                           "sample": "p=%d in full: receive rows by Algorithm 5, send rows gathered from them "
                                     "(one search per rank)" % pm},
    }


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
        elif args.mode == "shifted":
            oracle.shifted_table(p, args.blocks, 0, 0, per_step)
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
        "config": {"workload": workload_label(args.mode, p, q, args.blocks), "sampled": True},
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
        elif args.mode == "shifted":
            bs.bcast_schedule_shifted(p, 0, args.blocks, 0, p, recv, send, stream)
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
    total_ms = max_over_ranks(total_ms, world)
    ms_per_step = total_ms / args.steps
    value = whole_job_value(p, args.steps, world, total_ms)

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
            e2e_ms = max_over_ranks(e2e_ms, world)
            e2e = {"value": whole_job_value(p, e2e_steps, world, e2e_ms), "unit": UNIT,
                   "h2d_bytes_per_step": 0, "d2h_bytes_per_step": table_bytes, "steps": e2e_steps,
                   "ms_per_step": e2e_ms / e2e_steps,
                   "note": "bcast_schedule_host: tables land in pinned host memory; inputs are scalars"}
            del hrecv, hsend
        else:
            e2e = {"value": None, "unit": UNIT, "error": e2e_err}

    peak, peak_src = measured_peaks()
    store_only = None
    configs = None
    if world == 1 and args.mode == "broadcast":
        store_only = measure_store_ceiling(bs, torch, recv, send, stream)
        if not args.no_configs:
            configs = measure_configs(bs, torch, recv, send, stream, peak, statistics.mean(per_step_ms), p)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    kernel_ms = statistics.mean(per_step_ms)
    achieved = table_bytes / (kernel_ms * 1e-3) / 1e9
    traffic = scaled_traffic("schedule_table_kernel", "clean", table_bytes) if args.mode == "broadcast" else None

    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        v, dt, sample = time_oracle_sample(p, oracle_sample_size(p), args.mode, args.blocks)
        cpu_baseline = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample,
                        "seconds": dt, "host_cores_available": os.cpu_count(),
                        "mode": "window (q + 1 searches per rank: the oracle's slowest route)"}
        if args.mode == "broadcast":
            cpu_baseline.update(oracle_other_modes(p))

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
        "config": {"workload": workload_label(args.mode, p, q, args.blocks),
                   "bytes_per_step": table_bytes, "replicas": world,
                   "l2": "tables larger than L2" if flush is None else "L2 flushed between steps"},
        "entries_per_s": value * 2 * q,
        "hbm_write_gbs": achieved * world,
        "ms_per_step_min": min(per_step_ms), "ms_per_step_median": statistics.median(per_step_ms),
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": traffic, "peak_source": peak_src,
                     "kernel": "schedule_table_kernel", "bytes_per_launch": table_bytes,
                     "frac_of_nominal_8TBs": achieved / 8000.0,
                     "store_only_gbs": store_only,
                     "frac_of_store_only": achieved / store_only if store_only else None},
        "cpu_baseline": cpu_baseline,
        "e2e": e2e,
        "gpu_launches": args.steps,
        "clocks": clocks,
    }
    if configs is not None:
        line["configs"] = configs
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def time_launches(torch, stream, fn, pairs: int, per_pair: int = 1, before=None):
    """Mean and minimum device time in ms of one call of fn: `pairs` event pairs, each around `per_pair` calls
    back to back (short launches are timed many to a pair)."""
    times = []
    for _ in range(pairs):
        if before is not None:
            before()
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(per_pair):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1) / per_pair)
    return statistics.mean(times), min(times)


def measure_store_ceiling(bs, torch, recv, send, stream):
    """GB/s of bcast_store_ceiling over the same bytes as the headline tables (both buffers, one launch each)."""
    def fill():
        bs.bcast_store_ceiling(recv, recv.numel() * 4, 0, stream)
        bs.bcast_store_ceiling(send, send.numel() * 4, 0, stream)
    fill()
    torch.cuda.synchronize()
    mean_ms, _ = time_launches(torch, stream, fill, 5)
    return (recv.numel() + send.numel()) * 4 / (mean_ms * 1e-3) / 1e9


def measure_configs(bs, torch, recv, send, stream, peak, headline_ms, p_large):
    """The other benchmark configurations and the library's other table forms, measured in the same run (same
    device buffers, same clock sampling window is not repeated: short runs).  Each entry: mean ms per launch, the
    workload's own throughput, and the roofline fraction with its bound."""
    from paper_2407_18004_b200 import workloads
    flat_r, flat_s = recv.view(-1), send.view(-1)
    out = {}

    def tables(p):
        q = bs.bcast_q(p)
        return q, flat_r[:p * q].view(p, q), flat_s[:p * q].view(p, q)

    def table_entry(name, p, launch, pairs, per_pair, what):
        q, r, s_ = tables(p)
        fn = lambda: launch(p, q, r, s_)
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        mean_ms, min_ms = time_launches(torch, stream, fn, pairs, per_pair)
        nbytes = 8 * q * p
        gbs = nbytes / (mean_ms * 1e-3) / 1e9
        # the store pattern alone over the same two tables, launched the same way: what a launch of this size can reach
        def fill():
            bs.bcast_store_ceiling(r, r.numel() * 4, 0, stream)
            bs.bcast_store_ceiling(s_, s_.numel() * 4, 0, stream)
        fill()
        torch.cuda.synchronize()
        fill_ms, _ = time_launches(torch, stream, fill, 3, per_pair)
        store_gbs = nbytes / (fill_ms * 1e-3) / 1e9
        out[name] = {"workload": what % (p, q), "ms": mean_ms, "ms_min": min_ms, "launches_per_event_pair": per_pair,
                     "value": p / (mean_ms * 1e-3), "unit": UNIT, "bytes_per_launch": nbytes,
                     "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                                  "store_only_gbs": store_gbs, "frac_of_store_only": gbs / store_gbs}}
        return mean_ms

    table_entry("config2_p=2^20+1", workloads.P_MEDIUM,
                lambda p, q, r, s_: bs.bcast_schedule(p, 0, 0, p, r, s_, stream), 5, 60,
                "all ranks of p=%d (q=%d), root 0 (configuration 2); tables larger than L2, launches back to back")
    table_entry("ordinary_p=123456789", 123456789,
                lambda p, q, r, s_: bs.bcast_schedule(p, 0, 0, p, r, s_, stream), 10, 1,
                "all ranks of p=%d (q=%d), root 0: a p with no special form")
    ms_root = table_entry("root_p/3_p=2^27-1", p_large,
                          lambda p, q, r, s_: bs.bcast_schedule(p, p // 3, 0, p, r, s_, stream), 10, 1,
                          "all ranks of p=%d (q=%d), root floor(p/3)")
    out["root_p/3_p=2^27-1"]["ms_over_root_0"] = ms_root / headline_ms
    table_entry("allbroadcast_p=2^27-1", p_large,
                lambda p, q, r, s_: bs.bcast_allbroadcast_schedule(p, p // 3, 0, p, r, s_, stream), 10, 1,
                "Algorithm 7's tables of processor floor(p/3) for all roots of p=%d (q=%d)")
    table_entry("shifted_n=64_p=2^27-1", p_large,
                lambda p, q, r, s_: bs.bcast_schedule_shifted(p, 0, 64, 0, p, r, s_, stream), 10, 1,
                "all ranks of p=%d (q=%d), root 0, rows after Algorithm 1's preamble for n=64 blocks")

    # the tables in use: Algorithm 1 and its reversal by all processors of configuration 2's p, 64 blocks, on
    # tables left by a launch in the same buffers; state and scratch come out of the send buffer's tail
    p, n = workloads.P_MEDIUM, 64
    q, r, s_ = tables(p)
    bs.bcast_schedule(p, 0, 0, p, r, s_, stream)
    rounds = n - 1 + q
    spare = flat_s[(p * q + 3) // 4 * 4:]                  # from a 16-byte boundary on
    arrival = spare[:n * p].view(n, p)
    need = bs.bcast_simulate_scratch_bytes(p, n, True)
    n_words = 2 * n * p + n + 8 + (need + 7) // 8
    words = spare[n * p:n * p + 2 * n_words].view(torch.int64)     # n * p is a multiple of 4: still on a 16-byte boundary
    value, contrib = words[:n * p].view(n, p), words[n * p:2 * n * p].view(n, p)
    result, stats = words[2 * n * p:2 * n * p + n], words[2 * n * p + n:2 * n * p + n + 8]
    scratch = words[2 * n * p + n + 8:].view(torch.uint8)[:need]           # an even number of words in: 16-byte aligned
    contrib.random_(0, 2 ** 62)

    def reduce_step():
        value.copy_(contrib)
        bs.bcast_simulate_reduce(p, 0, n, r, s_, value, result, stats, scratch, stream)

    for name, fn, nbytes, what in (
            ("simulate_n=64_p=2^20+1", lambda: bs.bcast_simulate_broadcast(p, 0, n, r, s_, arrival, stats, scratch, stream),
             p * (10 * q + 8 * n + rounds * 14), "Algorithm 1 by all processors of p=%d (q=%d), 64 blocks, %d rounds"),
            ("reduce_n=64_p=2^20+1", reduce_step, p * (10 * q + 18 * n + rounds * 30),
             "Observation 1.3's reduction by all processors of p=%d (q=%d), 64 blocks, %d rounds, contributions copied in")):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        mean_ms, min_ms = time_launches(torch, stream, fn, 10)
        gbs = nbytes / (mean_ms * 1e-3) / 1e9
        out[name] = {"workload": what % (p, q, rounds), "ms": mean_ms, "ms_min": min_ms,
                     "value": (p - 1) * n / (mean_ms * 1e-3), "unit": "blocks/s", "bytes_per_step": nbytes,
                     "stats": stats.tolist(),
                     "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                                  "note": "algorithmic bytes of the whole step (all of its launches) over its time"}}

    # config 5: 2^24 independent queries (rows padded to 31), outputs in the same buffers
    nq = 2 ** 24
    hp, hr, ho = workloads.query_batch(nq, seed=0)
    dp, dr, do = [torch.from_numpy(a).cuda() for a in (hp, hr, ho)]
    brecv, bsend = flat_r[:nq * 31].view(nq, 31), flat_s[:nq * 31].view(nq, 31)
    bad = torch.zeros(1, dtype=torch.int32, device="cuda")
    batch = lambda: bs.bcast_schedule_batch(dp, dr, do, 31, brecv, bsend, bad, stream)
    for _ in range(3):
        batch()
    torch.cuda.synchronize()
    mean_ms, min_ms = time_launches(torch, stream, batch, 10)
    insts = scaled_instructions("schedule_batch_kernel", "batch", nq)
    ach = insts / (mean_ms * 1e-3) / 1e9 if insts else None
    out["config5_batch_2^24"] = {
        "workload": "2^24 queries, p log-uniform in [2, 2^31-1], rank and root uniform, seed 0, rows padded to 31 "
                    "(configuration 5)", "ms": mean_ms, "ms_min": min_ms, "value": nq / (mean_ms * 1e-3),
        "unit": "queries/s", "bytes_per_launch": nq * (2 * 31 * 4 + 12),
        "hbm_write_gbs": nq * 2 * 31 * 4 / (mean_ms * 1e-3) / 1e9,
        "roofline": {"bound": "alu", "achieved": ach, "peak": ISSUE_PEAK_GINST, "unit": "G warp-inst/s",
                     "frac": ach / ISSUE_PEAK_GINST if ach else None, "warp_instructions_per_launch": insts}}
    del dp, dr, do

    # config 4: the fused verification sweep
    lo, hi = 2, 65536
    checksum = torch.zeros(hi - lo + 1, dtype=torch.int64, device="cuda")
    fails = torch.zeros(8, dtype=torch.int32, device="cuda")
    need = bs.bcast_verify_sweep_scratch_bytes(lo, hi)
    scratch = flat_r.view(torch.uint8)[:need]
    sweep = lambda: bs.bcast_verify_sweep(lo, hi, checksum, fails, scratch, stream)
    sweep()
    torch.cuda.synchronize()
    mean_ms, min_ms = time_launches(torch, stream, sweep, 3)
    units = sum(range(lo, hi + 1))
    insts = scaled_instructions("verify_sweep_kernel", "sweep", units)
    ach = insts / (mean_ms * 1e-3) / 1e9 if insts else None
    out["config4_sweep_2_65536"] = {
        "workload": "every p in [2, 65536], all ranks, root 0: tables built and checked on the device, one checksum "
                    "per p (configuration 4)", "ms": mean_ms, "ms_min": min_ms, "value": units / (mean_ms * 1e-3),
        "unit": "rank-schedules/s", "fail_counts": fails.tolist(),
        "roofline": {"bound": "alu", "achieved": ach, "peak": ISSUE_PEAK_GINST, "unit": "G warp-inst/s",
                     "frac": ach / ISSUE_PEAK_GINST if ach else None, "warp_instructions_per_launch": insts}}
    return out


# ---------------------------------------------------------------------------------------------
# The other workloads: each a dict with its metric, one device step, the oracle on a bounded
# sample, and an end-to-end step that moves its inputs and results over PCIe.
OTHER_MODES = ("batch", "sweep", "simulate", "reduce")
ISSUE_PEAK_GINST = 148 * 4 * 1.965         # warp instructions per ns at one per scheduler and clock: 148 SMs x 4 x 1.965 GHz


def build_other(args, torch, bs):
    import numpy as np
    from paper_2407_18004_b200 import workloads
    stream = torch.cuda.current_stream()
    mode = args.mode
    if mode == "batch":
        nq = args.queries
        hp, hr, ho = workloads.query_batch(nq, seed=0)
        pin = [torch.from_numpy(a).pin_memory() for a in (hp, hr, ho)]
        dp, dr, do = [t.cuda() for t in pin]
        recv = torch.empty((nq, 31), dtype=torch.int32, device="cuda")
        send = torch.empty((nq, 31), dtype=torch.int32, device="cuda")
        bad = torch.zeros(1, dtype=torch.int32, device="cuda")
        host_out = {}

        def step():
            bs.bcast_schedule_batch(dp, dr, do, 31, recv, send, bad, stream)

        def e2e_step():
            if not host_out:
                host_out["r"] = torch.empty((nq, 31), dtype=torch.int32, pin_memory=True)
                host_out["s"] = torch.empty((nq, 31), dtype=torch.int32, pin_memory=True)
            for d, h in zip((dp, dr, do), pin):
                d.copy_(h, non_blocking=True)
            step()
            host_out["r"].copy_(recv, non_blocking=True)
            host_out["s"].copy_(send, non_blocking=True)

        def oracle_sample():
            import oracle
            m = min(nq, 2 ** 19)
            t0 = time.perf_counter()
            oracle.schedule_batch(hp[:m], hr[:m], ho[:m], 31)
            return m, time.perf_counter() - t0, ("the first %d queries: receive row by Algorithm 5, send row by "
                                                 "definition (q receive schedules)" % m)

        return dict(label="%d queries, p log-uniform in [2, 2^31-1], rank and root uniform, seed 0, rows padded to 31"
                          % nq, metric="schedule_queries_per_s", unit="queries/s", units=nq,
                    bytes=nq * (2 * 31 * 4 + 12), step=step, launches=1, kernel="schedule_batch_kernel",
                    bound="alu", e2e=e2e_step, h2d=12 * nq, d2h=2 * 31 * 4 * nq, oracle=oracle_sample,
                    extra=lambda: {"bad_queries": int(bad.item())})
    if mode == "sweep":
        lo, hi = args.sweep_lo, args.sweep_hi
        checksum = torch.zeros(hi - lo + 1, dtype=torch.int64, device="cuda")
        fails = torch.zeros(8, dtype=torch.int32, device="cuda")
        scratch = torch.empty(bs.bcast_verify_sweep_scratch_bytes(lo, hi), dtype=torch.uint8, device="cuda")
        units = sum(range(lo, hi + 1))
        host = {}

        def step():
            bs.bcast_verify_sweep(lo, hi, checksum, fails, scratch, stream)

        def e2e_step():
            if not host:
                host["c"] = torch.empty(hi - lo + 1, dtype=torch.int64, pin_memory=True)
                host["f"] = torch.empty(8, dtype=torch.int32, pin_memory=True)
            step()
            host["c"].copy_(checksum, non_blocking=True)
            host["f"].copy_(fails, non_blocking=True)

        def oracle_sample():
            import oracle
            ps = list(range(hi, lo - 1, -(hi - lo) // 96))[:96]
            t0 = time.perf_counter()
            for pp in ps:
                oracle.checksum(pp)
            return sum(ps), time.perf_counter() - t0, ("checksums of %d values of p spread evenly over [%d, %d] "
                                                       "(tables by Algorithm 5 and a gather, no condition checks)"
                                                       % (len(ps), lo, hi))

        return dict(label="every p in [%d, %d], all ranks, root 0: tables built and checked on the device, one "
                          "checksum per p" % (lo, hi), metric="verified_rank_schedules_per_s", unit="rank-schedules/s",
                    units=units, bytes=8 * (hi - lo + 1), step=step, launches=2, kernel="verify_sweep_kernel",
                    bound="alu", e2e=e2e_step, h2d=0, d2h=8 * (hi - lo + 1) + 32, oracle=oracle_sample,
                    extra=lambda: {"fail_counts": fails.tolist()})
    # simulate / reduce
    p = workload_of(args.workload)
    q = bs.bcast_q(p)
    n = args.blocks
    rounds = n - 1 + q
    bs.bcast_set_simulate_rounds({"auto": bs.BCAST_ROUNDS_AUTO, "launches": bs.BCAST_ROUNDS_LAUNCHES,
                                  "fused": bs.BCAST_ROUNDS_FUSED}[args.rounds])
    fused = args.rounds != "launches"
    round_launches = (rounds + 65535) // 65536 + 1 if fused else rounds     # fused: up to 65536 rounds a launch, and the seal
    form = "all rounds in cooperative launches" if fused else "one launch per round"
    recv = torch.empty((p, q), dtype=torch.int32, device="cuda")
    send = torch.empty((p, q), dtype=torch.int32, device="cuda")
    bs.bcast_schedule(p, 0, 0, p, recv, send, stream)
    stats = torch.zeros(8, dtype=torch.int64, device="cuda")
    scratch = torch.empty(bs.bcast_simulate_scratch_bytes(p, n, mode == "reduce"), dtype=torch.uint8, device="cuda")
    host = {}
    small_p = min(p, 2 ** 16 + 1)
    if mode == "simulate":
        arrival = torch.empty((n, p), dtype=torch.int32, device="cuda")

        def step():
            bs.bcast_simulate_broadcast(p, 0, n, recv, send, arrival, stats, scratch, stream)

        def e2e_step():
            if not host:
                host["s"] = torch.empty(8, dtype=torch.int64, pin_memory=True)
            bs.bcast_schedule(p, 0, 0, p, recv, send, stream)
            step()
            host["s"].copy_(stats, non_blocking=True)

        def oracle_sample():
            import oracle
            r, s = oracle.schedule_table(small_p, 0)
            t0 = time.perf_counter()
            oracle.simulate_broadcast(small_p, 0, n, r, s)
            return (small_p - 1) * n, time.perf_counter() - t0, ("the same %d blocks on p=%d processors (tables given)"
                                                                 % (n, small_p))

        # tables turned into bytes (8q read, 2q written per processor), arrival table set and counted (4 B per
        # cell each), and per round and processor two table bytes, two arrival reads and one arrival write
        nbytes = p * (10 * q + 8 * n + rounds * 14)
        return dict(label="Algorithm 1 by all processors of p=%d (q=%d), n=%d blocks, %d rounds (%s), tables on the device"
                          % (p, q, n, rounds, form), metric="simulated_block_deliveries_per_s", unit="blocks/s",
                    units=(p - 1) * n, bytes=nbytes, step=step, launches=round_launches + 4,
                    kernel="broadcast_rounds_kernel" if fused else "broadcast_round_kernel",
                    bound="hbm", e2e=e2e_step, h2d=0, d2h=64, oracle=oracle_sample,
                    extra=lambda: {"stats": stats.tolist()})
    gen = torch.Generator(device="cuda")
    gen.manual_seed(0)
    contrib = torch.randint(0, 2 ** 62, (n, p), dtype=torch.int64, device="cuda", generator=gen)
    value = torch.empty_like(contrib)
    result = torch.empty(n, dtype=torch.int64, device="cuda")

    def step():
        value.copy_(contrib)
        bs.bcast_simulate_reduce(p, 0, n, recv, send, value, result, stats, scratch, stream)

    def e2e_step():
        if not host:
            host["s"] = torch.empty(8, dtype=torch.int64, pin_memory=True)
            host["r"] = torch.empty(n, dtype=torch.int64, pin_memory=True)
        bs.bcast_schedule(p, 0, 0, p, recv, send, stream)
        step()
        host["s"].copy_(stats, non_blocking=True)
        host["r"].copy_(result, non_blocking=True)

    def oracle_sample():
        import numpy as np
        import oracle
        r, s = oracle.schedule_table(small_p, 0)
        v = np.random.default_rng(0).integers(0, 2 ** 62, size=(n, small_p), dtype=np.uint64)
        t0 = time.perf_counter()
        oracle.simulate_reduce(small_p, 0, n, r, s, v)
        return (small_p - 1) * n, time.perf_counter() - t0, ("the same %d blocks on p=%d processors (tables given)"
                                                             % (n, small_p))

    # contributions copied in (16 B per cell), sent counts cleared and read (2 B per cell), byte tables, and per
    # round and processor: three table bytes, the sender's value read, the own value read and written, sent
    # count read twice and written once
    nbytes = p * (10 * q + 18 * n + rounds * (3 + 8 + 16 + 3))
    return dict(label="Observation 1.3's reduction by all processors of p=%d (q=%d), n=%d blocks, %d rounds (%s)"
                      % (p, q, n, rounds, form), metric="simulated_partial_results_per_s", unit="blocks/s",
                units=(p - 1) * n, bytes=nbytes, step=step, launches=round_launches + 2,
                kernel="reduce_rounds_kernel" if fused else "reduce_round_kernel",
                bound="hbm", e2e=e2e_step, h2d=0, d2h=64 + 8 * n, oracle=oracle_sample,
                extra=lambda: {"stats": stats.tolist()})


def run_other(args):
    if args.impl == "reference":
        return run_other_reference(args)
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
    wl = build_other(args, torch, bs)
    stream = torch.cuda.current_stream()
    flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device="cuda")

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, flush_between):
        starts = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        stops = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        barrier()
        for i in range(steps):
            if flush_between:
                flush.zero_()
            starts[i].record(stream)
            fn()
            stops[i].record(stream)
        barrier()
        return [a.elapsed_time(b) for a, b in zip(starts, stops)]

    for _ in range(max(args.warmup, 3)):
        wl["step"]()
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.15)
    t0 = time.time()
    per_step_ms = timed(wl["step"], args.steps, True)
    t1 = time.time()
    clocks = sampler.stop(t0, t1)
    total_ms = sum(per_step_ms)
    total_ms = max_over_ranks(total_ms, world)
    value = whole_job_value(wl["units"], args.steps, world, total_ms)

    e2e = None
    if not args.no_e2e:
        wl["e2e"]()
        torch.cuda.synchronize()
        e2e_steps = max(1, min(args.steps, args.e2e_steps))
        e2e_ms = sum(timed(wl["e2e"], e2e_steps, False))
        e2e_ms = max_over_ranks(e2e_ms, world)
        e2e = {"value": whole_job_value(wl["units"], e2e_steps, world, e2e_ms), "unit": wl["unit"],
               "h2d_bytes_per_step": wl["h2d"], "d2h_bytes_per_step": wl["d2h"], "steps": e2e_steps,
               "ms_per_step": e2e_ms / e2e_steps}
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    mean_ms = statistics.mean(per_step_ms)
    if wl["bound"] == "hbm":
        peak, peak_src = measured_peaks()
        achieved = wl["bytes"] / (mean_ms * 1e-3) / 1e9
        roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                    "traffic": None, "peak_source": peak_src,
                    "kernel": wl["kernel"], "bytes_per_step": wl["bytes"],
                    "note": "algorithmic bytes of the whole step over the step's time (all of its launches)"}
    else:
        # bound by instruction issue: warp instructions of one launch (recorded from ncu while the sources
        # are unchanged) over its time, against one instruction per scheduler and clock
        insts = scaled_instructions(wl["kernel"], args.mode, wl["units"])
        achieved = insts / (mean_ms * 1e-3) / 1e9 if insts else None
        roofline = {"bound": "alu", "achieved": achieved, "peak": ISSUE_PEAK_GINST, "unit": "G warp-inst/s",
                    "frac": achieved / ISSUE_PEAK_GINST if achieved else None, "traffic": None,
                    "peak_source": "148 SMs x 4 schedulers x 1.965 GHz, one warp instruction per scheduler and clock",
                    "kernel": wl["kernel"], "warp_instructions_per_launch": insts,
                    "hbm_write_gbs": wl["bytes"] / (mean_ms * 1e-3) / 1e9}
    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        import oracle
        oracle.build()
        units, dt, sample = wl["oracle"]()
        cpu_baseline = {"value": units / dt, "unit": wl["unit"], "cores": 1, "kind": "oracle", "sample": sample,
                        "seconds": dt, "host_cores_available": os.cpu_count()}
    line = {
        "metric": wl["metric"], "value": value, "unit": wl["unit"], "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": total_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
        "config": {"workload": wl["label"], "bytes_per_step": wl["bytes"], "replicas": world,
                   "l2": "L2 flushed between steps"},
        "ms_per_step_min": min(per_step_ms), "ms_per_step_median": statistics.median(per_step_ms),
        "roofline": roofline, "cpu_baseline": cpu_baseline, "e2e": e2e,
        "gpu_launches": args.steps * wl["launches"], "clocks": clocks,
    }
    line.update(wl["extra"]())
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def run_other_reference(args):
    """The oracle's leg of the other workloads: its bounded sample, once per step."""
    if int(os.environ.get("RANK", "0")) != 0:
        return 0
    import oracle
    oracle.build()

    wl = reference_sample(args)
    for _ in range(args.warmup):
        wl()
    units = 0
    t0 = time.perf_counter()
    for _ in range(args.steps):
        u, _, sample = wl()
        units += u
    dt = time.perf_counter() - t0
    metric, unit = {"batch": ("schedule_queries_per_s", "queries/s"),
                    "sweep": ("verified_rank_schedules_per_s", "rank-schedules/s"),
                    "simulate": ("simulated_block_deliveries_per_s", "blocks/s"),
                    "reduce": ("simulated_partial_results_per_s", "blocks/s")}[args.mode]
    value = units / dt
    print(json.dumps({
        "impl": "reference", "metric": metric, "value": value, "unit": unit, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
        "config": {"workload": args.mode, "sampled": True},
        "cpu_baseline": {"value": value, "unit": unit, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))
    return 0


def reference_sample(args):
    """One step of the oracle's leg for the other workloads (sized for a run of a few minutes in all):
    a function returning (units processed, unused, description of the sample)."""
    import numpy as np
    import oracle
    from paper_2407_18004_b200 import workloads
    share = max(args.steps + args.warmup, 1)
    if args.mode == "batch":
        m = max(2 ** 19 // share, 1024)
        hp, hr, ho = workloads.query_batch(m, seed=0)

        def batch_step():
            oracle.schedule_batch(hp, hr, ho, 31)
            return m, 0.0, "each step: %d queries of the seed-0 batch" % m
        return batch_step
    if args.mode == "sweep":
        lo, hi = args.sweep_lo, args.sweep_hi
        count = max(96 // share, 2)
        ps = list(range(hi, lo - 1, -(hi - lo) // count))[:count]

        def sweep_step():
            for pp in ps:
                oracle.checksum(pp)
            return sum(ps), 0.0, "each step: checksums of p in %s" % ps
        return sweep_step
    p = min(workload_of(args.workload), 2 ** 16 + 1)
    n = args.blocks
    r, s = oracle.schedule_table(p, 0)
    v = np.random.default_rng(0).integers(0, 2 ** 62, size=(n, p), dtype=np.uint64)

    def simulate_step():
        if args.mode == "simulate":
            oracle.simulate_broadcast(p, 0, n, r, s)
        else:
            oracle.simulate_reduce(p, 0, n, r, s, v)
        return (p - 1) * n, 0.0, "each step: %d blocks on p=%d processors" % (n, p)
    return simulate_step


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="p=2^27-1")
    ap.add_argument("--mode", default="broadcast",
                    choices=["broadcast", "allbroadcast", "shifted", "batch", "sweep", "simulate", "reduce"],
                    help="broadcast: tables of all ranks for one root (the default, headline workload); "
                         "allbroadcast: Algorithm 7's tables of one processor for all roots; shifted: tables with "
                         "Algorithm 1's preamble for --blocks blocks; batch: 2^24 random (p, rank, root) queries; "
                         "sweep: fused verification of every p in [2, 65536]; simulate / reduce: Algorithm 1 and "
                         "its reversal run by all processors of --workload (default p=2^20+1) with --blocks blocks")
    ap.add_argument("--blocks", type=int, default=64, help="n, the number of blocks (shifted, simulate, reduce)")
    ap.add_argument("--rounds", default="auto", choices=["auto", "launches", "fused"],
                    help="simulate / reduce: one kernel launch per communication round, or all rounds in "
                         "cooperative launches (auto: fused where the device has them)")
    ap.add_argument("--queries", type=int, default=2 ** 24, help="number of queries (batch)")
    ap.add_argument("--sweep-lo", type=int, default=2, help="first p of the sweep")
    ap.add_argument("--sweep-hi", type=int, default=65536, help="last p of the sweep")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true",
                    help="skip the other benchmark configurations that the default run measures beside the headline")
    args = ap.parse_args()
    if args.mode in OTHER_MODES:
        if args.workload == "p=2^27-1":
            args.workload = "p=2^20+1"                     # the processors that simulate / reduce run on
        return run_other(args)
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
