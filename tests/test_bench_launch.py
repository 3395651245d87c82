"""The benchmark's reference arm under a two-process launch on CPU (gloo is not even needed: the
path has no exchange step): rank 0 alone prints the JSON line, the other rank exits 0 silently."""
import json
import os
import socket
import subprocess
import sys

from conftest import ROOT


def free_port() -> str:
    """A TCP port nobody listens on right now (two test runs side by side must not meet on a fixed one)."""
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        return str(sock.getsockname()[1])


def test_reference_arm_two_processes():
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", free_port(), os.path.join(ROOT, "bench.py"),
           "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0", "--workload", "p=1000"]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=300, env=env, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, out.stdout
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["d2h_bytes_per_step"] == 0


def test_reference_arm_single_process():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0", "--workload", "p=1000", "--mode", "allbroadcast"],
                         capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == "schedule_ranks_per_s"


def test_reference_arm_other_modes():
    # the oracle's leg of the other workloads, each on a small case
    for args, metric in [(["--mode", "shifted", "--workload", "p=1000", "--blocks", "8"], "schedule_ranks_per_s"),
                         (["--mode", "simulate", "--workload", "p=1000", "--blocks", "8"], "simulated_block_deliveries_per_s"),
                         (["--mode", "reduce", "--workload", "p=1000", "--blocks", "8"], "simulated_partial_results_per_s"),
                         (["--mode", "sweep", "--sweep-hi", "300"], "verified_rank_schedules_per_s"),
                         (["--mode", "batch"], "schedule_queries_per_s")]:
        out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                              "--warmup", "0"] + args, capture_output=True, text=True, timeout=300, cwd=ROOT)
        assert out.returncode == 0, out.stderr[-2000:]
        line = json.loads(out.stdout.strip().splitlines()[-1])
        assert line["impl"] == "reference" and line["metric"] == metric and line["value"] > 0
        assert line["cpu_baseline"]["kind"] == "oracle" and line["gpu_launches"] == 0


def test_max_over_ranks_and_whole_job_value_two_gloo_ranks():
    # the replicas of a multi-GPU run are timed as the slowest rank and counted together
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", free_port(), os.path.join(ROOT, "tests", "dist_worker.py")]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=300, env=env, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, out.stdout
    line = json.loads(lines[0])
    assert line["world"] == 2 and line["total_ms"] == 15.0
    assert abs(line["value"] - 2 * 1000 * 4 / 15e-3) < 1e-6
