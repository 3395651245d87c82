"""The benchmark's JSON line on a GPU: one short run of the default workload's code path on a smaller p, and the
keys every consumer of the line relies on."""
import json
import os
import subprocess
import sys

import pytest

from conftest import ROOT

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")


def run_bench(*args):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True,
                         timeout=900, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, out.stdout
    return json.loads(lines[0])


def test_default_mode_line_on_a_small_p():
    line = run_bench("--workload", "4194303", "--steps", "5", "--warmup", "3", "--no-configs")
    assert line["metric"] == "schedule_ranks_per_s" and line["unit"] == "ranks/s" and line["higher_is_better"]
    assert line["n_gpus"] == 1 and line["steps"] == 5 and line["warmup"] >= 3 and line["data"] == "synthetic"
    assert line["value"] > 0 and line["ms_per_step"] > 0 and line["gpu_launches"] == 5
    assert "workload" in line["config"] and line["vs_baseline"] is None
    roof = line["roofline"]
    assert roof["bound"] == "hbm" and roof["unit"] == "GB/s" and roof["kernel"] == "schedule_table_kernel"
    assert abs(roof["frac"] - roof["achieved"] / roof["peak"]) < 1e-9
    assert abs(roof["achieved"] - roof["bytes_per_launch"] / (line["ms_per_step"] * 1e-3) / 1e9) < 0.05 * roof["achieved"]
    cpu = line["cpu_baseline"]
    assert cpu["kind"] == "oracle" and cpu["value"] > 0 and cpu["cores"] == 1 and cpu["sample"]
    e2e = line["e2e"]
    assert e2e["value"] > 0 and e2e["d2h_bytes_per_step"] == roof["bytes_per_launch"] and e2e["value"] < line["value"]
    clocks = line["clocks"]
    assert clocks["sm_max_mhz"] >= clocks["sm_mhz"] > 0 and isinstance(clocks["reasons"], list)


def test_simulate_mode_line():
    line = run_bench("--mode", "simulate", "--workload", "70001", "--blocks", "16", "--steps", "3", "--warmup", "3")
    assert line["metric"] == "simulated_block_deliveries_per_s" and line["value"] > 0
    assert line["stats"] == [0, 0, 0, 0, 0, 0, 70000 * 16, 16 - 1 + 17]
    assert line["roofline"]["bound"] == "hbm" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["gpu_launches"] > 0
