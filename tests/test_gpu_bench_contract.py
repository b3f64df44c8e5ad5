"""bench.py prints one JSON line with the keys its contract names; checked on small workloads so
that a change to the library or to bench.py that breaks the line shows up in the GPU test run."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

REQUIRED = ["metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
            "vs_baseline", "dtype", "data", "config", "roofline", "e2e", "gpu_launches", "clocks"]


def run_bench(*args):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True, cwd=ROOT,
                         timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, out.stdout[-2000:]
    return json.loads(lines[0])


@pytest.mark.parametrize("args,bound", [
    (["--workload", "cfg1", "--steps", "40", "--warmup", "3", "--e2e-steps", "2", "--no-cpu-baseline", "--configs", "none"], "alu"),
    (["--workload", "cfg1", "--steps", "40", "--warmup", "3", "--e2e-steps", "2", "--no-cpu-baseline", "--configs", "none",
      "--fuse-rounds", "1"], "alu"),       # short vectors: one cooperative launch runs all 40 rounds
    (["--d", "400003", "--steps", "12", "--warmup", "3", "--e2e-steps", "2", "--no-cpu-baseline"], "alu"),
    (["--d", "400003", "--steps", "6", "--warmup", "3", "--e2e-steps", "2", "--no-cpu-baseline", "--fuse-rounds", "1"], "hbm"),
    (["--d", "800003", "--steps", "8", "--warmup", "3", "--e2e-steps", "1", "--no-cpu-baseline", "--storage", "bf16"], "alu"),
])
def test_bench_line_has_the_contract_keys(args, bound):
    line = run_bench(*args)
    for key in REQUIRED:
        assert key in line, key
    assert line["metric"] == "replica GB/s" and line["unit"] == "GB/s" and line["higher_is_better"] is True
    assert line["n_gpus"] == 1 and line["value"] > 0 and line["ms_per_step"] > 0 and line["gpu_launches"] > 0
    assert line["dtype"] == ("bf16 storage, f32 arithmetic" if "bf16" in args else "f32")
    assert line["data"] == "synthetic" and line["vs_baseline"] is None
    assert "workload" in line["config"] and "model" not in line["config"]
    roof = line["roofline"]
    for key in ("bound", "achieved", "peak", "unit", "frac", "traffic"):
        assert key in roof, key
    assert roof["bound"] == bound
    e2e = line["e2e"]
    assert e2e["value"] > 0 and e2e["h2d_bytes_per_step"] > 0 and e2e["d2h_bytes_per_step"] > 0
    assert e2e["value"] < line["value"]
    assert {"sm_mhz", "sm_max_mhz", "reasons"} <= set(line["clocks"])
    if bound == "alu" and roof["kernel"] == "fused_rounds_kernel":
        assert "one_launch_per_round" in line and line["one_launch_per_round"]["roofline"]["bound"] == "hbm"
    if bound == "hbm":
        assert roof["achieved"] == pytest.approx(0.75 * roof["replica_GBs"])       # 12 of the 16 bytes per element


def test_bench_line_carries_the_other_configs():
    line = run_bench("--workload", "cfg1", "--steps", "40", "--warmup", "3", "--e2e-steps", "1", "--no-cpu-baseline",
                     "--configs", "1,5")
    assert set(line["configs"]) == {"cfg1", "cfg5"}
    for entry in line["configs"].values():
        assert entry["ms_per_round"] > 0 and entry["replica_GBs"] > 0 and entry["launch_shape"]
        assert {"bound", "achieved", "peak", "frac", "traffic"} <= set(entry["roofline"])
    assert line["configs"]["cfg5"]["M"] == 4096 and "clocks" in line["configs"]["cfg5"]


def test_async_bench_line():
    line = run_bench("--mode", "async", "--d", "400003", "--steps", "64", "--warmup", "3")
    assert line["roofline"]["kernel"] == "step_kernel" and line["value"] > 0 and line["gpu_launches"] > 0
