"""bench.py on one GPU prints one JSON line with every key the benchmark contract names, and the
figures in it are consistent with one another."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bench_prints_one_consistent_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "5", "--warmup", "3", "--no-extras"],
                         cwd=ROOT, capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    line = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "roofline", "cpu_baseline", "e2e", "gpu_launches", "clocks"):
        assert key in line, key
    assert line["unit"] == "TOPS" and line["n_gpus"] == 1 and line["steps"] == 5 and line["warmup"] == 3
    assert line["higher_is_better"] is True and line["scaling"] == "weak" and line["vs_baseline"] is None
    assert line["data"] == "synthetic" and "workload" in line["config"] and "model" not in line["config"]
    M, N, K = line["config"]["M"], line["config"]["N"], line["config"]["K"]
    assert (M, N, K) == (8192, 8192, 8192)
    # value = 2 M N K / time per step
    assert abs(line["value"] - 2 * M * N * K / (line["ms_per_step"] * 1e-3) / 1e12) < 1e-6 * line["value"]
    roof = line["roofline"]
    assert roof["bound"] == "tensor" and roof["unit"] == "TFLOP/s" and roof["peak"] > 0
    assert abs(roof["frac"] - roof["achieved"] / roof["peak"]) < 1e-9
    assert 0.3 < roof["frac"] < 1.2
    # the six FP4 GEMMs of a step cannot take longer than the step
    assert roof["achieved"] * 1e12 * line["ms_per_step"] * 1e-3 > roof["flops_per_launch"]
    assert roof["traffic"] is None or roof["traffic"] > (M * K + K * N) * 3 + M * N * 4   # at least planes + C
    cpu = line["cpu_baseline"]
    assert cpu["kind"] == "oracle" and cpu["cores"] >= 1 and cpu["value"] > 0 and cpu["sample"]
    e2e = line["e2e"]
    assert e2e["unit"] == "TOPS" and e2e["h2d_bytes_per_step"] == M * K + K * N and e2e["d2h_bytes_per_step"] == 4 * M * N
    assert 0 < e2e["value"] < line["value"]
    assert line["gpu_launches"] >= 3 * line["steps"]
    clocks = line["clocks"]
    assert clocks["sm_max_mhz"] >= clocks["sm_mhz"] > 0 and isinstance(clocks["reasons"], list)
