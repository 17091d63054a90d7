"""bench.py's reference arm (the CPU oracle on a bounded sample) prints one JSON line with the agreed keys."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_the_contract_line():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "0", "--steps", "2", "--warmup", "1"],
                       capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    lines = [ln for ln in r.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"):
        assert key in d, key
    assert d["impl"] == "reference" and d["unit"] == "samples/s" and d["value"] > 0 and d["vs_baseline"] is None
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1 and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert "workload" in d["config"] and "model" not in d["config"]


import pytest


@pytest.mark.gpu
def test_own_arm_prints_the_contract_line_with_roofline_objects():
    """The ResNet-18-shaped workload at a reduced per-worker batch: the line carries every agreed key, the kernel passes
    ran (roofline of the dominant class at the timed grid size and with grids for the whole device) and the step entry."""
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--batch", "16", "--steps", "3", "--warmup", "3", "--no-cpu-baseline"],
                       capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling", "vs_baseline",
                "dtype", "data", "config", "clocks", "roofline", "e2e", "gpu_launches", "kernels"):
        assert key in d, key
    assert d["unit"] == "samples/s" and d["value"] > 0 and d["vs_baseline"] is None and d["dtype"] == "bf16" and d["steps"] == 3
    assert d["gpu_launches"] > 0 and d["e2e"]["value"] > 0 and d["e2e"]["h2d_bytes_per_step"] > 0 and d["e2e"]["d2h_bytes_per_step"] == 4
    assert "workload" in d["config"] and "model" not in d["config"] and d["config"]["grid_sms"] >= 1
    roof = d["roofline"]
    for key in ("bound", "achieved", "peak", "unit", "frac", "traffic", "kernel", "grid_sms", "avg_launch_ms", "launches_per_step", "step"):
        assert key in roof, key
    assert roof["bound"] in ("tensor", "hbm", "alu") and abs(roof["frac"] - roof["achieved"] / roof["peak"]) < 1e-9
    assert roof["grid_sms"] == d["config"]["grid_sms"]
    assert roof["avg_launch_ms"] * roof["launches_per_step"] <= d["ms_per_step"] * 3          # a class alone on a third of the SMs
    if roof["grid_sms"] != roof["device_sms"]:
        assert roof["all_sms"]["grid_sms"] == roof["device_sms"] and roof["all_sms"]["achieved"] > 0
    step = roof["step"]
    assert abs(step["frac"] - step["achieved"] / step["peak"]) < 1e-9 and abs(step["ms_per_step"] - d["ms_per_step"]) < 1e-9
