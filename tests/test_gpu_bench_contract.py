"""bench.py and the smoke entry point on a real GPU: the JSON line carries every key of the measurement
contract, for the CUDA arm and for the reference (oracle) arm."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run_bench(*extra):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *extra], capture_output=True, text=True,
                         timeout=900, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    return json.loads(out.stdout.strip().splitlines()[-1])


def test_bench_line_contract():
    d = run_bench("--steps", "5", "--warmup", "3", "--e2e-steps", "1", "--cpu-requests", "2")
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "roofline", "e2e", "cpu_baseline", "gpu_launches", "clocks"):
        assert key in d, key
    assert d["unit"] == "rounds/s" and d["n_gpus"] == 1 and d["steps"] == 5 and d["higher_is_better"] is True
    assert d["vs_baseline"] is None and d["data"] == "synthetic" and d["dtype"] == "bf16"
    assert "workload" in d["config"] and "model" not in d["config"]
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] > 0 and r["traffic"] >= r["algorithmic_bytes"]
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-3 and 0.3 < r["frac"] < 1.5
    assert d["value"] > 0 and d["gpu_launches"] == 4 * 5
    assert d["e2e"]["h2d_bytes_per_step"] > 2.6e9 and d["e2e"]["d2h_bytes_per_step"] > 0 and 0 < d["e2e"]["value"] < d["value"]
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] >= 1 and c["value"] > 0 and c["trees_match_gpu"] is True
    assert d["clocks"]["sm_max_mhz"] is None or d["clocks"]["sm_mhz"] <= d["clocks"]["sm_max_mhz"]


def test_reference_arm_line():
    d = run_bench("--impl", "reference", "--steps", "1", "--warmup", "0", "--cpu-requests", "2")
    assert d["impl"] == "reference" and d["unit"] == "rounds/s" and d["value"] > 0
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0 and d["e2e"]["value"] == d["value"]
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"]


def test_smoke_entry_point():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "__graft_entry__.py"), "--smoke"], capture_output=True,
                         text=True, timeout=900, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    assert "smoke ok" in out.stdout
