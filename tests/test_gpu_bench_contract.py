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
    d = run_bench("--workload", "c2", "--also", "c1", "--steps", "5", "--warmup", "3", "--e2e-steps", "1", "--cpu-requests", "2")
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "roofline", "roofline_softmax_topk", "kernel_ms", "other_workloads",
                "e2e", "cpu_baseline", "gpu_launches", "clocks"):
        assert key in d, key
    assert d["unit"] == "rounds/s" and d["n_gpus"] == 1 and d["steps"] == 5 and d["higher_is_better"] is True
    assert d["vs_baseline"] is None and d["data"] == "synthetic" and d["dtype"] == "bf16"
    assert "workload" in d["config"] and "model" not in d["config"]
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] > 0 and r["traffic"] >= r["algorithmic_bytes"]
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-3 and 0.3 < r["frac"] < 1.5
    # the dominant kernel's block is that kernel alone: its bytes over its own CUDA-event time
    assert r["kernel"] == "row_argmax" and abs(r["achieved"] - r["algorithmic_bytes"] / (r["ms"] * 1e-3) / 1e9) < 0.01 * r["achieved"]
    t = d["roofline_softmax_topk"]
    assert t["kernel"] == "softmax_topk_partial" and t["bound"] == "hbm" and t["algorithmic_bytes"] == 32 * 16 * 151936 * 2
    assert abs(t["frac"] - t["achieved"] / t["peak"]) < 1e-3 and 0.1 < t["frac"] < 1.5
    km = d["kernel_ms"]
    assert all(km[k] > 0 for k in ("softmax_topk_partial", "expand_emit", "row_argmax", "accept_walk"))
    assert "c1" in d["other_workloads"] and d["other_workloads"]["c1"]["value"] > 0
    assert set(d["config"]) == {"workload", "l2", "parallelism"}
    assert d["value"] > 0 and d["gpu_launches"] == 4 * 5
    assert d["e2e"]["h2d_bytes_per_step"] > 2.6e9 and d["e2e"]["d2h_bytes_per_step"] > 0 and 0 < d["e2e"]["value"] < d["value"]
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] >= 1 and c["value"] > 0 and c["trees_match_gpu"] is True
    assert c["single_thread_value"] > 0 and c["requests_differing_from_gpu"] == 0
    assert d["clocks"]["sm_max_mhz"] is None or d["clocks"]["sm_mhz"] <= d["clocks"]["sm_max_mhz"]


def test_reference_arm_line():
    d = run_bench("--impl", "reference", "--workload", "c2", "--steps", "1", "--warmup", "0", "--cpu-requests", "2")
    assert d["impl"] == "reference" and d["unit"] == "rounds/s" and d["value"] > 0
    assert set(d["config"]) == {"workload", "l2", "parallelism"}
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0 and d["e2e"]["value"] == d["value"]
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"]


def test_smoke_entry_point():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "__graft_entry__.py"), "--smoke"], capture_output=True,
                         text=True, timeout=900, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    assert "smoke ok" in out.stdout
