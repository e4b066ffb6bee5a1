"""The benchmark's output contract, checked on a small workload: one JSON line with the agreed
keys, a kernel-launch count that matches the steps, copies counted in the end-to-end figure."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*args):
    res = subprocess.run([sys.executable, "bench.py", *args], cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [x for x in res.stdout.splitlines() if x.strip().startswith("{")]
    assert len(lines) == 1, "exactly one JSON line on stdout"
    return json.loads(lines[0])


def test_bench_line_has_the_agreed_keys(cuda_device):
    d = _run("--workload", "resnet56", "--steps", "40", "--warmup", "3", "--cpu-sample", "200000")
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "clocks", "e2e", "gpu_launches", "roofline", "cpu_baseline"):
        assert key in d, key
    assert d["unit"] == "GB/s" and d["n_gpus"] == 1 and d["steps"] == 40 and d["warmup"] == 3
    assert d["higher_is_better"] is True and d["scaling"] == "weak" and d["vs_baseline"] is None
    assert d["dtype"] == "f32" and d["data"] == "synthetic" and "workload" in d["config"]
    assert d["gpu_launches"] == 40, "one kernel launch per timed step"
    assert d["value"] > 0 and abs(d["value"] - d["config"]["bytes_per_step"] / d["ms_per_step"] / 1e6) < 1e-6 * d["value"]
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] > 0 and r["achieved"] > 0
    assert r["frac"] is None and r["traffic"] is None, "a cache-resident set carries no HBM fraction"
    e = d["e2e"]
    P4 = 4 * (d["config"]["n_params"] + 0)  # arena padding makes the copies a little larger
    assert e["unit"] == "GB/s" and e["h2d_bytes_per_step"] >= d["config"]["n_workers"] * P4 and e["d2h_bytes_per_step"] >= P4
    assert 0 < e["value"] < d["value"], "the end-to-end figure includes the copies"
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] == 1 and c["unit"] == "GB/s" and c["value"] > 0 and c["sample"]
    assert set(d["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}


def test_reference_arm_line(cuda_device):
    d = _run("--impl", "reference", "--workload", "lenet5", "--steps", "3", "--warmup", "1", "--cpu-sample", "100000")
    assert d["impl"] == "reference" and d["gpu_launches"] == 0 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"] == {"value": d["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
