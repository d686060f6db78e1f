"""bench.py prints one JSON line with the keys its contract names (run on the tiny workload)."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*flags):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *flags], capture_output=True, text=True,
                         timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    return json.loads(lines[0])


def test_default_arm_line():
    r = _run("--workload", "tiny", "--steps", "4", "--warmup", "3")
    for k in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
              "vs_baseline", "dtype", "data", "config", "gpu_launches", "roofline", "e2e", "clocks", "cpu_baseline"):
        assert k in r, k
    assert r["n_gpus"] == 1 and r["steps"] == 4 and r["warmup"] == 3 and r["value"] > 0
    assert r["config"]["workload"] == "tiny" and r["vs_baseline"] is None and r["data"] == "synthetic"
    assert r["gpu_launches"] > 0
    rf = r["roofline"]
    assert rf["bound"] == "tensor" and rf["unit"] == "TFLOP/s" and rf["peak"] > 0
    assert abs(rf["frac"] - rf["achieved"] / rf["peak"]) < 1e-9
    e = r["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] == 4
    c = r["cpu_baseline"]
    assert c["kind"] == "oracle" and c["value"] > 0 and c["cores"] >= 1 and "tokens" in c["sample"]


def test_reference_arm_line():
    r = _run("--workload", "tiny", "--impl", "reference", "--steps", "2", "--warmup", "1")
    assert r["impl"] == "reference" and r["dtype"] == "f64" and r["value"] > 0
    assert r["cpu_baseline"]["kind"] == "oracle" and r["cpu_baseline"]["value"] == r["value"]
    assert r["e2e"] == dict(value=r["value"], unit=r["unit"], h2d_bytes_per_step=0, d2h_bytes_per_step=0)


def test_memory_bound_line():
    r = _run("--workload", "stress_grouped", "--steps", "3", "--warmup", "3")
    assert r["roofline"]["bound"] == "hbm" and r["unit"] == "GB/s" and r["value"] > 0
    assert r["config"]["candidate_order"].startswith("rollout order")
    assert r["loss_reduction"]["gbs"] > 0
