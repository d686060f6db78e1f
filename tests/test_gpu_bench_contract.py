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
    # the roofline is the whole step's: algorithmic 6*T*V*d over forward + backward time
    ph = r["phases_ms"]
    T, d, V = r["config"]["tokens_per_gpu"], r["config"]["d"], r["config"]["V"]
    want = 6.0 * T * V * d / ((ph["forward"] + ph["backward"]) * 1e-3) / 1e12
    assert abs(rf["achieved"] - want) <= 1e-6 * want and "all launches" in rf["kernel"]
    # by default the forward keeps the logits: the tensor cores execute T + 2*routed row passes, at most the algorithmic 3*T
    assert r["config"]["logits"].startswith("kept")
    assert 0 < rf["routed_rows"] <= T
    assert abs(rf["executed_frac"] / rf["frac"] - (T + 2.0 * rf["routed_rows"]) / (3.0 * T)) < 1e-6
    assert rf["frac_of_nominal_2250"] < rf["frac"] and rf["forward_frac"] > 0 and rf["backward_algorithmic_frac"] > 0
    assert rf["algorithmic_bytes"] == rf["algorithmic_bytes_forward"] + rf["algorithmic_bytes_backward"]
    assert rf["traffic"] is None or rf["traffic"] == rf["traffic_forward"] + rf["traffic_backward"]
    # the same line also carries the step with the logits recomputed (no [T, V] buffer) and kept the other way
    others = r["other_logits_modes"]
    assert set(others) == {"note", "recompute", "keep16" if r["config"]["logits"].startswith("kept: the forward stores [T, V] fp32") else "keep"}
    alt = others["recompute"]
    assert alt["value"] > 0 and alt["ms_per_step"] > 0 and alt["frac"] > 0 and alt["logits"].startswith("recomputed")
    assert abs(alt["executed_frac"] / alt["frac"] - (T + 3.0 * rf["routed_rows"]) / (3.0 * T)) < 1e-6
    e = r["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] == 4
    c = r["cpu_baseline"]
    assert c["kind"] == "oracle" and c["value"] > 0 and c["cores"] >= 1 and "tokens" in c["sample"]


def test_recompute_arm_line():
    # --logits recompute: no [T, V] buffer, the backward repeats the contraction on the routed rows
    r = _run("--workload", "tiny", "--steps", "3", "--warmup", "3", "--logits", "recompute", "--no-cpu-baseline")
    rf, T = r["roofline"], r["config"]["tokens_per_gpu"]
    assert r["config"]["logits"].startswith("recomputed") and r["value"] > 0
    assert set(r["other_logits_modes"]) == {"note", "keep", "keep16"}
    assert abs(rf["executed_frac"] / rf["frac"] - (T + 3.0 * rf["routed_rows"]) / (3.0 * T)) < 1e-6


def test_reference_arm_line():
    r = _run("--workload", "tiny", "--impl", "reference", "--steps", "2", "--warmup", "1")
    assert r["impl"] == "reference" and r["dtype"] == "f64" and r["value"] > 0 and r["n_gpus"] == 1
    assert r["cpu_baseline"]["kind"] == "oracle" and r["cpu_baseline"]["value"] == r["value"]
    assert r["e2e"] == dict(value=r["value"], unit=r["unit"], h2d_bytes_per_step=0, d2h_bytes_per_step=0)


def test_memory_bound_line():
    r = _run("--workload", "stress_grouped", "--steps", "3", "--warmup", "3")
    assert r["roofline"]["bound"] == "hbm" and r["unit"] == "GB/s" and r["value"] > 0
    assert r["config"]["candidate_order"].startswith("rollout order")
    assert r["loss_reduction"]["gbs"] > 0


def test_update_step_line():
    # one whole policy update at the paper's batch scale: two long-response micro-batches accumulated
    # into one dW, gradient norm, clipped AdamW
    r = _run("--workload", "batch128", "--steps", "1", "--warmup", "3")
    assert r["config"]["workload"] == "batch128" and r["config"]["responses"] == 128
    assert r["config"]["tokens"] > 100_000 and len(r["config"]["micro_batches"]) == 2
    assert r["value"] > 0 and r["phases_ms"]["gradient"] > r["phases_ms"]["optimizer"] > 0
    rf = r["roofline"]
    assert r["config"]["logits"].startswith("kept")
    assert rf["bound"] == "tensor" and 0 < rf["executed_frac"] <= rf["frac"] and rf["optimizer_gbs"] > 0
