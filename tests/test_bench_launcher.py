"""`python bench.py --gpus N` has to start its N ranks by itself (one process per GPU) and print
exactly one JSON line from rank 0.  Checked here without GPUs: --launcher-check makes every rank
join a gloo group instead of running the step."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(extra, env=None):
    e = dict(os.environ)
    for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT"):
        e.pop(k, None)
    e.update(env or {})
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--launcher-check", "--workload", "tiny",
                        "--steps", "2", "--warmup", "1"] + extra, capture_output=True, text=True, timeout=300, env=e)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, r.stdout
    return json.loads(lines[0])


def test_gpus_2_starts_two_ranks_and_prints_one_line():
    line = _run(["--gpus", "2"])
    assert line["n_gpus"] == 2 and line["launcher_check"] is True and line["value"] is None
    assert line["config"]["parallelism"] == "dp2"
    one = _run(["--gpus", "1"])
    assert one["n_gpus"] == 1
    # weak scaling: every rank brings its own batch
    assert line["config"]["tokens_all_ranks"] > 1.5 * one["config"]["tokens_all_ranks"]
