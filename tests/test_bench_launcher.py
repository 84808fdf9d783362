"""`python bench.py --gpus N` must itself start N ranks when it is not already running under torchrun.

Runs the launcher path on CPU (gloo, world size 2) with `--bootstrap-only`: ranks are spawned over 127.0.0.1, meet at a
barrier, reduce a stand-in elapsed time with MAX, and rank 0 prints the line.  No kernels are involved.
"""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(extra_args, extra_env=None):
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    env["CUDA_VISIBLE_DEVICES"] = ""                   # the CPU path (gloo), whatever the box has
    env.update(extra_env or {})
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + extra_args, env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, out.stdout                 # exactly one JSON line, from rank 0
    return json.loads(lines[0])


def test_gpus_2_starts_two_ranks_and_takes_the_max_over_them():
    line = _run(["--gpus", "2", "--bootstrap-only"])
    assert line["n_gpus"] == 2 and line["backend"] == "gloo"
    assert line["max_over_ranks"] == 2.0               # rank r contributes r + 1


def test_single_rank_needs_no_launcher():
    line = _run(["--gpus", "1", "--bootstrap-only"])
    assert line["n_gpus"] == 1 and line["backend"] is None
