"""bench.py --gpus N must run N ranks: started by a launcher, or by itself when there is none (CPU, gloo)."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(extra_env=None, args=()):
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    env.update(extra_env or {})
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], env=env, capture_output=True,
                         text=True, timeout=300)
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    return res, lines


def test_gpus_2_without_a_launcher_starts_two_ranks_and_takes_the_slowest():
    res, lines = _run(args=("--gpus", "2", "--backend", "gloo"))
    assert res.returncode == 0, res.stderr[-2000:]
    assert len(lines) == 1, res.stdout                      # rank 0 alone prints
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2
    # rank r works for (r + 1) * 10 ms: the reported time is the slowest rank's, not rank 0's own
    assert line["max_elapsed_s"] >= 0.02 > line["own_elapsed_s"]


def test_a_rank_count_that_contradicts_the_launcher_is_refused():
    env = {"WORLD_SIZE": "1", "RANK": "0", "LOCAL_RANK": "0"}
    res, _ = _run(env, args=("--gpus", "2", "--skip-cpu", "--skip-e2e"))
    assert res.returncode != 0
    assert "rank" in (res.stderr + res.stdout).lower() or "cuda" in (res.stderr + res.stdout).lower()
