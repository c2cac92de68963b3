"""bench.py's multi-rank entry on CPUs: `--gpus 2 --backend gloo --dry` must start two ranks by itself, run the
one exchange of the method (the average of the per-rank replica means, Eq. parle_x) between them, time it between
barriers as the max over ranks, and print exactly one JSON line, from rank 0, that says n_gpus = 2."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(extra, env=None):
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--backend", "gloo", "--dry", "--steps", "3"] + extra
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=300, env=env)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.strip().startswith("{")]
    assert len(lines) == 1, res.stdout
    return json.loads(lines[0])


def test_bench_starts_its_own_ranks_and_prints_one_line():
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    line = _run(["--gpus", "2"], env)
    assert line["n_gpus"] == 2 and line["dry"] is True and line["steps"] == 3
    assert line["exchanged_mean"] == 1.5                 # ranks hold 1 and 2: the mean of the per-rank means
    assert line["ms_per_step"] > 0 and line["scaling"] == "weak"


def test_bench_single_rank_dry_line():
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    line = _run(["--gpus", "1"], env)
    assert line["n_gpus"] == 1 and line["exchanged_mean"] == 1.0
