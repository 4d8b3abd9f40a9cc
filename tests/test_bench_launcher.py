"""`bench.py --gpus N` starts N ranks itself (one process per GPU); checked here without a GPU: two gloo
ranks whose 'step' is a sleep of known, rank-dependent length."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(extra, env=None):
    e = dict(os.environ)
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT"):
        e.pop(k, None)
    e.update(env or {})
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + extra, env=e, capture_output=True,
                          text=True, timeout=300)


def test_plain_start_with_two_gpus_launches_two_ranks_and_reports_the_slowest():
    r = _run(["--gpus", "2", "--steps", "5", "--warmup", "1", "--stub-step-ms", "20"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, r.stdout            # rank 0 alone prints
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["steps"] == 5
    # rank 0 sleeps 20 ms per step, rank 1 40 ms: the reported time is the maximum over the ranks
    assert 39.0 <= d["ms_per_step"] <= 60.0, d


def test_one_rank_needs_no_process_group():
    r = _run(["--gpus", "1", "--steps", "3", "--warmup", "1", "--stub-step-ms", "10"])
    assert r.returncode == 0, r.stderr[-2000:]
    d = json.loads([ln for ln in r.stdout.splitlines() if ln.startswith("{")][0])
    assert d["n_gpus"] == 1 and 9.0 <= d["ms_per_step"] <= 25.0


def test_gpus_flag_must_match_an_outer_launcher():
    r = _run(["--gpus", "4", "--stub-step-ms", "1"], env={"WORLD_SIZE": "2", "RANK": "0", "LOCAL_RANK": "0"})
    assert r.returncode != 0 and "does not match" in (r.stderr + r.stdout)
