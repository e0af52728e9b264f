"""`bench.py --gpus N` starts N ranks itself (one process per GPU) when no launcher did: checked on CPU with the
dry-run mode, in which every rank joins a gloo group and rank 0 reports the ranks that arrived."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(args, env=None):
    e = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    e.update(env or {})
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + args, env=e, capture_output=True, text=True,
                          timeout=300)


def test_gpus_2_starts_two_distinct_ranks():
    r = _run(["--gpus", "2", "--dry-run-ranks"])
    assert r.returncode == 0, r.stderr[-2000:]
    line = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(line) == 1, r.stdout                      # rank 0 alone prints
    rec = json.loads(line[0])
    assert rec["dry_run"] and rec["n_gpus"] == 2 and rec["ranks"] == [0, 1]


def test_row_sharded_mode_reaches_the_ranks_too():
    r = _run(["--gpus", "2", "--shard-rows", "--workload", "C1", "--dry-run-ranks"])
    assert r.returncode == 0, r.stderr[-2000:]
    rec = json.loads([l for l in r.stdout.splitlines() if l.startswith("{")][0])
    assert rec["ranks"] == [0, 1] and rec["shard_rows"] and rec["workload"] == "C1"


def test_world_size_must_match_gpus():
    r = _run(["--gpus", "3", "--dry-run-ranks"], env={"WORLD_SIZE": "2", "RANK": "0", "LOCAL_RANK": "0"})
    assert r.returncode != 0 and "WORLD_SIZE=2" in (r.stderr + r.stdout)


def test_single_process_default():
    r = _run(["--dry-run-ranks"])
    assert r.returncode == 0
    assert json.loads(r.stdout.strip().splitlines()[-1])["ranks"] == [0]
