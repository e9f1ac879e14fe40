"""`bench.py --gpus N` started without a launcher spawns its own ranks: one process per GPU with distinct rank variables."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_gpus_flag_spawns_one_rank_per_gpu():
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "3", "--print-rank-env"],
                         env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0, out.stderr
    ranks = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(ranks) == 3
    assert sorted(r["RANK"] for r in ranks) == ["0", "1", "2"]
    assert sorted(r["LOCAL_RANK"] for r in ranks) == ["0", "1", "2"]
    assert {r["WORLD_SIZE"] for r in ranks} == {"3"}
    assert {r["MASTER_ADDR"] for r in ranks} == {"127.0.0.1"} and len({r["MASTER_PORT"] for r in ranks}) == 1


def test_launcher_environment_is_respected():
    # under torchrun the ranks already exist: nothing is spawned, the process reports the launcher's variables
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT="29999")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--print-rank-env"],
                         env=env, capture_output=True, text=True, timeout=120)
    lines = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert out.returncode == 0 and len(lines) == 1 and lines[0]["RANK"] == "1" and lines[0]["WORLD_SIZE"] == "2"
