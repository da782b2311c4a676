"""`bench.py --gpus N` outside a torchrun environment starts its N ranks itself (one process per GPU
through torch.distributed.run on 127.0.0.1).  Checked here on CPU with the oracle arm of the small
configuration: two ranks start, rank 0 alone prints the one JSON line, the other exits 0 without work."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_gpus_flag_spawns_the_ranks():
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference", "--workload", "c1",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [json.loads(x) for x in res.stdout.splitlines() if x.startswith("{")]
    assert len(lines) == 1, res.stdout
    assert lines[0]["impl"] == "reference" and lines[0]["n_gpus"] == 2 and lines[0]["config"]["workload"].startswith("c1")


def test_rank_env_is_respected_without_spawning():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference", "--workload", "c1",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=600)
    assert res.returncode == 0 and res.stdout.strip() == ""        # ranks other than 0 print nothing
