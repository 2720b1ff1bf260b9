"""bench.py started as a plain script with --gpus N > 1 launches its own ranks; inside a rank environment it does not."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def dry_run(extra_env, *argv):
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE")}
    env.update(extra_env)
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--launch-dry-run", *argv], env=env, capture_output=True,
                         text=True, timeout=120)
    assert out.returncode == 0, out.stderr
    return json.loads(out.stdout.strip().splitlines()[-1])


def test_plain_start_with_several_gpus_becomes_the_launcher():
    r = dry_run({}, "--gpus", "8", "--steps", "5", "--warmup", "3")
    assert r["self_launch"] is True
    cmd = r["command"]
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"] and "--nproc-per-node=8" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-6:] == ["--gpus", "8", "--steps", "5", "--warmup", "3"] and cmd[-7].endswith("bench.py")
    assert "--launch-dry-run" not in cmd


def test_inside_a_rank_environment_or_on_one_gpu_it_runs_in_place():
    r = dry_run({"RANK": "3", "LOCAL_RANK": "3", "WORLD_SIZE": "8"}, "--gpus", "8")
    assert r["self_launch"] is False and r["command"] is None and r["env"]["RANK"] == "3"
    r = dry_run({}, "--gpus", "1")
    assert r["self_launch"] is False
