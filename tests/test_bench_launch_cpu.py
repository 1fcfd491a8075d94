"""`bench.py --gpus N` outside a launcher starts N ranks by itself.  Checked
here without a GPU: the launched ranks join a gloo group on the CPU, count
themselves with an all-reduce and rank 0 prints the count."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402


def _clean_env():
    env = dict(os.environ)
    for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT", "TORCHELASTIC_RUN_ID"):
        env.pop(k, None)
    return env


def test_gpus_2_starts_two_ranks():
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-spawn"],
                       capture_output=True, text=True, timeout=300, env=_clean_env())
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [l for l in p.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, p.stdout                      # rank 0 alone prints
    rec = json.loads(lines[0])
    assert rec["spawned_ranks"] == 2 and rec["world_size"] == 2


def test_launch_command_and_rank_environment():
    cmd = bench.spawn_command(4, ["--gpus", "4", "--steps", "20"])
    assert "--nproc-per-node=4" in cmd and "--master-addr" in cmd and cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-4:] == ["--gpus", "4", "--steps", "20"]
    # already under a launcher (WORLD_SIZE set), a single GPU, or the CPU arm: no second launcher
    args = bench.parse_args(["--gpus", "4"])
    old = os.environ.get("WORLD_SIZE")
    os.environ["WORLD_SIZE"] = "4"
    try:
        assert bench.maybe_spawn(args, ["--gpus", "4"]) is False
    finally:
        if old is None:
            del os.environ["WORLD_SIZE"]
        else:
            os.environ["WORLD_SIZE"] = old
    assert bench.maybe_spawn(bench.parse_args(["--gpus", "1"]), []) is False
    assert bench.maybe_spawn(bench.parse_args(["--gpus", "4", "--impl", "reference"]), []) is False


def test_rotation_period_divides_the_region():
    # 128 MiB per copy: 9 copies reach 1 GiB; a 20-step region rotates over 10 so that regions chain
    copies, closed = bench.pick_copies(128 << 20, 20)
    assert copies == 10 and closed
    copies, closed = bench.pick_copies(128 << 20, 2048)
    assert 2048 % copies == 0 and closed and copies * (128 << 20) >= (1 << 30)
    copies, closed = bench.pick_copies(2 << 30, 7)        # no divisor in reach: the caller flushes L2 instead
    assert copies == 2 and not closed
