"""Host logic of `bench.py --gpus N` (no GPU needed): how the flag is honoured with and without a
launcher, and that a contradiction between the flag and the launcher's world size is an error."""
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_launch_plan():
    import bench
    assert bench.launch_plan(1, {}, ["--steps", "3"]) == ("run", None)
    # started by torch.distributed.run: this process is one of the ranks
    assert bench.launch_plan(8, {"WORLD_SIZE": "8", "RANK": "3"}, []) == ("run", None)
    # --gpus N without a launcher: N local ranks, one per GPU, over 127.0.0.1
    kind, cmd = bench.launch_plan(4, {}, ["--gpus", "4", "--steps", "3"], port=29123)
    assert kind == "spawn"
    assert cmd[:3] == [sys.executable, "-m", "torch.distributed.run"]
    assert "--nproc-per-node=4" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[cmd.index("--master-port") + 1] == "29123"
    assert cmd[-5:] == [os.path.join(ROOT, "bench.py"), "--gpus", "4", "--steps", "3"]
    # the printed n_gpus must equal --gpus: a launcher with another world size is refused
    assert bench.launch_plan(2, {"WORLD_SIZE": "4"}, [])[0] == "error"
    assert bench.launch_plan(0, {}, [])[0] == "error"


def test_contradicting_world_size_exits_nonzero():
    env = dict(os.environ, WORLD_SIZE="3", RANK="0", LOCAL_RANK="0")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2"], env=env, capture_output=True,
                       text=True, timeout=120)
    assert r.returncode == 2 and "must agree" in r.stderr and r.stdout.strip() == ""


def test_strong_and_weak_ranges_cover_the_job():
    from paper_2301_13062_b200 import sharding
    n = 1_048_576
    for world in (1, 2, 3, 8):
        strong = [sharding.rank_env_range(n, r, world) for r in range(world)]
        assert strong[0][0] == 0 and strong[-1][1] == n and all(a[1] == b[0] for a, b in zip(strong, strong[1:]))
        weak = [sharding.weak_env_offset(n, r) for r in range(world)]
        assert weak == [r * n for r in range(world)]
