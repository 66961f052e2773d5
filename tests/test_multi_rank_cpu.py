"""World-size-2 (and 3) CPU test of the multi-GPU host logic over gloo: the env-range partition,
the totals all-reduce and the max-over-ranks timing reduction. The per-rank compute is the CPU
oracle standing in for a GPU's shard (tests may call it); the checks are that shards compose to
the single-process result and that no other exchange is needed."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

N, T, SEED = 1000, 60, 5


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, weak, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import cartpole_oracle as oracle
        from paper_2301_13062_b200 import sharding
        if weak:
            lo = sharding.weak_env_offset(N)
            hi = lo + N
        else:
            lo, hi = sharding.rank_env_range(N)
        r = oracle.rollout(hi - lo, T, SEED, env_offset=lo)
        totals = torch.from_numpy(r["totals"].view(np.int64).copy())
        sharding.reduce_totals(totals)
        slowest = sharding.max_over_ranks(float(rank + 1))
        np.savez(os.path.join(out_dir, f"rank{rank}.npz"), lo=lo, hi=hi, ret=r["ep_return_sum"],
                 cnt=r["ep_count"], totals=totals.numpy(), slowest=slowest)
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world,weak", [(2, False), (3, False), (2, True)])
def test_shards_compose_over_gloo(tmp_path, oracle, world, weak):
    port = _free_port()
    mp.start_processes(_worker, args=(world, port, weak, str(tmp_path)), nprocs=world, join=True, start_method="spawn")
    total_envs = N * world if weak else N
    whole = oracle.rollout(total_envs, T, SEED)
    covered = 0
    for rank in range(world):
        d = np.load(tmp_path / f"rank{rank}.npz")
        lo, hi = int(d["lo"]), int(d["hi"])
        assert np.array_equal(d["ret"], whole["ep_return_sum"][lo:hi])
        assert np.array_equal(d["cnt"], whole["ep_count"][lo:hi])
        assert np.array_equal(d["totals"].view(np.uint64), whole["totals"])  # every rank holds the global sum
        assert float(d["slowest"]) == float(world)
        covered += hi - lo
    assert covered == total_envs


def test_partition_properties():
    from paper_2301_13062_b200.inputs import shard_range
    for n in (1, 31, 32, 33, 1000, 1 << 20, (1 << 20) + 5):
        for world in (1, 2, 3, 8):
            ranges = [shard_range(n, r, world) for r in range(world)]
            assert ranges[0][0] == 0 and ranges[-1][1] == n
            for (a, b), (c, d) in zip(ranges, ranges[1:]):
                assert b == c and a <= b
            assert all(lo % 32 == 0 or lo == n for lo, _ in ranges)  # a done-bit word never spans two ranks
