"""The benchmark's multi-rank bookkeeping on CPU: two gloo ranks, replicas of one workload.

The path does not shard (one GPU, no data-path collective); `bench.py --gpus N` runs N independent
replicas and only the timing is reduced over ranks.  This checks that reduction: the slowest rank sets
the time and the whole-job value counts every rank's timesteps.
"""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    # rank r "measured" (r + 1) * 10 ms for 100 steps of 1000 timesteps
    times, value = bench.aggregate_over_ranks([10.0 * (rank + 1), 5.0 - rank], 100, 1000, world, dist)
    dist.barrier()
    out.put((rank, times, value))
    dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_two_gloo_ranks_take_the_slowest_time_and_sum_the_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=100) for _ in procs)
    for p in procs:
        p.join(30)
        assert p.exitcode == 0
    for rank, times, value in results:
        assert times == [20.0, 5.0]            # MAX over ranks, element by element
        assert value == pytest.approx(2 * 100 * 1000 / 20.0e-3)


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    times, value = bench.aggregate_over_ranks([4.0], 10, 50, 1)
    assert times == [4.0] and value == pytest.approx(10 * 50 / 4.0e-3)
