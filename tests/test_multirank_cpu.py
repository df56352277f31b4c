"""Multi-rank bookkeeping on CPU, two gloo ranks.

`bench.py --gpus N` runs N independent replicas of one workload and only the timing is reduced over
ranks: the slowest rank sets the time and the whole-job value counts every rank's timesteps.  The
data-parallel form of the loss (one batch split over ranks) needs contiguous shares and one sum of the
eight loss terms; its host logic is checked here with the oracle standing in for each rank's kernel.
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


def _shard_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import numpy as np
    import impact_inputs as ii
    import oracle
    from paper_1912_00167_b200.sharded import reduce_loss_terms, shard_bounds
    B, T, A = 7, 20, 6
    batch = ii.categorical_batch(B, T, A, seed=5)
    h = ii.LossHyper(clip_eps=0.3, kl_coef=0.1)
    lo, hi = shard_bounds(B, world, rank)
    mine = {k: np.ascontiguousarray(v[lo:hi]) for k, v in batch.items()}
    ref = oracle.loss_categorical(mine, h)
    # the oracle normalises by the share's own steps; the library would have been given the whole batch's M
    share = (hi - lo) * T / (B * T)
    terms = torch.from_numpy(ref["loss_terms"] * share)
    reduce_loss_terms(terms)
    out.put((rank, (lo, hi), terms.numpy().tolist(), (ref["dlogits"] * share).tolist()))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.timeout(180)
def test_two_gloo_ranks_share_a_batch_and_sum_their_loss_terms():
    """The host logic of the data-parallel form: contiguous shares, and one sum of eight numbers."""
    import numpy as np
    sys.path.insert(0, ROOT)
    import impact_inputs as ii
    import oracle
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 31500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_shard_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=150) for _ in procs)
    for p in procs:
        p.join(30)
        assert p.exitcode == 0
    B, T, A = 7, 20, 6
    batch = ii.categorical_batch(B, T, A, seed=5)
    whole = oracle.loss_categorical(batch, ii.LossHyper(clip_eps=0.3, kl_coef=0.1))
    assert [r[1] for r in results] == [(0, 4), (4, 7)]
    for _, _, terms, _ in results:
        np.testing.assert_allclose(terms, whole["loss_terms"], rtol=1e-12, atol=1e-14)
    dz = np.concatenate([np.asarray(r[3]) for r in results])
    np.testing.assert_allclose(dz, whole["dlogits"], rtol=1e-12, atol=1e-16)


def test_shard_bounds_cover_the_batch_once():
    sys.path.insert(0, ROOT)
    from paper_1912_00167_b200.sharded import shard_bounds
    for B in (0, 1, 7, 8, 1024):
        for world in (1, 2, 3, 8):
            spans = [shard_bounds(B, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == B
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    times, value = bench.aggregate_over_ranks([4.0], 10, 50, 1)
    assert times == [4.0] and value == pytest.approx(10 * 50 / 4.0e-3)
