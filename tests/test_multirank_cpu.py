"""CPU-only, world_size 2 over gloo: the multi-rank plumbing of bench.py (request sharding and the
max-over-ranks / sum-over-ranks reductions that turn per-rank device times into one job-wide number)."""
import os
import sys

import pytest

torch = pytest.importorskip("torch")
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    seeds = bench.shard_requests(rank, world, 4)
    ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    tokens = 1000.0 * (rank + 1)
    worst = bench.max_over_ranks(ms, world)
    total = bench.sum_over_ranks(tokens, world)
    dist.barrier()
    out[rank] = (seeds, worst, total)
    dist.destroy_process_group()


def test_sharding_and_reductions_over_two_ranks():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, 29517, out), nprocs=world, join=True)
    s0, w0, t0 = out[0]
    s1, w1, t1 = out[1]
    assert s0 == [0, 1, 2, 3] and s1 == [4, 5, 6, 7]       # disjoint request streams, same size (weak scaling)
    assert w0 == w1 == 15.0                                 # job time = slowest rank
    assert t0 == t1 == 3000.0                               # job work = all ranks
    value = t0 / (w0 * 1e-3)
    assert abs(value - 200000.0) < 1e-6


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1) == 3.5 and bench.sum_over_ranks(7.0, 1) == 7.0
    assert bench.shard_requests(0, 1, 3) == [0, 1, 2]


def _shard_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import numpy as np
    import torch.distributed as dist
    import paper_2510_15620_b200 as P
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    rng = np.random.default_rng(3)                       # same seed on every rank: same request
    lens = rng.integers(40, 600, size=101)
    owner = P.shard_candidates(lens, world)
    scores = rng.normal(size=101).astype(np.float32)
    mine = torch.from_numpy(np.where(owner == rank, scores, np.float32(0.0)))
    P.all_reduce_scores(mine)                            # what select_sharded's reduce does between probe and rule
    out[rank] = (owner.tolist(), mine.numpy().tobytes(), scores.tobytes(), int(lens[owner == rank].sum()))
    dist.barrier()
    dist.destroy_process_group()


def test_candidate_sharding_host_side_over_two_ranks():
    """The host side of candidate-sharded selection: every rank derives the same partition from the request,
    every candidate has exactly one owner, the loads differ by less than one sequence, and the SUM all-reduce of
    the owners' scores (zeros elsewhere) reproduces the full score vector bit for bit on every rank."""
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_shard_worker, args=(world, 29519, out), nprocs=world, join=True)
    o0, got0, want0, load0 = out[0]
    o1, got1, want1, load1 = out[1]
    assert o0 == o1 and set(o0) == {0, 1}
    assert got0 == want0 and got1 == want1
    assert abs(load0 - load1) < 600
