"""Multi-GPU path on CPU: two gloo ranks shard a batch by sample, run the selection stages
of their own samples with the oracle, and the gathered result equals the unsharded run.
Also checks the time aggregation bench.py uses (max over ranks)."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import oracle
    from paper_2412_03409_b200 import sharding, workloads as wl
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        L, N, n_samples = 4, 60, 5
        budget = L * N // 3
        mine = list(sharding.shard_batch(n_samples, rank, world))
        lens = {}
        for b in mine:                                   # no exchange: each sample stands alone
            scores = wl.synthetic_scores(L, N, seed=100 + b)
            _, _, res = oracle.select_sample(scores, budget)
            lens[b] = res.len
        gathered = [None] * world
        dist.all_gather_object(gathered, lens)           # test-only gather, not part of the path
        # weak-scaling ids are disjoint
        ids = sharding.samples_for_rank(rank, world, batch=3, replicas=2)
        all_ids = [None] * world
        dist.all_gather_object(all_ids, ids)
        slow = sharding.max_over_ranks(1.0 + rank)       # rank 1 is the slow one
        thr = sharding.aggregate_throughput(10.0, 1.0 + rank)
        if rank == 0:
            merged = {}
            for g in gathered:
                merged.update(g)
            np.save(os.path.join(out_dir, "lens.npy"), np.stack([merged[b] for b in range(n_samples)]))
            flat = [x for r in all_ids for rep in r for x in rep]
            np.save(os.path.join(out_dir, "ids.npy"), np.array(flat))
            np.save(os.path.join(out_dir, "agg.npy"), np.array([slow, thr]))
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_by_sample(tmp_path):
    import oracle
    from paper_2412_03409_b200 import workloads as wl
    oracle.build()
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    L, N, n_samples = 4, 60, 5
    ref = np.stack([oracle.select_sample(wl.synthetic_scores(L, N, seed=100 + b), L * N // 3)[2].len
                    for b in range(n_samples)])
    np.testing.assert_array_equal(np.load(tmp_path / "lens.npy"), ref)
    ids = np.load(tmp_path / "ids.npy")
    assert sorted(ids.tolist()) == list(range(world * 2 * 3))          # disjoint and dense
    slow, thr = np.load(tmp_path / "agg.npy")
    assert slow == 2.0 and thr == pytest.approx(world * 10.0 / 2.0)


def test_shard_helpers_single_process():
    from paper_2412_03409_b200 import sharding
    assert [list(sharding.shard_batch(5, r, 2)) for r in range(2)] == [[0, 1, 2], [3, 4]]
    assert [list(sharding.shard_batch(2, r, 4)) for r in range(4)] == [[0], [1], [], []]
    assert sharding.samples_for_rank(1, 4, batch=2) == [[2, 3]]
    assert sharding.max_over_ranks(3.5) == 3.5
    with pytest.raises(ValueError):
        sharding.samples_for_rank(2, 2, batch=1)
