"""Batch sharding across GPUs: which samples a rank owns, and how ranks' times combine.

Every stage of the path (score, sort, search, compact, decode) is independent per sample, so
N GPUs run N disjoint sets of samples with no exchange on the data path.  The only
communication is the benchmark's: a barrier and a max over ranks of the measured time.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def samples_for_rank(rank: int, world: int, batch: int, replicas: int = 1):
    """Global sample ids of each replica a rank runs: replicas lists of `batch` ids.

    Ids are disjoint across ranks and replicas; rank r, replica i, slot b gets
    (r * replicas + i) * batch + b, so the per-rank work is fixed as `world` grows.
    """
    if not (0 <= rank < world) or batch <= 0 or replicas <= 0:
        raise ValueError("bad sharding arguments")
    return [[(rank * replicas + i) * batch + b for b in range(batch)] for i in range(replicas)]


def shard_batch(n_samples: int, rank: int, world: int):
    """Contiguous slice of a fixed global batch for one rank (strong-scaling layout);
    the first n_samples % world ranks hold one extra sample."""
    if not (0 <= rank < world):
        raise ValueError("bad rank")
    q, r = divmod(n_samples, world)
    start = rank * q + min(rank, r)
    return range(start, start + q + (1 if rank < r else 0))


def max_over_ranks(value: float, device="cpu") -> float:
    """Max of a per-rank scalar (the slowest rank's time); identity without a process group."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, seconds: float, device="cpu") -> float:
    """Whole-job throughput: all ranks' units over the slowest rank's time."""
    world = dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1
    return world * units_per_rank / max_over_ranks(seconds, device)
