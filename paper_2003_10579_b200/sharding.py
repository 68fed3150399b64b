"""Replica sharding over ranks: replicas are independent, their global ids sit in the random
streams' counters, so rank r of W simply simulates a contiguous block of ids.  No data-path
collective; only timings are reduced (max over ranks)."""
from __future__ import annotations


def replica_block(rank: int, world: int, replicas_per_rank: int):
    """Weak scaling: every rank gets `replicas_per_rank` replicas; returns (replica_base, count)."""
    assert 0 <= rank < world
    return rank * replicas_per_rank, replicas_per_rank


def split_replicas(rank: int, world: int, total: int):
    """Strong scaling: `total` replicas split as evenly as possible; returns (replica_base, count)."""
    assert 0 <= rank < world
    q, rem = divmod(total, world)
    return rank * q + min(rank, rem), q + (1 if rank < rem else 0)


def max_over_ranks(value: float, device=None) -> float:
    """The slowest rank's time (a job is as slow as its slowest rank)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())
