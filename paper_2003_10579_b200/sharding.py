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


def gather_traces(trace: dict, group=None) -> dict:
    """The one exchange of a sharded simulation, after the run: every rank contributes the trace arrays of
    its replica block (a dict of tensors whose first dimension is the rank's replica count, as
    ``Simulation.trace(to_numpy=False)`` returns them, on the device for NCCL or on the host for gloo)
    and receives the arrays of all replicas, concatenated in rank order - which is global replica order
    when the blocks come from ``replica_block`` / ``split_replicas``.  Ranks may hold different numbers of
    replicas: shorter blocks are padded for the collective and trimmed afterwards.  Without an
    initialised process group (one rank) the input is returned unchanged."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return dict(trace)
    world = dist.get_world_size(group)
    first = next(iter(trace.values()))
    counts = [torch.zeros(1, dtype=torch.int64, device=first.device) for _ in range(world)]
    dist.all_gather(counts, torch.tensor([first.shape[0]], dtype=torch.int64, device=first.device), group=group)
    counts = [int(c.item()) for c in counts]
    top = max(counts)
    out = {}
    for key, t in trace.items():
        assert t.shape[0] == first.shape[0], "every trace array starts with the replica dimension"
        # bytes on the wire: the collectives' backends do not take every element type (unsigned 16- and 32-bit)
        wire = t.contiguous().reshape(t.shape[0], -1).view(torch.uint8)
        if wire.shape[0] < top:      # pad to the longest block
            pad = torch.zeros((top - wire.shape[0],) + tuple(wire.shape[1:]), dtype=wire.dtype, device=wire.device)
            wire = torch.cat([wire, pad])
        parts = [torch.empty_like(wire) for _ in range(world)]
        dist.all_gather(parts, wire, group=group)
        whole = torch.cat([p[:c] for p, c in zip(parts, counts)])
        out[key] = whole.view(t.dtype).reshape((whole.shape[0],) + tuple(t.shape[1:]))
    return out
