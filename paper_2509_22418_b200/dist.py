"""Multi-GPU plumbing: one process per GPU, replicas only.

Between outer syncs the replicas of Algorithm 1 never exchange data, so N GPUs run N disjoint
groups of replicas with no data-path collective; the only communication is the barrier and the
max-over-ranks of the measured times.
"""
from __future__ import annotations


def replica_group(n_replicas_per_rank: int, world: int, rank: int):
    """Global ids of the replicas rank `rank` simulates (contiguous block per rank)."""
    if not (0 <= rank < world):
        raise ValueError("rank outside the world")
    lo = rank * n_replicas_per_rank
    return list(range(lo, lo + n_replicas_per_rank))


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return list(values)
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()
