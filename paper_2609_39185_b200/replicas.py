"""Host-side logic of the multi-GPU mode: independent replicas over disjoint batch shards.

The path has no exchange step (every sequence and head is independent), so ranks never communicate on
the data path.  Two things keep N replicas equal to one big batch: thresholds are computed from GLOBAL
indices (each rank passes the global index of its first sequence), and timings are reduced with a
maximum over ranks.
"""
from __future__ import annotations


def shard_batch_base(rank: int, batch_per_rank: int) -> int:
    """Global index of the first sequence of `rank` when every rank holds `batch_per_rank` sequences."""
    return rank * batch_per_rank


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """Maximum of a scalar over all ranks (identity without a process group)."""
    if dist is None or not dist.is_initialized():
        return float(value)
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())
