"""Host-side logic of the multi-GPU mode: independent replicas over disjoint shards of the batch or of the heads.

The path has no exchange step (every sequence and head is independent), so ranks never communicate on
the data path.  Two things keep N replicas equal to one big problem: thresholds are computed from GLOBAL
indices (each rank passes the global index of its first sequence and, under a head split, of its first head
together with the layer's head count), and timings are reduced with a maximum over ranks.
"""
from __future__ import annotations


def shard_batch_base(rank: int, batch_per_rank: int) -> int:
    """Global index of the first sequence of `rank` when every rank holds `batch_per_rank` sequences."""
    return rank * batch_per_rank


def shard_head_range(rank: int, world: int, nheads_global: int) -> tuple[int, int]:
    """Heads [first, last) that `rank` holds when a layer's heads are split evenly over `world` ranks (tensor
    parallel); `first` is the descriptor's head_index_base.  The head count must divide evenly."""
    if nheads_global % world != 0:
        raise ValueError(f"{nheads_global} heads do not split evenly over {world} ranks")
    per = nheads_global // world
    return rank * per, (rank + 1) * per


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """Maximum of a scalar over all ranks (identity without a process group)."""
    if dist is None or not dist.is_initialized():
        return float(value)
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())
