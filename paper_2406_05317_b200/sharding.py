"""Host-side logic for running the path on several GPUs.

(sequence, head) units are independent (the conv weights are shared, the state is
not), so the forward path shards with no data-path collective.  Only the backward
pass of shared conv weights has an exchange step: one sum of dG over ranks.
The token axis does not shard: chunk n needs the cache of chunk n-1.
"""
from __future__ import annotations


def shard_range(n_items: int, world: int, rank: int) -> range:
    """Contiguous, balanced partition of n_items over `world` ranks."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    base, extra = divmod(n_items, world)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def weak_scaling_sequences(world: int, rank: int, per_rank: int = 1) -> range:
    """Weak scaling: every rank processes `per_rank` whole sequences of its own."""
    return range(rank * per_rank, (rank + 1) * per_rank)


def aggregate_throughput(dist, local_ms: float, local_units: float):
    """(max time over ranks in ms, total units over ranks). `dist` is torch.distributed
    (initialised) or None for a single process."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return local_ms, local_units
    import torch
    device = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    u = torch.tensor([local_units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def allreduce_weight_gradient(dist, dG):
    """Sum of the conv-weight gradient over ranks (the one exchange step of the backward
    pass when the heads of a layer share their weights)."""
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(dG, op=dist.ReduceOp.SUM)
    return dG
