"""Data-parallel sharding of the path over several GPUs (one process per GPU).

Every (batch, head) unit is independent: the sampled scores, the selection, mean(V) and the
attention of a unit read only that unit's Q, K, V (Sec. 3.2 defines everything per query against
its own keys).  So the batch is cut into contiguous ranges of sequences, one per rank, and no
collective touches the data path.  The only communication is the timing protocol of the
benchmark: a barrier and a max-over-ranks of the elapsed time.
"""
from __future__ import annotations


def shard_range(n_items: int, world: int, rank: int) -> tuple[int, int]:
    """Contiguous, balanced split of range(n_items): rank r gets [lo, hi); sizes differ by at most 1."""
    if world < 1 or not (0 <= rank < world):
        raise ValueError("bad world/rank")
    base, extra = divmod(n_items, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def rank_seed(base_seed: int, rank: int, buffer_set: int = 0) -> int:
    """Seed of the synthetic batch of one rank and buffer set (weak scaling: every rank draws its own batch)."""
    return int(base_seed) + 1000 * int(rank) + 17 * int(buffer_set)


def max_over_ranks(value: float, device=None) -> float:
    """Max of a per-rank number over the default process group (the value itself without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device=None) -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
