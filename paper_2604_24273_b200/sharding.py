"""Row sharding of a batch of states across ranks (one process per GPU).

Every token row is quantized and contracted independently with the same frozen weights, so a batch shards by
rows with a replica of the packed backbone on each rank and no collective on the data path.  The only
communication is plumbing: a barrier and a max-reduction of the per-rank step time.
"""
from __future__ import annotations


def shard_rows(M: int, world: int, rank: int) -> tuple[int, int]:
    """Contiguous, balanced split of M rows: returns (first_row, row_count) of `rank`; counts differ by <= 1."""
    if world < 1 or not (0 <= rank < world) or M < 0:
        raise ValueError("bad shard request")
    base, rem = divmod(M, world)
    start = rank * base + min(rank, rem)
    return start, base + (1 if rank < rem else 0)


def max_over_ranks(value: float, device=None) -> float:
    """Max of `value` over the default process group (identity without one)."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())
