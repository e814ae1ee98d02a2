"""Host-side helpers for running on several GPUs (one process per GPU).

The ops have no exchange step: output rows (m = (n,h,w)) are independent, so a problem is
sharded by giving each rank a contiguous slab of the outermost parallel iterator and the
whole (small) filter operand; no data-path collective is needed.  The only communication is
the max-reduction of a timing scalar in the benchmark.
"""
from __future__ import annotations


def row_slab(extent: int, rank: int, world: int):
    """[begin, end) of `extent` rows owned by `rank`: contiguous, balanced to within one row."""
    if world < 1 or not 0 <= rank < world or extent < 0:
        raise ValueError("bad slab request")
    base, rem = divmod(extent, world)
    begin = rank * base + min(rank, rem)
    return begin, begin + base + (1 if rank < rem else 0)


def max_over_ranks(value: float, device=None) -> float:
    """Max of a scalar over all ranks (identity when torch.distributed is not initialised)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())
