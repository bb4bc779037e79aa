"""Host-side helpers for running the path on several GPUs of one node.

Rows (tokens) are independent in every step of the path, so scale-out is plain sharding of M
with the weights replicated: no data-path collective.  torch.distributed is used only to agree
on a time (max over ranks) and for barriers.
"""
from __future__ import annotations

from typing import Tuple


def row_shard(M: int, rank: int, world: int, align: int = 1) -> Tuple[int, int]:
    """[begin, end) of the rows rank `rank` owns when M rows are split over `world` ranks in
    contiguous pieces whose sizes differ by less than 2 * `align` rows (pieces are multiples of
    `align` except possibly the last)."""
    if world < 1 or not (0 <= rank < world):
        raise ValueError("bad rank / world size")
    units = (M + align - 1) // align
    base, extra = divmod(units, world)
    begin_u = rank * base + min(rank, extra)
    end_u = begin_u + base + (1 if rank < extra else 0)
    return min(begin_u * align, M), min(end_u * align, M)


def max_over_ranks(value: float, device=None) -> float:
    """Max of a per-rank number over the default process group (identity without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_rate(units_per_rank: float, world: int, ms: float) -> float:
    """Whole-job rate: every rank processed `units_per_rank` in `ms` (already the max over ranks)."""
    return world * units_per_rank / (ms * 1e-3)
