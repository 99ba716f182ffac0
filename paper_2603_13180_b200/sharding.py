"""Data-parallel plumbing for the MXNorm path (one process per GPU, torch.distributed).

The forward path is row-independent: ranks own disjoint row slices and exchange nothing.  The only
quantity that sums over rows is the gain gradient of the backward; across ranks that is one
all-reduce of D floats.  Timing helpers take the maximum over ranks.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

TILE_ROWS = 128   # row granularity of the tiled scale layout


def shard_rows(T: int, rank: int, world: int, align: int = TILE_ROWS) -> tuple[int, int]:
    """[begin, end) of the rows owned by `rank`: contiguous, disjoint, covering [0, T), every boundary
    (except T itself) a multiple of `align` so that each shard's tiled scale buffer is a contiguous
    slice of the whole tensor's."""
    if not (0 <= rank < world) or T < 0 or align <= 0:
        raise ValueError("bad shard request")
    units = (T + align - 1) // align
    base, extra = divmod(units, world)
    b = rank * base + min(rank, extra)
    e = b + base + (1 if rank < extra else 0)
    return min(b * align, T), min(e * align, T)


def max_over_ranks(value: float, device="cpu") -> float:
    """Maximum of a per-rank scalar (device time of a timed region) over all ranks."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def allreduce_dgain(dgain: torch.Tensor) -> torch.Tensor:
    """Sums the per-rank gain gradients [D] in place (the one exchange step of the backward)."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(dgain, op=dist.ReduceOp.SUM)
    return dgain
