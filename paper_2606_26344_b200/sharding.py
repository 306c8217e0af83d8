"""Host-side logic for running the Gated MLP on several GPUs.

The operator is row-independent (each row of Y depends only on the same row of X), so the path
shards by rows: every rank holds all weights and a disjoint, contiguous range of rows, and there is
no collective on the data path.  ``torch.distributed`` is used for the rendezvous, the barrier around
a timed region and the max-over-ranks of the measured time only.
"""
from __future__ import annotations

from typing import Tuple


def row_range(M: int, rank: int, world: int) -> Tuple[int, int]:
    """Rows [start, stop) owned by `rank` when M rows are split over `world` ranks.

    Ranges are contiguous, disjoint, cover [0, M) and differ in length by at most one row.
    """
    if world <= 0 or not (0 <= rank < world) or M < 0:
        raise ValueError("bad rank/world/M")
    base, extra = divmod(M, world)
    start = rank * base + min(rank, extra)
    return start, start + base + (1 if rank < extra else 0)


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """The slowest rank's value (the time that bounds a multi-GPU step)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: int, world: int, ms_max: float) -> float:
    """Whole-job units per second when every rank processed `units_per_rank` in `ms_max` milliseconds."""
    return world * units_per_rank / (ms_max * 1e-3)
