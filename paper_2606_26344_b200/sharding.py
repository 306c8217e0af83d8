"""Host-side logic for running the Gated MLP on several GPUs.

The operator is row-independent (each row of Y depends only on the same row of X), so the path
shards by rows: every rank holds all weights and a disjoint, contiguous range of rows, and there is
no collective on the data path.  ``torch.distributed`` is used for the rendezvous, the barrier around
a timed region and the max-over-ranks of the measured time only.

The second way to cut the layer, by d_ff, is here as well: Y = H W_down sums over d_ff, so rank r may hold the
columns [a, b) of W_gate and W_up and the rows [a, b) of W_down, compute its fp32 partial product with one call of
the library, and the ranks exchange ONE all-reduce of M * d_model floats before the single rounding
(``dff_range``, ``forward_dff_partial``, ``forward_dff_sharded``).  Per-GPU weight bytes fall as 1 / world, which
is what matters for a handful of tokens.
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


def dff_range(d_ff: int, rank: int, world: int, multiple: int = 128) -> Tuple[int, int]:
    """Slice [start, stop) of d_ff owned by `rank`: contiguous, disjoint, covering [0, d_ff), every boundary except the
    last a multiple of `multiple` (the kernels' column tile), lengths as even as that allows."""
    if world <= 0 or not (0 <= rank < world) or d_ff <= 0 or multiple <= 0:
        raise ValueError("bad rank/world/d_ff")
    blocks = -(-d_ff // multiple)
    base, extra = divmod(blocks, world)
    first = rank * base + min(rank, extra)
    last = first + base + (1 if rank < extra else 0)
    return min(first * multiple, d_ff), min(last * multiple, d_ff)


def forward_dff_partial(X, Wg_s, Wu_s, Wd_s, gamma=None, eps: float = 1e-5, rmsnorm: bool = False, stream=None, P=None):
    """This rank's fp32 partial product [M, d_model] from its slice of the weights (Wg_s, Wu_s: [d_model, n],
    Wd_s: [n, d_model]; n may be 0 for a rank left without a slice).  One call of the library.  `P`: a float32
    [M, d_model] buffer to reuse (it is overwritten)."""
    import torch
    from . import gmlp
    M, d_model = X.shape
    if P is None:
        P = torch.zeros(M, d_model, dtype=torch.float32, device=X.device)
    if Wg_s.shape[1] > 0:
        gmlp.forward(X, Wg_s, Wu_s, Wd_s, P, gamma, eps, rmsnorm, stream=stream)
    else:
        P.zero_()
    return P


def forward_dff_sharded(X, Wg_s, Wu_s, Wd_s, dist=None, gamma=None, eps: float = 1e-5, rmsnorm: bool = False, stream=None,
                        P=None, Y=None):
    """The whole layer with d_ff cut over the ranks of `dist` (one process per GPU): partial product, one all-reduce
    (sum) of M * d_model floats, one rounding.  Every rank returns the full bf16 Y.  `P` / `Y`: buffers to reuse."""
    from . import gmlp
    P = forward_dff_partial(X, Wg_s, Wu_s, Wd_s, gamma, eps, rmsnorm, stream, P)
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(P)                                           # the path's only exchange
    return gmlp.sum_partials([P], Y, stream=stream)
