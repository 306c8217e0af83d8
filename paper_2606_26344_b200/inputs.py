"""Seeded synthetic inputs for the Gated-MLP workloads.

This module serves both the CPU oracle's tests and the CUDA path.  It holds none of the
operator's arithmetic: it only draws random numbers, scales them and rounds them once to
bf16.  Everything is generated on the host with a seeded ``torch.Generator`` so that the
oracle and the GPU receive exactly the same bf16 bits.

The workloads stand in for Llama-3 MLP layer shapes (no model weights or dataset items
are used): X ~ N(0,1); projection weights ~ N(0, 1/fan_in); the RMSNorm gain ~ U(0.5, 1.5);
in the 70B-shaped prefill case 1 % of the rows of X are scaled by 20 (outlier rows).
Draw order is fixed: X, [outlier permutation], [gain], W_gate, W_up, W_down.
"""
from __future__ import annotations

import dataclasses
from typing import Optional

import numpy as np
import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    M: int
    d_model: int
    d_ff: int
    seed: int
    rmsnorm: bool = False
    eps: float = 1e-5
    outlier_frac: float = 0.0
    outlier_scale: float = 20.0
    sample_rows: int = 256      # rows checked against the oracle when M is larger than this

    @property
    def flops(self) -> int:
        return 6 * self.M * self.d_model * self.d_ff

    @property
    def min_bytes(self) -> int:
        """Weights once, X once, Y once (+ gain); the intermediate H is not algorithmic traffic."""
        b = 2 * (3 * self.d_model * self.d_ff + 2 * self.M * self.d_model)
        if self.rmsnorm:
            b += 2 * self.d_model
        return b


def _ragged(M: int, seed: int, rmsnorm: bool) -> Workload:
    return Workload(f"ragged-M{M}-{'norm' if rmsnorm else 'plain'}", M, 2048, 5632, seed,
                    rmsnorm=rmsnorm, eps=1e-6)


WORKLOADS = {
    w.name: w for w in [
        Workload("tiny", 16, 256, 512, 0),
        Workload("llama3-8b-decode-M8", 8, 4096, 14336, 0),
        Workload("llama3-8b-batch-M64", 64, 4096, 14336, 0),      # not a stated config: the mid-M schedule on the same layer
        Workload("llama3-8b-prefill-M2048-rmsnorm", 2048, 4096, 14336, 0, rmsnorm=True, eps=1e-5),
        Workload("llama3-70b-prefill-M4096-outliers", 4096, 8192, 28672, 0, outlier_frac=0.01),
        *[_ragged(M, s, n) for (M, s) in zip((1, 7, 129, 1000, 8192), (1, 2, 3, 4, 5)) for n in (False, True)],
    ]
}


@dataclasses.dataclass
class Inputs:
    """bf16 tensors on the host (torch.bfloat16, contiguous).  ``gamma`` is None without RMSNorm."""
    workload: Workload
    X: torch.Tensor
    Wg: torch.Tensor
    Wu: torch.Tensor
    Wd: torch.Tensor
    gamma: Optional[torch.Tensor]
    outlier_rows: np.ndarray

    def bits(self, name: str) -> np.ndarray:
        """The tensor's bf16 bit patterns as a uint16 numpy array (what the oracle takes)."""
        t = getattr(self, name)
        return t.view(torch.int16).numpy().view(np.uint16)


def make_inputs(w: Workload) -> Inputs:
    g = torch.Generator(device="cpu").manual_seed(w.seed)
    X = torch.randn(w.M, w.d_model, generator=g, dtype=torch.float32)
    outliers = np.zeros(0, dtype=np.int64)
    if w.outlier_frac > 0.0:
        perm = torch.randperm(w.M, generator=g)
        n_out = int(round(w.outlier_frac * w.M))
        idx = perm[:n_out]
        X[idx] *= w.outlier_scale
        outliers = np.sort(idx.numpy().astype(np.int64))
    gamma = None
    if w.rmsnorm:
        gamma = (torch.rand(w.d_model, generator=g, dtype=torch.float32) + 0.5).to(torch.bfloat16)
    Wg = (torch.randn(w.d_model, w.d_ff, generator=g, dtype=torch.float32) * w.d_model ** -0.5).to(torch.bfloat16)
    Wu = (torch.randn(w.d_model, w.d_ff, generator=g, dtype=torch.float32) * w.d_model ** -0.5).to(torch.bfloat16)
    Wd = (torch.randn(w.d_ff, w.d_model, generator=g, dtype=torch.float32) * w.d_ff ** -0.5).to(torch.bfloat16)
    return Inputs(w, X.to(torch.bfloat16).contiguous(), Wg.contiguous(), Wu.contiguous(), Wd.contiguous(),
                  gamma, outliers)


def sample_rows(w: Workload, outlier_rows: np.ndarray) -> np.ndarray:
    """Rows compared with the oracle: all rows when M <= sample_rows, else a seeded sample.

    The sample is stratified so that outlier rows are represented in proportion
    (ceil(outlier_frac * sample_rows) of them); rows are independent, so any subset is a
    valid check of the whole.
    """
    if w.M <= w.sample_rows:
        return np.arange(w.M, dtype=np.int64)
    gs = torch.Generator(device="cpu").manual_seed(w.seed + 1000)
    n_out = 0
    picked = []
    if outlier_rows.size:
        n_out = min(int(np.ceil(w.outlier_frac * w.sample_rows)), outlier_rows.size)
        p = torch.randperm(outlier_rows.size, generator=gs).numpy()
        picked.append(outlier_rows[p[:n_out]])
    normal = np.setdiff1d(np.arange(w.M, dtype=np.int64), outlier_rows)
    p = torch.randperm(normal.size, generator=gs).numpy()
    picked.append(normal[p[: w.sample_rows - n_out]])
    return np.sort(np.concatenate(picked)).astype(np.int64)


def custom_inputs(M: int, d_model: int, d_ff: int, seed: int, rmsnorm: bool = False, eps: float = 1e-5) -> Inputs:
    """Same recipe on an arbitrary shape (used by the tile-boundary and edge-case tests)."""
    return make_inputs(Workload(f"custom-{M}x{d_model}x{d_ff}-s{seed}", M, d_model, d_ff, seed,
                                rmsnorm=rmsnorm, eps=eps))
