"""Shared helpers of the GPU parity tests: run the CUDA path through the C ABI and compare
with the CPU oracle element by element on the same seeded inputs.

Pass rule (stated by the benchmark spec): |y - y_ref| <= 2e-2 * max(1, |y_ref|) for every compared
element; y_ref is the oracle's fp64 value (H rounded to bf16 where the GPU rounds it).
"""
import numpy as np
import torch

import oracle
from paper_2606_26344_b200 import gmlp, inputs as I


def to_device(inp, dev="cuda"):
    d = dict(X=inp.X.to(dev), Wg=inp.Wg.to(dev), Wu=inp.Wu.to(dev), Wd=inp.Wd.to(dev))
    d["gamma"] = inp.gamma.to(dev) if inp.gamma is not None else None
    return d


def gpu_forward(inp, variant=gmlp.VARIANT_AUTO, dev_tensors=None, use_gamma=True, checked=True):
    w = inp.workload
    t = dev_tensors or to_device(inp)
    ws = gmlp.alloc_workspace(w.M, w.d_model, w.d_ff, w.rmsnorm, variant)
    Y = torch.full_like(t["X"], float("nan"))
    gmlp.forward(t["X"], t["Wg"], t["Wu"], t["Wd"], Y, gamma=t["gamma"] if (w.rmsnorm and use_gamma) else None,
                 eps=w.eps, rmsnorm=w.rmsnorm, variant=variant, workspace=ws, checked=checked)
    torch.cuda.synchronize()
    return Y


def oracle_rows(inp, rows, use_gamma=True, num_threads=0):
    w = inp.workload
    return oracle.gmlp_rows(inp.bits("X"), inp.bits("Wg"), inp.bits("Wu"), inp.bits("Wd"), rows=rows,
                            gamma=inp.bits("gamma") if (w.rmsnorm and use_gamma) else None,
                            eps=w.eps, rmsnorm=w.rmsnorm, num_threads=num_threads)


def err_over_tol(Y, y_ref, rows):
    y = Y[torch.as_tensor(rows, device=Y.device)].float().cpu().numpy().astype(np.float64)
    return np.abs(y - y_ref) / oracle.tolerance(y_ref), y


def check_case(inp, variant=gmlp.VARIANT_AUTO, label=""):
    """Full check of one case; returns max err/tol."""
    w = inp.workload
    rows = I.sample_rows(w, inp.outlier_rows)
    Y = gpu_forward(inp, variant)
    assert bool(torch.isfinite(Y.float()).all()), f"{label}: non-finite output"
    y_ref = oracle_rows(inp, rows)
    e, _ = err_over_tol(Y, y_ref, rows)
    worst = float(e.max()) if e.size else 0.0
    assert worst <= 1.0, (f"{label}: {int((e > 1).sum())} of {e.size} elements out of tolerance, "
                          f"max err/tol {worst:.3f} at {np.unravel_index(int(e.argmax()), e.shape)}")
    return worst
