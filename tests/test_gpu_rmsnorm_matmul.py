"""GPU parity of gmlp_rmsnorm_matmul (the paper's running example, Section 2) against the CPU oracle:
|z - z_ref| <= 2e-2 * max(1, |z_ref|) for the rewritten schedule (row scale after the matmul, squares
reduced from the MMA's own shared-memory tiles) and for the unfused one (RMSNorm kernel, then GEMM)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2606_26344_b200 import gmlp, inputs as I

pytestmark = pytest.mark.gpu


def _case(M, K, N, seed, unfused, gain, eps=1e-5):
    inp = I.custom_inputs(M, K, N, seed, rmsnorm=True, eps=eps)       # X [M,K], Wg [K,N], gamma [K]
    dev = torch.device("cuda")
    X, W = inp.X.to(dev), inp.Wg.to(dev)
    gamma = inp.gamma.to(dev) if gain else None
    Z = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=dev)
    gmlp.rmsnorm_matmul(X, W, Z, gamma=gamma, eps=eps, unfused=unfused, checked=True)
    torch.cuda.synchronize()
    assert bool(torch.isfinite(Z.float()).all())
    rows = I.sample_rows(inp.workload, inp.outlier_rows)
    z_ref = oracle.rmsnorm_matmul_rows(inp.bits("X"), inp.bits("Wg"), rows=rows,
                                       gamma=inp.bits("gamma") if gain else None, eps=eps)
    z = Z[torch.as_tensor(rows, device=dev)].float().cpu().numpy().astype(np.float64)
    err = np.abs(z - z_ref) / (2e-2 * np.maximum(1.0, np.abs(z_ref)))
    assert err.max() <= 1.0, f"max err/tol {err.max():.3f}"
    return err.max()


@pytest.mark.parametrize("shape", [(128, 64, 256), (1, 64, 128), (17, 72, 136), (129, 320, 392), (300, 512, 1024),
                                   (257, 1096, 648), (1030, 264, 520)])
@pytest.mark.parametrize("mode", ["rewritten", "unfused", "unfused+gain"])
def test_rmsnorm_matmul_small_and_ragged(shape, mode):
    M, K, N = shape
    _case(M, K, N, 800 + M, unfused=(mode != "rewritten"), gain=(mode == "unfused+gain"), eps=1e-6)


@pytest.mark.parametrize("mode", ["rewritten", "unfused"])
def test_rmsnorm_matmul_paper_sized(mode):
    # the paper sweeps {2K, 4K, 8K}^3; one mid-size point at full size, 256 sampled rows
    _case(2048, 4096, 4096, 5, unfused=(mode == "unfused"), gain=False)


def test_gain_is_routed_to_the_unfused_schedule_and_needs_a_workspace():
    inp = I.custom_inputs(40, 128, 256, 2, rmsnorm=True)
    dev = torch.device("cuda")
    X, W, gamma = inp.X.to(dev), inp.Wg.to(dev), inp.gamma.to(dev)
    import ctypes
    a = gmlp.GmlpRmsmmArgs()
    a.struct_bytes = ctypes.sizeof(gmlp.GmlpRmsmmArgs)
    Z = torch.empty(40, 256, dtype=torch.bfloat16, device=dev)
    a.X, a.W, a.Z, a.M, a.K, a.N = X.data_ptr(), W.data_ptr(), Z.data_ptr(), 40, 128, 256
    a.rms_gain, a.rms_eps = gamma.data_ptr(), 1e-5
    assert gmlp.lib().gmlp_rmsnorm_matmul(ctypes.byref(a)) == gmlp.ERR_WORKSPACE
    ws = torch.empty(4096, dtype=torch.uint8, device=dev)               # enough for the row scales, not for Xn
    a.workspace, a.workspace_bytes = ws.data_ptr(), 4096
    assert gmlp.lib().gmlp_rmsnorm_matmul(ctypes.byref(a)) == gmlp.ERR_WORKSPACE
    a.rms_gain = None
    assert gmlp.lib().gmlp_rmsnorm_matmul(ctypes.byref(a)) == gmlp.OK
    torch.cuda.synchronize()
