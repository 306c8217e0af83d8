"""GPU parity of gmlp_matmul_add_rmsnorm ("Matmul+Add+RMSNorm", Section 6.1) against the CPU oracle:
S = bf16(X W + R) and Z = bf16(RMSNorm(S) * gain), both within 2e-2 * max(1, |ref|), for the fused schedule
(residual and sum of squares in the GEMM epilogue, light normalise pass) and the unfused one."""
import ctypes
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2606_26344_b200 import gmlp, inputs as I

pytestmark = pytest.mark.gpu


def _inputs(M, K, N, seed):
    g = torch.Generator().manual_seed(seed)
    X = torch.randn(M, K, generator=g).to(torch.bfloat16)
    W = (torch.randn(K, N, generator=g) / math.sqrt(K)).to(torch.bfloat16)
    R = torch.randn(M, N, generator=g).to(torch.bfloat16)
    gam = (0.5 + torch.rand(N, generator=g)).to(torch.bfloat16)
    return X, W, R, gam


def _bits(t):
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def _check(M, K, N, seed, unfused, gain, eps=1e-5, in_place=False, max_rows=256):
    X, W, R, gam = _inputs(M, K, N, seed)
    dev = torch.device("cuda")
    Xd, Wd, Rd = X.to(dev), W.to(dev), R.to(dev)
    S = Rd if in_place else torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=dev)
    Z = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=dev)
    gmlp.matmul_add_rmsnorm(Xd, Wd, Rd, S, Z, gamma=gam.to(dev) if gain else None, eps=eps, unfused=unfused, checked=True)
    torch.cuda.synchronize()
    assert bool(torch.isfinite(S.float()).all()) and bool(torch.isfinite(Z.float()).all())
    rows = np.arange(M) if M <= max_rows else np.sort(np.random.default_rng(seed).choice(M, max_rows, replace=False))
    Sb, Sr, Zr = oracle.matmul_add_rmsnorm_rows(_bits(X), _bits(W), _bits(R), rows=rows,
                                                gamma=_bits(gam) if gain else None, eps=eps)
    idx = torch.as_tensor(rows, device=dev)
    s = S[idx].float().cpu().numpy().astype(np.float64)
    z = Z[idx].float().cpu().numpy().astype(np.float64)
    es = np.abs(s - Sr) / oracle.tolerance(Sr)
    ez = np.abs(z - Zr) / oracle.tolerance(Zr)
    assert es.max() <= 1.0 and ez.max() <= 1.0, f"S err/tol {es.max():.3f}, Z err/tol {ez.max():.3f}"
    if not unfused:
        # the fused epilogue rounds the fp32 sum once: the stored S is the oracle's bf16 S up to the rare
        # element whose fp32 and fp64 sums straddle a rounding boundary
        flips = float(np.mean(_bits(S[idx].cpu()) != Sb))
        assert flips < 0.02, f"S differs from the singly rounded reference on {flips:.3%} of elements"
    return ez.max()


@pytest.mark.parametrize("shape", [(128, 64, 256), (1, 64, 128), (17, 72, 136), (129, 320, 392), (300, 512, 1024),
                                   (257, 1096, 648), (1030, 264, 520), (1500, 128, 776)])
@pytest.mark.parametrize("mode", ["fused", "fused+gain", "unfused+gain"])
def test_small_and_ragged(shape, mode):
    M, K, N = shape
    _check(M, K, N, 40 + M, unfused=mode.startswith("unfused"), gain=mode.endswith("gain"), eps=1e-6)


@pytest.mark.parametrize("M", [129, 1030])
def test_in_place_residual_update(M):
    _check(M, 256, 520, 77, unfused=False, gain=True, in_place=True)


@pytest.mark.parametrize("mode", ["fused", "unfused"])
def test_paper_sized(mode):
    # the paper sweeps {2K, 4K, 8K}^3; one mid-size point at full size, 256 sampled rows
    _check(2048, 4096, 4096, 5, unfused=(mode == "unfused"), gain=True)


def test_fused_result_is_deterministic_and_z_matches_a_norm_of_the_stored_s():
    X, W, R, gam = _inputs(300, 256, 1024, 9)
    dev = torch.device("cuda")
    S1, Z1 = gmlp.matmul_add_rmsnorm(X.to(dev), W.to(dev), R.to(dev), gamma=gam.to(dev), checked=True)
    S2, Z2 = gmlp.matmul_add_rmsnorm(X.to(dev), W.to(dev), R.to(dev), gamma=gam.to(dev), checked=True)
    assert torch.equal(S1.view(torch.int16), S2.view(torch.int16)) and torch.equal(Z1.view(torch.int16), Z2.view(torch.int16))
    # Eq. (1) on the S that the GPU stored, in fp64: Z must be that value rounded, up to an ulp
    sd = S1.double().cpu()
    want = sd * torch.rsqrt((sd * sd).mean(dim=1, keepdim=True) + float(np.float32(1e-5))) * gam.double()
    got = Z1.double().cpu()
    assert bool(((got - want).abs() <= want.abs() * 2.0 ** -7 + 1e-30).all())


def test_argument_checks():
    dev = torch.device("cuda")
    X, W, R, _ = _inputs(40, 128, 256, 2)
    Xd, Wd, Rd = X.to(dev), W.to(dev), R.to(dev)
    S, Z = torch.empty_like(Rd), torch.empty_like(Rd)
    a = gmlp.make_mmaddnorm_args(Xd, Wd, Rd, S, Z)
    f = lambda: gmlp.lib().gmlp_matmul_add_rmsnorm(ctypes.byref(a))
    assert f() == gmlp.ERR_WORKSPACE
    ws = torch.empty(4096, dtype=torch.uint8, device=dev)
    a.workspace, a.workspace_bytes = ws.data_ptr(), 4096
    assert f() == gmlp.OK
    a.flags = gmlp.MMADDNORM_UNFUSED
    assert f() == gmlp.ERR_WORKSPACE                       # the unfused schedule needs M*N*2 bytes
    a.flags = 1 << 9
    assert f() == gmlp.ERR_FLAGS
    a.flags = 0
    a.R = None
    assert f() == gmlp.ERR_NULL
    a.R = Rd.data_ptr()
    a.N = 100
    assert f() == gmlp.ERR_SHAPE
    torch.cuda.synchronize()
    assert gmlp.device_status() == 0
