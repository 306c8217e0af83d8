"""Pins for the oracle's RMSNorm+MatMul (the paper's running example, Section 2): torch fp64, textbook
loops, the legal rewrite (X (.) r) W == (X W) (.) r of Section 5, scale invariance, closed forms."""
import math

import numpy as np
import torch

import oracle
from paper_2606_26344_b200 import inputs as I


def _bits(t):
    return t.to(torch.bfloat16).contiguous().view(torch.int16).numpy().view(np.uint16)


def test_against_torch_fp64_and_naive_loops():
    inp = I.custom_inputs(9, 72, 40, 81, rmsnorm=True)
    X, gam = inp.bits("X"), inp.bits("gamma")
    W = np.ascontiguousarray(inp.bits("Wg"))                      # [72, 40]
    eps = float(np.float32(1e-5))
    xd, wd, gd = inp.X.double(), inp.Wg.double(), inp.gamma.double()
    r = torch.rsqrt((xd * xd).mean(dim=1, keepdim=True) + eps)
    want = ((xd * r * gd) @ wd).numpy()
    Z = oracle.rmsnorm_matmul_rows(X, W, gamma=gam, eps=1e-5)
    assert np.allclose(Z, want, rtol=1e-12, atol=1e-13)
    naive = oracle.naive_matmul((xd * r * gd).numpy(), wd.numpy())
    assert np.allclose(Z, naive, rtol=1e-13, atol=1e-14)
    # gain-less form == gain of ones; subset of rows
    ones = _bits(torch.ones(72))
    assert np.array_equal(oracle.rmsnorm_matmul_rows(X, W, eps=1e-5), oracle.rmsnorm_matmul_rows(X, W, gamma=ones, eps=1e-5))
    assert np.array_equal(oracle.rmsnorm_matmul_rows(X, W, rows=np.array([7, 2]), gamma=gam), Z[[7, 2]])


def test_legal_rewrite_row_scale_after_the_matmul():
    # Section 5: MatMul(Multiply(X, rsqrt), W) == Multiply(MatMul(X, W), rsqrt) since rsqrt is invariant over k
    inp = I.custom_inputs(6, 96, 64, 82)
    X, W = inp.bits("X"), inp.bits("Wg")
    Z = oracle.rmsnorm_matmul_rows(X, W, eps=1e-6)
    xd, wd = inp.X.double().numpy(), inp.Wg.double().numpy()
    r = 1.0 / np.sqrt(np.mean(xd * xd, axis=1, keepdims=True) + float(np.float32(1e-6)))
    rewritten = oracle.naive_matmul(xd, wd) * r
    assert np.allclose(Z, rewritten, rtol=1e-12, atol=1e-14)


def test_invariances_and_closed_forms():
    inp = I.custom_inputs(4, 64, 48, 83, rmsnorm=True)
    W, gam = inp.bits("Wg"), inp.bits("gamma")
    base = oracle.rmsnorm_matmul_rows(inp.bits("X"), W, gamma=gam, eps=0.0)
    Xs = inp.X.clone(); Xs[0] *= 4.0; Xs[2] *= 0.125
    assert np.allclose(oracle.rmsnorm_matmul_rows(_bits(Xs), W, gamma=gam, eps=0.0), base, rtol=1e-14, atol=0)
    assert np.all(oracle.rmsnorm_matmul_rows(inp.bits("X"), np.zeros_like(W), gamma=gam) == 0.0)
    # constant row, eps = 0: xn = sign(c) * gamma  =>  z_n = sign(c) * sum_k gamma_k w_kn
    row = _bits(torch.full((1, 64), -3.0))
    z = oracle.rmsnorm_matmul_rows(row, W, gamma=gam, eps=0.0)[0]
    want = -(inp.gamma.double().numpy() @ inp.Wg.double().numpy())
    assert np.allclose(z, want, rtol=1e-13, atol=1e-14)
    # one-hot W picks a normalised column: z_n = x_n * r
    Wsel = np.zeros((64, 48), np.uint16); one = _bits(torch.ones(1))[0]
    for n in range(48):
        Wsel[n, n] = one
    xd = inp.X.double().numpy()
    r = 1.0 / np.sqrt(np.mean(xd * xd, axis=1, keepdims=True) + float(np.float32(1e-5)))
    assert np.allclose(oracle.rmsnorm_matmul_rows(inp.bits("X"), Wsel, eps=1e-5), (xd * r)[:, :48], rtol=1e-14, atol=0)
