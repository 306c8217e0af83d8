"""Pins for the oracle's MatMul+Add+RMSNorm ("Matmul+Add+RMSNorm" of the benchmark list, Section 6.1):
S = X W + R stored in bf16 with one rounding, Z = RMSNorm(S) by Eq. (1) on the stored S.
Expected values: torch fp64, the separately compiled textbook matmul, closed forms, invariants."""
import math

import numpy as np
import torch

import oracle
from paper_2606_26344_b200 import inputs as I


def _bits(t):
    return t.to(torch.bfloat16).contiguous().view(torch.int16).numpy().view(np.uint16)


def _case(M, K, N, seed):
    g = torch.Generator().manual_seed(seed)
    X = torch.randn(M, K, generator=g).to(torch.bfloat16)
    W = (torch.randn(K, N, generator=g) / math.sqrt(K)).to(torch.bfloat16)
    R = torch.randn(M, N, generator=g).to(torch.bfloat16)
    gam = (0.5 + torch.rand(N, generator=g)).to(torch.bfloat16)
    return X, W, R, gam


def test_against_torch_fp64_and_naive_loops():
    X, W, R, gam = _case(7, 40, 72, 3)
    eps = float(np.float32(1e-5))
    Sb, Sr, Z = oracle.matmul_add_rmsnorm_rows(_bits(X), _bits(W), _bits(R), gamma=_bits(gam), eps=1e-5)
    s_want = (X.double() @ W.double() + R.double()).numpy()
    assert np.allclose(Sr, s_want, rtol=1e-13, atol=1e-14)
    naive = oracle.naive_matmul(X.double().numpy(), W.double().numpy()) + R.double().numpy()
    assert np.allclose(Sr, naive, rtol=1e-14, atol=1e-15)
    # the stored S: one rounding of the fp64 sum (library conversion from the same fp64 values, away from ties)
    sb_t = torch.tensor(Sr).to(torch.bfloat16)
    assert np.array_equal(Sb, _bits(sb_t))
    # RMSNorm of the STORED S, with the gain
    sd = sb_t.double()
    r = torch.rsqrt((sd * sd).mean(dim=1, keepdim=True) + eps)
    assert np.allclose(Z, (sd * r * gam.double()).numpy(), rtol=1e-13, atol=1e-15)
    # gain of ones == no gain; row subsets
    ones = _bits(torch.ones(72))
    a = oracle.matmul_add_rmsnorm_rows(_bits(X), _bits(W), _bits(R), eps=1e-5)[2]
    b = oracle.matmul_add_rmsnorm_rows(_bits(X), _bits(W), _bits(R), gamma=ones, eps=1e-5)[2]
    assert np.array_equal(a, b)
    sub = oracle.matmul_add_rmsnorm_rows(_bits(X), _bits(W), _bits(R), rows=np.array([5, 0]), gamma=_bits(gam), eps=1e-5)
    assert np.array_equal(sub[2], Z[[5, 0]]) and np.array_equal(sub[0], Sb[[5, 0]])


def test_reduces_to_the_pinned_rmsnorm_row():
    # X = 0: S = R exactly, and Z is Eq. (1) on R, which the prologue oracle (pinned on its own) also computes
    X, W, R, gam = _case(5, 16, 64, 4)
    Sb, _, Z = oracle.matmul_add_rmsnorm_rows(_bits(torch.zeros_like(X)), _bits(W), _bits(R), gamma=_bits(gam), eps=1e-6)
    assert np.array_equal(Sb, _bits(R))
    for i in range(5):
        xn, r = oracle.rmsnorm_row(_bits(R[i]), _bits(gam), 1e-6)
        want = R[i].double().numpy() * r * gam.double().numpy()
        assert np.allclose(Z[i], want, rtol=1e-14, atol=1e-300)
        assert np.array_equal(oracle.bf16_rn(Z[i]), xn)
    # R = 0 and W = identity: S = X exactly
    Xs = torch.randn(4, 32, generator=torch.Generator().manual_seed(5)).to(torch.bfloat16)
    Sb2, _, Z2 = oracle.matmul_add_rmsnorm_rows(_bits(Xs), _bits(torch.eye(32)), _bits(torch.zeros(4, 32)), eps=1e-5)
    assert np.array_equal(Sb2, _bits(Xs))
    xd = Xs.double().numpy()
    assert np.allclose(Z2, xd / np.sqrt(np.mean(xd * xd, axis=1, keepdims=True) + float(np.float32(1e-5))), rtol=1e-14)


def test_unit_rms_scale_invariance_and_sign():
    X, W, R, _ = _case(6, 48, 128, 6)
    Sb, _, Z = oracle.matmul_add_rmsnorm_rows(_bits(X), _bits(W), _bits(R), eps=1e-6)
    sd = oracle.bf16_to_double(Sb)
    ms = np.mean(sd * sd, axis=1)
    rms = np.sqrt(np.mean(Z * Z, axis=1))
    assert np.allclose(rms, np.sqrt(ms / (ms + float(np.float32(1e-6)))), rtol=1e-13)
    # scaling X and R by 4 (exact in bf16) scales S by 4 exactly and leaves Z unchanged up to the eps term
    _, _, Z4 = oracle.matmul_add_rmsnorm_rows(_bits(X * 4), _bits(W), _bits(R * 4), eps=1e-6)
    assert np.allclose(Z4, Z, rtol=1e-5, atol=1e-7) and not np.array_equal(Z4, Z)
    # negating X and R negates Z
    _, _, Zn = oracle.matmul_add_rmsnorm_rows(_bits(-X), _bits(W), _bits(-R), eps=1e-6)
    assert np.array_equal(Zn, -Z)


def test_the_residual_is_added_before_the_norm_and_the_norm_runs_along_n():
    X, W, R, gam = _case(3, 24, 40, 8)
    _, _, Z = oracle.matmul_add_rmsnorm_rows(_bits(X), _bits(W), _bits(R), gamma=_bits(gam), eps=1e-5)
    # norm first, residual after (a wrong order) gives something else
    sd = (X.double() @ W.double())
    r = torch.rsqrt((sd * sd).mean(dim=1, keepdim=True) + 1e-5)
    wrong = (sd * r * gam.double() + R.double()).numpy()
    assert not np.allclose(Z, wrong, rtol=1e-2, atol=1e-2)
    # a norm along M instead of N gives something else
    s = (X.double() @ W.double() + R.double())
    wrong2 = (s * torch.rsqrt((s * s).mean(dim=0, keepdim=True) + 1e-5) * gam.double()).numpy()
    assert not np.allclose(Z, wrong2, rtol=1e-2, atol=1e-2)
    # transposed W would not even have the right shape unless square: use a square case
    Xq, Wq, Rq, _ = _case(3, 32, 32, 9)
    a = oracle.matmul_add_rmsnorm_rows(_bits(Xq), _bits(Wq), _bits(Rq))[1]
    b = oracle.matmul_add_rmsnorm_rows(_bits(Xq), _bits(Wq.t().contiguous()), _bits(Rq))[1]
    assert not np.allclose(a, b, rtol=1e-3, atol=1e-3)
    assert np.allclose(a, (Xq.double() @ Wq.double() + Rq.double()).numpy(), rtol=1e-13, atol=1e-14)


def test_integer_inputs_are_exact_and_bad_arguments_rejected():
    g = torch.Generator().manual_seed(10)
    X = torch.randint(-3, 4, (4, 16), generator=g).float()
    W = torch.randint(-2, 3, (16, 24), generator=g).float()
    R = torch.randint(-5, 6, (4, 24), generator=g).float()
    Sb, Sr, _ = oracle.matmul_add_rmsnorm_rows(_bits(X), _bits(W), _bits(R))
    want = (X.long() @ W.long() + R.long()).numpy()
    assert np.array_equal(Sr, want.astype(np.float64))
    assert np.array_equal(oracle.bf16_to_double(Sb), want.astype(np.float64))      # |S| < 256: exact in bf16
    import pytest
    with pytest.raises(ValueError):
        oracle.matmul_add_rmsnorm_rows(_bits(X), _bits(W), _bits(R[:, :8]))
    with pytest.raises(RuntimeError):
        oracle.matmul_add_rmsnorm_rows(_bits(X), _bits(W), _bits(R), rows=np.array([4]))
