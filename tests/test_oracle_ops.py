"""Pins for the oracle's SiLU and RMSNorm against closed forms and invariants.

silu(x) = x * sigmoid(x) (granular-operation table, Section 5); RMSNorm is Eq. (1) of
Section 2.  Expected values are mathematical facts or library routines, never the oracle.
"""
import math

import numpy as np
import torch

import oracle
from paper_2606_26344_b200 import inputs as I


def _bits(t):
    return t.to(torch.bfloat16).contiguous().view(torch.int16).numpy().view(np.uint16)


def test_silu_closed_forms():
    assert oracle.silu(np.array([0.0]))[0] == 0.0
    x = np.linspace(-40, 40, 4001)
    s = oracle.silu(x)
    # sigma(x) + sigma(-x) = 1  =>  silu(x) - silu(-x) = x
    assert np.allclose(s - oracle.silu(-x), x, rtol=0, atol=1e-13)
    # library routine
    want = torch.nn.functional.silu(torch.tensor(x, dtype=torch.float64)).numpy()
    assert np.allclose(s, want, rtol=1e-14, atol=1e-300)
    # textbook value at 1: 1/(1+e^-1)
    assert abs(oracle.silu(np.array([1.0]))[0] - 1.0 / (1.0 + math.exp(-1.0))) < 1e-16


def test_silu_minimum_and_tails():
    # The minimum of x*sigmoid(x) solves 1 + x + e^-x ... = 0 i.e. x = -(1 + W(1/e));
    # numerically x* = -1.2784645427610738, silu(x*) = -0.2784645427610738 (= x* + 1).
    xs = np.linspace(-1.3, -1.25, 200001)
    s = oracle.silu(xs)
    i = int(np.argmin(s))
    assert abs(xs[i] - (-1.2784645427610738)) < 1e-6
    assert abs(s[i] - (-0.2784645427610738)) < 1e-12
    assert abs(s[i] - (xs[i] + 1.0)) < 1e-6
    big = oracle.silu(np.array([50.0, 1e4, -1e4, -800.0]))
    assert big[0] == 50.0 / (1.0 + math.exp(-50.0)) and big[1] == 1e4
    assert big[2] == 0.0 and np.signbit(big[2]) and big[3] == 0.0        # -0, never NaN


def test_rmsnorm_unit_rms_before_gain():
    g = torch.Generator().manual_seed(3)
    for d, eps in ((4096, 1e-5), (2048, 1e-6), (256, 1e-5)):
        x = torch.randn(d, generator=g)
        xb = _bits(x)
        xd = oracle.bf16_to_double(xb)
        _, r = oracle.rmsnorm_row(xb, None, eps)
        ms = float(np.mean(xd * xd))
        # rms of x*r is sqrt(ms/(ms+eps)): one, up to the eps term
        rms = math.sqrt(float(np.mean((xd * r) ** 2)))
        assert abs(rms - math.sqrt(ms / (ms + float(np.float32(eps))))) < 1e-14
        assert abs(rms - 1.0) < 2 * eps
        # the rounded output has unit rms up to bf16 rounding noise (2^-9 relative per element)
        xn, _ = oracle.rmsnorm_row(xb, None, eps)
        rms_b = math.sqrt(float(np.mean(oracle.bf16_to_double(xn) ** 2)))
        assert abs(rms_b - 1.0) < 1e-3


def test_rmsnorm_against_torch_fp64_and_gain_position():
    g = torch.Generator().manual_seed(4)
    d, eps = 512, 1e-5
    x = torch.randn(d, generator=g).to(torch.bfloat16)
    gamma = (torch.rand(d, generator=g) + 0.5).to(torch.bfloat16)
    xd, gd = x.double(), gamma.double()
    eps32 = float(np.float32(eps))
    want_val = xd * torch.rsqrt((xd * xd).mean() + eps32) * gd
    xn, r = oracle.rmsnorm_row(_bits(x), _bits(gamma), eps)
    got = oracle.bf16_to_double(xn)
    # single rounding of the fp64 value: within half a bf16 ulp (at most 2^-8 relative) of it
    assert np.all(np.abs(got - want_val.numpy()) <= np.abs(want_val.numpy()) * 2.0 ** -8)
    assert abs(r - float(torch.rsqrt((xd * xd).mean() + eps32))) < 1e-15
    # gamma == None is gamma == 1
    ones = torch.ones(d, dtype=torch.bfloat16)
    a, _ = oracle.rmsnorm_row(_bits(x), None, eps)
    b, _ = oracle.rmsnorm_row(_bits(x), _bits(ones), eps)
    assert np.array_equal(a, b)


def test_rmsnorm_scale_invariance_and_constant_row():
    g = torch.Generator().manual_seed(5)
    x = torch.randn(384, generator=g).to(torch.bfloat16)
    base, _ = oracle.rmsnorm_row(_bits(x), None, 0.0)
    for p in (-3, 2, 7):
        scaled, _ = oracle.rmsnorm_row(_bits(x * (2.0 ** p)), None, 0.0)
        assert np.array_equal(base, scaled)
    for c in (3.0, -0.5):
        row = torch.full((128,), c).to(torch.bfloat16)
        out, _ = oracle.rmsnorm_row(_bits(row), None, 0.0)
        assert np.all(oracle.bf16_to_double(out) == math.copysign(1.0, c))
        eps = 1e-2
        out, _ = oracle.rmsnorm_row(_bits(row), None, eps)
        want = c / math.sqrt(c * c + float(np.float32(eps)))
        assert np.all(out == oracle.bf16_rn(np.array([want]))[0])


def test_tolerance_rule():
    y_ref = np.array([0.0, 0.5, -1.0, 10.0, -250.0])
    tol = oracle.tolerance(y_ref)
    assert np.allclose(tol, [0.02, 0.02, 0.02, 0.2, 5.0])


def test_workload_table_matches_the_stated_configs():
    w = I.WORKLOADS
    assert (w["tiny"].M, w["tiny"].d_model, w["tiny"].d_ff) == (16, 256, 512)
    d = w["llama3-8b-decode-M8"]
    assert (d.M, d.d_model, d.d_ff, d.rmsnorm) == (8, 4096, 14336, False)
    assert 3 * d.d_model * d.d_ff * 2 == 352321536            # "about 352 MB of weights"
    p = w["llama3-8b-prefill-M2048-rmsnorm"]
    assert (p.M, p.rmsnorm, p.eps) == (2048, True, 1e-5)
    q = w["llama3-70b-prefill-M4096-outliers"]
    assert (q.M, q.d_model, q.d_ff, q.outlier_frac) == (4096, 8192, 28672, 0.01)
    for M, s in zip((1, 7, 129, 1000, 8192), (1, 2, 3, 4, 5)):
        for n in ("plain", "norm"):
            r = w[f"ragged-M{M}-{n}"]
            assert (r.M, r.d_model, r.d_ff, r.seed, r.eps) == (M, 2048, 5632, s, 1e-6)


def test_inputs_are_seeded_and_have_the_stated_statistics():
    w = I.Workload("t", 300, 512, 768, 7, rmsnorm=True, outlier_frac=0.01)
    a, b = I.make_inputs(w), I.make_inputs(w)
    for n in ("X", "Wg", "Wu", "Wd", "gamma"):
        assert np.array_equal(a.bits(n), b.bits(n))
    assert a.outlier_rows.size == 3
    assert abs(a.Wg.float().std().item() - 512 ** -0.5) < 2e-3
    assert abs(a.Wd.float().std().item() - 768 ** -0.5) < 2e-3
    assert 0.5 <= a.gamma.float().min().item() and a.gamma.float().max().item() <= 1.5
    normal = np.setdiff1d(np.arange(300), a.outlier_rows)
    assert abs(a.X.float()[normal].std().item() - 1.0) < 0.02
    assert abs(a.X.float()[a.outlier_rows].std().item() - 20.0) < 2.0
    rows = I.sample_rows(w, a.outlier_rows)
    assert rows.size == 256 and np.unique(rows).size == 256
    assert np.intersect1d(rows, a.outlier_rows).size == 3
    assert np.array_equal(rows, I.sample_rows(w, a.outlier_rows))
    small = I.Workload("s", 16, 64, 64, 0)
    assert np.array_equal(I.sample_rows(small, np.zeros(0, dtype=np.int64)), np.arange(16))
