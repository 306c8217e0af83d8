"""Pins for the oracle's gate activations other than SiLU (the SwiGLU- and GLU-gated forms of the
benchmark list, Section 6.1): Swish-beta g*sigmoid(beta*g) and GLU sigmoid(g).

Expected values are closed forms, identities, extended-precision arithmetic or library
routines; the whole-operator checks rebuild H from the separately compiled naive matmul.
"""
import math
from decimal import Decimal, getcontext

import numpy as np
import pytest
import torch

import oracle


def _bits(t):
    return t.to(torch.bfloat16).contiguous().view(torch.int16).numpy().view(np.uint16)


def _rand(M, dm, dff, seed):
    g = torch.Generator().manual_seed(seed)
    X = torch.randn(M, dm, generator=g)
    Wg, Wu = torch.randn(dm, dff, generator=g) / math.sqrt(dm), torch.randn(dm, dff, generator=g) / math.sqrt(dm)
    Wd = torch.randn(dff, dm, generator=g) / math.sqrt(dff)
    return tuple(_bits(t) for t in (X, Wg, Wu, Wd))


def test_swish_with_beta_one_is_silu_and_beta_zero_is_half():
    x = np.linspace(-60, 60, 6001)
    assert np.array_equal(oracle.gate_act(x, "swish", 1.0), oracle.silu(x))
    assert np.array_equal(oracle.gate_act(x, "silu"), oracle.silu(x))
    assert np.array_equal(oracle.gate_act(x, "swish", 0.0), x / 2.0)


def test_swish_scaling_identity_and_relu_limit():
    # swish_beta(g) = silu(beta g) / beta
    x = np.linspace(-20, 20, 2001)
    for beta in (0.25, 1.702, 3.0, -0.5):
        assert np.allclose(oracle.gate_act(x, "swish", beta), oracle.silu(beta * x) / beta, rtol=1e-14, atol=1e-300)
    big = oracle.gate_act(np.array([1.0, -1.0, 0.0]), "swish", 60.0)
    assert abs(big[0] - 1.0) < 1e-25 + 2e-16 and abs(big[1] + math.exp(-60.0)) < 1e-40 and big[2] == 0.0


def test_sigmoid_gate_closed_forms():
    s = oracle.gate_act(np.array([0.0, math.log(3.0), -math.log(3.0), 800.0, -800.0]), "glu")
    assert s[0] == 0.5 and abs(s[1] - 0.75) < 1e-15 and abs(s[2] - 0.25) < 1e-15
    assert s[3] == 1.0 and s[4] == 0.0
    x = np.linspace(-40, 40, 4001)
    sg = oracle.gate_act(x, "glu")
    assert np.allclose(sg + oracle.gate_act(-x, "glu"), 1.0, rtol=0, atol=5e-16)       # sigma(x) + sigma(-x) = 1
    assert np.all(np.diff(sg) >= 0)
    assert np.allclose(sg, torch.sigmoid(torch.tensor(x, dtype=torch.float64)).numpy(), rtol=1e-14, atol=1e-300)
    # silu(x) = x * sigma(x) ties the two pinned functions together
    assert np.allclose(x * sg, oracle.silu(x), rtol=1e-15, atol=1e-300)


def test_against_fifty_digit_arithmetic():
    getcontext().prec = 50
    for g, beta in ((0.3, 1.702), (-2.75, 0.5), (5.125, 2.0), (-0.001, 10.0)):
        d = Decimal(g) / (Decimal(1) + (-(Decimal(beta) * Decimal(g))).exp())
        got = float(oracle.gate_act(np.array([g]), "swish", beta)[0])
        assert abs(got - float(d)) <= 2e-16 * abs(float(d))
        s = Decimal(1) / (Decimal(1) + (-Decimal(g)).exp())
        assert abs(float(oracle.gate_act(np.array([g]), "glu")[0]) - float(s)) <= 2e-16 * float(s)


@pytest.mark.parametrize("act,beta", [("swish", 1.702), ("swish", 0.0), ("glu", 1.0)])
def test_whole_operator_against_naive_loops(act, beta):
    """H rebuilt from the naive triple-loop matmul (another translation unit) and the formula typed here."""
    M, dm, dff = 5, 24, 40
    X, Wg, Wu, Wd = _rand(M, dm, dff, 31)
    xd, wg, wu, wd = (oracle.bf16_to_double(t) for t in (X, Wg, Wu, Wd))
    G, U = oracle.naive_matmul(xd, wg), oracle.naive_matmul(xd, wu)
    if act == "glu":
        a = np.array([[1.0 / (1.0 + math.exp(-v)) for v in row] for row in G])
    else:
        a = np.array([[v / (1.0 + math.exp(-(beta * v))) for v in row] for row in G])
    Hb = oracle.bf16_rn(a * U)
    want = oracle.naive_matmul(oracle.bf16_to_double(Hb), wd)
    Y, H = oracle.gmlp_rows(X, Wg, Wu, Wd, act=act, beta=beta, want_h=True)
    assert np.array_equal(H, Hb)
    assert np.array_equal(Y, want)
    P = oracle.gate_up_rows(X, Wg, Wu, act=act, beta=beta)
    assert np.array_equal(P, a * U)


def test_zero_gate_weights_give_the_value_of_the_activation_at_zero():
    # G = 0: GLU gates with sigma(0) = 1/2 (Y = (U/2) Wd, a linear map), SiLU and Swish gate with 0
    M, dm, dff = 4, 16, 32
    X, Wg, Wu, Wd = _rand(M, dm, dff, 7)
    Z = np.zeros_like(Wg)
    xd, wu, wd = (oracle.bf16_to_double(t) for t in (X, Wu, Wd))
    half_u = oracle.bf16_to_double(oracle.bf16_rn(0.5 * (xd @ wu)))
    Y = oracle.gmlp_rows(X, Z, Wu, Wd, act="glu")
    assert np.allclose(Y, half_u @ wd, rtol=1e-13, atol=1e-13)
    assert np.all(oracle.gmlp_rows(X, Z, Wu, Wd, act="swish", beta=3.0) == 0.0)


def test_the_three_gates_differ_where_they_should():
    M, dm, dff = 3, 16, 32
    X, Wg, Wu, Wd = _rand(M, dm, dff, 9)
    y_silu = oracle.gmlp_rows(X, Wg, Wu, Wd)
    assert np.array_equal(oracle.gmlp_rows(X, Wg, Wu, Wd, act="swish", beta=1.0), y_silu)
    assert not np.allclose(oracle.gmlp_rows(X, Wg, Wu, Wd, act="swish", beta=2.0), y_silu, rtol=1e-3, atol=1e-3)
    assert not np.allclose(oracle.gmlp_rows(X, Wg, Wu, Wd, act="glu"), y_silu, rtol=1e-3, atol=1e-3)


def test_gelu_closed_forms_identities_and_library_routines():
    """GELU g * Phi(g), Phi the standard normal distribution function (the exact form)."""
    gelu = lambda v: oracle.gate_act(np.asarray(v, dtype=np.float64), "gelu")
    assert gelu([0.0])[0] == 0.0
    # Phi(x) + Phi(-x) = 1  =>  gelu(x) - gelu(-x) = x
    x = np.linspace(-12, 12, 4801)
    assert np.allclose(gelu(x) - gelu(-x), x, rtol=0, atol=4e-16 * np.maximum(1.0, np.abs(x)))
    # tabulated values of Phi: Phi(1) = 0.8413447460685429, Phi(-2) = 0.0227501319481792, Phi(3) = 0.9986501019683699
    assert abs(gelu([1.0])[0] - 0.8413447460685429) < 2e-16
    assert abs(gelu([-2.0])[0] + 2 * 0.0227501319481792) < 1e-16
    assert abs(gelu([3.0])[0] - 3 * 0.9986501019683699) < 1e-15
    # tails: gelu(x) -> x, gelu(-x) -> -0 with the relative accuracy of erfc kept (Phi(-10) = 7.619853024160527e-24)
    assert gelu([40.0])[0] == 40.0 and gelu([-40.0])[0] == 0.0
    assert abs(gelu([-10.0])[0] / (-10 * 7.619853024160527e-24) - 1.0) < 1e-13
    # the one minimum: gelu'(x) = Phi(x) + x phi(x) = 0 at x* = -0.7517915...; there Phi(x*) = -x* phi(x*), so the
    # minimum is -x*^2 phi(x*) with phi the normal density - an expression without erf
    fine = np.linspace(-0.76, -0.74, 200001)
    v = gelu(fine)
    xs = fine[int(np.argmin(v))]
    assert abs(xs + 0.751791524693564) < 2e-7
    xstar = -0.751791524693564                      # (the grid point is within 1e-7 of it, and gelu is flat there)
    assert abs(v.min() + xstar * xstar * math.exp(-xstar * xstar / 2.0) / math.sqrt(2.0 * math.pi)) < 1e-13
    assert abs(v.min() + 0.1699712) < 1e-7
    assert np.all(np.diff(gelu(np.linspace(-0.75, 12, 2000))) > 0) and np.all(np.diff(gelu(np.linspace(-12, -0.76, 2000))) < 0)
    # library routines: math.erf / erfc and torch's gelu (exact form) in float64
    pts = np.array([-6.5, -3.25, -1.0, -0.3, 0.002, 0.7, 2.5, 9.0])
    want = np.array([0.5 * t * math.erfc(-t / math.sqrt(2.0)) for t in pts])
    assert np.allclose(gelu(pts), want, rtol=1e-14, atol=0)
    tg = torch.nn.functional.gelu(torch.tensor(x, dtype=torch.float64), approximate="none").numpy()
    # (torch evaluates x (1 + erf(x / sqrt 2)) / 2, which is absolutely, not relatively, accurate in the negative tail)
    assert np.all(np.abs(gelu(x) - tg) <= 1e-12 * np.abs(tg) + 2.3e-16 * np.maximum(1.0, np.abs(x)))
    # and it is NOT the tanh approximation (which differs by up to 5e-4 around |x| = 2)
    tt = torch.nn.functional.gelu(torch.tensor(x, dtype=torch.float64), approximate="tanh").numpy()
    assert np.abs(gelu(x) - tt).max() > 1e-4


def test_gelu_gated_operator_is_built_from_the_pinned_pieces():
    X, Wg, Wu, Wd = _rand(5, 48, 80, 21)
    y, H = oracle.gmlp_rows(X, Wg, Wu, Wd, want_h=True, act="gelu")
    G = oracle.naive_matmul(oracle.bf16_to_double(X), oracle.bf16_to_double(Wg))
    U = oracle.naive_matmul(oracle.bf16_to_double(X), oracle.bf16_to_double(Wu))
    h = oracle.bf16_to_double(oracle.bf16_rn(oracle.gate_act(G, "gelu") * U))
    assert np.array_equal(oracle.bf16_to_double(H), h)
    assert np.array_equal(y, oracle.naive_matmul(h, oracle.bf16_to_double(Wd)))
    # and differs from the SiLU-gated operator
    assert np.abs(y - oracle.gmlp_rows(X, Wg, Wu, Wd)).max() > 1e-3
