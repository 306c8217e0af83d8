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
