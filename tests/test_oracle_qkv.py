"""Pins for the oracle's plain matmul on selected rows and the QKV projection built from it (Section 6.1:
three matmuls that share X): the separately compiled textbook loops, torch fp64, closed forms."""
import math

import numpy as np
import pytest
import torch

import oracle


def _bits(t):
    return t.to(torch.bfloat16).contiguous().view(torch.int16).numpy().view(np.uint16)


def _case(M, K, Nq, Nkv, seed):
    g = torch.Generator().manual_seed(seed)
    X = torch.randn(M, K, generator=g).to(torch.bfloat16)
    Ws = [(torch.randn(K, n, generator=g) / math.sqrt(K)).to(torch.bfloat16) for n in (Nq, Nkv, Nkv)]
    return X, Ws


def test_matmul_rows_against_naive_loops_and_torch():
    X, (W, _, _) = _case(9, 40, 56, 8, 1)
    Z = oracle.matmul_rows(_bits(X), _bits(W))
    naive = oracle.naive_matmul(X.double().numpy(), W.double().numpy())
    assert np.array_equal(Z, naive)                     # same ascending-k sum, another translation unit
    assert np.allclose(Z, (X.double() @ W.double()).numpy(), rtol=1e-13, atol=1e-14)
    assert np.array_equal(oracle.matmul_rows(_bits(X), _bits(W), rows=np.array([8, 3, 3])), Z[[8, 3, 3]])
    # a transposed weight gives something else (square case)
    Xs, (Ws, _, _) = _case(4, 32, 32, 8, 2)
    a = oracle.matmul_rows(_bits(Xs), _bits(Ws))
    b = oracle.matmul_rows(_bits(Xs), _bits(Ws.t().contiguous()))
    assert not np.allclose(a, b, rtol=1e-3, atol=1e-3)


def test_matmul_rows_closed_forms():
    X, _ = _case(5, 24, 8, 8, 3)
    eye = torch.eye(24)
    assert np.array_equal(oracle.matmul_rows(_bits(X), _bits(eye)), X.double().numpy())
    ones = torch.ones(24, 8)
    assert np.allclose(oracle.matmul_rows(_bits(X), _bits(ones)), X.double().sum(dim=1, keepdim=True).expand(5, 8).numpy(),
                       rtol=1e-14, atol=1e-14)
    g = torch.Generator().manual_seed(4)
    Xi = torch.randint(-4, 5, (6, 16), generator=g).float()
    Wi = torch.randint(-3, 4, (16, 24), generator=g).float()
    assert np.array_equal(oracle.matmul_rows(_bits(Xi), _bits(Wi)), (Xi.long() @ Wi.long()).numpy().astype(np.float64))
    with pytest.raises(ValueError):
        oracle.matmul_rows(_bits(X), _bits(torch.ones(8, 8)))
    with pytest.raises(RuntimeError):
        oracle.matmul_rows(_bits(X), _bits(eye), rows=np.array([5]))


def test_qkv_is_three_independent_products_of_the_same_x():
    X, (Wq, Wk, Wv) = _case(7, 48, 64, 16, 5)
    Q, K, V = oracle.qkv_rows(_bits(X), _bits(Wq), _bits(Wk), _bits(Wv))
    assert Q.shape == (7, 64) and K.shape == (7, 16) and V.shape == (7, 16)
    # equal to one product with the column-concatenated weight, split again
    cat = torch.cat([Wq, Wk, Wv], dim=1)
    Z = (X.double() @ cat.double()).numpy()
    assert np.allclose(np.concatenate([Q, K, V], axis=1), Z, rtol=1e-13, atol=1e-14)
    # changing Wv changes V only
    Q2, K2, V2 = oracle.qkv_rows(_bits(X), _bits(Wq), _bits(Wk), _bits(Wv * 2))
    assert np.array_equal(Q2, Q) and np.array_equal(K2, K) and np.array_equal(V2, 2 * V)
