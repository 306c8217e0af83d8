"""Pins for the oracle's Group Query Attention (Section 6.1 names the kernel; the definition is the standard
one, no mask): a library routine in fp64, closed forms, invariants, and the head-to-group mapping."""
import math

import numpy as np
import pytest
import torch

import oracle


def _bits(t):
    return t.to(torch.bfloat16).contiguous().view(torch.int16).numpy().view(np.uint16)


def _case(M, S, Hq, Hkv, D, seed):
    g = torch.Generator().manual_seed(seed)
    Q = torch.randn(M, Hq * D, generator=g).to(torch.bfloat16)
    K = torch.randn(S, Hkv * D, generator=g).to(torch.bfloat16)
    V = torch.randn(S, Hkv * D, generator=g).to(torch.bfloat16)
    return Q, K, V


def _torch_ref(Q, K, V, Hq, Hkv):
    M, S = Q.shape[0], K.shape[0]
    D = Q.shape[1] // Hq
    q = Q.double().view(M, Hq, D).transpose(0, 1)                       # [Hq, M, D]
    k = K.double().view(S, Hkv, D).transpose(0, 1).repeat_interleave(Hq // Hkv, dim=0)
    v = V.double().view(S, Hkv, D).transpose(0, 1).repeat_interleave(Hq // Hkv, dim=0)
    o = torch.nn.functional.scaled_dot_product_attention(q, k, v)       # library routine, fp64
    return o.transpose(0, 1).reshape(M, Hq * D).numpy()


@pytest.mark.parametrize("shape", [(5, 7, 4, 2, 8), (3, 33, 8, 2, 16), (4, 16, 2, 2, 32), (2, 9, 6, 1, 8)])
def test_against_the_library_attention_in_fp64(shape):
    M, S, Hq, Hkv, D = shape
    Q, K, V = _case(*shape, seed=11)
    O = oracle.gqa_rows(_bits(Q), _bits(K), _bits(V), Hq, Hkv)
    assert np.allclose(O, _torch_ref(Q, K, V, Hq, Hkv), rtol=1e-12, atol=1e-13)
    sub = oracle.gqa_rows(_bits(Q), _bits(K), _bits(V), Hq, Hkv, rows=np.array([M - 1, 0]))
    assert np.array_equal(sub, O[[M - 1, 0]])


def test_closed_forms():
    M, S, Hq, Hkv, D = 3, 6, 4, 2, 8
    Q, K, V = _case(M, S, Hq, Hkv, D, 12)
    # zero queries: uniform weights, every output row is the mean of its group's V
    O = oracle.gqa_rows(_bits(torch.zeros_like(Q)), _bits(K), _bits(V), Hq, Hkv)
    vm = V.double().view(S, Hkv, D).mean(dim=0)                         # [Hkv, D]
    want = vm.repeat_interleave(Hq // Hkv, dim=0).reshape(1, Hq * D).expand(M, Hq * D).numpy()
    assert np.allclose(O, want, rtol=1e-14, atol=1e-15)
    # a single key: the output is that key's value, whatever the query
    O1 = oracle.gqa_rows(_bits(Q), _bits(K[:1]), _bits(V[:1]), Hq, Hkv)
    want1 = V[:1].double().view(1, Hkv, D).repeat_interleave(Hq // Hkv, dim=1).reshape(1, Hq * D).expand(M, Hq * D).numpy()
    assert np.allclose(O1, want1, rtol=1e-15, atol=0)
    # one dominant key (score far above the rest): the output is its value up to e^-gap
    Kd = torch.zeros(S, Hkv * D)
    Kd[2] = 64.0
    Qd = torch.ones(M, Hq * D)
    Od = oracle.gqa_rows(_bits(Qd), _bits(Kd), _bits(V), Hq, Hkv)
    want_d = V[2:3].double().view(1, Hkv, D).repeat_interleave(Hq // Hkv, dim=1).reshape(1, Hq * D).expand(M, Hq * D).numpy()
    assert np.allclose(Od, want_d, rtol=0, atol=1e-12)


def test_invariants():
    M, S, Hq, Hkv, D = 4, 12, 4, 2, 16
    Q, K, V = _case(M, S, Hq, Hkv, D, 13)
    O = oracle.gqa_rows(_bits(Q), _bits(K), _bits(V), Hq, Hkv)
    # outputs are convex combinations of the group's values
    v = V.double().view(S, Hkv, D)
    for h in range(Hq):
        lo, hi = v[:, h // 2].min(dim=0).values.numpy(), v[:, h // 2].max(dim=0).values.numpy()
        o = O[:, h * D:(h + 1) * D]
        assert np.all(o >= lo - 1e-12) and np.all(o <= hi + 1e-12)
    # permuting the keys and values together changes nothing; adding a constant to V shifts O by it
    perm = torch.randperm(S, generator=torch.Generator().manual_seed(1))
    Op = oracle.gqa_rows(_bits(Q), _bits(K[perm]), _bits(V[perm]), Hq, Hkv)
    assert np.allclose(Op, O, rtol=1e-13, atol=1e-14)
    Oc = oracle.gqa_rows(_bits(Q), _bits(K), _bits(V.float() + 2.0), Hq, Hkv)
    assert np.allclose(Oc, oracle.gqa_rows(_bits(Q), _bits(K), _bits((V.float() + 2.0)), Hq, Hkv))
    vshift = (V.float() + 2.0).to(torch.bfloat16).double() - V.double()  # what the shift is after bf16 rounding
    assert np.allclose(Oc - O, _torch_ref(Q, K, vshift, Hq, Hkv), rtol=1e-10, atol=1e-12)
    # the scale is 1/sqrt(D): doubling Q is not the same as no scale
    assert not np.allclose(oracle.gqa_rows(_bits(Q * 2), _bits(K), _bits(V), Hq, Hkv), O, rtol=1e-3, atol=1e-3)


def test_head_to_group_mapping_and_bad_arguments():
    M, S, Hq, Hkv, D = 2, 5, 4, 2, 8
    Q, K, V = _case(M, S, Hq, Hkv, D, 14)
    O = oracle.gqa_rows(_bits(Q), _bits(K), _bits(V), Hq, Hkv)
    # changing the second key/value head changes query heads 2 and 3 only (consecutive heads share a group)
    V2 = V.clone()
    V2[:, D:] = V2[:, D:] * 2
    O2 = oracle.gqa_rows(_bits(Q), _bits(K), _bits(V2), Hq, Hkv)
    assert np.array_equal(O2[:, :2 * D], O[:, :2 * D]) and np.allclose(O2[:, 2 * D:], 2 * O[:, 2 * D:], rtol=1e-14)
    # Hq == Hkv is ordinary multi-head attention
    Qm, Km, Vm = _case(3, 6, 2, 2, 8, 15)
    assert np.allclose(oracle.gqa_rows(_bits(Qm), _bits(Km), _bits(Vm), 2, 2), _torch_ref(Qm, Km, Vm, 2, 2), rtol=1e-12)
    with pytest.raises(RuntimeError):
        oracle.gqa_rows(_bits(Q), _bits(K[:, :D]), _bits(V[:, :D]), 4, 3 if False else 1, rows=np.array([9]))
    with pytest.raises(ValueError):
        oracle.gqa_rows(_bits(Q), _bits(K), _bits(V[:, :D]), Hq, Hkv)


def _torch_ref_causal(Q, K, V, Hq, Hkv):
    M, S = Q.shape[0], K.shape[0]
    D = Q.shape[1] // Hq
    q = Q.double().view(M, Hq, D).transpose(0, 1)
    k = K.double().view(S, Hkv, D).transpose(0, 1).repeat_interleave(Hq // Hkv, dim=0)
    v = V.double().view(S, Hkv, D).transpose(0, 1).repeat_interleave(Hq // Hkv, dim=0)
    mask = torch.arange(S)[None, :] <= (torch.arange(M)[:, None] + (S - M))          # bottom-right aligned
    o = torch.nn.functional.scaled_dot_product_attention(q, k, v, attn_mask=mask)
    return o.transpose(0, 1).reshape(M, Hq * D).numpy()


@pytest.mark.parametrize("shape", [(6, 6, 4, 2, 8), (3, 11, 2, 1, 16), (1, 5, 2, 2, 8)])
def test_causal_against_the_library_attention_and_closed_forms(shape):
    M, S, Hq, Hkv, D = shape
    Q, K, V = _case(*shape, seed=21)
    O = oracle.gqa_rows(_bits(Q), _bits(K), _bits(V), Hq, Hkv, causal=True)
    assert np.allclose(O, _torch_ref_causal(Q, K, V, Hq, Hkv), rtol=1e-12, atol=1e-13)
    if M == S:
        # the first query sees the first key only: its output is that key's value; the last one sees everything
        want0 = V[:1].double().view(1, Hkv, D).repeat_interleave(Hq // Hkv, dim=1).reshape(Hq * D).numpy()
        assert np.allclose(O[0], want0, rtol=1e-15, atol=0)
        full = oracle.gqa_rows(_bits(Q), _bits(K), _bits(V), Hq, Hkv)
        assert np.array_equal(O[-1], full[-1]) and not np.allclose(O[0], full[0], rtol=1e-3, atol=1e-3)
    # keys beyond a row's horizon do not matter to it
    K2, V2 = K.clone(), V.clone()
    K2[-1] += 3.0
    V2[-1] -= 5.0
    O2 = oracle.gqa_rows(_bits(Q), _bits(K2), _bits(V2), Hq, Hkv, causal=True)
    if M > 1:
        assert np.array_equal(O2[:-1], O[:-1])


def test_causal_needs_at_least_as_many_keys_as_queries():
    Q, K, V = _case(4, 3, 2, 1, 8, seed=22)
    with pytest.raises(RuntimeError):
        oracle.gqa_rows(_bits(Q), _bits(K), _bits(V), 2, 1, causal=True)
