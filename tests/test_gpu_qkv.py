"""GPU parity of gmlp_qkv_proj (the QKV projection of Section 6.1: three matmuls sharing X) against the CPU
oracle, one-launch and three-launch schedules, grouped-query shapes (Nkv < Nq) and ragged tails."""
import ctypes
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2606_26344_b200 import gmlp

pytestmark = pytest.mark.gpu


def _bits(t):
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def _case(M, K, Nq, Nkv, seed):
    g = torch.Generator().manual_seed(seed)
    X = torch.randn(M, K, generator=g).to(torch.bfloat16)
    Ws = [(torch.randn(K, n, generator=g) / math.sqrt(K)).to(torch.bfloat16) for n in (Nq, Nkv, Nkv)]
    return X, Ws


def _check(M, K, Nq, Nkv, seed, separate, max_rows=128):
    X, Ws = _case(M, K, Nq, Nkv, seed)
    dev = torch.device("cuda")
    outs = gmlp.qkv_proj(X.to(dev), *[w.to(dev) for w in Ws], separate=separate, checked=True)
    torch.cuda.synchronize()
    rows = np.arange(M) if M <= max_rows else np.sort(np.random.default_rng(seed).choice(M, max_rows, replace=False))
    refs = oracle.qkv_rows(_bits(X), *[_bits(w) for w in Ws], rows=rows)
    for name, o, r in zip("QKV", outs, refs):
        got = o[torch.as_tensor(rows, device=dev)].float().cpu().numpy().astype(np.float64)
        e = np.abs(got - r) / oracle.tolerance(r)
        assert np.isfinite(got).all() and e.max() <= 1.0, f"{name}: max err/tol {e.max():.3f}"
    return outs


@pytest.mark.parametrize("shape", [(128, 64, 256, 64), (1, 64, 128, 128), (17, 72, 136, 40), (129, 320, 520, 264),
                                   (300, 512, 1024, 256), (257, 1096, 648, 8), (1030, 264, 520, 136),
                                   (3100, 128, 776, 256)])
@pytest.mark.parametrize("separate", [False, True])
def test_small_and_ragged(shape, separate):
    _check(*shape, seed=20 + shape[0], separate=separate)


def test_llama_like_shape_and_schedules_agree_bit_for_bit():
    # 8B attention block: d_model 4096, 32 query heads and 8 key/value heads of 128
    a = _check(2048, 4096, 4096, 1024, 3, separate=False)
    b = _check(2048, 4096, 4096, 1024, 3, separate=True)
    for x, y in zip(a, b):
        assert torch.equal(x.view(torch.int16), y.view(torch.int16))       # same tiles, same order of the sums


def test_argument_checks():
    dev = torch.device("cuda")
    X, Ws = _case(40, 128, 256, 64, 2)
    Xd, (q, k, v) = X.to(dev), [w.to(dev) for w in Ws]
    Q = torch.empty(40, 256, dtype=torch.bfloat16, device=dev)
    K, V = torch.empty(40, 64, dtype=torch.bfloat16, device=dev), torch.empty(40, 64, dtype=torch.bfloat16, device=dev)
    a = gmlp.make_qkv_args(Xd, q, k, v, Q, K, V)
    f = lambda: gmlp.lib().gmlp_qkv_proj(ctypes.byref(a))
    assert f() == gmlp.OK
    a.flags = 1 << 9
    assert f() == gmlp.ERR_FLAGS
    a.flags = 0
    a.Wv = None
    assert f() == gmlp.ERR_NULL
    a.Wv = v.data_ptr()
    a.Nkv = 60
    assert f() == gmlp.ERR_SHAPE
    a.Nkv = 64
    a.reserved = 1
    assert f() == gmlp.ERR_FLAGS
    assert gmlp.lib().gmlp_qkv_proj(None) == gmlp.ERR_NULL
    torch.cuda.synchronize()
    assert gmlp.device_status() == 0
