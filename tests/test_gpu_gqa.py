"""GPU parity of gmlp_gqa_attention (Group Query Attention, Section 6.1) against the CPU oracle:
|o - o_ref| <= 2e-2 * max(1, |o_ref|), ragged M and S, several group sizes, and closed-form cases."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2606_26344_b200 import gmlp

pytestmark = pytest.mark.gpu
D = 128


def _bits(t):
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def _case(M, S, Hq, Hkv, seed, q_scale=1.0):
    g = torch.Generator().manual_seed(seed)
    Q = (torch.randn(M, Hq * D, generator=g) * q_scale).to(torch.bfloat16)
    K = torch.randn(S, Hkv * D, generator=g).to(torch.bfloat16)
    V = torch.randn(S, Hkv * D, generator=g).to(torch.bfloat16)
    return Q, K, V


def _check(M, S, Hq, Hkv, seed, q_scale=1.0, max_rows=64, causal=False):
    Q, K, V = _case(M, S, Hq, Hkv, seed, q_scale)
    dev = torch.device("cuda")
    O = torch.full((M, Hq * D), float("nan"), dtype=torch.bfloat16, device=dev)
    gmlp.gqa_attention(Q.to(dev), K.to(dev), V.to(dev), Hq, Hkv, O=O, checked=True, causal=causal)
    torch.cuda.synchronize()
    assert bool(torch.isfinite(O.float()).all())
    rows = np.arange(M) if M <= max_rows else np.sort(np.random.default_rng(seed).choice(M, max_rows, replace=False))
    if causal and M > max_rows:          # the first and the last rows of the mask matter most
        rows = np.unique(np.concatenate([rows, np.arange(4), np.arange(M - 4, M), np.array([127, 128, 255, 256])[:0 if M < 257 else 4]]))
    ref = oracle.gqa_rows(_bits(Q), _bits(K), _bits(V), Hq, Hkv, rows=rows, causal=causal)
    got = O[torch.as_tensor(rows, device=dev)].float().cpu().numpy().astype(np.float64)
    e = np.abs(got - ref) / oracle.tolerance(ref)
    assert e.max() <= 1.0, f"max err/tol {e.max():.3f}"
    return e.max()


@pytest.mark.parametrize("shape", [(128, 128, 2, 1), (1, 1, 1, 1), (1, 300, 4, 4), (17, 200, 4, 2), (300, 129, 8, 2),
                                   (129, 1000, 6, 3), (256, 1024, 4, 1), (1030, 64, 2, 2)])
def test_small_and_ragged(shape):
    _check(*shape, seed=50 + shape[0])


@pytest.mark.parametrize("shape", [(128, 128, 2, 1), (1, 1, 1, 1), (1, 300, 4, 4), (17, 200, 4, 2), (300, 300, 8, 2),
                                   (129, 1000, 6, 3), (256, 256, 4, 1), (700, 700, 2, 2), (1030, 1100, 2, 1)])
def test_causal_small_and_ragged(shape):
    _check(*shape, seed=150 + shape[0], causal=True)


def test_causal_llama_like_block_and_first_rows_exact():
    _check(2048, 2048, 32, 8, seed=4, causal=True)
    # row 0 sees key 0 only: its output is V[0] of its group exactly
    dev = torch.device("cuda")
    Q, K, V = _case(300, 300, 4, 2, 8)
    O = gmlp.gqa_attention(Q.to(dev), K.to(dev), V.to(dev), 4, 2, checked=True, causal=True).cpu()
    want = V[:1].view(1, 2, D).repeat_interleave(2, dim=1).reshape(4 * D)
    assert torch.equal(O[0].view(torch.int16), want.contiguous().view(torch.int16))
    # S < M is refused
    with pytest.raises(gmlp.GmlpError) as e:
        gmlp.gqa_attention(Q.to(dev), K[:200].to(dev), V[:200].to(dev), 4, 2, causal=True)
    assert e.value.status == gmlp.ERR_SHAPE


def test_peaked_softmax_and_large_scores():
    # queries scaled up: scores of +-100 and a softmax concentrated on a few keys (the running maximum moves a lot)
    _check(200, 700, 4, 2, seed=7, q_scale=6.0)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("slope", [0.02, 1.0, 20.0])
def test_scores_that_rise_along_the_keys_move_the_base_in_every_block(slope, causal):
    """Key j is (1 + slope * j) times one direction and every query is a multiple of it, so a row's scores rise along the
    keys: gently (a block's sum of exponentials with the old base stays moderate), by hundreds or by thousands of
    binary orders per block (the exponentials with the old base overflow and the block has to be redone with a new
    one).  Against the oracle, and against the closed form for the steepest case: the softmax is one-hot on the last
    key a row may see."""
    M, S, Hq, Hkv = 300, 700, 4, 2
    g = torch.Generator().manual_seed(11)
    u = torch.randn(D, generator=g)
    u = u / u.norm() * 4.0
    ramp = 1.0 + slope * torch.arange(S, dtype=torch.float32)
    K = (ramp[:, None] * u[None, :]).repeat(1, Hkv).to(torch.bfloat16)
    Q = ((1.0 + torch.rand(M, 1, generator=g)) * u[None, :]).repeat(1, Hq).to(torch.bfloat16)
    V = torch.randn(S, Hkv * D, generator=g).to(torch.bfloat16)
    dev = torch.device("cuda")
    O = torch.full((M, Hq * D), float("nan"), dtype=torch.bfloat16, device=dev)
    gmlp.gqa_attention(Q.to(dev), K.to(dev), V.to(dev), Hq, Hkv, O=O, checked=True, causal=causal)
    torch.cuda.synchronize()
    assert bool(torch.isfinite(O.float()).all())
    rows = np.array([0, 1, 127, 128, 129, 255, 256, 257, 298, 299])
    ref = oracle.gqa_rows(_bits(Q), _bits(K), _bits(V), Hq, Hkv, rows=rows, causal=causal)
    got = O[torch.as_tensor(rows, device=dev)].float().cpu().numpy().astype(np.float64)
    e = np.abs(got - ref) / oracle.tolerance(ref)
    assert e.max() <= 1.0, f"max err/tol {e.max():.3f}"
    if slope == 20.0:                                    # adjacent keys differ by more than 40 nats
        last = (rows + (S - M)) if causal else np.full(len(rows), S - 1)
        want = V.float().numpy().astype(np.float64)[last]                        # [rows, Hkv * D]
        for h in range(Hq):
            gsel = slice((h // (Hq // Hkv)) * D, (h // (Hq // Hkv)) * D + D)
            assert np.abs(got[:, h * D:(h + 1) * D] - want[:, gsel]).max() <= 2e-2 * max(1.0, np.abs(want).max())


def test_llama_like_block():
    # 8B attention block: 32 query heads, 8 key/value heads of 128; 2048 tokens; 64 sampled query rows
    _check(2048, 2048, 32, 8, seed=3)


def test_closed_forms_on_device():
    dev = torch.device("cuda")
    Q, K, V = _case(70, 333, 4, 2, 9)
    # zero queries: every output row is the mean of its group's values
    O = gmlp.gqa_attention(torch.zeros_like(Q).to(dev), K.to(dev), V.to(dev), 4, 2, checked=True).float().cpu()
    vm = V.float().view(333, 2, D).mean(dim=0).repeat_interleave(2, dim=0).reshape(1, 4 * D)
    assert bool(((O - vm).abs() <= 2e-2).all())
    # a single key: the output is that key's value exactly (P = 1, one rounding of a bf16 value)
    O1 = gmlp.gqa_attention(Q.to(dev), K[:1].to(dev), V[:1].to(dev), 4, 2, checked=True).cpu()
    want = V[:1].view(1, 2, D).repeat_interleave(2, dim=1).reshape(1, 4 * D).expand(70, 4 * D)
    assert torch.equal(O1.view(torch.int16), want.contiguous().view(torch.int16))
    # deterministic
    a = gmlp.gqa_attention(Q.to(dev), K.to(dev), V.to(dev), 4, 2, checked=True)
    b = gmlp.gqa_attention(Q.to(dev), K.to(dev), V.to(dev), 4, 2, checked=True)
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))


def test_argument_checks():
    dev = torch.device("cuda")
    Q, K, V = _case(40, 50, 4, 2, 2)
    Qd, Kd, Vd = Q.to(dev), K.to(dev), V.to(dev)
    O = torch.empty_like(Qd)
    a = gmlp.make_gqa_args(Qd, Kd, Vd, O, 4, 2)
    f = lambda: gmlp.lib().gmlp_gqa_attention(ctypes.byref(a))
    assert f() == gmlp.OK
    a.head_dim = 64
    assert f() == gmlp.ERR_UNSUPPORTED
    a.head_dim = 128
    a.n_kv_heads = 3
    assert f() == gmlp.ERR_SHAPE
    a.n_kv_heads = 2
    a.flags = 1 << 9
    assert f() == gmlp.ERR_FLAGS
    a.flags = 0
    a.V = None
    assert f() == gmlp.ERR_NULL
    assert gmlp.lib().gmlp_gqa_attention(None) == gmlp.ERR_NULL
    torch.cuda.synchronize()
    assert gmlp.device_status() == 0
