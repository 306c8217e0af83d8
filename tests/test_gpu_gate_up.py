"""GPU parity of gmlp_gate_up (the gate/up half alone: Matmul+Matmul+SiLU+Mul of the paper's benchmark
list) against the CPU oracle, element by element: |h - p_ref| <= 2e-2 * max(1, |p_ref|), and, tighter,
one bf16 rounding step of the fp64 value plus the effect of fp32 accumulation."""
import numpy as np
import pytest
import torch

import oracle
from paper_2606_26344_b200 import gmlp, inputs as I

pytestmark = pytest.mark.gpu


def _check(inp, variant, rows=None):
    w = inp.workload
    dev = torch.device("cuda")
    X, Wg, Wu = inp.X.to(dev), inp.Wg.to(dev), inp.Wu.to(dev)
    gamma = inp.gamma.to(dev) if w.rmsnorm else None
    ws = gmlp.alloc_workspace(w.M, w.d_model, w.d_ff, w.rmsnorm, variant)
    H = torch.full((w.M, w.d_ff), float("nan"), dtype=torch.bfloat16, device=dev)
    gmlp.gate_up(X, Wg, Wu, H, gamma=gamma, eps=w.eps, rmsnorm=w.rmsnorm, variant=variant, workspace=ws, checked=True)
    torch.cuda.synchronize()
    assert bool(torch.isfinite(H.float()).all())
    if rows is None:
        rows = I.sample_rows(w, inp.outlier_rows)
    P = oracle.gate_up_rows(inp.bits("X"), inp.bits("Wg"), inp.bits("Wu"), rows=rows,
                            gamma=inp.bits("gamma") if w.rmsnorm else None, eps=w.eps, rmsnorm=w.rmsnorm)
    h = H[torch.as_tensor(rows, device=dev)].float().cpu().numpy().astype(np.float64)
    err = np.abs(h - P)
    assert np.all(err <= 2e-2 * np.maximum(1.0, np.abs(P)))
    rms = np.sqrt(np.mean(P * P, axis=1, keepdims=True))
    assert np.all(err <= np.abs(P) * 2.0 ** -7 + rms * 2.0 ** -8)


@pytest.mark.parametrize("rmsnorm", [False, True])
@pytest.mark.parametrize("variant,shape", [
    (gmlp.VARIANT_SKINNY, (1, 256, 512)), (gmlp.VARIANT_SKINNY, (8, 1032, 2056)), (gmlp.VARIANT_SKINNY, (100, 328, 1992)),
    (gmlp.VARIANT_UMMA, (130, 320, 392)), (gmlp.VARIANT_UMMA, (300, 512, 1024)),
    (gmlp.VARIANT_PAIR, (300, 512, 1024)), (gmlp.VARIANT_PAIR, (1300, 264, 520)),
    (gmlp.VARIANT_AUTO, (16, 256, 512)), (gmlp.VARIANT_AUTO, (520, 1024, 2816))])
def test_gate_up_alone(variant, shape, rmsnorm):
    M, dm, dff = shape
    _check(I.custom_inputs(M, dm, dff, 700 + M, rmsnorm=rmsnorm, eps=1e-6), variant)


@pytest.mark.parametrize("name", ["llama3-8b-decode-M8", "llama3-8b-prefill-M2048-rmsnorm", "ragged-M1000-norm"])
def test_gate_up_alone_on_stated_shapes(name):
    _check(I.make_inputs(I.WORKLOADS[name]), gmlp.VARIANT_AUTO)


def test_gate_up_matches_the_h_of_the_full_call_and_rejects_other_schedules():
    inp = I.custom_inputs(200, 512, 768, 3)
    dev = torch.device("cuda")
    X, Wg, Wu, Wd = (t.to(dev) for t in (inp.X, inp.Wg, inp.Wu, inp.Wd))
    ws = gmlp.alloc_workspace(200, 512, 768, False, gmlp.VARIANT_UMMA)
    gmlp.forward(X, Wg, Wu, Wd, variant=gmlp.VARIANT_UMMA, workspace=ws, checked=True)
    H_full = ws[: 200 * 768 * 2].view(torch.bfloat16).view(200, 768).clone()
    H = gmlp.gate_up(X, Wg, Wu, variant=gmlp.VARIANT_UMMA, checked=True)
    assert torch.equal(H.view(torch.int16), H_full.view(torch.int16))
    with pytest.raises(gmlp.GmlpError) as ei:
        gmlp.gate_up(X, Wg, Wu, variant=gmlp.VARIANT_SIMT)
    assert ei.value.status == gmlp.ERR_UNSUPPORTED
