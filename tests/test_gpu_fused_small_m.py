"""GPU parity of the one-kernel ("fused") form of the small-M schedule against the CPU oracle: a thread-block cluster per
128-wide slice of d_ff runs gate/up, the activation and its rows of the down projection, and a second kernel adds the
slices' partial Y.  The form is forced on (and off, for the comparison) through the library's tuning variable, so that the
shapes below run it whether or not the default rule would take it."""
import numpy as np
import pytest
import torch

import oracle
from paper_2606_26344_b200 import gmlp, inputs as I

from _parity import to_device

pytestmark = pytest.mark.gpu

# (M, d_model, d_ff): clusters of 3 / 4 / 2 CTAs; a d_ff that ends inside a slice; a d_model that ends inside a k-block and
# inside a down tile; one token; the largest token count the form takes
SHAPES = [(7, 2048, 5632), (1, 2048, 5632), (16, 2048, 5632), (8, 1024, 4096), (5, 1536, 8960), (3, 2048, 5640),
          (9, 2056, 5632), (4, 3072, 8192),
          # drawn at random (multiples of 8) and kept for the cluster sizes they give: 8, 1, 6, 5, 4, 1 with the largest token
          # count, 6 with one token, 3 with twelve partial-Y tiles per CTA, 8 again with every dimension ragged
          (14, 1648, 1464), (6, 288, 11896), (7, 1104, 2296), (5, 2976, 2976), (9, 1768, 4192), (16, 272, 11792),
          (1, 2808, 2032), (12, 2512, 4320), (9, 2864, 1600)]


def _kernels_of(call):
    """Names of the kernels one call of the operator launches (the library's profiling marks)."""
    gmlp.profile_enable(True)
    try:
        call()
        torch.cuda.synchronize()
        return set(gmlp.profile_read())
    finally:
        gmlp.profile_enable(False)


def _forward(inp, rmsnorm, fused, monkeypatch, act="silu", beta=1.0, fp32=False, stream=None):
    monkeypatch.setenv("GMLP_SKINNY_FUSED", "1" if fused else "0")
    w = inp.workload
    t = to_device(inp)
    ws = gmlp.alloc_workspace(w.M, w.d_model, w.d_ff, rmsnorm, gmlp.VARIANT_SKINNY)
    Y = torch.full((w.M, w.d_model), float("nan"), dtype=torch.float32 if fp32 else torch.bfloat16, device="cuda")
    gmlp.forward(t["X"], t["Wg"], t["Wu"], t["Wd"], Y, gamma=t["gamma"] if rmsnorm else None, eps=w.eps, rmsnorm=rmsnorm,
                 variant=gmlp.VARIANT_SKINNY, workspace=ws, checked=True, act=act, beta=beta, stream=stream)
    torch.cuda.synchronize()
    return Y


def _reference(inp, rmsnorm, act="silu", beta=1.0):
    return oracle.gmlp_rows(inp.bits("X"), inp.bits("Wg"), inp.bits("Wu"), inp.bits("Wd"),
                            gamma=inp.bits("gamma") if rmsnorm else None, eps=inp.workload.eps, rmsnorm=rmsnorm, act=act, beta=beta)


@pytest.mark.parametrize("rmsnorm", [False, True])
@pytest.mark.parametrize("shape", SHAPES)
def test_fused_form_against_the_oracle(shape, rmsnorm, monkeypatch):
    M, dm, dff = shape
    assert gmlp.small_m_fused_plan(M, dm, dff)[0] >= 1, "the shape was chosen to have a fused plan"
    inp = I.custom_inputs(M, dm, dff, 700 + M, rmsnorm=rmsnorm, eps=1e-6)
    out = []
    names = _kernels_of(lambda: out.append(_forward(inp, rmsnorm, True, monkeypatch)))
    assert names == ({"rmsnorm", "fused", "sum"} if rmsnorm else {"fused", "sum"})        # that the form really ran
    Y = out[0]
    y_ref = _reference(inp, rmsnorm)
    e = np.abs(Y.float().cpu().numpy().astype(np.float64) - y_ref) / oracle.tolerance(y_ref)
    assert np.isfinite(Y.float().cpu().numpy()).all() and float(e.max()) <= 1.0, f"{shape}: max err/tol {float(e.max()):.3f}"
    # the same call again gives the same bits (the slices are added in a fixed order)
    Y2 = _forward(inp, rmsnorm, True, monkeypatch)
    assert torch.equal(Y.view(torch.int16), Y2.view(torch.int16))


@pytest.mark.parametrize("act,beta", [("swish", 1.702), ("glu", 1.0), ("gelu", 1.0)])
def test_fused_form_with_other_gate_activations(act, beta, monkeypatch):
    inp = I.custom_inputs(6, 2048, 5632, 731)
    Y = _forward(inp, False, True, monkeypatch, act=act, beta=beta)
    y_ref = _reference(inp, False, act=act, beta=beta)
    e = np.abs(Y.float().cpu().numpy().astype(np.float64) - y_ref) / oracle.tolerance(y_ref)
    assert float(e.max()) <= 1.0, f"{act}: max err/tol {float(e.max()):.3f}"


def test_fused_form_fp32_output_rounds_to_the_bf16_output(monkeypatch):
    inp = I.custom_inputs(7, 2048, 5632, 741)
    Yb = _forward(inp, False, True, monkeypatch)
    Yf = _forward(inp, False, True, monkeypatch, fp32=True)
    assert torch.equal(Yf.to(torch.bfloat16).view(torch.int16), Yb.view(torch.int16))
    y_ref = _reference(inp, False)
    e = np.abs(Yf.cpu().numpy().astype(np.float64) - y_ref) / oracle.tolerance(y_ref)
    assert float(e.max()) <= 1.0


def test_two_kernel_forms_still_run_where_the_fused_form_is_the_default(monkeypatch):
    M, dm, dff = 7, 2048, 5632
    assert gmlp.small_m_fused_plan(M, dm, dff)[4] == 1
    inp = I.custom_inputs(M, dm, dff, 751)
    out = []
    assert _kernels_of(lambda: out.append(_forward(inp, False, False, monkeypatch))) == {"gate_up", "down"}
    Y = out[0]
    y_ref = _reference(inp, False)
    e = np.abs(Y.float().cpu().numpy().astype(np.float64) - y_ref) / oracle.tolerance(y_ref)
    assert float(e.max()) <= 1.0


def test_fused_calls_on_two_streams_do_not_depend_on_each_other(monkeypatch):
    """Nothing in the fused kernel waits for another CTA of its grid through global memory, so two launches that share the
    GPU (each with its own workspace) both finish and both are right."""
    monkeypatch.setenv("GMLP_SKINNY_FUSED", "1")
    inps = [I.custom_inputs(7, 2048, 5632, 760 + i) for i in range(2)]
    ts = [to_device(i) for i in inps]
    streams = [torch.cuda.Stream() for _ in range(2)]
    wss = [gmlp.alloc_workspace(7, 2048, 5632, False, gmlp.VARIANT_SKINNY) for _ in range(2)]
    Ys = [torch.full_like(t["X"], float("nan")) for t in ts]
    torch.cuda.synchronize()
    for _ in range(20):
        for k in range(2):
            gmlp.forward(ts[k]["X"], ts[k]["Wg"], ts[k]["Wu"], ts[k]["Wd"], Ys[k], variant=gmlp.VARIANT_SKINNY,
                         workspace=wss[k], stream=streams[k])
    torch.cuda.synchronize()
    assert gmlp.device_status() == 0
    for k in range(2):
        y_ref = _reference(inps[k], False)
        e = np.abs(Ys[k].float().cpu().numpy().astype(np.float64) - y_ref) / oracle.tolerance(y_ref)
        assert float(e.max()) <= 1.0


def test_default_rule_takes_the_fused_form_on_the_small_layer():
    """The stated ragged workloads with one and seven tokens run as fused kernel + slice sum under AUTO."""
    for name in ("ragged-M1-plain", "ragged-M7-plain"):
        w = I.WORKLOADS[name]
        assert gmlp.pick_variant(w.M, w.d_model, w.d_ff) == gmlp.VARIANT_SKINNY
        inp = I.make_inputs(w)
        t = to_device(inp)
        Y = torch.empty_like(t["X"])
        assert _kernels_of(lambda: gmlp.forward(t["X"], t["Wg"], t["Wu"], t["Wd"], Y, checked=True)) == {"fused", "sum"}
        y_ref = _reference(inp, False)
        e = np.abs(Y.float().cpu().numpy().astype(np.float64) - y_ref) / oracle.tolerance(y_ref)
        assert float(e.max()) <= 1.0
