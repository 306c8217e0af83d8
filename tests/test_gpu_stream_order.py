"""GMLP_FLAG_WEIGHTS_IN_STREAM_ORDER: weights written by work enqueued on the same stream right before the call.  The
kernels of a call fetch weight tiles ahead of stream order (that is how a call's start overlaps its predecessor's tail);
with the flag the call's first kernel is launched in plain stream order and the call sees the new weights."""
import numpy as np
import pytest
import torch

import oracle
from paper_2606_26344_b200 import gmlp, inputs as I

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("shape,variant", [((7, 2048, 5632), gmlp.VARIANT_AUTO),        # the one-kernel small-M form
                                           ((8, 4096, 14336), gmlp.VARIANT_AUTO),       # two cluster-form kernels
                                           ((24, 1024, 20480), gmlp.VARIANT_SKINNY),    # stream-K gate/up
                                           ((300, 1024, 2048), gmlp.VARIANT_AUTO)])     # 128-row tiles
@pytest.mark.parametrize("rmsnorm", [False, True])
def test_weights_copied_on_the_same_stream_just_before_the_call(shape, variant, rmsnorm):
    M, dm, dff = shape
    dev = torch.device("cuda")
    a = I.custom_inputs(M, dm, dff, 31, rmsnorm=rmsnorm)
    b = I.custom_inputs(M, dm, dff, 32, rmsnorm=rmsnorm)
    X = a.X.to(dev)
    gamma = a.gamma.to(dev) if rmsnorm else None
    src = [tuple(t.to(dev) for t in (i.Wg, i.Wu, i.Wd)) for i in (a, b)]
    Wg, Wu, Wd = (torch.empty_like(t) for t in src[0])
    ws = gmlp.alloc_workspace(M, dm, dff, rmsnorm, variant)
    outs = []
    torch.cuda.synchronize()
    for k in range(12):                       # alternate the two weight sets; every call must see the set just copied
        for dst, s in zip((Wg, Wu, Wd), src[k % 2]):
            dst.copy_(s, non_blocking=True)   # device-to-device copies on the stream of the call
        Y = torch.empty_like(X)
        gmlp.forward(X, Wg, Wu, Wd, Y, gamma=gamma, eps=a.workload.eps, rmsnorm=rmsnorm, variant=variant, workspace=ws,
                     weights_in_stream_order=True)
        outs.append(Y)
    torch.cuda.synchronize()
    assert gmlp.device_status() == 0
    rows = np.unique(np.array([0, M // 2, M - 1]))
    refs = [oracle.gmlp_rows(a.bits("X"), i.bits("Wg"), i.bits("Wu"), i.bits("Wd"), rows=rows,
                             gamma=a.bits("gamma") if rmsnorm else None, eps=a.workload.eps, rmsnorm=rmsnorm) for i in (a, b)]
    for k, Y in enumerate(outs):
        y = Y[torch.as_tensor(rows, device=dev)].float().cpu().numpy().astype(np.float64)
        assert np.all(np.abs(y - refs[k % 2]) <= oracle.tolerance(refs[k % 2])), f"call {k} did not see the weights copied before it"
        assert torch.equal(Y.view(torch.int16), outs[k % 2].view(torch.int16))


def test_the_flag_changes_nothing_else():
    inp = I.custom_inputs(7, 2048, 5632, 33)
    dev = torch.device("cuda")
    X, Wg, Wu, Wd = (t.to(dev) for t in (inp.X, inp.Wg, inp.Wu, inp.Wd))
    plain = gmlp.forward(X, Wg, Wu, Wd, checked=True)
    ordered = gmlp.forward(X, Wg, Wu, Wd, checked=True, weights_in_stream_order=True)
    assert torch.equal(plain.view(torch.int16), ordered.view(torch.int16))
