"""GMLP_FLAG_Y_FP32: the down projection's fp32 accumulator is delivered without the final rounding; rounding it
gives the default bf16 output bit for bit, and it is closer to the oracle than the bf16 output."""
import numpy as np
import pytest
import torch

import oracle
from paper_2606_26344_b200 import gmlp, inputs as I

from _parity import oracle_rows, to_device

pytestmark = pytest.mark.gpu

V = gmlp
CASES = [(V.VARIANT_SKINNY, 1, 256, 512), (V.VARIANT_SKINNY, 8, 1024, 2056), (V.VARIANT_SKINNY, 100, 520, 1096),
         (V.VARIANT_UMMA, 9, 1024, 2048), (V.VARIANT_UMMA, 129, 320, 392), (V.VARIANT_UMMA, 77, 1024, 4096),
         (V.VARIANT_UMMA, 300, 512, 1024), (V.VARIANT_PAIR, 300, 512, 1088), (V.VARIANT_PAIR, 1030, 320, 392),
         (V.VARIANT_TENSOR, 520, 1024, 2816), (V.VARIANT_AUTO, 16, 256, 512), (V.VARIANT_AUTO, 1100, 1024, 2048)]


@pytest.mark.parametrize("case", CASES)
def test_fp32_output_rounds_to_the_bf16_output_and_is_within_tolerance(case):
    variant, M, dm, dff = case
    rmsnorm = M % 2 == 1
    inp = I.custom_inputs(M, dm, dff, 1400 + M, rmsnorm=rmsnorm)
    t = to_device(inp)
    kw = dict(gamma=t["gamma"] if rmsnorm else None, eps=inp.workload.eps, rmsnorm=rmsnorm, variant=variant, checked=True)
    Yb = gmlp.forward(t["X"], t["Wg"], t["Wu"], t["Wd"], **kw)
    buf = torch.full((M * dm + 64,), float("nan"), dtype=torch.float32, device="cuda")    # guard behind Y
    Yf = buf[:M * dm].view(M, dm)
    gmlp.forward(t["X"], t["Wg"], t["Wu"], t["Wd"], Yf, **kw)
    torch.cuda.synchronize()
    assert bool(torch.isfinite(Yf).all()) and bool(torch.isnan(buf[M * dm:]).all())
    assert torch.equal(Yf.to(torch.bfloat16).view(torch.int16), Yb.view(torch.int16))
    rows = I.sample_rows(inp.workload, inp.outlier_rows)
    y_ref = oracle_rows(inp, rows)
    idx = torch.as_tensor(rows, device="cuda")
    ef = np.abs(Yf[idx].double().cpu().numpy() - y_ref) / oracle.tolerance(y_ref)
    eb = np.abs(Yb[idx].double().cpu().numpy() - y_ref) / oracle.tolerance(y_ref)
    assert ef.max() <= 1.0
    assert np.mean(ef) <= np.mean(eb) + 1e-12          # no final rounding: not further from the reference on average


def test_cuda_core_schedules_and_the_gate_up_half_refuse_the_flag():
    inp = I.custom_inputs(5, 64, 128, 1)
    t = to_device(inp)
    Yf = torch.empty(5, 64, dtype=torch.float32, device="cuda")
    for v in (V.VARIANT_SIMT, V.VARIANT_STREAM):
        with pytest.raises(gmlp.GmlpError) as e:
            gmlp.forward(t["X"], t["Wg"], t["Wu"], t["Wd"], Yf, variant=v)
        assert e.value.status == gmlp.ERR_UNSUPPORTED
    import ctypes
    H = torch.empty(5, 128, dtype=torch.bfloat16, device="cuda")
    a = gmlp.make_args(t["X"], t["Wg"], t["Wu"], t["Wd"], torch.empty_like(t["X"]))
    a.Y = H.data_ptr()
    a.flags |= gmlp.FLAG_Y_FP32
    assert gmlp.lib().gmlp_gate_up(ctypes.byref(a)) == gmlp.ERR_FLAGS
