"""GMLP_FLAG_WEIGHTS_OUT_IN: weights stored [out, in] give the same result, bit for bit, as the same weights
stored [in, out] (the tensor-core kernels read them as K-major operands; tiles and sum order do not change),
and that result is within tolerance of the CPU oracle."""
import pytest
import torch

from paper_2606_26344_b200 import gmlp, inputs as I

from _parity import check_case, to_device

pytestmark = pytest.mark.gpu

V = gmlp
CASES = [(V.VARIANT_SKINNY, 1, 256, 512), (V.VARIANT_SKINNY, 8, 1024, 2056), (V.VARIANT_SKINNY, 100, 520, 1096),
         (V.VARIANT_UMMA, 9, 1024, 2048), (V.VARIANT_UMMA, 129, 320, 392), (V.VARIANT_UMMA, 77, 1024, 4096),
         (V.VARIANT_UMMA, 300, 512, 1024), (V.VARIANT_PAIR, 300, 512, 1088), (V.VARIANT_PAIR, 1030, 320, 392),
         (V.VARIANT_TENSOR, 520, 1024, 2816), (V.VARIANT_AUTO, 16, 256, 512), (V.VARIANT_AUTO, 2048, 1024, 2048)]


def _t(w):
    return w.t().contiguous()


@pytest.mark.parametrize("rmsnorm", [False, True])
@pytest.mark.parametrize("case", CASES)
def test_out_in_storage_matches_in_out_storage_bit_for_bit(case, rmsnorm):
    variant, M, dm, dff = case
    inp = I.custom_inputs(M, dm, dff, 1200 + M, rmsnorm=rmsnorm)
    t = to_device(inp)
    kw = dict(gamma=t["gamma"] if rmsnorm else None, eps=inp.workload.eps, rmsnorm=rmsnorm, variant=variant, checked=True)
    Y_io = gmlp.forward(t["X"], t["Wg"], t["Wu"], t["Wd"], **kw)
    Y_oi = gmlp.forward(t["X"], _t(t["Wg"]), _t(t["Wu"]), _t(t["Wd"]), weights_out_in=True, **kw)
    torch.cuda.synchronize()
    assert torch.equal(Y_io.view(torch.int16), Y_oi.view(torch.int16))
    check_case(inp, variant, f"in-out{case}")          # and the common value is the oracle's, within tolerance


@pytest.mark.parametrize("variant,M", [(V.VARIANT_SKINNY, 8), (V.VARIANT_UMMA, 100), (V.VARIANT_PAIR, 260)])
def test_gate_up_half_with_out_in_weights(variant, M):
    inp = I.custom_inputs(M, 512, 1096, 1300 + M)
    t = to_device(inp)
    H_io = gmlp.gate_up(t["X"], t["Wg"], t["Wu"], variant=variant, checked=True)
    H_oi = gmlp.gate_up(t["X"], _t(t["Wg"]), _t(t["Wu"]), variant=variant, checked=True, weights_out_in=True)
    torch.cuda.synchronize()
    assert torch.equal(H_io.view(torch.int16), H_oi.view(torch.int16))


def test_cuda_core_schedules_refuse_the_flag():
    inp = I.custom_inputs(5, 64, 128, 1)
    t = to_device(inp)
    for v in (V.VARIANT_SIMT, V.VARIANT_STREAM):
        with pytest.raises(gmlp.GmlpError) as e:
            gmlp.forward(t["X"], _t(t["Wg"]), _t(t["Wu"]), _t(t["Wd"]), variant=v, weights_out_in=True)
        assert e.value.status == gmlp.ERR_UNSUPPORTED
