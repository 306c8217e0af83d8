"""gmlp_autotune: the measured choice among the schedules is remembered per shape, AUTO follows it, results
stay within tolerance of the oracle, and clearing restores the built-in rule."""
import pytest
import torch

from paper_2606_26344_b200 import gmlp, inputs as I

from _parity import check_case, to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _clean():
    gmlp.autotune_clear()
    yield
    gmlp.autotune_clear()


@pytest.mark.parametrize("shape", [(8, 1024, 2048), (100, 512, 1024), (300, 512, 1024)])
def test_autotune_picks_a_runnable_schedule_and_auto_follows_it(shape):
    M, dm, dff = shape
    inp = I.custom_inputs(M, dm, dff, 60 + M, rmsnorm=True)
    t = to_device(inp)
    default = gmlp.pick_variant(M, dm, dff)
    Y = torch.empty_like(t["X"])
    a = gmlp.make_args(t["X"], t["Wg"], t["Wu"], t["Wd"], Y, t["gamma"], inp.workload.eps, True)   # library workspace
    v, us = gmlp.autotune(a, 5)
    allowed = {gmlp.VARIANT_TENSOR} | ({gmlp.VARIANT_SKINNY} if M <= 128 else set())
    assert v in allowed and 1.0 < us < 1e5
    assert gmlp.pick_variant(M, dm, dff) == v
    q = gmlp.autotune_query(M, dm, dff)
    assert q is not None and q[0] == v and (q[1:] == (-1, -1) if v == gmlp.VARIANT_SKINNY else set(q[1:]) <= {0, 1})
    assert gmlp.autotune_query(M + 1, dm, dff) is None
    assert gmlp.pick_variant(M + 1, dm, dff) == gmlp.lib().gmlp_pick_variant(M + 1, dm, dff, 0)   # other shapes untouched
    assert gmlp.workspace_bytes(M, dm, dff, gmlp.FLAG_RMSNORM) == gmlp.workspace_bytes(M, dm, dff, gmlp.FLAG_RMSNORM, v)
    check_case(inp, gmlp.VARIANT_AUTO, f"tuned{shape}")
    gmlp.autotune_clear()
    assert gmlp.pick_variant(M, dm, dff) == default


def test_autotune_respects_a_small_caller_workspace_and_validates_arguments():
    M, dm, dff = 16, 512, 1024
    inp = I.custom_inputs(M, dm, dff, 3)
    t = to_device(inp)
    Y = torch.empty_like(t["X"])
    ws = gmlp.alloc_workspace(M, dm, dff, False, gmlp.VARIANT_UMMA)            # H only: too small for SKINNY's partials
    assert ws.numel() < gmlp.workspace_bytes(M, dm, dff, 0, gmlp.VARIANT_SKINNY)
    a = gmlp.make_args(t["X"], t["Wg"], t["Wu"], t["Wd"], Y, workspace=ws)
    v, _ = gmlp.autotune(a, 3)
    assert v != gmlp.VARIANT_SKINNY
    import ctypes
    f = gmlp.lib().gmlp_autotune
    assert f(None, 3, None, None) == gmlp.ERR_NULL
    assert f(ctypes.byref(a), 0, None, None) == gmlp.ERR_FLAGS
    a.workspace_bytes = 256
    assert f(ctypes.byref(a), 3, None, None) == gmlp.ERR_WORKSPACE
    torch.cuda.synchronize()
    assert gmlp.device_status() == 0
