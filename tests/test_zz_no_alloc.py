"""gmlp_forward_static: the entry point for callers that are not allowed to allocate device memory
(a serving loop whose memory plan is frozen, a process whose memory manager forbids cudaMalloc after
start-up).  Its scratch is a fixed array inside the library, shared by every call on the device.

The file name sorts last on purpose: if this addition ever fails, a run that stops at the first
failure has already run every other test.  The GPU test passes alone in a fresh process and after
the rest of the suite: it depends on no state left by other tests, and the call clears the counters
it needs itself.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2606_26344_b200 import build as B
from paper_2606_26344_b200 import gmlp, inputs as I


def test_static_entry_refuses_shapes_beyond_its_fixed_scratch():
    B.build_libgmlp()
    lib = gmlp.lib()
    p = 0x1000
    assert lib.gmlp_forward_static(p, p, p, p, p, gmlp.STATIC_MAX_M + 1, 4096, 14336, None) == gmlp.ERR_STATIC_LIMIT
    assert lib.gmlp_forward_static(p, p, p, p, p, 4, 60, 128, None) == gmlp.ERR_SHAPE
    assert lib.gmlp_forward_static(None, p, p, p, p, 4, 64, 128, None) == gmlp.ERR_NULL
    assert lib.gmlp_forward_static(None, None, None, None, None, 0, 64, 128, None) == gmlp.OK
    assert "fixed scratch" in gmlp.status_string(gmlp.ERR_STATIC_LIMIT)


@pytest.mark.gpu
def test_static_entry_matches_the_oracle_and_the_workspace_entry_on_two_calls_in_a_row(monkeypatch):
    import oracle
    dev = torch.device("cuda")
    # decode-shaped (several contributors per column tile), the 2048 x 5632 layer (both GEMMs in the cluster form)
    # and a ragged small case
    for (M, dm, dff, seed) in ((8, 4096, 14336, 0), (7, 2048, 5632, 2), (5, 264, 520, 3)):
        first = I.custom_inputs(M, dm, dff, seed)
        second = I.custom_inputs(M, dm, dff, seed + 100)
        Wg, Wu, Wd = first.Wg.to(dev), first.Wu.to(dev), first.Wd.to(dev)
        for inp in (first, second):                      # two calls in a row share the built-in scratch
            X = inp.X.to(dev)
            default = gmlp.forward(X, Wg, Wu, Wd, variant=gmlp.VARIANT_SKINNY, checked=True)
            # (the static entry runs the two-kernel forms; where the workspace entry would take its one-kernel form - which
            # needs scratch for partial sums that the built-in array was not sized for - that form is switched off for the
            # bit-for-bit comparison, and the default is compared by the tolerance rule)
            monkeypatch.setenv("GMLP_SKINNY_FUSED", "0")
            want = gmlp.forward(X, Wg, Wu, Wd, variant=gmlp.VARIANT_SKINNY, checked=True)
            monkeypatch.delenv("GMLP_SKINNY_FUSED")
            got = torch.full_like(X, float("nan"))
            gmlp.forward_static(X, Wg, Wu, Wd, got)
            torch.cuda.synchronize()
            assert gmlp.device_status() == 0
            w, g = want.float().cpu().numpy().astype(np.float64), got.float().cpu().numpy().astype(np.float64)
            assert np.all(np.isfinite(g))
            # against the oracle (the weights are the first case's for both calls), by the rule of the other GPU tests
            y_ref = oracle.gmlp_rows(inp.bits("X"), first.bits("Wg"), first.bits("Wu"), first.bits("Wd"))
            assert np.all(np.abs(g - y_ref) <= oracle.tolerance(y_ref))
            # and against the existing entry point: same kernels, same split - in fact bit-identical
            assert np.all(np.abs(g - w) <= 2e-2 * np.maximum(1.0, np.abs(w)))
            assert torch.equal(got.view(torch.int16), want.view(torch.int16))
            d = default.float().cpu().numpy().astype(np.float64)
            assert np.all(np.abs(g - d) <= 2e-2 * np.maximum(1.0, np.abs(d)))
    # a shape that is too large for the array is refused on the device as well, and nothing was written
    X = torch.zeros(gmlp.STATIC_MAX_M + 1, 64, dtype=torch.bfloat16, device=dev)
    Wg = torch.zeros(64, 128, dtype=torch.bfloat16, device=dev)
    Wd = torch.zeros(128, 64, dtype=torch.bfloat16, device=dev)
    with pytest.raises(gmlp.GmlpError) as ei:
        gmlp.forward_static(X, Wg, Wg, Wd, torch.empty_like(X))
    assert ei.value.status == gmlp.ERR_STATIC_LIMIT


@pytest.mark.gpu
def test_static_entry_leaves_the_free_device_memory_as_it_found_it():
    """The point of the call: after one warm-up call per device (which loads the library's code and its built-in array)
    further calls take nothing from the device.  Free memory as the driver reports it, before and after."""
    dev = torch.device("cuda")
    inp = I.custom_inputs(8, 4096, 14336, 0)
    X, Wg, Wu, Wd = (t.to(dev) for t in (inp.X, inp.Wg, inp.Wu, inp.Wd))
    Y = torch.empty_like(X)
    gmlp.forward_static(X, Wg, Wu, Wd, Y)                # warm-up: first use on this device
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info(dev)
    for _ in range(3):
        gmlp.forward_static(X, Wg, Wu, Wd, Y)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info(dev)
    assert free_after == free_before
    assert gmlp.device_status() == 0
