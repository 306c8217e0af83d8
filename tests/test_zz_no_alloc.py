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
def test_static_entry_matches_the_workspace_entry_on_two_calls_in_a_row():
    dev = torch.device("cuda")
    # decode-shaped (several stream-K contributors per column tile) and a ragged small case
    for (M, dm, dff, seed) in ((8, 4096, 14336, 0), (5, 264, 520, 3)):
        first = I.custom_inputs(M, dm, dff, seed)
        second = I.custom_inputs(M, dm, dff, seed + 100)
        Wg, Wu, Wd = first.Wg.to(dev), first.Wu.to(dev), first.Wd.to(dev)
        for inp in (first, second):                      # two calls in a row share the built-in scratch
            X = inp.X.to(dev)
            want = gmlp.forward(X, Wg, Wu, Wd, variant=gmlp.VARIANT_SKINNY, checked=True)
            got = torch.full_like(X, float("nan"))
            gmlp.forward_static(X, Wg, Wu, Wd, got)
            torch.cuda.synchronize()
            assert gmlp.device_status() == 0
            w, g = want.float().cpu().numpy().astype(np.float64), got.float().cpu().numpy().astype(np.float64)
            assert np.all(np.isfinite(g))
            # the parity rule of the other GPU tests, taken around the existing entry point's output
            assert np.all(np.abs(g - w) <= 2e-2 * np.maximum(1.0, np.abs(w)))
            # same kernels, same split: in fact bit-identical
            assert torch.equal(got.view(torch.int16), want.view(torch.int16))
    # a shape that is too large for the array is refused on the device as well, and nothing was written
    X = torch.zeros(gmlp.STATIC_MAX_M + 1, 64, dtype=torch.bfloat16, device=dev)
    Wg = torch.zeros(64, 128, dtype=torch.bfloat16, device=dev)
    Wd = torch.zeros(128, 64, dtype=torch.bfloat16, device=dev)
    with pytest.raises(gmlp.GmlpError) as ei:
        gmlp.forward_static(X, Wg, Wg, Wd, torch.empty_like(X))
    assert ei.value.status == gmlp.ERR_STATIC_LIMIT
