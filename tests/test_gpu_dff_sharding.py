"""The d_ff-sharded Gated MLP on one GPU: the shards of 2, 3 or 4 "ranks" run one after the other (each a complete
call of the library that leaves an fp32 partial product), gmlp_sum_partials adds them in rank order and rounds once;
the result is checked against the CPU oracle of the whole layer like any other output."""
import numpy as np
import pytest
import torch

import oracle
from paper_2606_26344_b200 import gmlp, inputs as I, sharding

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("world", [2, 3, 4])
@pytest.mark.parametrize("shape", [(8, 1024, 4096), (77, 512, 1000), (300, 1024, 2816)])
def test_shards_of_dff_sum_to_the_layer(shape, world):
    M, dm, dff = shape
    inp = I.custom_inputs(M, dm, dff, 21)
    dev = torch.device("cuda")
    X, Wg, Wu, Wd = (t.to(dev) for t in (inp.X, inp.Wg, inp.Wu, inp.Wd))
    parts = []
    for r in range(world):
        a, b = sharding.dff_range(dff, r, world)
        parts.append(sharding.forward_dff_partial(X, Wg[:, a:b].contiguous(), Wu[:, a:b].contiguous(), Wd[a:b].contiguous()))
    Y = gmlp.sum_partials(parts)
    torch.cuda.synchronize()
    assert gmlp.device_status() == 0
    rows = np.arange(M) if M <= 64 else np.sort(np.random.default_rng(3).choice(M, 64, replace=False))
    ref = oracle.gmlp_rows(inp.bits("X")[rows], inp.bits("Wg"), inp.bits("Wu"), inp.bits("Wd"))
    got = Y[torch.as_tensor(rows, device=dev)].float().cpu().numpy().astype(np.float64)
    e = np.abs(got - ref) / oracle.tolerance(ref)
    assert e.max() <= 1.0, f"max err/tol {e.max():.3f}"
    # one shard is the whole layer: the same bits as the ordinary call
    whole = gmlp.sum_partials([sharding.forward_dff_partial(X, Wg, Wu, Wd)])
    assert torch.equal(whole, gmlp.forward(X, Wg, Wu, Wd))


def test_single_process_path_of_the_sharded_call_and_argument_checks():
    inp = I.custom_inputs(16, 256, 512, 2)
    dev = torch.device("cuda")
    X, Wg, Wu, Wd = (t.to(dev) for t in (inp.X, inp.Wg, inp.Wu, inp.Wd))
    Y = sharding.forward_dff_sharded(X, Wg, Wu, Wd, dist=None)
    assert torch.equal(Y, gmlp.forward(X, Wg, Wu, Wd))
    with pytest.raises(ValueError):
        gmlp.sum_partials([])
    with pytest.raises(ValueError):
        gmlp.sum_partials([torch.zeros(4, 8, device=dev), torch.zeros(4, 16, device=dev)])
    with pytest.raises(gmlp.GmlpError) as e:
        gmlp.sum_partials([torch.zeros(1, 4, device=dev)])           # count not a multiple of 8
    assert e.value.status == gmlp.ERR_SHAPE
