"""Multi-rank host logic on CPU (gloo, world size 2): row sharding covers the batch exactly once with
no exchange of data, the oracle on a rank's rows equals the oracle on the whole batch restricted to
those rows (row independence), and step times aggregate as the maximum over ranks."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2606_26344_b200 import sharding


def test_row_ranges_partition_the_batch():
    for M in (0, 1, 7, 8, 129, 1000, 4096):
        for world in (1, 2, 3, 8):
            spans = [sharding.row_range(M, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == M
            assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
            lens = [b - a for a, b in spans]
            assert max(lens) - min(lens) <= 1
    with pytest.raises(ValueError):
        sharding.row_range(8, 2, 2)
    assert sharding.job_throughput(8, 4, 0.5) == 4 * 8 / 0.5e-3


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    sys.path.insert(0, root)
    import oracle
    from paper_2606_26344_b200 import inputs as I
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        inp = I.custom_inputs(11, 64, 96, 5)                      # every rank builds the same seeded batch
        a, b = sharding.row_range(11, rank, world)
        X, Wg, Wu, Wd = (inp.bits(n) for n in ("X", "Wg", "Wu", "Wd"))
        mine = oracle.gmlp_rows(X[a:b], Wg, Wu, Wd, num_threads=1)       # this rank's rows only, weights replicated
        whole = oracle.gmlp_rows(X, Wg, Wu, Wd, num_threads=1)
        ok = np.array_equal(mine, whole[a:b])
        counts = torch.zeros(11, dtype=torch.int64)
        counts[a:b] += 1
        dist.all_reduce(counts)                                   # test bookkeeping only, not the data path
        t = sharding.max_over_ranks(10.0 + rank, dist)
        dist.barrier()
        if rank == 0:
            out.put((ok, counts.tolist(), t))
        else:
            out.put((ok, None, t))
    finally:
        dist.destroy_process_group()


def test_two_ranks_cover_rows_once_and_take_the_slowest_time():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    results = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert all(r[0] for r in results)
    assert all(r[2] == 11.0 for r in results)
    counts = [r[1] for r in results if r[1] is not None][0]
    assert counts == [1] * 11


def test_dff_ranges_partition_the_hidden_dimension():
    for d_ff in (128, 512, 5632, 14336, 1000, 72):
        for world in (1, 2, 3, 8):
            spans = [sharding.dff_range(d_ff, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == d_ff
            assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
            assert all(a % 128 == 0 or a == d_ff for a, _ in spans) and all(b % 128 == 0 or b == d_ff for _, b in spans)
            lens = [b - a for a, b in spans]
            assert max(lens) - min(l for l in lens) <= 128 + (128 - d_ff % 128) % 128
    with pytest.raises(ValueError):
        sharding.dff_range(512, 2, 2)


def _dff_worker(rank, world, port, out):
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    sys.path.insert(0, root)
    import oracle
    from paper_2606_26344_b200 import inputs as I
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        M, dm, dff = 6, 64, 320
        inp = I.custom_inputs(M, dm, dff, 9)
        X, Wg, Wu, Wd = (inp.bits(n) for n in ("X", "Wg", "Wu", "Wd"))
        a, b = sharding.dff_range(dff, rank, world)
        # this rank's partial product: its columns of W_gate / W_up, its rows of W_down (the oracle leaves Y unrounded)
        part = oracle.gmlp_rows(X, np.ascontiguousarray(Wg[:, a:b]), np.ascontiguousarray(Wu[:, a:b]),
                                np.ascontiguousarray(Wd[a:b, :]), num_threads=1)
        t = torch.from_numpy(np.ascontiguousarray(part))
        dist.all_reduce(t)                                          # the d_ff split's one exchange
        whole = oracle.gmlp_rows(X, Wg, Wu, Wd, num_threads=1)
        err = float(np.abs(t.numpy() - whole).max() / max(1.0, float(np.abs(whole).max())))
        dist.barrier()
        out.put((rank, a, b, err))
    finally:
        dist.destroy_process_group()


def test_two_ranks_split_dff_and_one_all_reduce_restores_the_layer():
    world = 2
    port = _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_dff_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0][1] == 0 and res[0][2] == res[1][1] and res[1][2] == 320          # the slices tile d_ff
    assert all(r[3] < 1e-13 for r in res)                                          # fp64 sums differ by rounding order only
