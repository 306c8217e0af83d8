"""The file that keeps tuned schedule choices between processes: its format, what a load takes and what it skips, and a
save / load round trip.  No GPU is needed for any of it (without a CUDA device the choices attach to device 0)."""
import os

import pytest
import torch

from paper_2606_26344_b200 import build as B
from paper_2606_26344_b200 import gmlp


def _lines(path):
    return [l.rstrip("\n") for l in open(path) if l.strip() and not l.startswith("#")]


def test_load_takes_matching_lines_only_and_save_writes_them_back(tmp_path):
    B.build_libgmlp()
    gmlp.autotune_clear()
    v = gmlp.lib().gmlp_version()
    good = [f"gmlp-tune-v1\t{v}\tNVIDIA B200\t8\t4096\t14336\t4\t-1\t-1\t0\t0",
            f"gmlp-tune-v1\t{v}\tNVIDIA B200\t2048\t4096\t14336\t6\t1\t0\t0\t12",
            f"gmlp-tune-v1\t{v}\tNVIDIA B200\t129\t2048\t5632\t6\t0\t0\t2\t4",
            f"gmlp-tune-v1\t{v}\tNVIDIA B200\t7\t2048\t5632\t4\t-1\t-1\t2\t1"]     # SKINNY with its own forms: two kernels, half-size rings
    skipped = [f"gmlp-tune-v1\t{v}\tNVIDIA H100\t8\t4096\t14336\t4\t-1\t-1\t0\t0",          # another GPU model
               f"gmlp-tune-v1\t{v + 1}\tNVIDIA B200\t16\t4096\t14336\t4\t-1\t-1\t0\t0",      # another library version
               f"gmlp-tune-v1\t{v}\tNVIDIA B200\t8\t4097\t14336\t4\t-1\t-1\t0\t0",           # d_model not a multiple of 8
               f"gmlp-tune-v1\t{v}\tNVIDIA B200\t8\t4096\t14336\t2\t-1\t-1\t0\t0",           # not a schedule tuning may keep
               f"gmlp-tune-v1\t{v}\tNVIDIA B200\t8\t4096\t14336\t6\t1\t1\t3\t0",             # gate/up form 3 does not exist
               f"gmlp-tune-v1\t{v}\tNVIDIA B200\t8\t4096\t14336\t6\t1\t1\t0\t5",             # down form 5 does not exist
               f"gmlp-tune-v1\t{v}\tNVIDIA B200\t9\t4096\t14336\t4\t-1\t-1\t3\t0",           # SKINNY: one-kernel form 3 does not exist
               f"gmlp-tune-v1\t{v}\tNVIDIA B200\t9\t4096\t14336\t4\t-1\t-1\t0\t4",           # SKINNY: ring form 4 does not exist
               f"gmlp-tune-v1\t{v}\tNVIDIA B200\t8\t4096\tx\t6\t1\t1\t0\t0",                 # not a number
               f"gmlp-tune-v1\t{v}\tNVIDIA B200\t8\t4096",                                   # too few fields
               f"gmlp-tune-v0\t{v}\tNVIDIA B200\t8\t4096\t14336\t4\t-1\t-1\t0\t0"]           # another format
    src = tmp_path / "tuned.txt"
    src.write_text("# a comment\n\n" + "\n".join(good[:1] + skipped + good[1:]) + "\n")
    assert gmlp.autotune_load(str(src), "NVIDIA B200") == 4
    out = tmp_path / "saved.txt"
    assert gmlp.autotune_save(str(out)) == 4
    assert sorted(_lines(out)) == sorted(good)
    assert open(out).readline().startswith("#")
    # a later line for the same shape replaces the earlier one; loading twice does not duplicate
    newer = f"gmlp-tune-v1\t{v}\tNVIDIA B200\t8\t4096\t14336\t6\t0\t0\t0\t0"
    src.write_text(newer + "\n")
    assert gmlp.autotune_load(str(src), "NVIDIA B200") == 1
    assert gmlp.autotune_save(str(out)) == 4 and newer in _lines(out) and good[0] not in _lines(out)
    # round trip: clear, load what was saved, save again - the same lines
    before = sorted(_lines(out))
    gmlp.autotune_clear()
    assert gmlp.autotune_save(str(tmp_path / "empty.txt")) == 0
    assert gmlp.autotune_load(str(out), "NVIDIA B200") == 4
    again = tmp_path / "again.txt"
    assert gmlp.autotune_save(str(again)) == 4 and sorted(_lines(again)) == before
    gmlp.autotune_clear()
    with pytest.raises(gmlp.GmlpError):
        gmlp.autotune_load(str(tmp_path / "missing.txt"), "NVIDIA B200")


@pytest.mark.gpu
def test_a_tuned_choice_survives_through_the_file(tmp_path):
    from paper_2606_26344_b200 import inputs as I
    dev = torch.device("cuda")
    gmlp.autotune_clear()
    inp = I.custom_inputs(40, 1024, 2048, 4)
    X, Wg, Wu, Wd = (t.to(dev) for t in (inp.X, inp.Wg, inp.Wu, inp.Wd))
    Y = torch.empty_like(X)
    a = gmlp.make_args(X, Wg, Wu, Wd, Y, None, 1e-5, False, gmlp.VARIANT_AUTO, None, torch.cuda.current_stream())
    gmlp.autotune(a, 8)
    kept = gmlp.autotune_query(40, 1024, 2048)
    assert kept is not None
    path = tmp_path / "tuned.txt"
    assert gmlp.autotune_save(str(path)) == 1
    assert torch.cuda.get_device_name(dev) in open(path).read()
    gmlp.autotune_clear()
    assert gmlp.autotune_query(40, 1024, 2048) is None
    assert gmlp.autotune_load(str(path)) == 1                      # the current device's name
    assert gmlp.autotune_query(40, 1024, 2048) == kept
    assert gmlp.autotune_load(str(path), "some other GPU") == 0
    gmlp.autotune_clear()
    # with GMLP_TUNE_CACHE set, tuning rewrites the file by itself
    auto = tmp_path / "auto.txt"
    os.environ["GMLP_TUNE_CACHE"] = str(auto)
    try:
        gmlp.autotune(a, 4)
    finally:
        os.environ.pop("GMLP_TUNE_CACHE", None)
    assert len(_lines(auto)) == 1 and _lines(auto)[0].split("\t")[3:6] == ["40", "1024", "2048"]
    gmlp.autotune_clear()


@pytest.mark.gpu
def test_a_tuned_small_m_form_is_what_runs(tmp_path):
    """A kept SKINNY choice carries its own forms: the one-kernel form on or off, and the ring size."""
    from paper_2606_26344_b200 import inputs as I
    dev = torch.device("cuda")
    inp = I.custom_inputs(7, 2048, 5632, 5)
    X, Wg, Wu, Wd = (t.to(dev) for t in (inp.X, inp.Wg, inp.Wu, inp.Wd))
    name, v = torch.cuda.get_device_name(dev), gmlp.lib().gmlp_version()

    def kernels():
        gmlp.profile_enable(True)
        try:
            Y = gmlp.forward(X, Wg, Wu, Wd, checked=True)
            torch.cuda.synchronize()
            return set(gmlp.profile_read()), Y
        finally:
            gmlp.profile_enable(False)

    gmlp.autotune_clear()
    by_rule, Y0 = kernels()
    assert by_rule == {"fused", "sum"}
    path = tmp_path / "t.txt"
    path.write_text(f"gmlp-tune-v1\t{v}\t{name}\t7\t2048\t5632\t4\t-1\t-1\t2\t2\n")      # two kernels, full-size rings
    assert gmlp.autotune_load(str(path)) == 1
    tuned, Y1 = kernels()
    assert tuned == {"gate_up", "down"}
    path.write_text(f"gmlp-tune-v1\t{v}\t{name}\t7\t2048\t5632\t4\t-1\t-1\t1\t0\n")      # the one-kernel form
    assert gmlp.autotune_load(str(path)) == 1
    assert kernels()[0] == {"fused", "sum"}
    gmlp.autotune_clear()
    import numpy as np
    import oracle
    y_ref = oracle.gmlp_rows(inp.bits("X"), inp.bits("Wg"), inp.bits("Wu"), inp.bits("Wd"))
    for Y in (Y0, Y1):
        assert np.all(np.abs(Y.float().cpu().numpy().astype(np.float64) - y_ref) <= oracle.tolerance(y_ref))
