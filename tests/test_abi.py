"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol
the header declares, and rejects bad arguments with the documented codes before any device
work."""
import ctypes
import os
import re

import pytest
import torch

from paper_2606_26344_b200 import build as B
from paper_2606_26344_b200 import gmlp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "gmlp.h")


@pytest.fixture(scope="module")
def lib():
    B.build_libgmlp()
    return gmlp.lib()


def declared_symbols():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gmlp_[a-z_]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = declared_symbols()
    assert "gmlp_forward" in names and "gmlp_forward_ex" in names and "gmlp_workspace_bytes" in names
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in gmlp.h but not exported"


def test_struct_layout_matches_header(lib):
    # 2 x u32, 5 pointers, 3 x i64, pointer, float, i32, 2 pointers, u64, float, u32 on LP64
    assert ctypes.sizeof(gmlp.GmlpArgs) == 8 + 5 * 8 + 3 * 8 + 8 + 4 + 4 + 8 + 8 + 8 + 4 + 4


def test_version_and_status_strings(lib):
    assert lib.gmlp_version() >= 100
    for code in range(-9, 1):
        assert gmlp.status_string(code) and gmlp.status_string(code) != "unknown status"
    assert gmlp.status_string(-99) == "unknown status"


def _args(**kw):
    a = gmlp.GmlpArgs()
    a.struct_bytes = ctypes.sizeof(gmlp.GmlpArgs)
    a.X = a.Wg = a.Wu = a.Wd = a.Y = 0x1000
    a.M, a.d_model, a.d_ff = 4, 64, 128
    for k, v in kw.items():
        setattr(a, k, v)
    return a


def test_argument_validation_happens_before_device_work(lib):
    f = lambda a: lib.gmlp_forward_ex(ctypes.byref(a))
    assert lib.gmlp_forward_ex(None) == gmlp.ERR_NULL
    assert f(_args(struct_bytes=8)) == gmlp.ERR_FLAGS
    assert f(_args(flags=1 << 11)) == gmlp.ERR_FLAGS
    assert f(_args(variant=17)) == gmlp.ERR_FLAGS
    assert f(_args(flags=gmlp.FLAG_ACT_SWISH | gmlp.FLAG_ACT_GLU, act_beta=1.0)) == gmlp.ERR_FLAGS
    assert f(_args(flags=gmlp.FLAG_ACT_GELU | gmlp.FLAG_ACT_GLU, act_beta=1.0)) == gmlp.ERR_FLAGS
    assert f(_args(flags=gmlp.FLAG_ACT_GELU | gmlp.FLAG_ACT_SWISH, act_beta=1.0)) == gmlp.ERR_FLAGS
    assert f(_args(flags=gmlp.FLAG_ACT_SWISH, act_beta=float("nan"))) == gmlp.ERR_FLAGS
    assert f(_args(flags=gmlp.FLAG_ACT_SWISH, act_beta=float("inf"))) == gmlp.ERR_FLAGS
    assert f(_args(reserved=1)) == gmlp.ERR_FLAGS
    assert f(_args(variant=-1)) == gmlp.ERR_FLAGS
    assert f(_args(M=-1)) == gmlp.ERR_SHAPE
    assert f(_args(d_model=60)) == gmlp.ERR_SHAPE
    assert f(_args(d_ff=0)) == gmlp.ERR_SHAPE
    assert f(_args(d_ff=12)) == gmlp.ERR_SHAPE
    assert f(_args(X=None)) == gmlp.ERR_NULL
    assert f(_args(Y=None)) == gmlp.ERR_NULL
    assert f(_args(Wd=0x1008)) == gmlp.ERR_ALIGN
    assert f(_args(workspace=0x1010, workspace_bytes=1 << 20)) == gmlp.ERR_ALIGN
    assert lib.gmlp_forward(None, 0x1000, 0x1000, 0x1000, 0x1000, 4, 64, 128, 0) == gmlp.ERR_NULL
    assert lib.gmlp_forward_host(None, 0x1000, 0x1000) == gmlp.ERR_NULL
    assert lib.gmlp_forward_host(ctypes.byref(_args()), None, 0x1000) == gmlp.ERR_NULL
    assert lib.gmlp_autotune(None, 5, None, None) == gmlp.ERR_NULL
    assert lib.gmlp_autotune(ctypes.byref(_args()), 0, None, None) == gmlp.ERR_FLAGS
    assert lib.gmlp_autotune(ctypes.byref(_args(M=0)), 5, None, None) == gmlp.ERR_SHAPE
    lib.gmlp_autotune_clear()
    assert lib.gmlp_matmul_add_rmsnorm(None) == gmlp.ERR_NULL
    assert lib.gmlp_set_default_eps(-1.0) == gmlp.ERR_FLAGS
    assert lib.gmlp_set_default_eps(1e-5) == gmlp.OK


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-device behaviour")
def test_no_device_means_arch_error_not_fallback(lib):
    assert lib.gmlp_forward_ex(ctypes.byref(_args())) == gmlp.ERR_ARCH
    assert lib.gmlp_device_status() == gmlp.ERR_ARCH


def test_workspace_sizes_and_variant_choice(lib):
    wb = gmlp.workspace_bytes
    assert wb(0, 64, 128) >= 256 and wb(-1, 64, 128) == 0 and wb(4, 60, 128) == 0
    M, dm, dff = 2048, 4096, 14336
    h = M * dff * 2
    assert wb(M, dm, dff, 0, gmlp.VARIANT_UMMA) >= h
    assert wb(M, dm, dff, gmlp.FLAG_RMSNORM, gmlp.VARIANT_UMMA) >= h + M * dm * 2
    assert wb(M, dm, dff, 0, gmlp.VARIANT_UMMA) < h + 4096
    assert wb(8, dm, dff, 0, gmlp.VARIANT_STREAM) > wb(8, dm, dff, 0, gmlp.VARIANT_SIMT)     # split-K partials
    assert wb(8, dm, dff, 0, gmlp.VARIANT_STREAM) < 64 << 20
    # AUTO: the operand-swapped stream-K schedule for a handful of tokens, else the 128-row tensor-core tiles
    # with a per-GEMM kernel choice
    assert gmlp.pick_variant(1, 2048, 5632) == gmlp.VARIANT_SKINNY
    assert gmlp.pick_variant(16, 2048, 5632) == gmlp.VARIANT_SKINNY
    # (up to 32 tokens everywhere; on a layer whose two GEMMs both have the operand-swapped schedule's cluster form up to 96,
    # and up to 200 where d_model >= 3072, because the 128-row tiles pay for a second row block from 129 tokens on)
    assert gmlp.pick_variant(32, 2048, 5632) == gmlp.VARIANT_SKINNY and gmlp.pick_variant(32, 8192, 28672) == gmlp.VARIANT_SKINNY
    assert gmlp.pick_variant(96, 2048, 5632) == gmlp.VARIANT_SKINNY and gmlp.pick_variant(97, 2048, 5632) == gmlp.VARIANT_TENSOR
    assert gmlp.pick_variant(33, 8192, 28672) == gmlp.VARIANT_TENSOR and gmlp.pick_variant(33, 4096, 20480) == gmlp.VARIANT_TENSOR
    assert gmlp.pick_variant(8, dm, dff) == gmlp.VARIANT_SKINNY
    assert gmlp.pick_variant(128, dm, dff) == gmlp.VARIANT_SKINNY and gmlp.pick_variant(200, dm, dff) == gmlp.VARIANT_SKINNY
    assert gmlp.pick_variant(201, dm, dff) == gmlp.VARIANT_TENSOR and gmlp.pick_variant(129, 3072, 8192) == gmlp.VARIANT_SKINNY
    assert gmlp.pick_variant(129, 2048, 5632) == gmlp.VARIANT_TENSOR
    assert gmlp.pick_variant(2048, dm, dff) == gmlp.VARIANT_TENSOR
    assert gmlp.pick_variant(4096, 8192, 28672) == gmlp.VARIANT_TENSOR
    assert wb(300, dm, dff, 0, gmlp.VARIANT_TENSOR) == wb(300, dm, dff, 0, gmlp.VARIANT_UMMA)
    assert gmlp.pick_variant(4, 60, 128) == gmlp.ERR_SHAPE


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    monkeypatch.setattr(gmlp, "_lib", None)
    monkeypatch.setattr(gmlp, "_LIB_PATH", str(tmp_path / "libgmlp.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        gmlp.lib()


def test_header_is_plain_c(tmp_path):
    """The boundary is a C header: it must compile as C99 on its own (no C++, no CUDA, no torch types)."""
    import subprocess
    src = tmp_path / "t.c"
    src.write_text('#include "gmlp.h"\nint main(void) { gmlp_args a; gmlp_qkv_args q; gmlp_gqa_args g; (void)a; (void)q; (void)g; '
                   'return GMLP_OK + GMLP_VARIANT_TENSOR - GMLP_VARIANT_TENSOR; }\n')
    r = subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-fsyntax-only",
                        "-I", os.path.join(ROOT, "include"), str(src)], capture_output=True, text=True)
    assert r.returncode == 0, r.stderr


def test_small_m_plan_per_gemm_form(lib):
    """Host arithmetic of the operand-swapped schedule: which GEMMs split K over a cluster per column tile (and how), which
    keep stream-K.  148 SMs (a B200 holds 74 / 45 / 33 / 26 / 22 / 15 / 15 clusters of 2 .. 8 CTAs at once)."""
    plan = lambda *a: gmlp.small_m_plan(*a, 148)
    # 2048 x 5632: gate/up 44 tiles x 3 CTAs (132 SMs); down 16 tiles x 6 (eight would need 16 clusters of 8: 15 fit)
    assert plan(7, 2048, 5632) == ((3, 128, 44), (6, 128, 16))
    # 8B: gate/up has 112 tiles, 76 % of the SMs with one CTA each (no reduction); down 32 tiles x 4
    assert plan(8, 4096, 14336) == ((1, 128, 112), (4, 128, 32))
    # 70B: 224 gate/up tiles exceed the SMs: stream-K; down 64 tiles x 2
    gu, down = plan(8, 8192, 28672)
    assert gu[0] == 0 and down == (2, 128, 64)
    # every cluster plan fills at least a quarter of the SMs (80 % with 64-column tiles) and fits one wave
    capacity = {1: 148, 2: 74, 3: 45, 4: 33, 5: 26, 6: 22, 7: 15, 8: 15}
    for (M, dm, dff) in ((1, 2048, 5632), (16, 1024, 4096), (24, 3072, 8192), (96, 4096, 11008), (5, 264, 520), (200, 2048, 5632)):
        for c, cols, tiles in plan(M, dm, dff):
            if c >= 1:
                assert cols in (64, 128) and tiles * c <= 148 and tiles <= capacity[c]
                assert tiles * c * 100 >= 148 * (25 if cols == 128 else 80)
    # more than 128 tokens run only where both GEMMs have the cluster form; shapes are validated
    assert lib.gmlp_small_m_plan(7, 60, 128, 148, (ctypes.c_int32 * 6)()) == gmlp.ERR_SHAPE
    assert lib.gmlp_small_m_plan(7, 64, 128, 148, None) == gmlp.ERR_NULL


def test_small_m_fused_plan(lib):
    """Host arithmetic of the one-kernel form of the operand-swapped schedule: one cluster per 128-wide slice of d_ff, the
    largest cluster that fits one wave, TMEM for gate, up and a CTA's share of the partial-Y tiles."""
    plan = lambda *a: gmlp.small_m_fused_plan(*a, 148)
    # 2048 x 5632: 44 slices x 3 CTAs (132 SMs; four would need 176); (2 + ceil(16 / 3)) x 16 = 128 TMEM columns; the default
    assert plan(7, 2048, 5632)[:2] == (3, 44) and plan(7, 2048, 5632)[3:] == (128, 1)
    assert plan(1, 2048, 5632)[2] >= plan(16, 2048, 5632)[2] >= 4      # fewer tokens: smaller exchange area, more ring stages
    # at most 16 tokens; 8B and 70B layers do not apply (the partial-Y tiles of a CTA would not fit TMEM / too many slices)
    assert plan(17, 2048, 5632)[0] == 0 and plan(8, 4096, 14336)[0] == 0 and plan(8, 8192, 28672)[0] == 0
    # applies but is not the default: more than 90 MB of weights, or more than six down tiles per CTA
    assert plan(8, 1536, 8960)[0] == 2 and plan(8, 1536, 8960)[4] == 1 and plan(8, 2048, 8192)[:2] == (2, 64) and plan(8, 2048, 8192)[4] == 0
    assert plan(8, 4096, 5632)[0] == 3 and plan(8, 4096, 5632)[4] == 0
    assert plan(8, 1024, 4096) [:2] == (4, 32) and plan(8, 1024, 4096)[4] == 1
    capacity = {1: 148, 2: 74, 3: 45, 4: 33, 5: 26, 6: 22, 7: 15, 8: 15}
    for (M, dm, dff) in ((1, 2048, 5632), (16, 1024, 4096), (5, 3072, 8192), (8, 2560, 6912), (2, 1024, 16384), (16, 256, 512)):
        c, slices, stages, cols, _ = plan(M, dm, dff)
        if c >= 1:
            assert slices == -(-dff // 128) and slices * c <= 148 and slices <= capacity[c] and slices * c * 10 >= 148 * 6
            assert 2 <= stages <= 12 and cols in (32, 64, 128, 256, 512) and cols >= (2 + -(-(-(-dm // 128)) // c)) * 16
    # the workspace holds the slices' partial Y
    assert gmlp.workspace_bytes(7, 2048, 5632, 0, gmlp.VARIANT_SKINNY) >= 44 * 7 * 2048 * 4
    assert lib.gmlp_small_m_fused_plan(7, 60, 128, 148, (ctypes.c_int32 * 5)()) == gmlp.ERR_SHAPE
    assert lib.gmlp_small_m_fused_plan(7, 64, 128, 148, None) == gmlp.ERR_NULL
