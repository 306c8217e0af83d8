"""Thin ctypes binding over ``libgmlp.so`` (argument marshalling only).

Every step of the operator runs in the library's CUDA kernels; torch is used here for
device memory and streams.  The names mirror ``include/gmlp.h``.  If the library has not
been built this module raises on first use: there is no CPU or eager fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

OK = 0
ERR_NULL, ERR_SHAPE, ERR_ALIGN, ERR_FLAGS, ERR_WORKSPACE, ERR_ARCH, ERR_LAUNCH, ERR_TIMEOUT, ERR_UNSUPPORTED = \
    -1, -2, -3, -4, -5, -6, -7, -8, -9
ERR_STATIC_LIMIT = -10
STATIC_MAX_M = 16
STATIC_SCRATCH_BYTES = 12 << 20
FLAG_RMSNORM = 1 << 0
FLAG_CHECKED = 1 << 2
FLAG_ACT_SWISH = 1 << 5
FLAG_ACT_GLU = 1 << 6
FLAG_WEIGHTS_OUT_IN = 1 << 7
FLAG_Y_FP32 = 1 << 8
FLAG_ACT_GELU = 1 << 9
FLAG_WEIGHTS_IN_STREAM_ORDER = 1 << 10
ACT_FLAGS = {"silu": 0, "swish": FLAG_ACT_SWISH, "glu": FLAG_ACT_GLU, "gelu": FLAG_ACT_GELU}
VARIANT_AUTO, VARIANT_SIMT, VARIANT_STREAM, VARIANT_UMMA, VARIANT_SKINNY, VARIANT_PAIR, VARIANT_TENSOR = 0, 1, 2, 3, 4, 5, 6

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libgmlp.so")
_lib = None


class GmlpArgs(ctypes.Structure):
    _fields_ = [
        ("struct_bytes", ctypes.c_uint32), ("flags", ctypes.c_uint32),
        ("X", ctypes.c_void_p), ("Wg", ctypes.c_void_p), ("Wu", ctypes.c_void_p), ("Wd", ctypes.c_void_p),
        ("Y", ctypes.c_void_p),
        ("M", ctypes.c_int64), ("d_model", ctypes.c_int64), ("d_ff", ctypes.c_int64),
        ("rms_gain", ctypes.c_void_p), ("rms_eps", ctypes.c_float), ("variant", ctypes.c_int32),
        ("stream", ctypes.c_void_p), ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_uint64),
        ("act_beta", ctypes.c_float), ("reserved", ctypes.c_uint32),
    ]


class GmlpRmsmmArgs(ctypes.Structure):
    _fields_ = [
        ("struct_bytes", ctypes.c_uint32), ("flags", ctypes.c_uint32),
        ("X", ctypes.c_void_p), ("W", ctypes.c_void_p), ("Z", ctypes.c_void_p),
        ("M", ctypes.c_int64), ("K", ctypes.c_int64), ("N", ctypes.c_int64),
        ("rms_gain", ctypes.c_void_p), ("rms_eps", ctypes.c_float), ("reserved", ctypes.c_int32),
        ("stream", ctypes.c_void_p), ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_uint64),
    ]


RMSMM_UNFUSED = 1 << 4
MMADDNORM_UNFUSED = 1 << 4
QKV_SEPARATE = 1 << 4
GQA_CAUSAL = 1 << 4


class GmlpGqaArgs(ctypes.Structure):
    _fields_ = [
        ("struct_bytes", ctypes.c_uint32), ("flags", ctypes.c_uint32),
        ("Q", ctypes.c_void_p), ("K", ctypes.c_void_p), ("V", ctypes.c_void_p), ("O", ctypes.c_void_p),
        ("M", ctypes.c_int64), ("S", ctypes.c_int64),
        ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
        ("reserved", ctypes.c_int32), ("stream", ctypes.c_void_p),
    ]


class GmlpQkvArgs(ctypes.Structure):
    _fields_ = [
        ("struct_bytes", ctypes.c_uint32), ("flags", ctypes.c_uint32),
        ("X", ctypes.c_void_p), ("Wq", ctypes.c_void_p), ("Wk", ctypes.c_void_p), ("Wv", ctypes.c_void_p),
        ("Q", ctypes.c_void_p), ("Kout", ctypes.c_void_p), ("V", ctypes.c_void_p),
        ("M", ctypes.c_int64), ("K", ctypes.c_int64), ("Nq", ctypes.c_int64), ("Nkv", ctypes.c_int64),
        ("stream", ctypes.c_void_p), ("reserved", ctypes.c_uint64),
    ]


class GmlpMmAddNormArgs(ctypes.Structure):
    _fields_ = [
        ("struct_bytes", ctypes.c_uint32), ("flags", ctypes.c_uint32),
        ("X", ctypes.c_void_p), ("W", ctypes.c_void_p), ("R", ctypes.c_void_p), ("S", ctypes.c_void_p),
        ("Z", ctypes.c_void_p),
        ("M", ctypes.c_int64), ("K", ctypes.c_int64), ("N", ctypes.c_int64),
        ("rms_gain", ctypes.c_void_p), ("rms_eps", ctypes.c_float), ("reserved", ctypes.c_int32),
        ("stream", ctypes.c_void_p), ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_uint64),
    ]


class GmlpError(RuntimeError):
    def __init__(self, status: int):
        self.status = status
        super().__init__(f"libgmlp error {status}: {status_string(status)}")


def lib() -> ctypes.CDLL:
    """Loads libgmlp.so (once).  Raises if it is missing: build it with ``__graft_entry__.build()``."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} not found: the CUDA library must be built first "
                               "(python -m paper_2606_26344_b200.build); there is no fallback path")
        L = ctypes.CDLL(_LIB_PATH)
        vp, i64, u32, u64, i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_uint32, ctypes.c_uint64, ctypes.c_int32
        L.gmlp_forward.restype = ctypes.c_int
        L.gmlp_forward.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, u32]
        L.gmlp_forward_ex.restype = ctypes.c_int
        L.gmlp_forward_ex.argtypes = [ctypes.POINTER(GmlpArgs)]
        L.gmlp_rmsnorm_matmul.restype = ctypes.c_int
        L.gmlp_rmsnorm_matmul.argtypes = [ctypes.POINTER(GmlpRmsmmArgs)]
        L.gmlp_gate_up.restype = ctypes.c_int
        L.gmlp_gate_up.argtypes = [ctypes.POINTER(GmlpArgs)]
        L.gmlp_forward_host.restype = ctypes.c_int
        L.gmlp_forward_host.argtypes = [ctypes.POINTER(GmlpArgs), vp, vp]
        L.gmlp_forward_static.restype = ctypes.c_int
        L.gmlp_forward_static.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, vp]
        L.gmlp_workspace_bytes.restype = u64
        L.gmlp_workspace_bytes.argtypes = [i64, i64, i64, u32, i32]
        L.gmlp_matmul_add_rmsnorm.restype = ctypes.c_int
        L.gmlp_matmul_add_rmsnorm.argtypes = [ctypes.POINTER(GmlpMmAddNormArgs)]
        L.gmlp_gqa_attention.restype = ctypes.c_int
        L.gmlp_gqa_attention.argtypes = [ctypes.POINTER(GmlpGqaArgs)]
        L.gmlp_qkv_proj.restype = ctypes.c_int
        L.gmlp_qkv_proj.argtypes = [ctypes.POINTER(GmlpQkvArgs)]
        L.gmlp_autotune.restype = ctypes.c_int
        L.gmlp_autotune.argtypes = [ctypes.POINTER(GmlpArgs), ctypes.c_int, ctypes.POINTER(ctypes.c_int32),
                                    ctypes.POINTER(ctypes.c_float)]
        L.gmlp_autotune_query.restype = ctypes.c_int
        L.gmlp_autotune_query.argtypes = [i64, i64, i64] + [ctypes.POINTER(ctypes.c_int32)] * 3
        L.gmlp_autotune_clear.restype = None
        L.gmlp_autotune_clear.argtypes = []
        L.gmlp_autotune_save.restype = ctypes.c_int
        L.gmlp_autotune_save.argtypes = [ctypes.c_char_p]
        L.gmlp_autotune_load.restype = ctypes.c_int
        L.gmlp_autotune_load.argtypes = [ctypes.c_char_p, ctypes.c_char_p]
        L.gmlp_sum_partials.restype = ctypes.c_int
        L.gmlp_sum_partials.argtypes = [ctypes.POINTER(ctypes.c_void_p), ctypes.c_int32, ctypes.c_void_p, ctypes.c_uint64,
                                        ctypes.c_void_p]
        L.gmlp_workspace_forget.restype = ctypes.c_int
        L.gmlp_workspace_forget.argtypes = [ctypes.c_void_p, ctypes.c_uint64]
        L.gmlp_pick_variant.restype = ctypes.c_int
        L.gmlp_pick_variant.argtypes = [i64, i64, i64, u32]
        L.gmlp_device_status.restype = ctypes.c_int
        L.gmlp_device_status.argtypes = []
        L.gmlp_selftest_wait_timeout.restype = ctypes.c_int
        L.gmlp_selftest_wait_timeout.argtypes = [vp]
        L.gmlp_launch_count.restype = u64
        L.gmlp_launch_count.argtypes = []
        L.gmlp_reset_launch_count.restype = None
        L.gmlp_reset_launch_count.argtypes = []
        L.gmlp_profile_enable.restype = ctypes.c_int
        L.gmlp_profile_enable.argtypes = [ctypes.c_int]
        L.gmlp_profile_read.restype = ctypes.c_int
        L.gmlp_profile_read.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.c_int, ctypes.POINTER(ctypes.c_int)]
        L.gmlp_profile_kernel_name.restype = ctypes.c_char_p
        L.gmlp_profile_kernel_name.argtypes = [ctypes.c_int]
        L.gmlp_status_string.restype = ctypes.c_char_p
        L.gmlp_status_string.argtypes = [ctypes.c_int]
        L.gmlp_version.restype = ctypes.c_int
        L.gmlp_version.argtypes = []
        L.gmlp_set_stream.restype = ctypes.c_int
        L.gmlp_set_stream.argtypes = [vp]
        L.gmlp_set_default_eps.restype = ctypes.c_int
        L.gmlp_set_default_eps.argtypes = [ctypes.c_float]
        L.gmlp_shutdown.restype = None
        L.gmlp_shutdown.argtypes = []
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().gmlp_status_string(int(status)).decode()


def workspace_bytes(M: int, d_model: int, d_ff: int, flags: int = 0, variant: int = VARIANT_AUTO) -> int:
    return int(lib().gmlp_workspace_bytes(M, d_model, d_ff, flags, variant))


def small_m_plan(M: int, d_model: int, d_ff: int, sm_count: int = 0):
    """gmlp_small_m_plan: ((cluster, tile columns, tiles) of the gate/up GEMM, the same of the down projection) as
    GMLP_VARIANT_SKINNY would run the shape; cluster 0 = stream-K."""
    out = (ctypes.c_int32 * 6)()
    L = lib()
    L.gmlp_small_m_plan.restype = ctypes.c_int
    L.gmlp_small_m_plan.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_int32, ctypes.POINTER(ctypes.c_int32)]
    rc = L.gmlp_small_m_plan(M, d_model, d_ff, sm_count, out)
    if rc != OK:
        raise GmlpError(rc)
    return tuple(out[0:3]), tuple(out[3:6])


def small_m_fused_plan(M: int, d_model: int, d_ff: int, sm_count: int = 0):
    """gmlp_small_m_fused_plan: (CTAs per cluster, slices, ring stages, TMEM columns, taken by default) of the one-kernel
    form of GMLP_VARIANT_SKINNY; cluster 0 = the form does not apply."""
    out = (ctypes.c_int32 * 5)()
    L = lib()
    L.gmlp_small_m_fused_plan.restype = ctypes.c_int
    L.gmlp_small_m_fused_plan.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_int32, ctypes.POINTER(ctypes.c_int32)]
    rc = L.gmlp_small_m_fused_plan(M, d_model, d_ff, sm_count, out)
    if rc != OK:
        raise GmlpError(rc)
    return tuple(out[0:5])


def pick_variant(M: int, d_model: int, d_ff: int, flags: int = 0) -> int:
    return int(lib().gmlp_pick_variant(M, d_model, d_ff, flags))


def device_status() -> int:
    return int(lib().gmlp_device_status())


def selftest_wait_timeout() -> int:
    """Runs the bounded-wait self-test on torch's current stream; ERR_TIMEOUT is the expected result."""
    st = torch.cuda.current_stream()
    return int(lib().gmlp_selftest_wait_timeout(st.cuda_stream))


def launch_count() -> int:
    return int(lib().gmlp_launch_count())


def reset_launch_count() -> None:
    lib().gmlp_reset_launch_count()


def profile_enable(on: bool) -> None:
    lib().gmlp_profile_enable(1 if on else 0)


def profile_read() -> dict:
    """Average durations (ms) of the kernels of the calls recorded since profile_enable(True), by kernel name."""
    ms = (ctypes.c_float * 8)()
    n = ctypes.c_int(0)
    rc = lib().gmlp_profile_read(ms, 8, ctypes.byref(n))
    if rc != OK:
        raise GmlpError(rc)
    return {lib().gmlp_profile_kernel_name(i).decode(): float(ms[i]) for i in range(n.value)}


def _check_bf16_cuda(t: torch.Tensor, name: str) -> None:
    if not (t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()):
        raise TypeError(f"{name}: expected a contiguous CUDA bfloat16 tensor")


def make_args(X, Wg, Wu, Wd, Y, gamma=None, eps: float = 1e-5, rmsnorm: bool = False, variant: int = VARIANT_AUTO,
              workspace: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None,
              checked: bool = False, act: str = "silu", beta: float = 1.0, weights_out_in: bool = False,
              weights_in_stream_order: bool = False) -> GmlpArgs:
    for t, n in ((X, "X"), (Wg, "Wg"), (Wu, "Wu"), (Wd, "Wd")):
        _check_bf16_cuda(t, n)
    y_fp32 = Y.dtype == torch.float32              # a float32 Y asks for the unrounded down projection
    if not (Y.is_cuda and Y.is_contiguous() and Y.dtype in (torch.bfloat16, torch.float32)):
        raise TypeError("Y: expected a contiguous CUDA bfloat16 or float32 tensor")
    M, d_model = X.shape
    d_ff = Wg.shape[0] if weights_out_in else Wg.shape[1]
    w_up, w_down = ((d_ff, d_model), (d_model, d_ff)) if weights_out_in else ((d_model, d_ff), (d_ff, d_model))
    if Wg.shape != w_up or Wu.shape != w_up or Wd.shape != w_down or Y.shape != X.shape:
        raise ValueError("shape mismatch")
    flags = (FLAG_RMSNORM if rmsnorm else 0) | (FLAG_CHECKED if checked else 0) | ACT_FLAGS[act] | \
        (FLAG_WEIGHTS_OUT_IN if weights_out_in else 0) | (FLAG_Y_FP32 if y_fp32 else 0) | \
        (FLAG_WEIGHTS_IN_STREAM_ORDER if weights_in_stream_order else 0)
    if gamma is not None:
        _check_bf16_cuda(gamma, "gamma")
    st = stream if stream is not None else torch.cuda.current_stream(X.device)
    a = GmlpArgs()
    a.struct_bytes = ctypes.sizeof(GmlpArgs)
    a.flags = flags
    a.X, a.Wg, a.Wu, a.Wd, a.Y = X.data_ptr(), Wg.data_ptr(), Wu.data_ptr(), Wd.data_ptr(), Y.data_ptr()
    a.M, a.d_model, a.d_ff = M, d_model, d_ff
    a.rms_gain = gamma.data_ptr() if gamma is not None else None
    a.rms_eps = eps
    a.variant = variant
    a.stream = st.cuda_stream
    a.workspace = workspace.data_ptr() if workspace is not None else None
    a.workspace_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    a.act_beta = beta
    a.reserved = 0
    return a


def alloc_workspace(M: int, d_model: int, d_ff: int, rmsnorm: bool = False, variant: int = VARIANT_AUTO,
                    device="cuda") -> torch.Tensor:
    n = workspace_bytes(M, d_model, d_ff, FLAG_RMSNORM if rmsnorm else 0, variant)
    ws = torch.empty(n + 256, dtype=torch.uint8, device=device)[:n] if n else torch.empty(256, dtype=torch.uint8, device=device)
    # the caching allocator may hand out memory the library saw as a workspace before and that other tensors have
    # written since: what the library remembers about it (counters it left at zero) no longer holds
    with torch.cuda.device(ws.device):
        lib().gmlp_workspace_forget(ws.data_ptr(), ws.numel())
    return ws


def forward_ex(args: GmlpArgs) -> None:
    rc = lib().gmlp_forward_ex(ctypes.byref(args))
    if rc != OK:
        raise GmlpError(rc)


def forward(X, Wg, Wu, Wd, Y=None, gamma=None, eps: float = 1e-5, rmsnorm: bool = False,
            variant: int = VARIANT_AUTO, workspace=None, stream=None, checked: bool = False,
            act: str = "silu", beta: float = 1.0, weights_out_in: bool = False,
            weights_in_stream_order: bool = False) -> torch.Tensor:
    """Y = (act(Xn Wg) * (Xn Wu)) Wd on the GPU; asynchronous on ``stream`` (default: torch's current stream).

    ``act``: "silu" (the paper's operator), "swish" (g * sigmoid(beta * g)) or "glu" (sigmoid(g)).
    ``weights_out_in``: the weights are stored [out, in] (Wg, Wu [d_ff, d_model], Wd [d_model, d_ff]).
    ``weights_in_stream_order``: the weights are produced by work enqueued just before on the same stream (the call
    otherwise may fetch weight tiles while that work is still running)."""
    if Y is None:
        Y = torch.empty_like(X)
    with torch.cuda.device(X.device):
        forward_ex(make_args(X, Wg, Wu, Wd, Y, gamma, eps, rmsnorm, variant, workspace, stream, checked, act, beta,
                             weights_out_in, weights_in_stream_order))
    return Y


def forward_host(args: GmlpArgs, X_host: torch.Tensor, Y_host: torch.Tensor) -> None:
    """gmlp_forward_host: X_host / Y_host are host (ideally pinned) bf16 tensors; args.X / args.Y device staging."""
    rc = lib().gmlp_forward_host(ctypes.byref(args), X_host.data_ptr(), Y_host.data_ptr())
    if rc != OK:
        raise GmlpError(rc)


def forward_simple(X, Wg, Wu, Wd, Y, flags: int = 0) -> None:
    """The nine-argument call exactly as the operator is stated."""
    M, d_model = X.shape
    with torch.cuda.device(X.device):
        rc = lib().gmlp_forward(X.data_ptr(), Wg.data_ptr(), Wu.data_ptr(), Wd.data_ptr(), Y.data_ptr(),
                                M, d_model, Wg.shape[1], flags)
    if rc != OK:
        raise GmlpError(rc)


def forward_static(X, Wg, Wu, Wd, Y, stream=None) -> None:
    """gmlp_forward_static: the operator for callers that may not allocate device memory.

    Scratch comes from a fixed array inside the library (M <= STATIC_MAX_M, no RMSNorm); nothing is
    allocated.  Calls that can overlap on the GPU race on that array: keep them on one stream.
    """
    for t, n in ((X, "X"), (Wg, "Wg"), (Wu, "Wu"), (Wd, "Wd"), (Y, "Y")):
        _check_bf16_cuda(t, n)
    M, d_model = X.shape
    st = stream if stream is not None else torch.cuda.current_stream(X.device)
    with torch.cuda.device(X.device):
        rc = lib().gmlp_forward_static(X.data_ptr(), Wg.data_ptr(), Wu.data_ptr(), Wd.data_ptr(), Y.data_ptr(),
                                       M, d_model, Wg.shape[1], st.cuda_stream)
    if rc != OK:
        raise GmlpError(rc)


def gate_up(X, Wg, Wu, H=None, gamma=None, eps: float = 1e-5, rmsnorm: bool = False, variant: int = VARIANT_AUTO,
            workspace=None, stream=None, checked: bool = False, act: str = "silu", beta: float = 1.0,
            weights_out_in: bool = False) -> torch.Tensor:
    """gmlp_gate_up: H = bf16(act(Xn Wg) * (Xn Wu)), the gate/up half alone; H is [M, d_ff]."""
    for t, n in ((X, "X"), (Wg, "Wg"), (Wu, "Wu")):
        _check_bf16_cuda(t, n)
    M, d_model = X.shape
    d_ff = Wg.shape[0] if weights_out_in else Wg.shape[1]
    w_up = (d_ff, d_model) if weights_out_in else (d_model, d_ff)
    if Wg.shape != w_up or Wu.shape != w_up:
        raise ValueError("shape mismatch")
    if H is None:
        H = torch.empty(M, d_ff, dtype=torch.bfloat16, device=X.device)
    _check_bf16_cuda(H, "H")
    if gamma is not None:
        _check_bf16_cuda(gamma, "gamma")
    st = stream if stream is not None else torch.cuda.current_stream(X.device)
    a = GmlpArgs()
    a.struct_bytes = ctypes.sizeof(GmlpArgs)
    a.flags = (FLAG_RMSNORM if rmsnorm else 0) | (FLAG_CHECKED if checked else 0) | ACT_FLAGS[act] | \
        (FLAG_WEIGHTS_OUT_IN if weights_out_in else 0)
    a.act_beta = beta
    a.X, a.Wg, a.Wu, a.Wd, a.Y = X.data_ptr(), Wg.data_ptr(), Wu.data_ptr(), None, H.data_ptr()
    a.M, a.d_model, a.d_ff = M, d_model, d_ff
    a.rms_gain = gamma.data_ptr() if gamma is not None else None
    a.rms_eps = eps
    a.variant = variant
    a.stream = st.cuda_stream
    a.workspace = workspace.data_ptr() if workspace is not None else None
    a.workspace_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    with torch.cuda.device(X.device):
        rc = lib().gmlp_gate_up(ctypes.byref(a))
    if rc != OK:
        raise GmlpError(rc)
    return H


def rmsnorm_matmul(X, W, Z=None, gamma=None, eps: float = 1e-5, unfused: bool = False, stream=None,
                   checked: bool = False) -> torch.Tensor:
    """gmlp_rmsnorm_matmul: Z = RMSNorm(X) @ W.  Default: the rewritten schedule (row scale in the GEMM epilogue)."""
    for t, n in ((X, "X"), (W, "W")):
        _check_bf16_cuda(t, n)
    M, K = X.shape
    N = W.shape[1]
    if W.shape[0] != K:
        raise ValueError("shape mismatch")
    if Z is None:
        Z = torch.empty(M, N, dtype=torch.bfloat16, device=X.device)
    _check_bf16_cuda(Z, "Z")
    nbytes = M * K * 2 if (unfused or gamma is not None) else M * 4
    ws = torch.empty(((nbytes + 255) // 256 + 1) * 256, dtype=torch.uint8, device=X.device)
    st = stream if stream is not None else torch.cuda.current_stream(X.device)
    a = GmlpRmsmmArgs()
    a.struct_bytes = ctypes.sizeof(GmlpRmsmmArgs)
    a.flags = (FLAG_CHECKED if checked else 0) | (RMSMM_UNFUSED if unfused else 0)
    a.X, a.W, a.Z = X.data_ptr(), W.data_ptr(), Z.data_ptr()
    a.M, a.K, a.N = M, K, N
    a.rms_gain = gamma.data_ptr() if gamma is not None else None
    a.rms_eps = eps
    a.reserved = 0
    a.stream = st.cuda_stream
    a.workspace = ws.data_ptr() if ws is not None else None
    a.workspace_bytes = ws.numel() if ws is not None else 0
    with torch.cuda.device(X.device):
        rc = lib().gmlp_rmsnorm_matmul(ctypes.byref(a))
    if rc != OK:
        raise GmlpError(rc)
    return Z


def make_mmaddnorm_args(X, W, R, S, Z, gamma=None, eps: float = 1e-5, unfused: bool = False, workspace=None,
                        stream=None, checked: bool = False) -> GmlpMmAddNormArgs:
    for t, n in ((X, "X"), (W, "W"), (R, "R"), (S, "S"), (Z, "Z")):
        _check_bf16_cuda(t, n)
    M, K = X.shape
    N = W.shape[1]
    if W.shape[0] != K or R.shape != (M, N) or S.shape != (M, N) or Z.shape != (M, N):
        raise ValueError("shape mismatch")
    st = stream if stream is not None else torch.cuda.current_stream(X.device)
    a = GmlpMmAddNormArgs()
    a.struct_bytes = ctypes.sizeof(GmlpMmAddNormArgs)
    a.flags = (FLAG_CHECKED if checked else 0) | (MMADDNORM_UNFUSED if unfused else 0)
    a.X, a.W, a.R, a.S, a.Z = X.data_ptr(), W.data_ptr(), R.data_ptr(), S.data_ptr(), Z.data_ptr()
    a.M, a.K, a.N = M, K, N
    a.rms_gain = gamma.data_ptr() if gamma is not None else None
    a.rms_eps = eps
    a.reserved = 0
    a.stream = st.cuda_stream
    a.workspace = workspace.data_ptr() if workspace is not None else None
    a.workspace_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    return a


def mmaddnorm_workspace(M: int, N: int, unfused: bool = False, device="cuda") -> torch.Tensor:
    nbytes = M * N * 2 if unfused else ((N + 255) // 256) * M * 4
    return torch.empty(((nbytes + 255) // 256 + 1) * 256, dtype=torch.uint8, device=device)


def matmul_add_rmsnorm_ex(args: GmlpMmAddNormArgs) -> None:
    rc = lib().gmlp_matmul_add_rmsnorm(ctypes.byref(args))
    if rc != OK:
        raise GmlpError(rc)


def matmul_add_rmsnorm(X, W, R, S=None, Z=None, gamma=None, eps: float = 1e-5, unfused: bool = False, stream=None,
                       checked: bool = False):
    """gmlp_matmul_add_rmsnorm: S = X @ W + R, Z = RMSNorm(S) * gamma.  Returns (S, Z); S may be R (in place)."""
    M, N = X.shape[0], W.shape[1]
    if S is None:
        S = torch.empty(M, N, dtype=torch.bfloat16, device=X.device)
    if Z is None:
        Z = torch.empty(M, N, dtype=torch.bfloat16, device=X.device)
    ws = mmaddnorm_workspace(M, N, unfused, X.device)
    with torch.cuda.device(X.device):
        matmul_add_rmsnorm_ex(make_mmaddnorm_args(X, W, R, S, Z, gamma, eps, unfused, ws, stream, checked))
    return S, Z


def autotune(args: GmlpArgs, iters: int = 20):
    """gmlp_autotune: time every schedule that can run args' shape, remember the fastest for AUTO.
    Returns (variant, microseconds per call)."""
    v, us = ctypes.c_int32(0), ctypes.c_float(0.0)
    rc = lib().gmlp_autotune(ctypes.byref(args), iters, ctypes.byref(v), ctypes.byref(us))
    if rc != OK:
        raise GmlpError(rc)
    return int(v.value), float(us.value)


def autotune_clear() -> None:
    lib().gmlp_autotune_clear()


def autotune_save(path: str) -> int:
    """gmlp_autotune_save: the tuned choices of this process as a text file; returns the number of shapes written."""
    n = lib().gmlp_autotune_save(os.fsencode(path))
    if n < 0:
        raise GmlpError(n)
    return n


def autotune_load(path: str, device_name: Optional[str] = None) -> int:
    """gmlp_autotune_load: takes the file's lines for this library version and `device_name` (default: the current
    device's name); returns the number of shapes taken."""
    n = lib().gmlp_autotune_load(os.fsencode(path), None if device_name is None else device_name.encode())
    if n < 0:
        raise GmlpError(n)
    return n


def autotune_query(M: int, d_model: int, d_ff: int):
    """(variant, gate_up_pair, down_pair) kept by autotune for this shape on the current device, or None."""
    v, g, d = ctypes.c_int32(0), ctypes.c_int32(0), ctypes.c_int32(0)
    if not lib().gmlp_autotune_query(M, d_model, d_ff, ctypes.byref(v), ctypes.byref(g), ctypes.byref(d)):
        return None
    return int(v.value), int(g.value), int(d.value)


def make_qkv_args(X, Wq, Wk, Wv, Q, K, V, separate: bool = False, stream=None, checked: bool = False) -> GmlpQkvArgs:
    for t, n in ((X, "X"), (Wq, "Wq"), (Wk, "Wk"), (Wv, "Wv"), (Q, "Q"), (K, "K"), (V, "V")):
        _check_bf16_cuda(t, n)
    M, Kd = X.shape
    Nq, Nkv = Wq.shape[1], Wk.shape[1]
    if Wq.shape[0] != Kd or Wk.shape != (Kd, Nkv) or Wv.shape != (Kd, Nkv) or Q.shape != (M, Nq) or K.shape != (M, Nkv) \
            or V.shape != (M, Nkv):
        raise ValueError("shape mismatch")
    st = stream if stream is not None else torch.cuda.current_stream(X.device)
    a = GmlpQkvArgs()
    a.struct_bytes = ctypes.sizeof(GmlpQkvArgs)
    a.flags = (FLAG_CHECKED if checked else 0) | (QKV_SEPARATE if separate else 0)
    a.X, a.Wq, a.Wk, a.Wv = X.data_ptr(), Wq.data_ptr(), Wk.data_ptr(), Wv.data_ptr()
    a.Q, a.Kout, a.V = Q.data_ptr(), K.data_ptr(), V.data_ptr()
    a.M, a.K, a.Nq, a.Nkv = M, Kd, Nq, Nkv
    a.stream = st.cuda_stream
    a.reserved = 0
    return a


def qkv_proj_ex(args: GmlpQkvArgs) -> None:
    rc = lib().gmlp_qkv_proj(ctypes.byref(args))
    if rc != OK:
        raise GmlpError(rc)


def qkv_proj(X, Wq, Wk, Wv, separate: bool = False, stream=None, checked: bool = False):
    """gmlp_qkv_proj: (Q, K, V) = (X @ Wq, X @ Wk, X @ Wv), one launch unless ``separate``."""
    M = X.shape[0]
    Q = torch.empty(M, Wq.shape[1], dtype=torch.bfloat16, device=X.device)
    K = torch.empty(M, Wk.shape[1], dtype=torch.bfloat16, device=X.device)
    V = torch.empty(M, Wv.shape[1], dtype=torch.bfloat16, device=X.device)
    with torch.cuda.device(X.device):
        qkv_proj_ex(make_qkv_args(X, Wq, Wk, Wv, Q, K, V, separate, stream, checked))
    return Q, K, V


def make_gqa_args(Q, K, V, O, n_q_heads: int, n_kv_heads: int, stream=None, checked: bool = False,
                  causal: bool = False) -> GmlpGqaArgs:
    for t, n in ((Q, "Q"), (K, "K"), (V, "V"), (O, "O")):
        _check_bf16_cuda(t, n)
    M, S = Q.shape[0], K.shape[0]
    D = Q.shape[1] // n_q_heads
    if Q.shape[1] != n_q_heads * D or K.shape != (S, n_kv_heads * D) or V.shape != K.shape or O.shape != Q.shape:
        raise ValueError("shape mismatch")
    st = stream if stream is not None else torch.cuda.current_stream(Q.device)
    a = GmlpGqaArgs()
    a.struct_bytes = ctypes.sizeof(GmlpGqaArgs)
    a.flags = (FLAG_CHECKED if checked else 0) | (GQA_CAUSAL if causal else 0)
    a.Q, a.K, a.V, a.O = Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr()
    a.M, a.S = M, S
    a.n_q_heads, a.n_kv_heads, a.head_dim, a.reserved = n_q_heads, n_kv_heads, D, 0
    a.stream = st.cuda_stream
    return a


def gqa_attention_ex(args: GmlpGqaArgs) -> None:
    rc = lib().gmlp_gqa_attention(ctypes.byref(args))
    if rc != OK:
        raise GmlpError(rc)


def gqa_attention(Q, K, V, n_q_heads: int, n_kv_heads: int, O=None, stream=None, checked: bool = False,
                  causal: bool = False) -> torch.Tensor:
    """gmlp_gqa_attention: O_h = softmax(Q_h K_g^T / sqrt(D)) V_g, D = 128; no mask, or causal (queries = last M positions)."""
    if O is None:
        O = torch.empty_like(Q)
    with torch.cuda.device(Q.device):
        gqa_attention_ex(make_gqa_args(Q, K, V, O, n_q_heads, n_kv_heads, stream, checked, causal))
    return O


def sum_partials(parts, Y=None, stream=None) -> "torch.Tensor":
    """gmlp_sum_partials: Y = bf16(parts[0] + parts[1] + ...) over fp32 partial products of equal shape (the last
    step of a d_ff-sharded Gated MLP); the sum runs in the order given."""
    if not parts:
        raise ValueError("no partial products")
    for t in parts:
        if not (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous() and t.shape == parts[0].shape):
            raise ValueError("partial products must be contiguous float32 CUDA tensors of one shape")
    if Y is None:
        Y = torch.empty(parts[0].shape, dtype=torch.bfloat16, device=parts[0].device)
    _check_bf16_cuda(Y, "Y")
    ptrs = (ctypes.c_void_p * len(parts))(*[t.data_ptr() for t in parts])
    st = stream.cuda_stream if stream is not None else torch.cuda.current_stream(Y.device).cuda_stream
    with torch.cuda.device(Y.device):
        rc = lib().gmlp_sum_partials(ptrs, len(parts), Y.data_ptr(), Y.numel(), st)
    if rc != OK:
        raise GmlpError(rc)
    return Y
