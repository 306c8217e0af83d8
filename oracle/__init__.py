"""CPU oracle for the Gated MLP — TEST INFRASTRUCTURE ONLY.

Python face of ``gmlp_oracle.c`` / ``naive_matmul.c`` (plain C, fp64, OpenMP over rows).
Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package.  The CUDA library and its Python binding never do, and nothing here imports them.

Arrays are numpy; bf16 values travel as ``uint16`` bit patterns so that the oracle sees
exactly the bits the GPU is given.

The shared object is compiled for the CPU it runs on (``-march=native``) and therefore
carries a tag derived from the CPU's feature flags in its file name: a copy built on a
different machine is ignored and rebuilt.
"""
from __future__ import annotations

import ctypes
import hashlib
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SOURCES = ("gmlp_oracle.c", "naive_matmul.c")
_lock = threading.Lock()
_lib = None


def _cpu_tag() -> str:
    flags = ""
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    flags = line
                    break
    except OSError:
        pass
    return hashlib.sha1(flags.encode()).hexdigest()[:10]


def lib_path() -> str:
    return os.path.join(_HERE, f"liboracle.{_cpu_tag()}.so")


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc if the shared object is missing or older than its sources."""
    out = lib_path()
    srcs = [os.path.join(_HERE, s) for s in _SOURCES]
    if not force and os.path.exists(out):
        if all(os.path.getmtime(out) >= os.path.getmtime(s) for s in srcs):
            return out
    tmp = out + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
           "-shared", "-fPIC", "-o", tmp, *srcs, "-lm"]
    subprocess.run(cmd, check=True, capture_output=True, text=True)
    os.replace(tmp, out)
    return out


def _load():
    global _lib
    with _lock:
        if _lib is not None:
            return _lib
        lib = ctypes.CDLL(build())
        u16p = ctypes.POINTER(ctypes.c_uint16)
        f64p = ctypes.POINTER(ctypes.c_double)
        i64p = ctypes.POINTER(ctypes.c_int64)
        lib.gmlp_oracle_bf16_to_double.restype = ctypes.c_double
        lib.gmlp_oracle_bf16_to_double.argtypes = [ctypes.c_uint16]
        lib.gmlp_oracle_bf16_rn.restype = ctypes.c_uint16
        lib.gmlp_oracle_bf16_rn.argtypes = [ctypes.c_double]
        lib.gmlp_oracle_silu.restype = ctypes.c_double
        lib.gmlp_oracle_silu.argtypes = [ctypes.c_double]
        lib.gmlp_oracle_rmsnorm_row.restype = None
        lib.gmlp_oracle_rmsnorm_row.argtypes = [u16p, u16p, ctypes.c_float, ctypes.c_int64, u16p, f64p]
        lib.gmlp_oracle_rows.restype = ctypes.c_int
        lib.gmlp_oracle_rows.argtypes = [u16p, u16p, u16p, u16p, u16p, ctypes.c_float, ctypes.c_int,
                                         ctypes.c_int64, ctypes.c_int64, ctypes.c_int64,
                                         i64p, ctypes.c_int64, f64p, u16p, u16p, ctypes.c_int]
        lib.gmlp_oracle_rows_act.restype = ctypes.c_int
        lib.gmlp_oracle_rows_act.argtypes = lib.gmlp_oracle_rows.argtypes + [ctypes.c_int, ctypes.c_double]
        lib.gmlp_oracle_gate_act.restype = ctypes.c_double
        lib.gmlp_oracle_gate_act.argtypes = [ctypes.c_double, ctypes.c_int, ctypes.c_double]
        lib.gmlp_oracle_gate_act_array.restype = None
        lib.gmlp_oracle_gate_act_array.argtypes = [f64p, f64p, ctypes.c_int64, ctypes.c_int, ctypes.c_double]
        lib.gmlp_oracle_gate_up_rows.restype = ctypes.c_int
        lib.gmlp_oracle_gate_up_rows.argtypes = [u16p, u16p, u16p, u16p, ctypes.c_float, ctypes.c_int,
                                                 ctypes.c_int64, ctypes.c_int64, ctypes.c_int64,
                                                 i64p, ctypes.c_int64, f64p, ctypes.c_int]
        lib.gmlp_oracle_matmul_add_rmsnorm_rows.restype = ctypes.c_int
        lib.gmlp_oracle_matmul_add_rmsnorm_rows.argtypes = [u16p, u16p, u16p, u16p, ctypes.c_float, ctypes.c_int64,
                                                            ctypes.c_int64, ctypes.c_int64, i64p, ctypes.c_int64,
                                                            u16p, f64p, f64p, ctypes.c_int]
        lib.gmlp_oracle_matmul_rows.restype = ctypes.c_int
        lib.gmlp_oracle_matmul_rows.argtypes = [u16p, u16p, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, i64p,
                                                ctypes.c_int64, f64p, ctypes.c_int]
        lib.gmlp_oracle_gqa_rows.restype = ctypes.c_int
        lib.gmlp_oracle_gqa_rows.argtypes = [u16p, u16p, u16p] + [ctypes.c_int64] * 5 + [i64p, ctypes.c_int64, f64p, ctypes.c_int,
                                             ctypes.c_int]
        lib.gmlp_oracle_gate_up_rows_act.restype = ctypes.c_int
        lib.gmlp_oracle_gate_up_rows_act.argtypes = lib.gmlp_oracle_gate_up_rows.argtypes + [ctypes.c_int, ctypes.c_double]
        lib.gmlp_oracle_rmsnorm_matmul_rows.restype = ctypes.c_int
        lib.gmlp_oracle_rmsnorm_matmul_rows.argtypes = [u16p, u16p, u16p, ctypes.c_float, ctypes.c_int64, ctypes.c_int64,
                                                        ctypes.c_int64, i64p, ctypes.c_int64, f64p, ctypes.c_int]
        lib.gmlp_oracle_bf16_rn_array.restype = None
        lib.gmlp_oracle_bf16_rn_array.argtypes = [f64p, u16p, ctypes.c_int64]
        lib.gmlp_oracle_silu_array.restype = None
        lib.gmlp_oracle_silu_array.argtypes = [f64p, f64p, ctypes.c_int64]
        lib.gmlp_oracle_max_threads.restype = ctypes.c_int
        lib.gmlp_oracle_max_threads.argtypes = []
        lib.naive_matmul_f64.restype = None
        lib.naive_matmul_f64.argtypes = [f64p, f64p, f64p, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64]
        _lib = lib
        return lib


def _u16(a, name):
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint16:
        raise TypeError(f"{name}: expected uint16 bf16 bit patterns, got {a.dtype}")
    return a


def _p(a, ty):
    return a.ctypes.data_as(ctypes.POINTER(ty))


def bf16_to_double(bits) -> np.ndarray:
    """bf16 bit patterns (uint16) -> float64, exact (numpy shift; no C involved)."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def bf16_rn(values) -> np.ndarray:
    """float64 -> bf16 bit patterns with the C oracle's single round-to-nearest-even."""
    lib = _load()
    v = np.ascontiguousarray(values, dtype=np.float64)
    out = np.empty(v.shape, dtype=np.uint16)
    lib.gmlp_oracle_bf16_rn_array(_p(v, ctypes.c_double), _p(out, ctypes.c_uint16), v.size)
    return out


def silu(values) -> np.ndarray:
    lib = _load()
    v = np.ascontiguousarray(values, dtype=np.float64)
    out = np.empty_like(v)
    lib.gmlp_oracle_silu_array(_p(v, ctypes.c_double), _p(out, ctypes.c_double), v.size)
    return out


ACT_KINDS = {"silu": 0, "swish": 1, "glu": 2, "gelu": 3}


def gate_act(values, act: str = "silu", beta: float = 1.0) -> np.ndarray:
    """The gate activation of the gated unit: silu g*sigmoid(g), swish g*sigmoid(beta*g), glu sigmoid(g), gelu g*Phi(g)."""
    lib = _load()
    v = np.ascontiguousarray(values, dtype=np.float64)
    out = np.empty_like(v)
    lib.gmlp_oracle_gate_act_array(_p(v, ctypes.c_double), _p(out, ctypes.c_double), v.size, ACT_KINDS[act], float(beta))
    return out


def rmsnorm_row(x_bits, gamma_bits=None, eps: float = 1e-5):
    """One row of the RMSNorm prologue.  Returns (xn bf16 bits, r as float64)."""
    lib = _load()
    x = _u16(x_bits, "x").reshape(-1)
    g = None if gamma_bits is None else _u16(gamma_bits, "gamma").reshape(-1)
    out = np.empty_like(x)
    r = ctypes.c_double(0.0)
    lib.gmlp_oracle_rmsnorm_row(_p(x, ctypes.c_uint16), None if g is None else _p(g, ctypes.c_uint16),
                                ctypes.c_float(eps), x.size, _p(out, ctypes.c_uint16), ctypes.byref(r))
    return out, r.value


def max_threads() -> int:
    return int(_load().gmlp_oracle_max_threads())


def gmlp_rows(X, Wg, Wu, Wd, rows=None, gamma=None, eps: float = 1e-5, rmsnorm: bool = False,
              num_threads: int = 0, want_h: bool = False, want_xn: bool = False, act: str = "silu", beta: float = 1.0):
    """Reference Y (float64, not rounded) for the selected rows of X.

    X [M, d_model], Wg/Wu [d_model, d_ff], Wd [d_ff, d_model]: uint16 bf16 bit patterns.
    Returns Y_ref [len(rows), d_model]; with want_h / want_xn also the bf16 bits of H / Xn.
    """
    lib = _load()
    X, Wg, Wu, Wd = _u16(X, "X"), _u16(Wg, "Wg"), _u16(Wu, "Wu"), _u16(Wd, "Wd")
    M, d_model = X.shape
    d_ff = Wg.shape[1]
    if Wg.shape != (d_model, d_ff) or Wu.shape != (d_model, d_ff) or Wd.shape != (d_ff, d_model):
        raise ValueError("shape mismatch")
    if rows is None:
        rows = np.arange(M, dtype=np.int64)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    g = None
    if gamma is not None:
        g = _u16(gamma, "gamma").reshape(-1)
        if g.size != d_model:
            raise ValueError("gamma size")
    R = rows.size
    Y = np.zeros((R, d_model), dtype=np.float64)
    H = np.zeros((R, d_ff), dtype=np.uint16) if want_h else None
    Xn = np.zeros((R, d_model), dtype=np.uint16) if want_xn else None
    common = (_p(X, ctypes.c_uint16), _p(Wg, ctypes.c_uint16), _p(Wu, ctypes.c_uint16),
              _p(Wd, ctypes.c_uint16), None if g is None else _p(g, ctypes.c_uint16),
              ctypes.c_float(eps), int(bool(rmsnorm)), M, d_model, d_ff,
              _p(rows, ctypes.c_int64), R, _p(Y, ctypes.c_double),
              None if H is None else _p(H, ctypes.c_uint16),
              None if Xn is None else _p(Xn, ctypes.c_uint16), int(num_threads))
    if act == "silu":
        rc = lib.gmlp_oracle_rows(*common)
    else:
        rc = lib.gmlp_oracle_rows_act(*common, ACT_KINDS[act], float(beta))
    if rc != 0:
        raise RuntimeError(f"gmlp_oracle_rows failed ({rc})")
    out = [Y]
    if want_h:
        out.append(H)
    if want_xn:
        out.append(Xn)
    return out[0] if len(out) == 1 else tuple(out)


def gate_up_rows(X, Wg, Wu, rows=None, gamma=None, eps: float = 1e-5, rmsnorm: bool = False,
                 num_threads: int = 0, act: str = "silu", beta: float = 1.0) -> np.ndarray:
    """Reference silu(Xn Wg) * (Xn Wu) (float64, not rounded) for the selected rows: the gate/up half alone."""
    lib = _load()
    X, Wg, Wu = _u16(X, "X"), _u16(Wg, "Wg"), _u16(Wu, "Wu")
    M, d_model = X.shape
    d_ff = Wg.shape[1]
    if Wg.shape != (d_model, d_ff) or Wu.shape != (d_model, d_ff):
        raise ValueError("shape mismatch")
    if rows is None:
        rows = np.arange(M, dtype=np.int64)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    g = None
    if gamma is not None:
        g = _u16(gamma, "gamma").reshape(-1)
        if g.size != d_model:
            raise ValueError("gamma size")
    P = np.zeros((rows.size, d_ff), dtype=np.float64)
    common = (_p(X, ctypes.c_uint16), _p(Wg, ctypes.c_uint16), _p(Wu, ctypes.c_uint16),
              None if g is None else _p(g, ctypes.c_uint16), ctypes.c_float(eps),
              int(bool(rmsnorm)), M, d_model, d_ff, _p(rows, ctypes.c_int64), rows.size,
              _p(P, ctypes.c_double), int(num_threads))
    if act == "silu":
        rc = lib.gmlp_oracle_gate_up_rows(*common)
    else:
        rc = lib.gmlp_oracle_gate_up_rows_act(*common, ACT_KINDS[act], float(beta))
    if rc != 0:
        raise RuntimeError(f"gmlp_oracle_gate_up_rows failed ({rc})")
    return P


def rmsnorm_matmul_rows(X, W, rows=None, gamma=None, eps: float = 1e-5, num_threads: int = 0) -> np.ndarray:
    """Reference RMSNorm(X) @ W (float64, no intermediate rounding) for the selected rows."""
    lib = _load()
    X, W = _u16(X, "X"), _u16(W, "W")
    M, K = X.shape
    if W.shape[0] != K:
        raise ValueError("shape mismatch")
    N = W.shape[1]
    if rows is None:
        rows = np.arange(M, dtype=np.int64)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    g = None
    if gamma is not None:
        g = _u16(gamma, "gamma").reshape(-1)
        if g.size != K:
            raise ValueError("gamma size")
    Z = np.zeros((rows.size, N), dtype=np.float64)
    rc = lib.gmlp_oracle_rmsnorm_matmul_rows(_p(X, ctypes.c_uint16), _p(W, ctypes.c_uint16),
                                             None if g is None else _p(g, ctypes.c_uint16), ctypes.c_float(eps),
                                             M, K, N, _p(rows, ctypes.c_int64), rows.size, _p(Z, ctypes.c_double),
                                             int(num_threads))
    if rc != 0:
        raise RuntimeError(f"gmlp_oracle_rmsnorm_matmul_rows failed ({rc})")
    return Z


def matmul_add_rmsnorm_rows(X, W, R, rows=None, gamma=None, eps: float = 1e-5, num_threads: int = 0):
    """Reference for S = X @ W + R, Z = RMSNorm(bf16(S)) on the selected rows.

    Returns (S_bits uint16 [rows, N], S_ref float64 unrounded, Z float64)."""
    lib = _load()
    X, W, R = _u16(X, "X"), _u16(W, "W"), _u16(R, "R")
    M, K = X.shape
    N = W.shape[1]
    if W.shape[0] != K or R.shape != (M, N):
        raise ValueError("shape mismatch")
    if rows is None:
        rows = np.arange(M, dtype=np.int64)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    g = None
    if gamma is not None:
        g = _u16(gamma, "gamma").reshape(-1)
        if g.size != N:
            raise ValueError("gamma size")
    Sb = np.zeros((rows.size, N), dtype=np.uint16)
    Sr = np.zeros((rows.size, N), dtype=np.float64)
    Z = np.zeros((rows.size, N), dtype=np.float64)
    rc = lib.gmlp_oracle_matmul_add_rmsnorm_rows(_p(X, ctypes.c_uint16), _p(W, ctypes.c_uint16), _p(R, ctypes.c_uint16),
                                                 None if g is None else _p(g, ctypes.c_uint16), ctypes.c_float(eps),
                                                 M, K, N, _p(rows, ctypes.c_int64), rows.size,
                                                 _p(Sb, ctypes.c_uint16), _p(Sr, ctypes.c_double), _p(Z, ctypes.c_double),
                                                 int(num_threads))
    if rc != 0:
        raise RuntimeError(f"gmlp_oracle_matmul_add_rmsnorm_rows failed ({rc})")
    return Sb, Sr, Z


def matmul_rows(X, W, rows=None, num_threads: int = 0) -> np.ndarray:
    """Reference X @ W (float64) for the selected rows; bf16 bit patterns in."""
    lib = _load()
    X, W = _u16(X, "X"), _u16(W, "W")
    M, K = X.shape
    if W.shape[0] != K:
        raise ValueError("shape mismatch")
    N = W.shape[1]
    if rows is None:
        rows = np.arange(M, dtype=np.int64)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    Z = np.zeros((rows.size, N), dtype=np.float64)
    rc = lib.gmlp_oracle_matmul_rows(_p(X, ctypes.c_uint16), _p(W, ctypes.c_uint16), M, K, N, _p(rows, ctypes.c_int64),
                                     rows.size, _p(Z, ctypes.c_double), int(num_threads))
    if rc != 0:
        raise RuntimeError(f"gmlp_oracle_matmul_rows failed ({rc})")
    return Z


def qkv_rows(X, Wq, Wk, Wv, rows=None, num_threads: int = 0):
    """Reference (Q, K, V) = (X @ Wq, X @ Wk, X @ Wv) for the selected rows: the QKV projection."""
    return tuple(matmul_rows(X, W, rows, num_threads) for W in (Wq, Wk, Wv))


def gqa_rows(Q, K, V, n_q_heads: int, n_kv_heads: int, rows=None, num_threads: int = 0, causal: bool = False) -> np.ndarray:
    """Reference group query attention (float64) for the selected query rows.

    Q [M, Hq*D], K and V [S, Hkv*D] bf16 bit patterns; returns O_ref [len(rows), Hq*D]."""
    lib = _load()
    Q, K, V = _u16(Q, "Q"), _u16(K, "K"), _u16(V, "V")
    M, S = Q.shape[0], K.shape[0]
    if Q.shape[1] % n_q_heads:
        raise ValueError("Q width is not a multiple of the head count")
    D = Q.shape[1] // n_q_heads
    if K.shape != (S, n_kv_heads * D) or V.shape != K.shape:
        raise ValueError("shape mismatch")
    if rows is None:
        rows = np.arange(M, dtype=np.int64)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    O = np.zeros((rows.size, n_q_heads * D), dtype=np.float64)
    rc = lib.gmlp_oracle_gqa_rows(_p(Q, ctypes.c_uint16), _p(K, ctypes.c_uint16), _p(V, ctypes.c_uint16), M, S,
                                  n_q_heads, n_kv_heads, D, _p(rows, ctypes.c_int64), rows.size, _p(O, ctypes.c_double),
                                  int(num_threads), int(bool(causal)))
    if rc != 0:
        raise RuntimeError(f"gmlp_oracle_gqa_rows failed ({rc})")
    return O


def naive_matmul(A, B) -> np.ndarray:
    """Textbook triple-loop matmul on float64 arrays (separate translation unit; tiny shapes only)."""
    lib = _load()
    A = np.ascontiguousarray(A, dtype=np.float64)
    B = np.ascontiguousarray(B, dtype=np.float64)
    M, K = A.shape
    K2, N = B.shape
    if K != K2:
        raise ValueError("inner dimensions differ")
    C = np.empty((M, N), dtype=np.float64)
    lib.naive_matmul_f64(_p(A, ctypes.c_double), _p(B, ctypes.c_double), _p(C, ctypes.c_double), M, K, N)
    return C


def tolerance(y_ref) -> np.ndarray:
    """Per-element bound of the parity rule: |y - y_ref| <= 2e-2 * max(1, |y_ref|)."""
    return 2e-2 * np.maximum(1.0, np.abs(np.asarray(y_ref, dtype=np.float64)))
