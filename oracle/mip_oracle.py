"""ctypes front end of the CPU oracle (``mip_oracle.c``).

TEST INFRASTRUCTURE ONLY: nothing in the product package may import this
module.  It compiles the plain-C oracle with gcc on first use (OpenMP over
output rows) and exposes it on NumPy arrays.  The arithmetic lives in the C
file; this module only marshals arguments.

Definitions followed: exact INT8 x INT8 -> INT32 GEMM (paper Section 5
opening, Section 7.3, Figure 1) and the convolution operator of Section 7.2.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mip_oracle.c")
# MIP_ORACLE_SANITIZE=1 selects a second build of the same source with gcc's address and undefined-
# behaviour sanitizers (-O1), used by the oracle's own unit tests: an out-of-bounds index or a signed
# overflow inside the oracle then aborts the test process instead of passing by luck.  The process must
# have the sanitizer runtime preloaded (see sanitizer_env()).
SANITIZED = os.environ.get("MIP_ORACLE_SANITIZE") == "1"
_LIB = os.path.join(_HERE, "libmip_oracle_san.so" if SANITIZED else "libmip_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle shared object next to its source; returns its path."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".tmp.%d" % os.getpid()
            opt = ["-O1", "-g", "-fsanitize=address,undefined", "-fno-sanitize-recover=undefined",
                   "-fno-omit-frame-pointer"] if SANITIZED else ["-O3", "-march=native"]
            cmd = ["gcc"] + opt + ["-fopenmp", "-fPIC", "-shared", "-std=c11", "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def sanitizer_env() -> dict:
    """Environment for a child process that should load the sanitized oracle build."""
    env = dict(os.environ)
    asan = subprocess.run(["gcc", "-print-file-name=libasan.so"], capture_output=True, text=True, check=True).stdout.strip()
    env.update(MIP_ORACLE_SANITIZE="1", LD_PRELOAD=asan,
               ASAN_OPTIONS="detect_leaks=0:abort_on_error=1", UBSAN_OPTIONS="halt_on_error=1:print_stacktrace=1")
    return env


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        i64, vp, ci = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int
        lib.mip_oracle_gemm.restype = i64
        lib.mip_oracle_gemm.argtypes = [ci, i64, i64, i64, vp, i64, vp, i64, vp, i64, ci]
        lib.mip_oracle_gemm_ex.restype = i64
        lib.mip_oracle_gemm_ex.argtypes = [ci, ci, i64, i64, i64, vp, i64, vp, i64, vp, i64, ci]
        lib.mip_oracle_conv.restype = i64
        lib.mip_oracle_conv.argtypes = [i64] * 13 + [vp, vp, vp, ci]
        lib.mip_oracle_dequant.restype = None
        lib.mip_oracle_dequant.argtypes = [vp, i64, ctypes.c_double, vp]
        lib.mip_oracle_requant.restype = None
        lib.mip_oracle_requant.argtypes = [vp, i64, ctypes.c_float, ctypes.c_int32, ctypes.c_int32, vp]
        lib.mip_oracle_add_bias.restype = i64
        lib.mip_oracle_add_bias.argtypes = [vp, i64, i64, vp, vp]
        lib.mip_oracle_threads.restype = ci
        lib.mip_oracle_threads.argtypes = []
        _lib = lib
    return _lib


def threads() -> int:
    """Number of OpenMP threads the oracle will use."""
    return int(_load().mip_oracle_threads())


class OracleOverflow(ArithmeticError):
    """The exact result of some cell does not fit int32."""


def _ptr(a: np.ndarray) -> int:
    return a.ctypes.data


def gemm(A: np.ndarray, B: np.ndarray, M: int, N: int, K: int, *, lda: int | None = None,
         ldb: int | None = None, C: np.ndarray | None = None, ldc: int | None = None,
         accumulate: bool = False, allow_overflow: bool = False) -> np.ndarray:
    """C = [C +] A * B, exact.

    ``A``: flat or 2-D C-contiguous buffer of int8 (signed mode) or uint8
    (unsigned mode), row-major M x K with pitch ``lda``.  ``B``: int8 (or uint8) buffer,
    column-major K x N, i.e. N runs of K bytes with pitch ``ldb``.  ``C``:
    int32 buffer with pitch ``ldc`` (allocated, zero-filled, when omitted); it is
    updated in place and returned.  Raises :class:`OracleOverflow` if any exact
    value leaves the int32 range, unless ``allow_overflow``.
    """
    if A.dtype == np.int8:
        a_unsigned = 0
    elif A.dtype == np.uint8:
        a_unsigned = 1
    else:
        raise TypeError("A must be int8 or uint8")
    if B.dtype == np.int8:
        b_unsigned = 0
    elif B.dtype == np.uint8:
        b_unsigned = 1
    else:
        raise TypeError("B must be int8 or uint8")
    lda = K if lda is None else lda
    ldb = K if ldb is None else ldb
    ldc = N if ldc is None else ldc
    if C is None:
        C = np.zeros(max(M, 0) * ldc, dtype=np.int32)
    if C.dtype != np.int32:
        raise TypeError("C must be int32")
    for arr in (A, B, C):
        if not arr.flags["C_CONTIGUOUS"]:
            raise ValueError("buffers must be C-contiguous")
    if M > 0 and N > 0:
        if K > 0 and (A.size < (M - 1) * lda + K or B.size < (N - 1) * ldb + K):
            raise ValueError("A or B buffer too small for the stated pitch")
        if C.size < (M - 1) * ldc + N:
            raise ValueError("C buffer too small for the stated pitch")
    rc = _load().mip_oracle_gemm_ex(a_unsigned, b_unsigned, M, N, K, _ptr(A), lda, _ptr(B), ldb, _ptr(C), ldc,
                                    1 if accumulate else 0)
    if rc < 0:
        raise ValueError("mip_oracle_gemm rejected its arguments")
    if rc > 0 and not allow_overflow:
        raise OracleOverflow("%d cells do not fit int32" % rc)
    return C


def conv_out_hw(H, W, R, S, stride, pad, dil):
    """Output extent of the convolution (paper Section 7.2 shapes)."""
    Ho = (H + 2 * pad[0] - dil[0] * (R - 1) - 1) // stride[0] + 1
    Wo = (W + 2 * pad[1] - dil[1] * (S - 1) - 1) // stride[1] + 1
    return Ho, Wo


def conv(X: np.ndarray, Wt: np.ndarray, *, stride=(1, 1), pad=(0, 0), dil=(1, 1),
         Y: np.ndarray | None = None, accumulate: bool = False,
         allow_overflow: bool = False) -> np.ndarray:
    """Y = [Y +] Conv(Wt, X): X uint8 [Nb][H][W][Cin], Wt int8 [Cout][R][S][Cin],
    Y int32 [Nb][Ho][Wo][Cout]; out-of-image taps contribute zero."""
    if X.dtype != np.uint8 or Wt.dtype != np.int8:
        raise TypeError("X must be uint8 and Wt int8")
    Nb, H, W, Cin = X.shape
    Cout, R, S, Cin2 = Wt.shape
    if Cin != Cin2:
        raise ValueError("channel mismatch")
    Ho, Wo = conv_out_hw(H, W, R, S, stride, pad, dil)
    X = np.ascontiguousarray(X)
    Wt = np.ascontiguousarray(Wt)
    if Y is None:
        Y = np.zeros((Nb, Ho, Wo, Cout), dtype=np.int32)
    if Y.dtype != np.int32 or Y.shape != (Nb, Ho, Wo, Cout) or not Y.flags["C_CONTIGUOUS"]:
        raise ValueError("Y must be a contiguous int32 [Nb][Ho][Wo][Cout] array")
    rc = _load().mip_oracle_conv(Nb, H, W, Cin, Cout, R, S, stride[0], stride[1], pad[0], pad[1],
                                 dil[0], dil[1], _ptr(X), _ptr(Wt), _ptr(Y), 1 if accumulate else 0)
    if rc < 0:
        raise ValueError("mip_oracle_conv rejected its arguments")
    if rc > 0 and not allow_overflow:
        raise OracleOverflow("%d cells do not fit int32" % rc)
    return Y


def dequant(Cq: np.ndarray, scale: float) -> np.ndarray:
    """C^r = scale * C^q (paper Section 7.3) in binary64, element by element; same shape as Cq."""
    if Cq.dtype != np.int32:
        raise TypeError("Cq must be int32")
    flat = np.ascontiguousarray(Cq).reshape(-1)
    out = np.empty(flat.size, dtype=np.float64)
    _load().mip_oracle_dequant(_ptr(flat), flat.size, float(scale), _ptr(out))
    return out.reshape(Cq.shape)


def requant(Cq: np.ndarray, scale: float, lo: int, hi: int) -> np.ndarray:
    """8-bit codes min(max(rne(fl32(fl32(Cq) * scale)), lo), hi) as an int32 array of Cq's shape."""
    if Cq.dtype != np.int32:
        raise TypeError("Cq must be int32")
    if not np.isfinite(np.float32(scale)):
        raise ValueError("scale must be finite")
    flat = np.ascontiguousarray(Cq).reshape(-1)
    out = np.empty(flat.size, dtype=np.int32)
    _load().mip_oracle_requant(_ptr(flat), flat.size, float(np.float32(scale)), int(lo), int(hi), _ptr(out))
    return out.reshape(Cq.shape)


def add_bias(Cq: np.ndarray, bias: np.ndarray, allow_overflow: bool = False) -> np.ndarray:
    """Cq(..., j) + bias[j], exact (int64, range-checked into int32); the last axis of Cq is the channel axis."""
    if Cq.dtype != np.int32 or bias.dtype != np.int32:
        raise TypeError("Cq and bias must be int32")
    cols = Cq.shape[-1]
    if bias.shape != (cols,):
        raise ValueError("bias must have one entry per output channel")
    flat = np.ascontiguousarray(Cq).reshape(-1, cols)
    bias = np.ascontiguousarray(bias)
    out = np.empty_like(flat)
    rc = _load().mip_oracle_add_bias(_ptr(flat), flat.shape[0], cols, _ptr(bias), _ptr(out))
    if rc < 0:
        raise ValueError("mip_oracle_add_bias rejected its arguments")
    if rc > 0 and not allow_overflow:
        raise OracleOverflow("%d cells do not fit int32" % rc)
    return out.reshape(Cq.shape)
