"""Thin ctypes binding of ``libmipgemm.so``: same names as ``include/mipgemm.h``.

Argument marshalling only -- every step of the method runs in the CUDA kernels
behind the C ABI.  Tensors are ``torch`` CUDA tensors (or raw device addresses as
``int``); PyTorch is used for device memory and streams, nothing else.  There is
no CPU fallback: if the shared library has not been built, importing this module
raises.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmipgemm.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        "libmipgemm.so is missing (%s). Build it with `python -m paper_2506_11728_b200.build` "
        "or `__graft_entry__.build()`; there is no fallback path." % LIB_PATH)

_lib = ctypes.CDLL(LIB_PATH)

_i64, _int, _vp, _sz = ctypes.c_int64, ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t

OK, ERR_INVALID_ARG, ERR_K_TOO_LARGE, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(7)
ERR_STATIC_SCRATCH_LIMIT = 7
STATIC_SCRATCH_BYTES = 8 << 20
PATH_NONE, PATH_DENSE, PATH_DENSE_PAIR, PATH_SKINNY, PATH_TRIVIAL = range(5)
PATH_MASK = 0xFF
PATH_REPACK, PATH_SPLITK, PATH_IM2COL_TMA, PATH_IM2COL_EXPLICIT = 0x100, 0x200, 0x400, 0x800
PATH_BATCHED = 0x1000
PATH_IM2COL_GATHER = 0x2000

#: every symbol include/mipgemm.h declares, with (restype, argtypes)
SIGNATURES = {
    "mipgemm_s8s8s32": (_int, [_i64, _i64, _i64, _vp, _i64, _vp, _i64, _vp, _i64, _int, _vp]),
    "mipgemm_u8s8s32": (_int, [_i64, _i64, _i64, _vp, _i64, _vp, _i64, _vp, _i64, _int, _vp]),
    "mipgemm_conv_u8s8s32": (_int, [_i64] * 5 + [_int] * 8 + [_vp, _vp, _vp, _int, _vp]),
    "mipgemm_gemm_ex": (_int, [_int] * 5 + [_i64, _i64, _i64, _vp, _i64, _vp, _i64, _vp, _i64, _int, _vp]),
    "mipgemm_batched_s8s8s32": (_int, [_i64] * 4 + [_vp, _i64, _i64, _vp, _i64, _i64, _vp, _i64, _i64, _int, _vp]),
    "mipgemm_batched_u8s8s32": (_int, [_i64] * 4 + [_vp, _i64, _i64, _vp, _i64, _i64, _vp, _i64, _i64, _int, _vp]),
    "mipgemm_s8s8f32_dequant": (_int, [_i64, _i64, _i64, _vp, _i64, _vp, _i64, _vp, _i64, ctypes.c_float, _vp]),
    "mipgemm_u8s8f32_dequant": (_int, [_i64, _i64, _i64, _vp, _i64, _vp, _i64, _vp, _i64, ctypes.c_float, _vp]),
    "mipgemm_conv_u8s8f32_dequant": (_int, [_i64] * 5 + [_int] * 8 + [_vp, _vp, _vp, ctypes.c_float, _vp]),
    "mipgemm_s8s8s8_requant": (_int, [_i64, _i64, _i64, _vp, _i64, _vp, _i64, _vp, _i64, ctypes.c_float, _int, _vp]),
    "mipgemm_u8s8u8_requant": (_int, [_i64, _i64, _i64, _vp, _i64, _vp, _i64, _vp, _i64, ctypes.c_float, _vp]),
    "mipgemm_conv_u8s8u8_requant": (_int, [_i64] * 5 + [_int] * 8 + [_vp, _vp, _vp, ctypes.c_float, _vp]),
    "mipgemm_s8s8f32_dequant_bias": (_int, [_i64, _i64, _i64, _vp, _i64, _vp, _i64, _vp, _i64, ctypes.c_float, _vp, _vp]),
    "mipgemm_u8s8f32_dequant_bias": (_int, [_i64, _i64, _i64, _vp, _i64, _vp, _i64, _vp, _i64, ctypes.c_float, _vp, _vp]),
    "mipgemm_conv_u8s8f32_dequant_bias": (_int, [_i64] * 5 + [_int] * 8 + [_vp, _vp, _vp, ctypes.c_float, _vp, _vp]),
    "mipgemm_s8s8s8_requant_bias": (_int, [_i64, _i64, _i64, _vp, _i64, _vp, _i64, _vp, _i64, ctypes.c_float, _int, _vp, _vp]),
    "mipgemm_u8s8u8_requant_bias": (_int, [_i64, _i64, _i64, _vp, _i64, _vp, _i64, _vp, _i64, ctypes.c_float, _vp, _vp]),
    "mipgemm_conv_u8s8u8_requant_bias": (_int, [_i64] * 5 + [_int] * 8 + [_vp, _vp, _vp, ctypes.c_float, _vp, _vp]),
    "mipgemm_host_s8s8s32": (_int, [_i64, _i64, _i64, _vp, _i64, _vp, _i64, _vp, _i64, _int, _vp]),
    "mipgemm_host_u8s8s32": (_int, [_i64, _i64, _i64, _vp, _i64, _vp, _i64, _vp, _i64, _int, _vp]),
    "mipgemm_s8s8s32_static_scratch": (_int, [_i64, _i64, _i64, _vp, _i64, _vp, _i64, _vp, _i64, _int, _vp]),
    "mipgemm_launch_count": (ctypes.c_uint64, []),
    "mipgemm_device_status": (_int, [_vp]),
    "mipgemm_set_workspace": (_int, [_vp, _sz]),
    "mipgemm_workspace_query_gemm": (_sz, [_i64, _i64, _i64, _vp, _i64, _vp, _i64, _vp, _i64, _int]),
    "mipgemm_workspace_query_conv": (_sz, [_i64] * 5 + [_int] * 8),
    "mipgemm_last_path": (_int, []),
    "mipgemm_last_cuda_error": (_int, []),
    "mipgemm_status_string": (ctypes.c_char_p, [_int]),
    "mipgemm_version": (_int, []),
    "mipgemm_probe_i8_peak": (_int, [_int, ctypes.POINTER(_int), ctypes.POINTER(ctypes.c_double), _vp, _vp]),
    "mipgemm_set_tuning": (_int, [_int, _int, _int, _int]),
    "mipgemm_set_weights_constant": (_int, [_int]),
    "mipgemm_register_constant_weights": (_int, [_vp, _sz]),
    "mipgemm_unregister_constant_weights": (_int, [_vp]),
    "mipgemm_static_scratch_status": (_int, [_vp]),
    "mipgemm_release_staging": (_int, []),
    "mipgemm_debug_set": (_int, [_int, ctypes.c_ulonglong]),
    "mipgemm_plan_cache_stats": (_int, [ctypes.POINTER(ctypes.c_uint64), ctypes.POINTER(ctypes.c_uint64)]),
}
for _name, (_res, _args) in SIGNATURES.items():
    _fn = getattr(_lib, _name)
    _fn.restype = _res
    _fn.argtypes = _args


class MipGemmError(RuntimeError):
    def __init__(self, status: int):
        self.status = status
        super().__init__("libmipgemm: %s (status %d, cuda error %d)" % (
            mipgemm_status_string(status), status, mipgemm_last_cuda_error()))


def _ptr(x) -> int:
    if x is None:
        return 0
    if isinstance(x, int):
        return x
    return x.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _check(status: int, check: bool) -> int:
    if check and status != OK:
        raise MipGemmError(status)
    return status


def mipgemm_s8s8s32(M, N, K, A, lda, B, ldb, C, ldc, accumulate=0, stream=None, check=True) -> int:
    """C[int32, MxN, pitch ldc] (+)= A[int8, MxK row-major, pitch lda] * B[int8, KxN column-major, pitch ldb]."""
    return _check(_lib.mipgemm_s8s8s32(M, N, K, _ptr(A), lda, _ptr(B), ldb, _ptr(C), ldc,
                                       int(bool(accumulate)), _stream(stream)), check)


def mipgemm_u8s8s32(M, N, K, A, lda, B, ldb, C, ldc, accumulate=0, stream=None, check=True) -> int:
    """Same with unsigned 8-bit A."""
    return _check(_lib.mipgemm_u8s8s32(M, N, K, _ptr(A), lda, _ptr(B), ldb, _ptr(C), ldc,
                                       int(bool(accumulate)), _stream(stream)), check)


def mipgemm_conv_u8s8s32(Nb, H, W, Cin, Cout, R, S, stride_h, stride_w, pad_h, pad_w, dil_h, dil_w,
                         X, Wt, Y, accumulate=0, stream=None, check=True) -> int:
    """Y[int32 NHWC] (+)= Conv(Wt[int8 KRSC], X[uint8 NHWC])."""
    return _check(_lib.mipgemm_conv_u8s8s32(Nb, H, W, Cin, Cout, R, S, stride_h, stride_w, pad_h, pad_w,
                                            dil_h, dil_w, _ptr(X), _ptr(Wt), _ptr(Y),
                                            int(bool(accumulate)), _stream(stream)), check)


K_CONTIGUOUS, MN_CONTIGUOUS = 0, 1


def mipgemm_gemm_ex(a_unsigned, b_unsigned, a_order, b_order, c_col_major, M, N, K, A, lda, B, ldb, C, ldc,
                    accumulate=0, stream=None, check=True) -> int:
    """General GEMM: any signedness pair, either storage order for A and B, row- or column-major C."""
    return _check(_lib.mipgemm_gemm_ex(int(a_unsigned), int(b_unsigned), int(a_order), int(b_order),
                                       int(c_col_major), M, N, K, _ptr(A), lda, _ptr(B), ldb, _ptr(C), ldc,
                                       int(bool(accumulate)), _stream(stream)), check)


def mipgemm_batched_s8s8s32(batch, M, N, K, A, lda, stride_a, B, ldb, stride_b, C, ldc, stride_c,
                            accumulate=0, stream=None, check=True) -> int:
    """C_b (+)= A_b * B_b for b < batch; member b of X starts stride_x elements after member b-1."""
    return _check(_lib.mipgemm_batched_s8s8s32(batch, M, N, K, _ptr(A), lda, stride_a, _ptr(B), ldb, stride_b,
                                               _ptr(C), ldc, stride_c, int(bool(accumulate)), _stream(stream)), check)


def mipgemm_batched_u8s8s32(batch, M, N, K, A, lda, stride_a, B, ldb, stride_b, C, ldc, stride_c,
                            accumulate=0, stream=None, check=True) -> int:
    return _check(_lib.mipgemm_batched_u8s8s32(batch, M, N, K, _ptr(A), lda, stride_a, _ptr(B), ldb, stride_b,
                                               _ptr(C), ldc, stride_c, int(bool(accumulate)), _stream(stream)), check)


def mipgemm_s8s8s8_requant(M, N, K, A, lda, B, ldb, C, ldc, scale, relu=0, stream=None, check=True) -> int:
    """C[int8] = sat(rne(scale * (A * B))) (clamped at 0 from below with relu)."""
    return _check(_lib.mipgemm_s8s8s8_requant(M, N, K, _ptr(A), lda, _ptr(B), ldb, _ptr(C), ldc,
                                              float(scale), int(bool(relu)), _stream(stream)), check)


def mipgemm_u8s8u8_requant(M, N, K, A, lda, B, ldb, C, ldc, scale, stream=None, check=True) -> int:
    """C[uint8] = sat(rne(scale * (A * B))), A unsigned."""
    return _check(_lib.mipgemm_u8s8u8_requant(M, N, K, _ptr(A), lda, _ptr(B), ldb, _ptr(C), ldc,
                                              float(scale), _stream(stream)), check)


def mipgemm_conv_u8s8u8_requant(Nb, H, W, Cin, Cout, R, S, stride_h, stride_w, pad_h, pad_w, dil_h, dil_w,
                                X, Wt, Y, scale, stream=None, check=True) -> int:
    """Y[uint8 NHWC] = sat(rne(scale * Conv(Wt, X)))."""
    return _check(_lib.mipgemm_conv_u8s8u8_requant(Nb, H, W, Cin, Cout, R, S, stride_h, stride_w, pad_h, pad_w,
                                                   dil_h, dil_w, _ptr(X), _ptr(Wt), _ptr(Y), float(scale),
                                                   _stream(stream)), check)


def mipgemm_s8s8f32_dequant_bias(M, N, K, A, lda, B, ldb, C, ldc, scale, bias, stream=None, check=True) -> int:
    """C[float32] = scale * (A * B + bias[column])."""
    return _check(_lib.mipgemm_s8s8f32_dequant_bias(M, N, K, _ptr(A), lda, _ptr(B), ldb, _ptr(C), ldc,
                                                    float(scale), _ptr(bias), _stream(stream)), check)


def mipgemm_u8s8f32_dequant_bias(M, N, K, A, lda, B, ldb, C, ldc, scale, bias, stream=None, check=True) -> int:
    """C[float32] = scale * (A * B + bias[column]), A unsigned."""
    return _check(_lib.mipgemm_u8s8f32_dequant_bias(M, N, K, _ptr(A), lda, _ptr(B), ldb, _ptr(C), ldc,
                                                    float(scale), _ptr(bias), _stream(stream)), check)


def mipgemm_conv_u8s8f32_dequant_bias(Nb, H, W, Cin, Cout, R, S, stride_h, stride_w, pad_h, pad_w, dil_h, dil_w,
                                      X, Wt, Y, scale, bias, stream=None, check=True) -> int:
    """Y[float32 NHWC] = scale * (Conv(Wt, X) + bias[channel])."""
    return _check(_lib.mipgemm_conv_u8s8f32_dequant_bias(Nb, H, W, Cin, Cout, R, S, stride_h, stride_w, pad_h, pad_w,
                                                         dil_h, dil_w, _ptr(X), _ptr(Wt), _ptr(Y), float(scale),
                                                         _ptr(bias), _stream(stream)), check)


def mipgemm_s8s8s8_requant_bias(M, N, K, A, lda, B, ldb, C, ldc, scale, bias, relu=0, stream=None, check=True) -> int:
    """C[int8] = sat(rne(scale * (A * B + bias[column]))) (clamped at 0 from below with relu)."""
    return _check(_lib.mipgemm_s8s8s8_requant_bias(M, N, K, _ptr(A), lda, _ptr(B), ldb, _ptr(C), ldc,
                                                   float(scale), int(bool(relu)), _ptr(bias), _stream(stream)), check)


def mipgemm_u8s8u8_requant_bias(M, N, K, A, lda, B, ldb, C, ldc, scale, bias, stream=None, check=True) -> int:
    """C[uint8] = sat(rne(scale * (A * B + bias[column]))), A unsigned."""
    return _check(_lib.mipgemm_u8s8u8_requant_bias(M, N, K, _ptr(A), lda, _ptr(B), ldb, _ptr(C), ldc,
                                                   float(scale), _ptr(bias), _stream(stream)), check)


def mipgemm_conv_u8s8u8_requant_bias(Nb, H, W, Cin, Cout, R, S, stride_h, stride_w, pad_h, pad_w, dil_h, dil_w,
                                     X, Wt, Y, scale, bias, stream=None, check=True) -> int:
    """Y[uint8 NHWC] = sat(rne(scale * (Conv(Wt, X) + bias[channel])))."""
    return _check(_lib.mipgemm_conv_u8s8u8_requant_bias(Nb, H, W, Cin, Cout, R, S, stride_h, stride_w, pad_h, pad_w,
                                                        dil_h, dil_w, _ptr(X), _ptr(Wt), _ptr(Y), float(scale),
                                                        _ptr(bias), _stream(stream)), check)


def mipgemm_s8s8f32_dequant(M, N, K, A, lda, B, ldb, C, ldc, scale, stream=None, check=True) -> int:
    """C[float32] = scale * (A * B): the exact int32 sum, converted and scaled in the epilogue."""
    return _check(_lib.mipgemm_s8s8f32_dequant(M, N, K, _ptr(A), lda, _ptr(B), ldb, _ptr(C), ldc,
                                               float(scale), _stream(stream)), check)


def mipgemm_u8s8f32_dequant(M, N, K, A, lda, B, ldb, C, ldc, scale, stream=None, check=True) -> int:
    return _check(_lib.mipgemm_u8s8f32_dequant(M, N, K, _ptr(A), lda, _ptr(B), ldb, _ptr(C), ldc,
                                               float(scale), _stream(stream)), check)


def mipgemm_conv_u8s8f32_dequant(Nb, H, W, Cin, Cout, R, S, stride_h, stride_w, pad_h, pad_w, dil_h, dil_w,
                                 X, Wt, Y, scale, stream=None, check=True) -> int:
    return _check(_lib.mipgemm_conv_u8s8f32_dequant(Nb, H, W, Cin, Cout, R, S, stride_h, stride_w, pad_h, pad_w,
                                                    dil_h, dil_w, _ptr(X), _ptr(Wt), _ptr(Y), float(scale),
                                                    _stream(stream)), check)


def mipgemm_host_s8s8s32(M, N, K, A, lda, B, ldb, C, ldc, accumulate=0, stream=None, check=True) -> int:
    """Host-buffer variant: A, B, C are host tensors/arrays (``data_ptr()``) or raw host addresses;
    copies in, computes on the device, copies C back and synchronises."""
    return _check(_lib.mipgemm_host_s8s8s32(M, N, K, _ptr(A), lda, _ptr(B), ldb, _ptr(C), ldc,
                                            int(bool(accumulate)), _stream(stream)), check)


def mipgemm_host_u8s8s32(M, N, K, A, lda, B, ldb, C, ldc, accumulate=0, stream=None, check=True) -> int:
    return _check(_lib.mipgemm_host_u8s8s32(M, N, K, _ptr(A), lda, _ptr(B), ldb, _ptr(C), ldc,
                                            int(bool(accumulate)), _stream(stream)), check)


def mipgemm_s8s8s32_static_scratch(M, N, K, A, lda, B, ldb, C, ldc, accumulate=0, stream=None, check=True) -> int:
    """mipgemm_s8s8s32 for callers that may not allocate device memory: re-pitching scratch comes from
    a fixed STATIC_SCRATCH_BYTES array inside the library (one per GPU, shared by all calls -- calls
    that can overlap on the GPU race on it).  Returns ERR_STATIC_SCRATCH_LIMIT, having launched
    nothing, when the operands need more than that.  Make the first call on a device outside any
    stream capture."""
    return _check(_lib.mipgemm_s8s8s32_static_scratch(M, N, K, _ptr(A), lda, _ptr(B), ldb, _ptr(C), ldc,
                                                      int(bool(accumulate)), _stream(stream)), check)


def mipgemm_launch_count() -> int:
    return int(_lib.mipgemm_launch_count())


def mipgemm_device_status(stream=None) -> int:
    return _lib.mipgemm_device_status(_stream(stream))


def mipgemm_set_workspace(buf, nbytes: int = 0) -> int:
    return _lib.mipgemm_set_workspace(_ptr(buf), nbytes)


def mipgemm_workspace_query_gemm(M, N, K, A, lda, B, ldb, C, ldc, accumulate=0) -> int:
    return _lib.mipgemm_workspace_query_gemm(M, N, K, _ptr(A), lda, _ptr(B), ldb, _ptr(C), ldc,
                                             int(bool(accumulate)))


def mipgemm_workspace_query_conv(Nb, H, W, Cin, Cout, R, S, stride_h, stride_w, pad_h, pad_w,
                                 dil_h, dil_w) -> int:
    return _lib.mipgemm_workspace_query_conv(Nb, H, W, Cin, Cout, R, S, stride_h, stride_w, pad_h, pad_w,
                                             dil_h, dil_w)


def mipgemm_last_path() -> int:
    return _lib.mipgemm_last_path()


def mipgemm_last_cuda_error() -> int:
    return _lib.mipgemm_last_cuda_error()


def mipgemm_status_string(status: int) -> str:
    return _lib.mipgemm_status_string(status).decode()


def mipgemm_version() -> int:
    return _lib.mipgemm_version()


def mipgemm_probe_i8_peak(iters: int, sink, stream=None):
    """Launches the tensor-pipe probe; returns (grid, ops_per_launch)."""
    grid = _int(0)
    ops = ctypes.c_double(0.0)
    st = _lib.mipgemm_probe_i8_peak(iters, ctypes.byref(grid), ctypes.byref(ops), _ptr(sink), _stream(stream))
    _check(st, True)
    return grid.value, ops.value


def mipgemm_set_weights_constant(on) -> int:
    """Promise that B of later M <= 16 calls is never written by work still pending on the stream."""
    return _check(_lib.mipgemm_set_weights_constant(int(bool(on))), True)


def mipgemm_register_constant_weights(buf, nbytes: int = 0, check=True) -> int:
    """Declares [buf, buf + nbytes) constant: M <= 16 calls whose B lies inside it may fetch it early.
    ``nbytes`` defaults to the tensor's size."""
    if not nbytes and hasattr(buf, "numel"):
        nbytes = buf.numel() * buf.element_size()
    return _check(_lib.mipgemm_register_constant_weights(_ptr(buf), nbytes), check)


def mipgemm_unregister_constant_weights(buf, check=True) -> int:
    return _check(_lib.mipgemm_unregister_constant_weights(_ptr(buf)), check)


def mipgemm_release_staging() -> int:
    """Frees the device staging buffer the host-buffer entry points keep between calls."""
    return _check(_lib.mipgemm_release_staging(), True)


def mipgemm_debug_set(flags=0, wait_budget_ns=0) -> int:
    """Test hook: withhold a device-side signal (bit 0) and set the limit of device-side waits (0 = 4 s)."""
    return _check(_lib.mipgemm_debug_set(int(flags), int(wait_budget_ns)), True)


def mipgemm_plan_cache_stats():
    """(enabled, hits, misses) of the plan / tensor-map cache."""
    hits, misses = ctypes.c_uint64(0), ctypes.c_uint64(0)
    on = _lib.mipgemm_plan_cache_stats(ctypes.byref(hits), ctypes.byref(misses))
    return bool(on), hits.value, misses.value


def mipgemm_static_scratch_status(stream=None) -> int:
    """Allocation-free status query of mipgemm_s8s8s32_static_scratch (synchronises the stream)."""
    return _lib.mipgemm_static_scratch_status(_stream(stream))


def mipgemm_set_tuning(block_n=0, stages=0, split_k=0, force_path=0) -> int:
    return _check(_lib.mipgemm_set_tuning(block_n, stages, split_k, force_path), True)
