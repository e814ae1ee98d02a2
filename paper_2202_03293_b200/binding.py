"""Thin ctypes binding of libsg.so: argument marshalling only.

Every function here has the name and argument order of its C entry point
(see include/sg.h) and takes torch tensors that already live on the GPU;
pointers, element strides and the current CUDA stream are extracted and
passed through.  Nothing is computed on the Python side and there is no
fallback: if the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libsg.so")
_lib = None

SG_OK = 0
SG_F32, SG_BF16 = 0, 1
SG_OVERWRITE, SG_ACCUMULATE = 0, 1
SG_KERNEL_AUTO, SG_KERNEL_FFMA, SG_KERNEL_TENSOR, SG_KERNEL_CONV_STRIP, SG_KERNEL_TMA_MOVE = 0, 1, 2, 3, 4

EXPORTS = [
    "sg_matmul", "sg_conv1d_nwc_wcf", "sg_conv2d_nhwc_hwcf", "sg_depthwise_conv1d_nwc_wc",
    "sg_depthwise_conv2d_nhwc_hwc", "sg_copy2d", "sg_transpose2d", "sg_colred2d", "sg_rowred2d", "sg_check", "sg_status_string",
    "sg_version", "sg_last_kernel", "sg_launch_count", "sg_set_kernel_override", "sg_set_tile_override",
    "sg_last_tile_choice", "sg_last_stream_k", "sg_shutdown", "sg_last_kernel_name", "sg_selftest_wait_timeout",
    "sg_tensor_map_cache_stats", "sg_matmul_bias_act",
]


class SgError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: status {code} ({status_string(code)})")


def lib() -> ctypes.CDLL:
    """Loads libsg.so (built in-tree by paper_2202_03293_b200.build); raises if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: run `python -m paper_2202_03293_b200.build` first "
                               "(there is no non-CUDA fallback)")
        L = ctypes.CDLL(_LIB_PATH)
        i64, vp, ci = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int
        p64 = ctypes.POINTER(ctypes.c_int64)
        L.sg_matmul.argtypes = [i64, i64, i64, vp, i64, i64, vp, i64, i64, vp, i64, i64, ci, ci, vp]
        L.sg_matmul.restype = ci
        L.sg_matmul_bias_act.argtypes = [i64, i64, i64, vp, i64, i64, vp, i64, i64, vp, i64, ci, vp, i64, i64, ci, vp]
        L.sg_matmul_bias_act.restype = ci
        L.sg_conv1d_nwc_wcf.argtypes = [i64] * 8 + [vp, p64, vp, p64, vp, p64, ci, ci, vp]
        L.sg_conv1d_nwc_wcf.restype = ci
        L.sg_conv2d_nhwc_hwcf.argtypes = [i64] * 13 + [vp, p64, vp, p64, vp, p64, ci, ci, vp]
        L.sg_conv2d_nhwc_hwcf.restype = ci
        L.sg_depthwise_conv2d_nhwc_hwc.argtypes = [i64] * 12 + [vp, p64, vp, p64, vp, p64, ci, ci, vp]
        L.sg_depthwise_conv2d_nhwc_hwc.restype = ci
        L.sg_depthwise_conv1d_nwc_wc.argtypes = [i64] * 7 + [vp, p64, vp, p64, vp, p64, ci, ci, vp]
        L.sg_depthwise_conv1d_nwc_wc.restype = ci
        for fn in (L.sg_copy2d, L.sg_transpose2d):
            fn.argtypes = [i64, i64, vp, i64, i64, vp, i64, i64, ci, vp]
            fn.restype = ci
        for fn in (L.sg_colred2d, L.sg_rowred2d):
            fn.argtypes = [i64, i64, vp, i64, i64, vp, i64, ci, ci, vp]
            fn.restype = ci
        L.sg_check.argtypes = [vp]
        L.sg_check.restype = ci
        L.sg_status_string.argtypes = [ci]
        L.sg_status_string.restype = ctypes.c_char_p
        L.sg_version.restype = ci
        L.sg_last_kernel.restype = ci
        L.sg_launch_count.restype = i64
        L.sg_set_kernel_override.argtypes = [ci]
        L.sg_set_kernel_override.restype = ci
        L.sg_set_tile_override.argtypes = [ci, ci, ci]
        L.sg_set_tile_override.restype = ci
        L.sg_last_tile_choice.argtypes = [ctypes.POINTER(ctypes.c_int)]
        L.sg_last_tile_choice.restype = None
        L.sg_last_stream_k.argtypes = [ctypes.POINTER(ctypes.c_int)]
        L.sg_last_stream_k.restype = None
        L.sg_shutdown.restype = None
        L.sg_last_kernel_name.restype = ctypes.c_char_p
        L.sg_selftest_wait_timeout.argtypes = [i64, vp]
        L.sg_selftest_wait_timeout.restype = ci
        L.sg_tensor_map_cache_stats.argtypes = [p64]
        L.sg_tensor_map_cache_stats.restype = None
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().sg_status_string(int(code)).decode()


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return SG_F32
    if t.dtype == torch.bfloat16:
        return SG_BF16
    raise TypeError(f"unsupported input dtype {t.dtype}")


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return getattr(stream, "cuda_stream", stream)


def _arr(vals):
    return (ctypes.c_int64 * len(vals))(*[int(v) for v in vals])


def _ptr(t: torch.Tensor):
    if not t.is_cuda:
        raise ValueError("tensors must live on a CUDA device")
    return ctypes.c_void_p(t.data_ptr())


def sg_matmul_raw(M, N, K, A, a_sm, a_sk, B, b_sk, b_sn, C, c_sm, c_sn, dtype, mode, stream) -> int:
    """Direct call with integer pointers; returns the status code without raising."""
    return lib().sg_matmul(M, N, K, A, a_sm, a_sk, B, b_sk, b_sn, C, c_sm, c_sn, dtype, mode, stream)


def sg_matmul(A: torch.Tensor, B: torch.Tensor, C: torch.Tensor, mode: int = SG_OVERWRITE, stream=None) -> torch.Tensor:
    """C[m,n] (+)= sum_k A[m,k]*B[k,n]; A, B bf16 or f32 (same dtype), C f32, any strides."""
    M, K = A.shape
    K2, N = B.shape
    if K != K2 or tuple(C.shape) != (M, N) or C.dtype != torch.float32 or A.dtype != B.dtype:
        raise ValueError("shape or dtype mismatch")
    rc = lib().sg_matmul(M, N, K, _ptr(A), A.stride(0), A.stride(1), _ptr(B), B.stride(0), B.stride(1),
                         _ptr(C), C.stride(0), C.stride(1), _dtype_code(A), mode, _stream(stream))
    if rc != SG_OK:
        raise SgError(rc, "sg_matmul")
    return C


SG_ACT_NONE, SG_ACT_RELU = 0, 1


def sg_matmul_bias_act(A: torch.Tensor, B: torch.Tensor, bias, C: torch.Tensor, act: int = SG_ACT_NONE, stream=None) -> torch.Tensor:
    """C[m,n] = act(sum_k A[m,k]*B[k,n] + bias[n]); bias an f32 vector of N values or None; C is overwritten."""
    M, K = A.shape
    K2, N = B.shape
    if K != K2 or tuple(C.shape) != (M, N) or C.dtype != torch.float32 or A.dtype != B.dtype:
        raise ValueError("shape or dtype mismatch")
    if bias is not None and (tuple(bias.shape) != (N,) or bias.dtype != torch.float32):
        raise ValueError("bias must be an f32 vector of N values")
    rc = lib().sg_matmul_bias_act(M, N, K, _ptr(A), A.stride(0), A.stride(1), _ptr(B), B.stride(0), B.stride(1),
                                  _ptr(bias) if bias is not None else None, bias.stride(0) if bias is not None else 0, int(act),
                                  _ptr(C), C.stride(0), C.stride(1), _dtype_code(A), _stream(stream))
    if rc != SG_OK:
        raise SgError(rc, "sg_matmul_bias_act")
    return C


def sg_conv1d_nwc_wcf(I: torch.Tensor, Kf: torch.Tensor, O: torch.Tensor, stride_w: int = 1, dilation_w: int = 1,
                      mode: int = SG_OVERWRITE, stream=None) -> torch.Tensor:
    """O[n,w,f] (+)= sum_{kw,c} I[n, w*stride_w + kw*dilation_w, c] * Kf[kw,c,f]."""
    N, W_in, C = I.shape
    KW, C2, F = Kf.shape
    N2, W_out, F2 = O.shape
    if C != C2 or N != N2 or F != F2 or O.dtype != torch.float32 or I.dtype != Kf.dtype:
        raise ValueError("shape or dtype mismatch")
    rc = lib().sg_conv1d_nwc_wcf(N, W_out, F, KW, C, W_in, stride_w, dilation_w, _ptr(I), _arr(I.stride()),
                                 _ptr(Kf), _arr(Kf.stride()), _ptr(O), _arr(O.stride()), _dtype_code(I), mode,
                                 _stream(stream))
    if rc != SG_OK:
        raise SgError(rc, "sg_conv1d_nwc_wcf")
    return O


def sg_conv2d_nhwc_hwcf(I: torch.Tensor, Kf: torch.Tensor, O: torch.Tensor, stride=(1, 1), dilation=(1, 1),
                        mode: int = SG_OVERWRITE, stream=None) -> torch.Tensor:
    """O[n,h,w,f] (+)= sum_{kh,kw,c} I[n, h*sh+kh*dh, w*sw+kw*dw, c] * Kf[kh,kw,c,f]."""
    N, H_in, W_in, C = I.shape
    KH, KW, C2, F = Kf.shape
    N2, H_out, W_out, F2 = O.shape
    if C != C2 or N != N2 or F != F2 or O.dtype != torch.float32 or I.dtype != Kf.dtype:
        raise ValueError("shape or dtype mismatch")
    rc = lib().sg_conv2d_nhwc_hwcf(N, H_out, W_out, F, KH, KW, C, H_in, W_in, stride[0], stride[1], dilation[0],
                                   dilation[1], _ptr(I), _arr(I.stride()), _ptr(Kf), _arr(Kf.stride()), _ptr(O),
                                   _arr(O.stride()), _dtype_code(I), mode, _stream(stream))
    if rc != SG_OK:
        raise SgError(rc, "sg_conv2d_nhwc_hwcf")
    return O


def sg_depthwise_conv2d_nhwc_hwc(I: torch.Tensor, Kf: torch.Tensor, O: torch.Tensor, stride=(1, 1), dilation=(1, 1),
                                 mode: int = SG_OVERWRITE, stream=None) -> torch.Tensor:
    """O[n,h,w,c] (+)= sum_{kh,kw} I[n, h*sh+kh*dh, w*sw+kw*dw, c] * Kf[kh,kw,c]."""
    N, H_in, W_in, C = I.shape
    KH, KW, C2 = Kf.shape
    N2, H_out, W_out, C3 = O.shape
    if C != C2 or C != C3 or N != N2 or O.dtype != torch.float32 or I.dtype != Kf.dtype:
        raise ValueError("shape or dtype mismatch")
    rc = lib().sg_depthwise_conv2d_nhwc_hwc(N, H_out, W_out, C, KH, KW, H_in, W_in, stride[0], stride[1], dilation[0],
                                            dilation[1], _ptr(I), _arr(I.stride()), _ptr(Kf), _arr(Kf.stride()), _ptr(O),
                                            _arr(O.stride()), _dtype_code(I), mode, _stream(stream))
    if rc != SG_OK:
        raise SgError(rc, "sg_depthwise_conv2d_nhwc_hwc")
    return O


def sg_depthwise_conv1d_nwc_wc(I: torch.Tensor, Kf: torch.Tensor, O: torch.Tensor, stride: int = 1, dilation: int = 1,
                               mode: int = SG_OVERWRITE, stream=None) -> torch.Tensor:
    """O[n,w,c] (+)= sum_kw I[n, w*sw+kw*dw, c] * Kf[kw,c]."""
    N, W_in, C = I.shape
    KW, C2 = Kf.shape
    N2, W_out, C3 = O.shape
    if C != C2 or C != C3 or N != N2 or O.dtype != torch.float32 or I.dtype != Kf.dtype:
        raise ValueError("shape or dtype mismatch")
    rc = lib().sg_depthwise_conv1d_nwc_wc(N, W_out, C, KW, W_in, stride, dilation, _ptr(I), _arr(I.stride()), _ptr(Kf),
                                          _arr(Kf.stride()), _ptr(O), _arr(O.stride()), _dtype_code(I), mode, _stream(stream))
    if rc != SG_OK:
        raise SgError(rc, "sg_depthwise_conv1d_nwc_wc")
    return O


def _move2d(fn, name, src: torch.Tensor, dst: torch.Tensor, want_shape, stream):
    if src.dim() != 2 or tuple(dst.shape) != tuple(want_shape) or src.dtype != dst.dtype:
        raise ValueError(f"{name}: shape or dtype mismatch")
    R, C = src.shape
    rc = fn(R, C, _ptr(src), src.stride(0), src.stride(1), _ptr(dst), dst.stride(0), dst.stride(1), _dtype_code(src),
            _stream(stream))
    if rc != SG_OK:
        raise SgError(rc, name)
    return dst


def sg_copy2d(src: torch.Tensor, dst: torch.Tensor, stream=None) -> torch.Tensor:
    """dst[i,j] = src[i,j]."""
    return _move2d(lib().sg_copy2d, "sg_copy2d", src, dst, src.shape, stream)


def sg_transpose2d(src: torch.Tensor, dst: torch.Tensor, stream=None) -> torch.Tensor:
    """dst[j,i] = src[i,j]; dst is C x R."""
    return _move2d(lib().sg_transpose2d, "sg_transpose2d", src, dst, (src.shape[1], src.shape[0]), stream)


def _reduce2d(fn, name, A: torch.Tensor, out: torch.Tensor, n_out, mode, stream):
    if A.dim() != 2 or out.dim() != 1 or out.shape[0] != n_out or out.dtype != torch.float32:
        raise ValueError(f"{name}: shape or dtype mismatch")
    R, C = A.shape
    rc = fn(R, C, _ptr(A), A.stride(0), A.stride(1), _ptr(out), out.stride(0), _dtype_code(A), int(mode), _stream(stream))
    if rc != SG_OK:
        raise SgError(rc, name)
    return out


def sg_colred2d(A: torch.Tensor, out: torch.Tensor, mode: int = SG_OVERWRITE, stream=None) -> torch.Tensor:
    """out[j] (+)= sum_i A[i,j]."""
    return _reduce2d(lib().sg_colred2d, "sg_colred2d", A, out, A.shape[1], mode, stream)


def sg_rowred2d(A: torch.Tensor, out: torch.Tensor, mode: int = SG_OVERWRITE, stream=None) -> torch.Tensor:
    """out[i] (+)= sum_j A[i,j]."""
    return _reduce2d(lib().sg_rowred2d, "sg_rowred2d", A, out, A.shape[0], mode, stream)


def sg_check(stream=None) -> None:
    rc = lib().sg_check(_stream(stream))
    if rc != SG_OK:
        raise SgError(rc, "sg_check")


def sg_version() -> int:
    return int(lib().sg_version())


def sg_last_kernel() -> int:
    return int(lib().sg_last_kernel())


def sg_launch_count() -> int:
    return int(lib().sg_launch_count())


def sg_set_kernel_override(kernel_family: int) -> None:
    rc = lib().sg_set_kernel_override(int(kernel_family))
    if rc != SG_OK:
        raise SgError(rc, "sg_set_kernel_override")


def sg_set_tile_override(tile_n: int = 0, ctas_per_tile: int = 0, k_splits: int = 0) -> None:
    rc = lib().sg_set_tile_override(int(tile_n), int(ctas_per_tile), int(k_splits))
    if rc != SG_OK:
        raise SgError(rc, "sg_set_tile_override")


def sg_last_tile_choice():
    out = (ctypes.c_int * 3)()
    lib().sg_last_tile_choice(out)
    return out[0], out[1], out[2]


def sg_last_stream_k():
    out = (ctypes.c_int * 2)()
    lib().sg_last_stream_k(out)
    return out[0], out[1]


def sg_shutdown() -> None:
    lib().sg_shutdown()


def sg_last_kernel_name() -> str:
    return lib().sg_last_kernel_name().decode()


def sg_selftest_wait_timeout(budget_cycles: int = 2_000_000, stream=None) -> None:
    rc = lib().sg_selftest_wait_timeout(int(budget_cycles), _stream(stream))
    if rc != SG_OK:
        raise SgError(rc, "sg_selftest_wait_timeout")


def sg_tensor_map_cache_stats():
    """(hits, misses) of the tensor-map cache since the library was loaded."""
    out = (ctypes.c_int64 * 2)()
    lib().sg_tensor_map_cache_stats(out)
    return int(out[0]), int(out[1])
