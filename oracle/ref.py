"""ctypes front end of the CPU oracle (``sg_ref.c``).

TEST INFRASTRUCTURE ONLY: the product (the CUDA library and its Python binding)
never imports this module.  It marshals NumPy arrays into the plain-C loop
nests, which evaluate the op definitions of the paper (Section 3 index
notation for conv_1d_nwc_wcf; Section 4.6.1 for matmul; Section 4.6.2 for the
strided/dilated 1-D and 2-D convolutions) with f64 accumulation.

All functions take f32 NumPy arrays (any strides) and return
``(out_f64, sum_abs_f64)`` where ``sum_abs`` is sum |a*b| per output element.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sg_ref.c")
_LIB = os.path.join(_HERE, "libsgref.so")
_lock = threading.Lock()
_lib = None

_i64 = ctypes.c_int64
_p = ctypes.c_void_p


def build(force: bool = False) -> str:
    """Compile sg_ref.c into libsgref.so with gcc (no CUDA involved)."""
    newest = max(os.path.getmtime(_SRC), os.path.getmtime(os.path.join(_HERE, "sg_ref.h")))
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < newest:
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def lib():
    global _lib
    with _lock:
        if _lib is None:
            build()
            _lib = ctypes.CDLL(_LIB)
            _lib.sg_ref_max_threads.restype = ctypes.c_int
    return _lib


def max_threads() -> int:
    return int(lib().sg_ref_max_threads())


def _f32(a):
    a = np.asarray(a)
    if a.dtype != np.float32:
        raise TypeError("oracle inputs must be float32 arrays")
    return a


def _estrides(a):
    return [s // a.itemsize for s in a.strides]


def _i64arr(v):
    return (ctypes.c_int64 * len(v))(*[int(x) for x in v])


def _ptr(a):
    return ctypes.c_void_p(a.ctypes.data)


def matmul(A, B, C_in=None, threads=0):
    """C[m,n] = (C_in[m,n]) + sum_k A[m,k]*B[k,n]."""
    A, B = _f32(A), _f32(B)
    M, K = A.shape
    K2, N = B.shape
    assert K == K2
    mode = 0 if C_in is None else 1
    C = np.zeros((M, N), np.float64) if C_in is None else np.array(C_in, dtype=np.float64, order="C")
    S = np.zeros((M, N), np.float64)
    sa, sb = _estrides(A), _estrides(B)
    rc = lib().sg_ref_matmul(_i64(M), _i64(N), _i64(K), _ptr(A), _i64(sa[0]), _i64(sa[1]),
                             _ptr(B), _i64(sb[0]), _i64(sb[1]), _ptr(C), _i64(N), _i64(1),
                             _ptr(S), ctypes.c_int(mode), ctypes.c_int(threads))
    if rc:
        raise ValueError("sg_ref_matmul rejected its arguments")
    return C, S


def matmul_bias_act(A, B, bias=None, act="none", threads=0):
    """C[m,n] = act(sum_k A[m,k]*B[k,n] + bias[n]); act "none" or "relu".  Returns (C, S) with S = sum|a*b| + |bias|."""
    A, B = _f32(A), _f32(B)
    M, K = A.shape
    K2, N = B.shape
    assert K == K2
    code = {"none": 0, "relu": 1}[act]
    C = np.zeros((M, N), np.float64)
    S = np.zeros((M, N), np.float64)
    sa, sb = _estrides(A), _estrides(B)
    if bias is not None:
        bias = _f32(bias)
        assert bias.shape == (N,)
        bp, bs = _ptr(bias), _estrides(bias)[0]
    else:
        bp, bs = ctypes.c_void_p(0), 0
    rc = lib().sg_ref_matmul_bias_act(_i64(M), _i64(N), _i64(K), _ptr(A), _i64(sa[0]), _i64(sa[1]),
                                      _ptr(B), _i64(sb[0]), _i64(sb[1]), bp, _i64(bs), ctypes.c_int(code),
                                      _ptr(C), _i64(N), _i64(1), _ptr(S), ctypes.c_int(threads))
    if rc:
        raise ValueError("sg_ref_matmul_bias_act rejected its arguments")
    return C, S


def matmul_points(A, B, pm, pn, threads=0):
    A, B = _f32(A), _f32(B)
    K = A.shape[1]
    pm = np.ascontiguousarray(pm, np.int64)
    pn = np.ascontiguousarray(pn, np.int64)
    out = np.zeros(pm.shape[0], np.float64)
    sab = np.zeros(pm.shape[0], np.float64)
    sa, sb = _estrides(A), _estrides(B)
    lib().sg_ref_matmul_points(_i64(K), _ptr(A), _i64(sa[0]), _i64(sa[1]), _ptr(B), _i64(sb[0]),
                               _i64(sb[1]), _i64(pm.shape[0]), _ptr(pm), _ptr(pn), _ptr(out),
                               _ptr(sab), ctypes.c_int(threads))
    return out, sab


def conv1d_nwc_wcf(I, Kf, stride=1, dilation=1, O_in=None, W_out=None, threads=0):
    """O[n,w,f] = (O_in) + sum_{kw,c} I[n, w*stride + kw*dilation, c] * Kf[kw,c,f]."""
    I, Kf = _f32(I), _f32(Kf)
    N, W_in, C = I.shape
    KW, C2, F = Kf.shape
    assert C == C2
    if W_out is None:
        W_out = (W_in - (KW - 1) * dilation - 1) // stride + 1
    mode = 0 if O_in is None else 1
    O = np.zeros((N, W_out, F), np.float64) if O_in is None else np.array(O_in, dtype=np.float64, order="C")
    S = np.zeros((N, W_out, F), np.float64)
    rc = lib().sg_ref_conv1d_nwc_wcf(_i64(N), _i64(W_out), _i64(F), _i64(KW), _i64(C), _i64(W_in),
                                     _i64(stride), _i64(dilation), _ptr(I), _i64arr(_estrides(I)),
                                     _ptr(Kf), _i64arr(_estrides(Kf)), _ptr(O),
                                     _i64arr([W_out * F, F, 1]), _ptr(S), ctypes.c_int(mode),
                                     ctypes.c_int(threads))
    if rc:
        raise ValueError("sg_ref_conv1d_nwc_wcf rejected its arguments")
    return O, S


def conv2d_nhwc_hwcf(I, Kf, stride=(1, 1), dilation=(1, 1), O_in=None, out_hw=None, threads=0):
    """O[n,h,w,f] = (O_in) + sum_{kh,kw,c} I[n,h*sh+kh*dh,w*sw+kw*dw,c] * Kf[kh,kw,c,f]."""
    I, Kf = _f32(I), _f32(Kf)
    N, H_in, W_in, C = I.shape
    KH, KW, C2, F = Kf.shape
    assert C == C2
    sh, sw = stride
    dh, dw = dilation
    if out_hw is None:
        out_hw = ((H_in - (KH - 1) * dh - 1) // sh + 1, (W_in - (KW - 1) * dw - 1) // sw + 1)
    Ho, Wo = out_hw
    mode = 0 if O_in is None else 1
    O = np.zeros((N, Ho, Wo, F), np.float64) if O_in is None else np.array(O_in, dtype=np.float64, order="C")
    S = np.zeros((N, Ho, Wo, F), np.float64)
    rc = lib().sg_ref_conv2d_nhwc_hwcf(_i64(N), _i64(Ho), _i64(Wo), _i64(F), _i64(KH), _i64(KW),
                                       _i64(C), _i64(H_in), _i64(W_in), _i64(sh), _i64(sw),
                                       _i64(dh), _i64(dw), _ptr(I), _i64arr(_estrides(I)),
                                       _ptr(Kf), _i64arr(_estrides(Kf)), _ptr(O),
                                       _i64arr([Ho * Wo * F, Wo * F, F, 1]), _ptr(S),
                                       ctypes.c_int(mode), ctypes.c_int(threads))
    if rc:
        raise ValueError("sg_ref_conv2d_nhwc_hwcf rejected its arguments")
    return O, S


def conv2d_points(I, Kf, pn, ph, pw, pf, stride=(1, 1), dilation=(1, 1), threads=0):
    I, Kf = _f32(I), _f32(Kf)
    KH, KW, C, _ = Kf.shape
    pts = [np.ascontiguousarray(p, np.int64) for p in (pn, ph, pw, pf)]
    n = pts[0].shape[0]
    out = np.zeros(n, np.float64)
    sab = np.zeros(n, np.float64)
    lib().sg_ref_conv2d_points(_i64(KH), _i64(KW), _i64(C), _i64(stride[0]), _i64(stride[1]),
                               _i64(dilation[0]), _i64(dilation[1]), _ptr(I),
                               _i64arr(_estrides(I)), _ptr(Kf), _i64arr(_estrides(Kf)), _i64(n),
                               _ptr(pts[0]), _ptr(pts[1]), _ptr(pts[2]), _ptr(pts[3]), _ptr(out),
                               _ptr(sab), ctypes.c_int(threads))
    return out, sab


def depthwise_conv2d_nhwc_hwc(I, Kf, stride=(1, 1), dilation=(1, 1), O_in=None, out_hw=None, threads=0):
    """O[n,h,w,c] = (O_in) + sum_{kh,kw} I[n,h*sh+kh*dh,w*sw+kw*dw,c] * Kf[kh,kw,c]  (Section 4.6.3)."""
    I, Kf = _f32(I), _f32(Kf)
    N, H_in, W_in, C = I.shape
    KH, KW, C2 = Kf.shape
    assert C == C2
    sh, sw = stride
    dh, dw = dilation
    if out_hw is None:
        out_hw = ((H_in - (KH - 1) * dh - 1) // sh + 1, (W_in - (KW - 1) * dw - 1) // sw + 1)
    Ho, Wo = out_hw
    mode = 0 if O_in is None else 1
    O = np.zeros((N, Ho, Wo, C), np.float64) if O_in is None else np.array(O_in, dtype=np.float64, order="C")
    S = np.zeros((N, Ho, Wo, C), np.float64)
    rc = lib().sg_ref_depthwise_conv2d_nhwc_hwc(_i64(N), _i64(Ho), _i64(Wo), _i64(C), _i64(KH), _i64(KW),
                                                _i64(H_in), _i64(W_in), _i64(sh), _i64(sw), _i64(dh), _i64(dw),
                                                _ptr(I), _i64arr(_estrides(I)), _ptr(Kf), _i64arr(_estrides(Kf)),
                                                _ptr(O), _i64arr([Ho * Wo * C, Wo * C, C, 1]), _ptr(S),
                                                ctypes.c_int(mode), ctypes.c_int(threads))
    if rc:
        raise ValueError("sg_ref_depthwise_conv2d_nhwc_hwc rejected its arguments")
    return O, S


def depthwise_conv1d_nwc_wc(I, Kf, stride=1, dilation=1, O_in=None, W_out=None, threads=0):
    """O[n,w,c] = (O_in) + sum_kw I[n,w*sw+kw*dw,c] * Kf[kw,c]: the 2-D op with H = KH = 1."""
    I, Kf = _f32(I), _f32(Kf)
    N, W_in, C = I.shape
    O_in4 = None if O_in is None else np.asarray(O_in)[:, None]
    out_hw = None if W_out is None else (1, W_out)
    O, S = depthwise_conv2d_nhwc_hwc(I[:, None], Kf[None], (1, stride), (1, dilation), O_in4, out_hw, threads)
    return O[:, 0], S[:, 0]


def _elem_view(a):
    """Bit-pattern view of a 2-D array of 2- or 4-byte elements (copy/transpose move bits)."""
    a = np.asarray(a)
    if a.ndim != 2 or a.itemsize not in (2, 4):
        raise TypeError("expected a 2-D array of 2- or 4-byte elements")
    return a.view(np.uint16 if a.itemsize == 2 else np.uint32)


def copy2d(src):
    """dst[i,j] = src[i,j] (Section 4.4, Copy2D); returns a dense array of src's dtype."""
    v = _elem_view(src)
    R, C = v.shape
    dst = np.zeros((R, C), v.dtype)
    ss = _estrides(v)
    rc = lib().sg_ref_copy2d(_i64(R), _i64(C), _i64(v.itemsize), _ptr(v), _i64(ss[0]), _i64(ss[1]),
                             _ptr(dst), _i64(C), _i64(1))
    if rc:
        raise ValueError("sg_ref_copy2d rejected its arguments")
    return dst.view(np.asarray(src).dtype)


def transpose2d(src):
    """dst[j,i] = src[i,j] (Section 4.4, Transpose2D); returns a dense C x R array."""
    v = _elem_view(src)
    R, C = v.shape
    dst = np.zeros((C, R), v.dtype)
    ss = _estrides(v)
    rc = lib().sg_ref_transpose2d(_i64(R), _i64(C), _i64(v.itemsize), _ptr(v), _i64(ss[0]), _i64(ss[1]),
                                  _ptr(dst), _i64(R), _i64(1))
    if rc:
        raise ValueError("sg_ref_transpose2d rejected its arguments")
    return dst.view(np.asarray(src).dtype)


def _reduce2d(fn, A, n_out, out_in, threads):
    A = _f32(A)
    R, C = A.shape
    mode = 0 if out_in is None else 1
    out = np.zeros(n_out, np.float64) if out_in is None else np.array(out_in, dtype=np.float64, order="C")
    assert out.shape == (n_out,)
    S = np.zeros(n_out, np.float64)
    sa = _estrides(A)
    rc = fn(_i64(R), _i64(C), _ptr(A), _i64(sa[0]), _i64(sa[1]), _ptr(out), _ptr(S),
            ctypes.c_int(mode), ctypes.c_int(threads))
    if rc:
        raise ValueError("the 2-D reduction rejected its arguments")
    return out, S


def colred2d(A, out_in=None, threads=0):
    """out[j] = (out_in[j]) + sum_i A[i,j]: C outputs (Section 4.4, ColRed2D)."""
    return _reduce2d(lib().sg_ref_colred2d, A, np.asarray(A).shape[1], out_in, threads)


def rowred2d(A, out_in=None, threads=0):
    """out[i] = (out_in[i]) + sum_j A[i,j]: R outputs (Section 4.4, RowRed2D)."""
    return _reduce2d(lib().sg_ref_rowred2d, A, np.asarray(A).shape[0], out_in, threads)
