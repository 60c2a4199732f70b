"""CPU oracle: direct convolution (fp64) and the glue ops that chain layers.

TEST INFRASTRUCTURE ONLY -- never imported by the product path.

`direct_conv` is the definition of a convolution layer's result (cross-
correlation, zero padding, floor output size), evaluated in fp64 by the plain
C loops in direct_conv.c.  `direct_conv_py` is the same definition as pure
Python/numpy loops for tiny shapes.  The paper treats all kernels of one
operator as computing this same function (its Section 3.1.1, "general" kernel
of Table 2, and its zero-accuracy-loss principle in Section 3).
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "liboracle_conv.so")
_SRC = os.path.join(_HERE, "direct_conv.c")
_lib = None


def build(force=False):
    """Compile direct_conv.c into liboracle_conv.so with gcc (OpenMP)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", _SO, _SRC])
    return _SO


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_SO)
        ip = ctypes.c_int
        for name, xt in (("oracle_direct_conv", ctypes.c_float), ("oracle_direct_conv_f64", ctypes.c_double)):
            fn = getattr(_lib, name)
            fn.restype = None
            fn.argtypes = [ctypes.POINTER(xt), ctypes.POINTER(ctypes.c_float),
                           ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_double)] + [ip] * 9
    return _lib


def out_size(H, W, R, S, stride, pad):
    return (H + 2 * pad - R) // stride + 1, (W + 2 * pad - S) // stride + 1


def direct_conv(x, w, bias=None, stride=1, pad=0, groups=1):
    """fp64 direct convolution.  x: (C,H,W) fp32 or fp64; w: (K,C/groups,R,S) fp32.

    Returns Y (K,OH,OW) fp64.
    """
    lib = _load()
    w = np.ascontiguousarray(w, dtype=np.float32)
    K, Cg, R, S = w.shape
    C, H, W = x.shape
    assert C == Cg * groups and K % groups == 0
    OH, OW = out_size(H, W, R, S, stride, pad)
    y = np.empty((K, OH, OW), dtype=np.float64)
    bptr = None
    if bias is not None:
        bias = np.ascontiguousarray(bias, dtype=np.float32)
        bptr = bias.ctypes.data_as(ctypes.POINTER(ctypes.c_float))
    if x.dtype == np.float32:
        x = np.ascontiguousarray(x)
        fn, xp = lib.oracle_direct_conv, x.ctypes.data_as(ctypes.POINTER(ctypes.c_float))
    else:
        x = np.ascontiguousarray(x, dtype=np.float64)
        fn, xp = lib.oracle_direct_conv_f64, x.ctypes.data_as(ctypes.POINTER(ctypes.c_double))
    fn(xp, w.ctypes.data_as(ctypes.POINTER(ctypes.c_float)), bptr,
       y.ctypes.data_as(ctypes.POINTER(ctypes.c_double)),
       C, H, W, K, R, S, stride, pad, groups)
    return y


def direct_conv_py(x, w, bias=None, stride=1, pad=0, groups=1):
    """The same definition as explicit Python loops (tiny shapes only)."""
    x = np.asarray(x, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    K, Cg, R, S = w.shape
    C, H, W = x.shape
    Kg = K // groups
    OH, OW = out_size(H, W, R, S, stride, pad)
    y = np.zeros((K, OH, OW), dtype=np.float64)
    for k in range(K):
        g = k // Kg
        for oh in range(OH):
            for ow in range(OW):
                acc = float(bias[k]) if bias is not None else 0.0
                for cc in range(Cg):
                    for r in range(R):
                        for s in range(S):
                            ih, iw = oh * stride + r - pad, ow * stride + s - pad
                            if 0 <= ih < H and 0 <= iw < W:
                                acc += x[g * Cg + cc, ih, iw] * w[k, cc, r, s]
                y[k, oh, ow] = acc
    return y


def activation(y, act):
    """act: 0 none, 1 ReLU, 2 ReLU6."""
    if act == 1:
        return np.maximum(y, 0.0)
    if act == 2:
        return np.minimum(np.maximum(y, 0.0), 6.0)
    return y


def maxpool(x, R, stride, pad):
    """Max over R x R windows; padded positions never win (treated as -inf)."""
    C, H, W = x.shape
    OH, OW = out_size(H, W, R, R, stride, pad)
    y = np.full((C, OH, OW), -np.inf, dtype=x.dtype)
    for oh in range(OH):
        for ow in range(OW):
            for r in range(R):
                for s in range(R):
                    ih, iw = oh * stride + r - pad, ow * stride + s - pad
                    if 0 <= ih < H and 0 <= iw < W:
                        y[:, oh, ow] = np.maximum(y[:, oh, ow], x[:, ih, iw])
    return y


def gavgpool(x):
    """Mean over the spatial grid, output (C,1,1)."""
    C, H, W = x.shape
    return (x.reshape(C, H * W).sum(axis=1) / float(H * W)).reshape(C, 1, 1)
