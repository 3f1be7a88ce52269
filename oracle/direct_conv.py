"""ORACLE — test infrastructure only (tests, the smoke check and the benchmark's
CPU-baseline leg may import this; the product path never does).

Python face of ``direct_conv.c``: 2-D convolution by its plain definition in
fp64 (the "sliding window" scheme of Section 3.2 and the right-hand side that
Eq. 6 must equal).  ``build()`` compiles the C file with gcc; the functions
below marshal NumPy arrays and nothing else.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "direct_conv.c")
_LIB = os.path.join(_HERE, "liboracle_conv.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile direct_conv.c (plain C, -O2, OpenMP over (n, co))."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", _SRC, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i, p, ll = ctypes.c_int, ctypes.c_void_p, ctypes.c_longlong
        lib.oracle_conv_out_extent.argtypes = [i] * 5
        lib.oracle_conv_out_extent.restype = i
        lib.oracle_threads.restype = i
        lib.oracle_direct_conv_f64.argtypes = [p, p, p, p] + [i] * 11
        lib.oracle_direct_conv_f64.restype = i
        lib.oracle_direct_conv_f64_images.argtypes = [p, p, p, p, p, i] + [i] * 11
        lib.oracle_direct_conv_f64_images.restype = i
        lib.oracle_direct_conv_f64_at.argtypes = [p, p, p, p, ll, p] + [i] * 11
        lib.oracle_direct_conv_f64_at.restype = i
        lib.oracle_direct_conv_rect_f64.argtypes = [p, p, p, p] + [i] * 10
        lib.oracle_direct_conv_rect_f64.restype = i
        _lib = lib
    return _lib


def threads() -> int:
    """Host threads the C oracle uses (OpenMP's maximum)."""
    return int(_load().oracle_threads())


def out_extent(size: int, k: int, stride: int, pad: int, dil: int) -> int:
    if size <= 0 or k <= 0 or stride <= 0 or pad < 0 or dil <= 0:
        raise ValueError("size, k, stride, dil must be positive and pad non-negative")
    return int(_load().oracle_conv_out_extent(size, k, stride, pad, dil))


def _prep(x, w, bias, groups):
    x = np.ascontiguousarray(x, dtype=np.float32)
    w = np.ascontiguousarray(w, dtype=np.float32)
    if x.ndim != 4 or w.ndim != 4 or w.shape[2] != w.shape[3]:
        raise ValueError("x must be [N,Cin,H,W], w [Cout,Cin/groups,k,k]")
    N, Cin, H, W = x.shape
    Cout, cpg, k, _ = w.shape
    if Cin % groups or Cout % groups or cpg != Cin // groups:
        raise ValueError("channel counts do not match groups")
    if bias is not None:
        bias = np.ascontiguousarray(bias, dtype=np.float32)
        if bias.shape != (Cout,):
            raise ValueError("bias must be [Cout]")
    return x, w, bias, (N, Cin, Cout, H, W, k)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def direct_conv(x, w, bias=None, stride=1, pad=0, dil=1, groups=1, relu=False) -> np.ndarray:
    """Whole output, fp64 [N,Cout,OH,OW]."""
    x, w, bias, (N, Cin, Cout, H, W, k) = _prep(x, w, bias, groups)
    OH, OW = out_extent(H, k, stride, pad, dil), out_extent(W, k, stride, pad, dil)
    y = np.empty((N, Cout, OH, OW), dtype=np.float64)
    rc = _load().oracle_direct_conv_f64(_ptr(x), _ptr(w), _ptr(bias), _ptr(y), N, Cin, Cout, H, W, k,
                                        stride, pad, dil, groups, int(bool(relu)))
    if rc != 0:
        raise ValueError("oracle_direct_conv_f64 rejected its arguments")
    return y


def direct_conv_images(x, w, bias, images, stride=1, pad=0, dil=1, groups=1, relu=False) -> np.ndarray:
    """Only the listed images, fp64 [len(images),Cout,OH,OW]."""
    x, w, bias, (N, Cin, Cout, H, W, k) = _prep(x, w, bias, groups)
    images = np.ascontiguousarray(images, dtype=np.int32)
    OH, OW = out_extent(H, k, stride, pad, dil), out_extent(W, k, stride, pad, dil)
    y = np.empty((len(images), Cout, OH, OW), dtype=np.float64)
    rc = _load().oracle_direct_conv_f64_images(_ptr(x), _ptr(w), _ptr(bias), _ptr(y), _ptr(images), len(images),
                                               N, Cin, Cout, H, W, k, stride, pad, dil, groups, int(bool(relu)))
    if rc != 0:
        raise ValueError("oracle_direct_conv_f64_images rejected its arguments")
    return y


def direct_conv_at(x, w, bias, flat_indices, stride=1, pad=0, dil=1, groups=1, relu=False) -> np.ndarray:
    """Only the listed output elements (flat indices into [N,Cout,OH,OW]), fp64."""
    x, w, bias, (N, Cin, Cout, H, W, k) = _prep(x, w, bias, groups)
    flat = np.ascontiguousarray(flat_indices, dtype=np.int64)
    out = np.empty(flat.shape, dtype=np.float64)
    rc = _load().oracle_direct_conv_f64_at(_ptr(x), _ptr(w), _ptr(bias), _ptr(flat), flat.size, _ptr(out),
                                           N, Cin, Cout, H, W, k, stride, pad, dil, groups, int(bool(relu)))
    if rc != 0:
        raise ValueError("oracle_direct_conv_f64_at rejected its arguments")
    return out


def direct_conv_rect(x, w, bias=None, pad_h=0, pad_w=0, relu=False) -> np.ndarray:
    """Rectangular kernel w [Cout,Cin,kh,kw], stride 1, its own padding per axis; fp64 [N,Cout,OH,OW]."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    w = np.ascontiguousarray(w, dtype=np.float32)
    if x.ndim != 4 or w.ndim != 4 or w.shape[1] != x.shape[1]:
        raise ValueError("x must be [N,Cin,H,W], w [Cout,Cin,kh,kw]")
    N, Cin, H, W = x.shape
    Cout, _, kh, kw = w.shape
    if bias is not None:
        bias = np.ascontiguousarray(bias, dtype=np.float32)
        if bias.shape != (Cout,):
            raise ValueError("bias must be [Cout]")
    OH, OW = H + 2 * pad_h - kh + 1, W + 2 * pad_w - kw + 1
    if OH <= 0 or OW <= 0:
        raise ValueError("the kernel does not fit the padded input")
    y = np.empty((N, Cout, OH, OW), dtype=np.float64)
    rc = _load().oracle_direct_conv_rect_f64(_ptr(x), _ptr(w), _ptr(bias), _ptr(y), N, Cin, Cout, H, W, kh, kw,
                                             pad_h, pad_w, int(bool(relu)))
    if rc != 0:
        raise ValueError("oracle_direct_conv_rect_f64 rejected its arguments")
    return y
