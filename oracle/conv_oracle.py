"""ctypes front end of the C oracle (conv_ref.c) plus the data-movement definitions.

Test infrastructure only.  Nothing here is shared with, or imported by, the CUDA path.
Arrays cross as numpy float16 (or their uint16 bit patterns); all arithmetic happens in C.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "conv_ref.c")
_LIB = os.path.join(_HERE, "libconvref.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile conv_ref.c with gcc (OpenMP) into libconvref.so beside it."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off",
             "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _CParams(ctypes.Structure):
    _fields_ = [(f, ctypes.c_int32) for f in (
        "n", "c", "h", "w", "k", "r", "s", "pad_h", "pad_w", "stride_h", "stride_w",
        "dil_h", "dil_w", "group")]


@dataclass(frozen=True)
class ConvParams:
    """Layer description: input NCHW, weights K x C/group x R x S."""
    n: int
    c: int
    h: int
    w: int
    k: int
    r: int
    s: int
    pad_h: int = 0
    pad_w: int = 0
    stride_h: int = 1
    stride_w: int = 1
    dil_h: int = 1
    dil_w: int = 1
    group: int = 1

    def _c(self) -> _CParams:
        return _CParams(self.n, self.c, self.h, self.w, self.k, self.r, self.s, self.pad_h,
                        self.pad_w, self.stride_h, self.stride_w, self.dil_h, self.dil_w,
                        self.group)


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u16p = ctypes.POINTER(ctypes.c_uint16)
        pp = ctypes.POINTER(_CParams)
        lib.ref_half_to_double.restype = ctypes.c_double
        lib.ref_half_to_double.argtypes = [ctypes.c_uint16]
        lib.ref_double_to_half.restype = ctypes.c_uint16
        lib.ref_double_to_half.argtypes = [ctypes.c_double]
        lib.ref_out_dim.restype = ctypes.c_int64
        lib.ref_out_dim.argtypes = [ctypes.c_int64] * 5
        lib.ref_conv_check.restype = ctypes.c_int
        lib.ref_conv_check.argtypes = [pp]
        for name in ("ref_conv_naive", "ref_conv_fast"):
            fn = getattr(lib, name)
            fn.restype = ctypes.c_int
            fn.argtypes = [pp, u16p, u16p, u16p, u16p, ctypes.c_int]
        lib.ref_conv_points.restype = ctypes.c_int
        lib.ref_conv_points.argtypes = [pp, u16p, u16p, u16p, ctypes.c_int,
                                        ctypes.POINTER(ctypes.c_int64), ctypes.c_int64, u16p]
        lib.ref_num_threads.restype = ctypes.c_int
        lib.ref_cast_f32_to_f16.restype = ctypes.c_int64
        lib.ref_cast_f32_to_f16.argtypes = [ctypes.POINTER(ctypes.c_float), u16p, ctypes.c_int64]
        lib.ref_inner_product.restype = None
        lib.ref_inner_product.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, u16p, u16p, u16p, u16p,
                                          ctypes.c_int]
        f64p = ctypes.POINTER(ctypes.c_double)
        lib.ref_batchnorm.restype = None
        lib.ref_batchnorm.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, u16p, ctypes.c_double,
                                      ctypes.c_int, f64p, f64p, u16p]
        lib.ref_bn_fold.restype = None
        lib.ref_bn_fold.argtypes = [ctypes.c_int64, ctypes.c_int64, u16p, u16p, f64p, f64p, f64p, f64p,
                                    ctypes.c_double, u16p, u16p]
        _lib = lib
    return _lib


def _bits(a, shape=None) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype == np.float16:
        a = a.view(np.uint16)
    if a.dtype != np.uint16:
        raise TypeError("oracle inputs are float16 arrays (or their uint16 bits)")
    if shape is not None and tuple(a.shape) != tuple(shape):
        raise ValueError(f"expected shape {tuple(shape)}, got {tuple(a.shape)}")
    return a


def _u16(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_uint16))


def half_bits_to_double(bits: int) -> float:
    return float(_load().ref_half_to_double(int(bits)))


def double_to_half_bits(v: float) -> int:
    return int(_load().ref_double_to_half(float(v)))


def out_dim(size: int, kernel: int, pad: int, stride: int, dil: int) -> int:
    """Output extent along one axis (may be <= 0 for an invalid layer)."""
    return int(_load().ref_out_dim(size, kernel, pad, stride, dil))


def num_threads() -> int:
    return int(_load().ref_num_threads())


def _out_shape(p: ConvParams):
    return (p.n, p.k, out_dim(p.h, p.r, p.pad_h, p.stride_h, p.dil_h),
            out_dim(p.w, p.s, p.pad_w, p.stride_w, p.dil_w))


def _run(name, p: ConvParams, x, w, bias, relu):
    lib = _load()
    cp = p._c()
    if lib.ref_conv_check(ctypes.byref(cp)):
        raise ValueError(f"invalid convolution parameters: {p}")
    xb = _bits(x, (p.n, p.c, p.h, p.w))
    wb = _bits(w, (p.k, p.c // p.group, p.r, p.s))
    bb = _bits(bias, (p.k,)) if bias is not None else None
    y = np.empty(_out_shape(p), dtype=np.uint16)
    rc = getattr(lib, name)(ctypes.byref(cp), _u16(xb), _u16(wb),
                            _u16(bb) if bb is not None else None, _u16(y), int(bool(relu)))
    if rc:
        raise RuntimeError(f"{name} failed with code {rc}")
    return y.view(np.float16)


def conv_naive(p: ConvParams, x, w, bias=None, relu=False) -> np.ndarray:
    """The definition as a literal loop nest.  Returns float16 [N,K,P,Q]."""
    return _run("ref_conv_naive", p, x, w, bias, relu)


def conv_fast(p: ConvParams, x, w, bias=None, relu=False) -> np.ndarray:
    """Same additions in the same order, row-wise and multi-threaded."""
    return _run("ref_conv_fast", p, x, w, bias, relu)


def conv_points(p: ConvParams, x, w, bias, relu, coords) -> np.ndarray:
    """The definition at chosen outputs.  coords: int64 [npoints,4] rows (n,k,p,q)."""
    lib = _load()
    cp = p._c()
    if lib.ref_conv_check(ctypes.byref(cp)):
        raise ValueError(f"invalid convolution parameters: {p}")
    xb = _bits(x, (p.n, p.c, p.h, p.w))
    wb = _bits(w, (p.k, p.c // p.group, p.r, p.s))
    bb = _bits(bias, (p.k,)) if bias is not None else None
    coords = np.ascontiguousarray(coords, dtype=np.int64).reshape(-1, 4)
    out = np.empty(coords.shape[0], dtype=np.uint16)
    rc = lib.ref_conv_points(ctypes.byref(cp), _u16(xb), _u16(wb),
                             _u16(bb) if bb is not None else None, int(bool(relu)),
                             coords.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)),
                             coords.shape[0], _u16(out))
    if rc:
        raise RuntimeError(f"ref_conv_points failed with code {rc}")
    return out.view(np.float16)


# ---- data-movement steps: their definitions are permutations ----------------------------

def cast_f32_to_f16(src: np.ndarray):
    """(float16 array, number of finite inputs that became infinite): the converter's cast."""
    lib = _load()
    a = np.ascontiguousarray(src, dtype=np.float32)
    out = np.empty(a.shape, dtype=np.uint16)
    n_over = lib.ref_cast_f32_to_f16(a.ctypes.data_as(ctypes.POINTER(ctypes.c_float)),
                                     out.ctypes.data_as(ctypes.POINTER(ctypes.c_uint16)), a.size)
    return out.view(np.float16), int(n_over)


def inner_product(x, w, bias=None, relu=False) -> np.ndarray:
    """x [N,C], w [K,C], bias [K] or None (float16) -> y [N,K] float16."""
    lib = _load()
    xb, wb = _bits(x), _bits(w)
    n, c = xb.shape
    k = wb.shape[0]
    assert wb.shape == (k, c)
    bb = None if bias is None else _bits(bias, (k,))
    y = np.empty((n, k), dtype=np.uint16)
    lib.ref_inner_product(n, c, k, _u16(xb), _u16(wb), None if bb is None else _u16(bb), _u16(y), int(bool(relu)))
    return y.view(np.float16)


def _f64(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def batchnorm(x, eps, mean=None, var=None):
    """Batch norm of x [N,C,H,W] (float16), Section 3.1: per channel over N*H*W,
    y = (x - mean) / sqrt(var + eps) with the biased variance.  mean/var None: computed from x;
    else the stored statistics (float64 [C]).  Returns (y float16, mean float64, var float64)."""
    lib = _load()
    xb = _bits(x)
    n, c = xb.shape[0], xb.shape[1]
    hw = int(np.prod(xb.shape[2:], dtype=np.int64))
    stored = mean is not None
    if stored != (var is not None):
        raise ValueError("give both mean and var, or neither")
    m = np.ascontiguousarray(mean, dtype=np.float64).copy() if stored else np.zeros(c, dtype=np.float64)
    v = np.ascontiguousarray(var, dtype=np.float64).copy() if stored else np.zeros(c, dtype=np.float64)
    if m.shape != (c,) or v.shape != (c,):
        raise ValueError("mean and var have one entry per channel")
    y = np.empty(xb.shape, dtype=np.uint16)
    lib.ref_batchnorm(n, c, hw, _u16(xb), float(eps), int(stored), _f64(m), _f64(v), _u16(y))
    return y.view(np.float16), m, v


def bn_fold(w, bias, mean, var, eps, gamma=None, beta=None):
    """Stored statistics (and an optional per-channel scale gamma / shift beta) folded into the
    convolution before the batch norm: returns (w' float16 like w, b' float16 [K])."""
    lib = _load()
    wb = _bits(w)
    k = wb.shape[0]
    per_k = int(np.prod(wb.shape[1:], dtype=np.int64))
    bb = None if bias is None else _bits(bias, (k,))
    m = np.ascontiguousarray(mean, dtype=np.float64)
    v = np.ascontiguousarray(var, dtype=np.float64)
    ga = None if gamma is None else np.ascontiguousarray(gamma, dtype=np.float64)
    be = None if beta is None else np.ascontiguousarray(beta, dtype=np.float64)
    for a in (m, v, ga, be):
        if a is not None and a.shape != (k,):
            raise ValueError("per-channel vectors have K entries")
    wo = np.empty(wb.shape, dtype=np.uint16)
    bo = np.empty(k, dtype=np.uint16)
    lib.ref_bn_fold(k, per_k, _u16(wb), None if bb is None else _u16(bb), _f64(m), _f64(v),
                    None if ga is None else _f64(ga), None if be is None else _f64(be), float(eps), _u16(wo), _u16(bo))
    return wo.view(np.float16), bo.view(np.float16)


def nchw_to_nhwc(x: np.ndarray, c_pad: int) -> np.ndarray:
    """x[n][c][h][w] -> x'[n][h][w][c], channels zero-filled up to c_pad."""
    n, c, h, w = x.shape
    out = np.zeros((n, h, w, c_pad), dtype=x.dtype)
    out[..., :c] = np.transpose(x, (0, 2, 3, 1))
    return out


def nhwc_to_nchw(xp: np.ndarray, c: int) -> np.ndarray:
    """Inverse of nchw_to_nhwc: drop the channel padding, channels back to axis 1."""
    return np.ascontiguousarray(np.transpose(xp[..., :c], (0, 3, 1, 2)))


def repack_weights(w: np.ndarray, group: int, c_pad: int) -> np.ndarray:
    """w[K][C/g][R][S] -> w'[g][K/g][R][S][c_pad] with zero fill beyond C/g."""
    k, cg, r, s = w.shape
    out = np.zeros((group, k // group, r, s, c_pad), dtype=w.dtype)
    out[..., :cg] = np.transpose(w.reshape(group, k // group, cg, r, s), (0, 1, 3, 4, 2))
    return out
