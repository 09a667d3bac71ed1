"""ctypes front end of the CPU oracle (test infrastructure, not product code).

Only the test-suite, the smoke check and the benchmark's cpu-baseline leg may
import this package.  It compiles ``oracle.cpp`` with g++ on first use and
exposes its functions on numpy arrays.  Nothing here touches CUDA or the
product library.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib: Optional[ctypes.CDLL] = None


class Shape(ctypes.Structure):
    """Problem statement of the paper's Notation section plus a zero padding."""

    _fields_ = [(k, ctypes.c_int32) for k in ("N", "C", "H", "W", "Co", "Kh", "Kw", "stride", "pad")]


def build(force: bool = False) -> str:
    """Compile the oracle (g++ -O3 -fopenmp, no fast-math, no contraction, no -march: the
    library is built once and may run on another host); returns the path of the library."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".{os.getpid()}.tmp"
        cmd = ["g++", "-std=c++17", "-O3", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off",
               _SRC, "-o", tmp]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load() -> ctypes.CDLL:
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    P = ctypes.POINTER
    sp = P(Shape)
    lib.oracle_out_dims.argtypes = [sp, P(ctypes.c_int32), P(ctypes.c_int32)]
    lib.oracle_out_dims.restype = ctypes.c_int
    lib.oracle_window_elems.argtypes = [sp]
    lib.oracle_window_elems.restype = ctypes.c_int64
    lib.oracle_im2col_elems.argtypes = [sp]
    lib.oracle_im2col_elems.restype = ctypes.c_int64
    lib.oracle_num_threads.restype = ctypes.c_int
    lib.oracle_transform.argtypes = [ctypes.c_void_p, ctypes.c_void_p, sp, ctypes.c_int32]
    lib.oracle_transform.restype = ctypes.c_int
    for name in ("oracle_conv_direct", "oracle_conv_im2win"):
        fn = getattr(lib, name)
        fn.argtypes = [ctypes.c_void_p, ctypes.c_void_p, sp, ctypes.c_void_p, ctypes.c_void_p]
        fn.restype = ctypes.c_int
    lib.oracle_conv_im2win_range.argtypes = [ctypes.c_void_p, ctypes.c_void_p, sp, ctypes.c_int32,
                                             ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p]
    lib.oracle_conv_im2win_range.restype = ctypes.c_int
    lib.oracle_conv_direct_points.argtypes = [ctypes.c_void_p, ctypes.c_void_p, sp, ctypes.c_void_p,
                                              ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p]
    lib.oracle_conv_direct_points.restype = ctypes.c_int
    lib.oracle_round_to_f16.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p]
    lib.oracle_round_to_f16.restype = None
    lib.oracle_f16_bits_to_f64.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p]
    lib.oracle_f16_bits_to_f64.restype = None
    lib.oracle_round_f64_to_f16.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p]
    lib.oracle_round_f64_to_f16.restype = None
    lib.oracle_epilogue.argtypes = [ctypes.c_void_p, ctypes.c_void_p, sp, ctypes.c_void_p, ctypes.c_int32,
                                    ctypes.c_int32, ctypes.c_void_p]
    lib.oracle_epilogue.restype = ctypes.c_int
    lib.oracle_window_elems_nhwc.argtypes = [sp, ctypes.c_int32]
    lib.oracle_window_elems_nhwc.restype = ctypes.c_int64
    lib.oracle_transform_nhwc.argtypes = [ctypes.c_void_p, ctypes.c_void_p, sp, ctypes.c_int32, ctypes.c_int32,
                                          ctypes.c_int32]
    lib.oracle_transform_nhwc.restype = ctypes.c_int
    lib.oracle_conv_im2win_nhwc_range.argtypes = [ctypes.c_void_p, ctypes.c_void_p, sp, ctypes.c_int32, ctypes.c_int32,
                                                  ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p]
    lib.oracle_conv_im2win_nhwc_range.restype = ctypes.c_int
    _lib = lib
    return lib


def make_shape(N, C, H, W, Co, Kh, Kw, stride, pad) -> Shape:
    return Shape(int(N), int(C), int(H), int(W), int(Co), int(Kh), int(Kw), int(stride), int(pad))


def _as_shape(shape) -> Shape:
    if isinstance(shape, Shape):
        return shape
    if isinstance(shape, dict):
        return make_shape(**shape)
    return make_shape(*shape)


def out_dims(shape) -> Tuple[int, int]:
    s = _as_shape(shape)
    ho, wo = ctypes.c_int32(), ctypes.c_int32()
    if _load().oracle_out_dims(ctypes.byref(s), ctypes.byref(ho), ctypes.byref(wo)):
        raise ValueError("invalid convolution shape")
    return ho.value, wo.value


def window_elems(shape) -> int:
    n = _load().oracle_window_elems(ctypes.byref(_as_shape(shape)))
    if n < 0:
        raise ValueError("invalid convolution shape")
    return n


def im2col_elems(shape) -> int:
    n = _load().oracle_im2col_elems(ctypes.byref(_as_shape(shape)))
    if n < 0:
        raise ValueError("invalid convolution shape")
    return n


def num_threads() -> int:
    return _load().oracle_num_threads()


def _ptr(a: np.ndarray) -> ctypes.c_void_p:
    return ctypes.c_void_p(a.ctypes.data)


def transform(x: np.ndarray, shape) -> np.ndarray:
    """Eq. 2 on a [N,C,H,W] array of a 2- or 4-byte dtype; bit patterns are copied verbatim.

    Returns the im2win tensor as a [N, C, Ho, Kh*(W+2p)] array of the same dtype.
    """
    s = _as_shape(shape)
    x = np.ascontiguousarray(x)
    assert x.shape == (s.N, s.C, s.H, s.W), (x.shape, shape)
    assert x.dtype.itemsize in (2, 4)
    ho, _ = out_dims(s)
    out = np.empty((s.N, s.C, ho, s.Kh * (s.W + 2 * s.pad)), dtype=x.dtype)
    rc = _load().oracle_transform(_ptr(x), _ptr(out), ctypes.byref(s), x.dtype.itemsize)
    if rc:
        raise ValueError(f"oracle_transform failed ({rc})")
    return out


def _conv(fn_name: str, x, f, shape, want_a=True):
    s = _as_shape(shape)
    x = np.ascontiguousarray(x, dtype=np.float32)
    f = np.ascontiguousarray(f, dtype=np.float32)
    assert x.shape == (s.N, s.C, s.H, s.W) and f.shape == (s.Co, s.C, s.Kh, s.Kw)
    ho, wo = out_dims(s)
    y = np.empty((s.N, s.Co, ho, wo), dtype=np.float64)
    a = np.empty_like(y)
    rc = getattr(_load(), fn_name)(_ptr(x), _ptr(f), ctypes.byref(s), _ptr(y), _ptr(a))
    if rc:
        raise ValueError(f"{fn_name} failed ({rc})")
    return y, a


def conv_direct(x, f, shape):
    """Eq. 1 by seven nested loops; returns (y, a) with a = sum |x||f| per output."""
    return _conv("oracle_conv_direct", x, f, shape)


def conv_im2win(x, f, shape):
    """Eq. 2 then Eq. 3 (the im2win route); returns (y, a)."""
    return _conv("oracle_conv_im2win", x, f, shape)


def conv_im2win_range(x, f, shape, n_begin: int, n_end: int):
    """The im2win route on images [n_begin, n_end) only; returns (y, a) for those images."""
    s = _as_shape(shape)
    x = np.ascontiguousarray(x, dtype=np.float32)
    f = np.ascontiguousarray(f, dtype=np.float32)
    ho, wo = out_dims(s)
    y = np.zeros((s.N, s.Co, ho, wo), dtype=np.float64)
    a = np.zeros_like(y)
    rc = _load().oracle_conv_im2win_range(_ptr(x), _ptr(f), ctypes.byref(s), n_begin, n_end, _ptr(y), _ptr(a))
    if rc:
        raise ValueError(f"oracle_conv_im2win_range failed ({rc})")
    return y[n_begin:n_end], a[n_begin:n_end]


def conv_direct_points(x, f, shape, flat_indices: Sequence[int]):
    """Eq. 1 at the given flat indices of the [N,Co,Ho,Wo] output; returns (y, a)."""
    s = _as_shape(shape)
    x = np.ascontiguousarray(x, dtype=np.float32)
    f = np.ascontiguousarray(f, dtype=np.float32)
    idx = np.ascontiguousarray(flat_indices, dtype=np.int64)
    y = np.empty(idx.shape, dtype=np.float64)
    a = np.empty_like(y)
    rc = _load().oracle_conv_direct_points(_ptr(x), _ptr(f), ctypes.byref(s), _ptr(idx), idx.size, _ptr(y), _ptr(a))
    if rc:
        raise ValueError(f"oracle_conv_direct_points failed ({rc})")
    return y, a


def round_to_f16(v: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Round float32 values to binary16 (nearest, ties to even, subnormals kept).

    Returns (bits as uint16, rounded values as float32).
    """
    v = np.ascontiguousarray(v, dtype=np.float32)
    bits = np.empty(v.shape, dtype=np.uint16)
    back = np.empty(v.shape, dtype=np.float32)
    _load().oracle_round_to_f16(_ptr(v), v.size, _ptr(bits), _ptr(back))
    return bits, back


def f16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.empty(bits.shape, dtype=np.float64)
    _load().oracle_f16_bits_to_f64(_ptr(bits), bits.size, _ptr(out))
    return out


# ------------------------------------------------- epilogue options (Algorithm 1, last step) ----
def round_f64_to_f16(v: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Round float64 values to binary16 in ONE rounding (nearest, ties to even).

    Returns (bits as uint16, rounded values as float64).
    """
    v = np.ascontiguousarray(v, dtype=np.float64)
    bits = np.empty(v.shape, dtype=np.uint16)
    back = np.empty(v.shape, dtype=np.float64)
    _load().oracle_round_f64_to_f16(_ptr(v), v.size, _ptr(bits), _ptr(back))
    return bits, back


def epilogue(y: np.ndarray, a: np.ndarray, shape, bias=None, relu=False, out16=False, nhwc=False):
    """Bias, ReLU and the store rounding applied to a convolution result (y, a as returned by the
    conv_* functions, [N,Co,Ho,Wo] float64).  Returns (y', a') with a' = a + |bias|; y' is
    [N,Ho,Wo,Co] when nhwc is set.  The inputs are not modified."""
    s = _as_shape(shape)
    y2 = np.array(y, dtype=np.float64, order="C", copy=True)
    a2 = np.array(a, dtype=np.float64, order="C", copy=True)
    ho, wo = out_dims(s)
    assert y2.shape == (s.N, s.Co, ho, wo) and a2.shape == y2.shape
    b = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
    assert b is None or b.shape == (s.Co,)
    yn = np.empty((s.N, ho, wo, s.Co), dtype=np.float64) if nhwc else None
    rc = _load().oracle_epilogue(_ptr(y2), _ptr(a2), ctypes.byref(s), None if b is None else _ptr(b),
                                 int(bool(relu)), int(bool(out16)), None if yn is None else _ptr(yn))
    if rc:
        raise ValueError(f"oracle_epilogue failed ({rc})")
    if nhwc:
        return yn, np.ascontiguousarray(a2.transpose(0, 2, 3, 1))
    return y2, a2


# ------------------------------------------------- channel-innermost (NHWC) im2win tensor ----
def window_elems_nhwc(shape, cp: int) -> int:
    n = _load().oracle_window_elems_nhwc(ctypes.byref(_as_shape(shape)), int(cp))
    if n < 0:
        raise ValueError("invalid convolution shape or channel padding")
    return n


def transform_nhwc(x: np.ndarray, shape, x_layout: str = "nchw", cp: Optional[int] = None) -> np.ndarray:
    """Channel-innermost im2win tensor [N, Ho, W+2p, Kh, Cp] of a 2- or 4-byte array x given as
    [N,C,H,W] (x_layout "nchw") or [N,H,W,C] ("nhwc"); bit patterns copied verbatim, zeros for the
    padding and for channels C..Cp-1."""
    s = _as_shape(shape)
    cp = s.C if cp is None else int(cp)
    x = np.ascontiguousarray(x)
    want = (s.N, s.C, s.H, s.W) if x_layout == "nchw" else (s.N, s.H, s.W, s.C)
    assert x.shape == want and x.dtype.itemsize in (2, 4)
    ho, _ = out_dims(s)
    out = np.empty((s.N, ho, s.W + 2 * s.pad, s.Kh, cp), dtype=x.dtype)
    rc = _load().oracle_transform_nhwc(_ptr(x), _ptr(out), ctypes.byref(s), x.dtype.itemsize,
                                       0 if x_layout == "nchw" else 1, cp)
    if rc:
        raise ValueError(f"oracle_transform_nhwc failed ({rc})")
    return out


def conv_im2win_nhwc(x, f, shape, x_layout: str = "nchw", cp: Optional[int] = None, n_begin: int = 0,
                     n_end: Optional[int] = None):
    """The NHWC im2win route on images [n_begin, n_end); returns (y, a) as [n, Co, Ho, Wo] float64."""
    s = _as_shape(shape)
    cp = s.C if cp is None else int(cp)
    n_end = s.N if n_end is None else n_end
    x = np.ascontiguousarray(x, dtype=np.float32)
    f = np.ascontiguousarray(f, dtype=np.float32)
    want = (s.N, s.C, s.H, s.W) if x_layout == "nchw" else (s.N, s.H, s.W, s.C)
    assert x.shape == want and f.shape == (s.Co, s.C, s.Kh, s.Kw)
    ho, wo = out_dims(s)
    y = np.zeros((s.N, s.Co, ho, wo), dtype=np.float64)
    a = np.zeros_like(y)
    rc = _load().oracle_conv_im2win_nhwc_range(_ptr(x), _ptr(f), ctypes.byref(s), 0 if x_layout == "nchw" else 1,
                                               cp, n_begin, n_end, _ptr(y), _ptr(a))
    if rc:
        raise ValueError(f"oracle_conv_im2win_nhwc_range failed ({rc})")
    return y[n_begin:n_end], a[n_begin:n_end]
