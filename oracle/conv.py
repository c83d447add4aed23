"""ctypes front end of the C oracle convolution (test infrastructure only).

The arithmetic lives in conv_oracle.c (Eq. 4 / Eq. 6 of the paper, fp64, no output
rounding); this file only marshals numpy arrays.
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass

import numpy as np

from . import build as _build


@dataclass(frozen=True)
class ConvShape:
    N: int
    H: int
    W: int
    C_in: int
    C_out: int
    KH: int
    KW: int
    stride: tuple = (1, 1)
    pad: tuple = (0, 0)
    dil: tuple = (1, 1)
    relu: bool = False


class _CShape(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "N", "H", "W", "C_in", "C_out", "KH", "KW", "stride_h", "stride_w",
        "pad_h", "pad_w", "dil_h", "dil_w", "relu")]


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        lib.oracle_out_shape.restype = ctypes.c_int32
        lib.oracle_conv2d_f64.restype = ctypes.c_int32
        lib.oracle_conv2d_f64_sample.restype = ctypes.c_int32
        lib.oracle_threads.restype = ctypes.c_int32
        _lib = lib
    return _lib


def _cshape(s: ConvShape) -> _CShape:
    return _CShape(s.N, s.H, s.W, s.C_in, s.C_out, s.KH, s.KW, s.stride[0], s.stride[1],
                   s.pad[0], s.pad[1], s.dil[0], s.dil[1], 1 if s.relu else 0)


def threads() -> int:
    return int(_load().oracle_threads())


def out_shape(s: ConvShape):
    h = ctypes.c_int32()
    w = ctypes.c_int32()
    _load().oracle_out_shape(ctypes.byref(_cshape(s)), ctypes.byref(h), ctypes.byref(w))
    return int(h.value), int(w.value)


def _ptr(a, ctype):
    return a.ctypes.data_as(ctypes.POINTER(ctype)) if a is not None else None


def _prep(s, x_bits, w_bits, mask, bias):
    x = np.ascontiguousarray(x_bits, dtype=np.uint16)
    w = np.ascontiguousarray(w_bits, dtype=np.uint16)
    assert x.size == s.N * s.H * s.W * s.C_in, "x must be [N,H,W,C_in]"
    assert w.size == s.C_out * s.KH * s.KW * s.C_in, "w must be [C_out,KH,KW,C_in]"
    m = None if mask is None else np.ascontiguousarray(mask, dtype=np.uint8)
    if m is not None:
        assert m.size == w.size
    b = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
    if b is not None:
        assert b.size == s.C_out
    return x, w, m, b


def conv2d_f64(s: ConvShape, x_bits, w_bits, mask=None, bias=None) -> np.ndarray:
    """y [N,H_out,W_out,C_out] in fp64: act(bias + conv(x, mask .* w)), unrounded."""
    x, w, m, b = _prep(s, x_bits, w_bits, mask, bias)
    ho, wo = out_shape(s)
    y = np.empty((s.N, ho, wo, s.C_out), dtype=np.float64)
    rc = _load().oracle_conv2d_f64(ctypes.byref(_cshape(s)), _ptr(x, ctypes.c_uint16),
                                   _ptr(w, ctypes.c_uint16), _ptr(m, ctypes.c_uint8),
                                   _ptr(b, ctypes.c_float), _ptr(y, ctypes.c_double))
    if rc != 0:
        raise MemoryError("oracle_conv2d_f64 failed")
    return y


def conv2d_f64_sample(s: ConvShape, x_bits, w_bits, flat_idx, mask=None, bias=None) -> np.ndarray:
    """The same values at the given flat indices of y [N,H_out,W_out,C_out]."""
    x, w, m, b = _prep(s, x_bits, w_bits, mask, bias)
    idx = np.ascontiguousarray(flat_idx, dtype=np.int64)
    out = np.empty(idx.shape, dtype=np.float64)
    rc = _load().oracle_conv2d_f64_sample(ctypes.byref(_cshape(s)), _ptr(x, ctypes.c_uint16),
                                          _ptr(w, ctypes.c_uint16), _ptr(m, ctypes.c_uint8),
                                          _ptr(b, ctypes.c_float), _ptr(idx, ctypes.c_int64),
                                          ctypes.c_int64(idx.size), _ptr(out, ctypes.c_double))
    if rc != 0:
        raise MemoryError("oracle_conv2d_f64_sample failed")
    return out
