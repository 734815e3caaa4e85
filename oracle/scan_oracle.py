"""Result oracle: the prefix sum by its definition, in int64 / fp64.

TEST INFRASTRUCTURE ONLY.  The arithmetic is the sequential loop in
``scan_oracle.c``; this module only widens the inputs exactly and marshals
arrays.  It shares no code with the CUDA library.

Definition followed (paper, Section 1, notation paragraph): "prefix sum" is the
inclusive prefix sum under +; the exclusive form shifts the result right by one
and puts the identity 0 in front.  Input types and the widening rules are not
in the paper; they are this library's: int8 is summed exactly in int64 and then
reported modulo 2**32 as a two's-complement int32, fp16 / bf16 are widened
exactly to fp64 and summed in fp64.
"""
from __future__ import annotations

import ctypes

import numpy as np

from . import build as _build

_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        c_sz, c_int, c_i64, c_dbl, vp = (ctypes.c_size_t, ctypes.c_int, ctypes.c_int64,
                                         ctypes.c_double, ctypes.c_void_p)
        lib.oracle_scan_i8_i64.argtypes = [vp, c_sz, c_int, c_i64, vp]
        lib.oracle_scan_i8_i64.restype = None
        lib.oracle_scan_f64.argtypes = [vp, c_sz, c_int, c_dbl, vp, vp]
        lib.oracle_scan_f64.restype = None
        lib.oracle_scan_rows_i8_i64.argtypes = [vp, c_sz, c_sz, c_int, vp]
        lib.oracle_scan_rows_i8_i64.restype = None
        lib.oracle_scan_rows_f64.argtypes = [vp, c_sz, c_sz, c_int, vp, vp]
        lib.oracle_scan_rows_f64.restype = None
        lib.oracle_scan_segments_i8_i64.argtypes = [vp, vp, c_sz, c_int, vp]
        lib.oracle_scan_segments_i8_i64.restype = None
        lib.oracle_scan_segments_f64.argtypes = [vp, vp, c_sz, c_int, vp, vp]
        lib.oracle_scan_segments_f64.restype = None
        _lib = lib
    return _lib


def _ptr(a: np.ndarray):
    return ctypes.c_void_p(a.ctypes.data)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns (uint16) exactly to fp64.

    A bfloat16 is the upper half of an IEEE fp32, so placing the 16 bits in the
    high half of a 32-bit word gives the same value as an fp32.
    """
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def widen(x: np.ndarray, dtype: str) -> np.ndarray:
    """Exact widening of an input array to the oracle's accumulation type.

    dtype: "i8" (-> int8, accumulated in int64 by the C loop), "f16" (np.float16 -> fp64),
    "bf16" (uint16 bit patterns -> fp64).
    """
    if dtype == "i8":
        return np.ascontiguousarray(x, dtype=np.int8)
    if dtype == "f16":
        assert x.dtype == np.float16
        return np.ascontiguousarray(x.astype(np.float64))
    if dtype == "bf16":
        return np.ascontiguousarray(bf16_bits_to_f64(x))
    raise ValueError(dtype)


def scan_i8(x: np.ndarray, exclusive: bool = False, init: int = 0) -> np.ndarray:
    """Sequential int64 scan of an int8 array (1-D, or 2-D = independent rows)."""
    x = np.ascontiguousarray(x, dtype=np.int8)
    y = np.empty(x.shape, dtype=np.int64)
    lib = _load()
    if x.ndim == 1:
        lib.oracle_scan_i8_i64(_ptr(x), x.size, int(exclusive), int(init), _ptr(y))
    elif x.ndim == 2:
        assert init == 0
        lib.oracle_scan_rows_i8_i64(_ptr(x), x.shape[0], x.shape[1], int(exclusive), _ptr(y))
    else:
        raise ValueError("1-D or 2-D input expected")
    return y


def scan_f64(x64: np.ndarray, exclusive: bool = False, init: float = 0.0):
    """Sequential fp64 scan of an already widened array.

    Returns (y, a): the scan and the running sum of |x| over the same index
    range as each y[i] (the quantity the floating-point tolerance is scaled by).
    """
    x64 = np.ascontiguousarray(x64, dtype=np.float64)
    y = np.empty(x64.shape, dtype=np.float64)
    a = np.empty(x64.shape, dtype=np.float64)
    lib = _load()
    if x64.ndim == 1:
        lib.oracle_scan_f64(_ptr(x64), x64.size, int(exclusive), float(init), _ptr(y), _ptr(a))
    elif x64.ndim == 2:
        assert init == 0.0
        lib.oracle_scan_rows_f64(_ptr(x64), x64.shape[0], x64.shape[1], int(exclusive), _ptr(y), _ptr(a))
    else:
        raise ValueError("1-D or 2-D input expected")
    return y, a


def wrap_int32(y64: np.ndarray) -> np.ndarray:
    """Exact int64 sums reduced modulo 2**32 and read as two's-complement int32.

    This is what an int32 accumulator holds whatever the order of the additions,
    because addition modulo 2**32 is associative.
    """
    return (y64.astype(np.int64) & np.int64(0xFFFFFFFF)).astype(np.uint32).view(np.int32)


def scan(x: np.ndarray, dtype: str, exclusive: bool = False):
    """Scan an input in one of the library's input types.

    Returns a dict with "y" (int64 or fp64 result), and either "y32" (the
    wrapped int32 view, integer input) or "a" (abs-prefix for the tolerance,
    floating-point input).
    """
    if dtype == "i8":
        y = scan_i8(x, exclusive)
        return {"y": y, "y32": wrap_int32(y)}
    y, a = scan_f64(widen(x, dtype), exclusive)
    return {"y": y, "a": a}


def scan_segments(x: np.ndarray, dtype: str, offsets, exclusive: bool = False):
    """Segmented scan of a 1-D input: piece k is x[offsets[k]:offsets[k+1]], scanned from zero on its own.

    ``offsets`` has one more entry than there are pieces, starts at 0, ends at len(x) and never decreases.
    Returns the same dict as ``scan``; "a" restarts with every piece as well.
    """
    off = np.ascontiguousarray(offsets, dtype=np.uint64)
    assert x.ndim == 1 and off.ndim == 1 and off.size >= 1
    assert int(off[0]) == 0 and int(off[-1]) == x.size and bool((off[1:] >= off[:-1]).all())
    lib = _load()
    if dtype == "i8":
        xi = np.ascontiguousarray(x, dtype=np.int8)
        y = np.empty(xi.shape, dtype=np.int64)
        lib.oracle_scan_segments_i8_i64(_ptr(xi), _ptr(off), off.size - 1, int(exclusive), _ptr(y))
        return {"y": y, "y32": wrap_int32(y)}
    x64 = widen(x, dtype)
    y = np.empty(x64.shape, dtype=np.float64)
    a = np.empty(x64.shape, dtype=np.float64)
    lib.oracle_scan_segments_f64(_ptr(x64), _ptr(off), off.size - 1, int(exclusive), _ptr(y), _ptr(a))
    return {"y": y, "a": a}


def float_tolerance(a: np.ndarray) -> np.ndarray:
    """Per-element bound 1e-5 * sum|x| + 1e-6 used for fp32 outputs."""
    return 1e-5 * a + 1e-6
