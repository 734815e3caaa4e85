"""ctypes binding of the C-ABI library (``include/tcu_scan.h``): same names, argument
marshalling only.  Every step of the scan runs in the library's CUDA kernels; PyTorch is
used by callers for device memory and streams.  There is no fallback: if the compiled
library is missing, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libtcu_scan.so")

TCU_OK, TCU_ERR_INVALID_ARG, TCU_ERR_UNSUPPORTED, TCU_ERR_WORKSPACE, TCU_ERR_CUDA, TCU_ERR_TIMEOUT, TCU_ERR_TOO_LARGE = range(7)
TCU_SCAN_NOALLOC_MAX_ELEMENTS = 1 << 26
TCU_I8_I32, TCU_F16_F32, TCU_BF16_F32 = range(3)
DTYPES = {"i8": TCU_I8_I32, "f16": TCU_F16_F32, "bf16": TCU_BF16_F32}

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2411_17887_b200.build` "
        "(there is no CPU or PyTorch fallback)")

_lib = ctypes.CDLL(LIB_PATH)


class TcuScanStats(ctypes.Structure):
    _fields_ = [("rows", ctypes.c_uint64), ("cols", ctypes.c_uint64),
                ("s", ctypes.c_uint32), ("dtype", ctypes.c_uint32), ("exclusive", ctypes.c_uint32),
                ("variant", ctypes.c_uint32), ("upper_level_path", ctypes.c_uint32),
                ("tiles", ctypes.c_uint64), ("mma_instructions", ctypes.c_uint64), ("sxs_products", ctypes.c_uint64),
                ("levels_used", ctypes.c_uint32), ("depth_bound", ctypes.c_uint32),
                ("grid", ctypes.c_uint32), ("smem_bytes", ctypes.c_uint32), ("in_stages", ctypes.c_uint32),
                ("tail_elements", ctypes.c_uint32), ("down_sweep_path", ctypes.c_uint32)]


_vp, _sz, _int = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
_lib.tcu_scan_workspace_bytes.argtypes = [_sz, _sz, _int, _int]
_lib.tcu_scan_workspace_bytes.restype = _sz
_lib.tcu_scan_workspace_init.argtypes = [_vp, _sz, _vp]
_lib.tcu_scan_workspace_init.restype = _int
for _name in ("tcu_scan_inclusive", "tcu_scan_exclusive", "tcu_scan_level0_debug", "tcu_scan_inclusive_twosweep"):
    getattr(_lib, _name).argtypes = [_vp, _vp, _sz, _int, _int, _vp, _sz, _vp]
    getattr(_lib, _name).restype = _int
_lib.tcu_scan_inclusive_noalloc.argtypes = [_vp, _vp, _sz, _int, _int, _vp]
_lib.tcu_scan_inclusive_noalloc.restype = _int
_lib.tcu_scan_batched.argtypes = [_vp, _vp, _sz, _sz, _int, _int, _int, _vp, _sz, _vp]
_lib.tcu_scan_batched.restype = _int
_lib.tcu_scan_host.argtypes = [_vp, _vp, _sz, _int, _int, _int, _vp, _vp, _vp, _sz, _vp]
_lib.tcu_scan_host.restype = _int
_lib.tcu_scan_device_status.argtypes = [_vp, _vp]
_lib.tcu_scan_device_status.restype = _int
_lib.tcu_scan_selftest_timeout.argtypes = [_vp, _sz, ctypes.c_uint, _vp]
_lib.tcu_scan_selftest_timeout.restype = _int
_lib.tcu_sort_tmp_bytes.argtypes = [_sz]
_lib.tcu_sort_tmp_bytes.restype = _sz
_lib.tcu_sort_u32.argtypes = [_vp, _vp, _sz, _vp, _sz, _vp, _sz, _vp]
_lib.tcu_sort_u32.restype = _int
_lib.tcu_scan_set_down_sweep_path.argtypes = [_int]
_lib.tcu_scan_set_down_sweep_path.restype = _int
_lib.tcu_scan_set_upper_level_path.argtypes = [_int]
_lib.tcu_scan_set_upper_level_path.restype = _int
_lib.tcu_scan_set_max_ctas.argtypes = [_int]
_lib.tcu_scan_set_max_ctas.restype = _int
_lib.tcu_scan_last_stats.argtypes = [ctypes.POINTER(TcuScanStats)]
_lib.tcu_scan_last_stats.restype = _int
_lib.tcu_status_string.argtypes = [_int]
_lib.tcu_status_string.restype = ctypes.c_char_p


def _p(x):
    """Device/host pointer of a tensor-like (``data_ptr()``), an int, or None."""
    if x is None:
        return None
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    return int(x)


def tcu_status_string(st: int) -> str:
    return _lib.tcu_status_string(int(st)).decode()


def tcu_scan_workspace_bytes(rows: int, cols: int, dt: int, s: int) -> int:
    return int(_lib.tcu_scan_workspace_bytes(rows, cols, dt, s))


def tcu_scan_workspace_init(d_ws, ws_bytes: int, stream=0) -> int:
    return _lib.tcu_scan_workspace_init(_p(d_ws), ws_bytes, stream)


def tcu_scan_inclusive(d_in, d_out, n: int, dt: int, s: int, d_ws, ws_bytes: int, stream=0) -> int:
    return _lib.tcu_scan_inclusive(_p(d_in), _p(d_out), n, dt, s, _p(d_ws), ws_bytes, stream)


def tcu_scan_inclusive_noalloc(d_in, d_out, n: int, dt: int, s: int, stream=0) -> int:
    """Inclusive scan that takes no workspace: the carry records live in an array built into the
    library (at most TCU_SCAN_NOALLOC_MAX_ELEMENTS elements; calls must not overlap on the GPU)."""
    return _lib.tcu_scan_inclusive_noalloc(_p(d_in), _p(d_out), n, dt, s, stream)


def tcu_scan_inclusive_twosweep(d_in, d_out, n: int, dt: int, s: int, d_ws, ws_bytes: int, stream=0) -> int:
    return _lib.tcu_scan_inclusive_twosweep(_p(d_in), _p(d_out), n, dt, s, _p(d_ws), ws_bytes, stream)


def tcu_scan_exclusive(d_in, d_out, n: int, dt: int, s: int, d_ws, ws_bytes: int, stream=0) -> int:
    return _lib.tcu_scan_exclusive(_p(d_in), _p(d_out), n, dt, s, _p(d_ws), ws_bytes, stream)


def tcu_scan_level0_debug(d_in, d_out, n: int, dt: int, s: int, d_ws, ws_bytes: int, stream=0) -> int:
    return _lib.tcu_scan_level0_debug(_p(d_in), _p(d_out), n, dt, s, _p(d_ws), ws_bytes, stream)


def tcu_scan_batched(d_in, d_out, rows: int, cols: int, dt: int, s: int, exclusive: int, d_ws, ws_bytes: int,
                     stream=0) -> int:
    return _lib.tcu_scan_batched(_p(d_in), _p(d_out), rows, cols, dt, s, int(exclusive), _p(d_ws), ws_bytes, stream)


def tcu_scan_host(h_in, h_out, n: int, dt: int, s: int, exclusive: int, d_in, d_out, d_ws, ws_bytes: int,
                  stream=0) -> int:
    return _lib.tcu_scan_host(_p(h_in), _p(h_out), n, dt, s, int(exclusive), _p(d_in), _p(d_out), _p(d_ws),
                              ws_bytes, stream)


def tcu_scan_device_status(d_ws, stream=0) -> int:
    return _lib.tcu_scan_device_status(_p(d_ws), stream)


def tcu_scan_selftest_timeout(d_ws, ws_bytes: int, limit_ms: int, stream=0) -> int:
    return _lib.tcu_scan_selftest_timeout(_p(d_ws), ws_bytes, int(limit_ms), stream)


def tcu_sort_tmp_bytes(n: int) -> int:
    return int(_lib.tcu_sort_tmp_bytes(n))


def tcu_sort_u32(d_keys_in, d_keys_out, n: int, d_tmp, tmp_bytes: int, d_ws, ws_bytes: int, stream=0) -> int:
    return _lib.tcu_sort_u32(_p(d_keys_in), _p(d_keys_out), n, _p(d_tmp), tmp_bytes, _p(d_ws), ws_bytes, stream)


def tcu_scan_set_down_sweep_path(path: int) -> int:
    return _lib.tcu_scan_set_down_sweep_path(int(path))


def tcu_scan_set_upper_level_path(path: int) -> int:
    return _lib.tcu_scan_set_upper_level_path(int(path))


def tcu_scan_set_max_ctas(max_ctas: int) -> int:
    return _lib.tcu_scan_set_max_ctas(int(max_ctas))


def tcu_scan_last_stats() -> dict:
    st = TcuScanStats()
    rc = _lib.tcu_scan_last_stats(ctypes.byref(st))
    if rc != TCU_OK:
        raise RuntimeError(tcu_status_string(rc))
    return {name: int(getattr(st, name)) for name, _ in TcuScanStats._fields_}


def check(rc: int) -> None:
    if rc != TCU_OK:
        raise RuntimeError(f"tcu_scan: {tcu_status_string(rc)} (status {rc})")
