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
                ("tail_elements", ctypes.c_uint32), ("down_sweep_path", ctypes.c_uint32),
                ("segments_path", ctypes.c_uint32)]


class TcuScanOptions(ctypes.Structure):
    _fields_ = [("struct_bytes", ctypes.c_uint32), ("exclusive", ctypes.c_uint32), ("variant", ctypes.c_uint32),
                ("upper_level_path", ctypes.c_uint32), ("down_sweep_path", ctypes.c_uint32),
                ("max_ctas", ctypes.c_uint32), ("d_carry_in", ctypes.c_void_p), ("d_carry_out", ctypes.c_void_p),
                ("d_stamps", ctypes.c_void_p)]


TCU_SCAN_STAMPS_PER_CTA = 16
STAMP_NAMES = ("entry", "setup_done", "previous_kernel_done", "first_tile_claimed", "first_tile_landed",
               "first_total_published", "first_carry_known", "first_tile_stored", "role_loops_done",
               "all_warps_done", "exit")


_vp, _sz, _int = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
_lib.tcu_scan_workspace_bytes.argtypes = [_sz, _sz, _int, _int]
_lib.tcu_scan_workspace_bytes.restype = _sz
_lib.tcu_scan_workspace_init.argtypes = [_vp, _sz, _vp]
_lib.tcu_scan_workspace_init.restype = _int
for _name in ("tcu_scan_inclusive", "tcu_scan_exclusive", "tcu_scan_level0_debug"):
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
_lib.tcu_scan_selftest_timeout.argtypes = [_vp, _vp, _sz, _int, _int, _sz, ctypes.c_uint, _int, _int, _vp, _sz, _vp]
_lib.tcu_scan_selftest_timeout.restype = _int
_lib.tcu_scan_noalloc_status.argtypes = [_vp]
_lib.tcu_scan_noalloc_status.restype = _int
_lib.tcu_scan_ex.argtypes = [_vp, _vp, _sz, _sz, _int, _int, ctypes.POINTER(TcuScanOptions), ctypes.POINTER(TcuScanStats),
                             _vp, _sz, _vp]
_lib.tcu_scan_ex.restype = _int
_lib.tcu_scan_segmented_workspace_bytes.argtypes = [_sz, _int, _int]
_lib.tcu_scan_segmented_workspace_bytes.restype = _sz
_lib.tcu_scan_segmented.argtypes = [_vp, _vp, _sz, _vp, _sz, _int, _int, _int, _vp, _sz, _vp]
_lib.tcu_scan_segmented.restype = _int
_lib.tcu_reduce_total.argtypes = [_vp, _sz, _int, _vp, _vp, _sz, _vp]
_lib.tcu_reduce_total.restype = _int
_lib.tcu_carry_exclusive_prefix.argtypes = [_vp, _sz, _sz, _int, _vp, _vp]
_lib.tcu_carry_exclusive_prefix.restype = _int
_lib.tcu_sort_tmp_bytes.argtypes = [_sz]
_lib.tcu_sort_tmp_bytes.restype = _sz
_lib.tcu_sort_u32.argtypes = [_vp, _vp, _sz, _vp, _sz, _vp, _sz, _vp]
_lib.tcu_sort_u32.restype = _int
_lib.tcu_widen_copy.argtypes = [_vp, _vp, _sz, _int, _vp]
_lib.tcu_widen_copy.restype = _int
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


def tcu_scan_noalloc_status(stream=0) -> int:
    """TCU_OK, or TCU_ERR_TIMEOUT if the most recent noalloc call on this device gave up a wait (syncs `stream`)."""
    return _lib.tcu_scan_noalloc_status(stream)


def _stats_dict(st: TcuScanStats) -> dict:
    return {name: int(getattr(st, name)) for name, _ in TcuScanStats._fields_}


def tcu_scan_ex(d_in, d_out, rows: int, cols: int, dt: int, s: int, d_ws, ws_bytes: int, stream=0, *,
                exclusive: int = 0, variant: int = 0, upper_level_path: int = 0, down_sweep_path: int = 0,
                max_ctas: int = 0, d_carry_in=None, d_carry_out=None, d_stamps=None, stats: dict = None) -> int:
    """The general call: every per-call choice of ``tcu_scan_options_t`` as a keyword.  If ``stats`` is a dict
    it is filled with the call's ``tcu_scan_stats_t``."""
    opt = TcuScanOptions(ctypes.sizeof(TcuScanOptions), int(exclusive), int(variant), int(upper_level_path),
                         int(down_sweep_path), int(max_ctas), _p(d_carry_in), _p(d_carry_out), _p(d_stamps))
    st = TcuScanStats()
    rc = _lib.tcu_scan_ex(_p(d_in), _p(d_out), rows, cols, dt, s, ctypes.byref(opt), ctypes.byref(st), _p(d_ws),
                          ws_bytes, stream)
    if stats is not None and rc == TCU_OK:
        stats.update(_stats_dict(st))
    return rc


def tcu_scan_segmented_workspace_bytes(n: int, dt: int, s: int) -> int:
    return int(_lib.tcu_scan_segmented_workspace_bytes(n, dt, s))


def tcu_scan_segmented(d_in, d_out, n: int, d_offsets, num_segments: int, dt: int, s: int, exclusive: int, d_ws,
                       ws_bytes: int, stream=0) -> int:
    return _lib.tcu_scan_segmented(_p(d_in), _p(d_out), n, _p(d_offsets), num_segments, dt, s, int(exclusive),
                                   _p(d_ws), ws_bytes, stream)


def tcu_reduce_total(d_in, n: int, dt: int, d_total, d_ws, ws_bytes: int, stream=0) -> int:
    return _lib.tcu_reduce_total(_p(d_in), n, dt, _p(d_total), _p(d_ws), ws_bytes, stream)


def tcu_carry_exclusive_prefix(d_totals, count: int, index: int, dt: int, d_carry, stream=0) -> int:
    return _lib.tcu_carry_exclusive_prefix(_p(d_totals), count, index, dt, _p(d_carry), stream)


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


def tcu_scan_selftest_timeout(d_in, d_out, n: int, dt: int, s: int, skip_tile: int, limit_ms: int, d_ws,
                              ws_bytes: int, stream=0, *, upper_level_path: int = 0, down_sweep_path: int = 0) -> int:
    return _lib.tcu_scan_selftest_timeout(_p(d_in), _p(d_out), n, dt, s, int(skip_tile), int(limit_ms),
                                          int(upper_level_path), int(down_sweep_path), _p(d_ws), ws_bytes, stream)


def tcu_sort_tmp_bytes(n: int) -> int:
    return int(_lib.tcu_sort_tmp_bytes(n))


def tcu_sort_u32(d_keys_in, d_keys_out, n: int, d_tmp, tmp_bytes: int, d_ws, ws_bytes: int, stream=0) -> int:
    return _lib.tcu_sort_u32(_p(d_keys_in), _p(d_keys_out), n, _p(d_tmp), tmp_bytes, _p(d_ws), ws_bytes, stream)


def tcu_widen_copy(d_in, d_out, n: int, dt: int, stream=0) -> int:
    return _lib.tcu_widen_copy(_p(d_in), _p(d_out), n, dt, stream)


def tcu_scan_last_stats() -> dict:
    st = TcuScanStats()
    rc = _lib.tcu_scan_last_stats(ctypes.byref(st))
    if rc != TCU_OK:
        raise RuntimeError(tcu_status_string(rc))
    return _stats_dict(st)


def check(rc: int) -> None:
    if rc != TCU_OK:
        raise RuntimeError(f"tcu_scan: {tcu_status_string(rc)} (status {rc})")
