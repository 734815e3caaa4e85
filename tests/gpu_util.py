"""Helpers for the GPU parity tests: move seeded inputs to the device, call the C-ABI
library through the ctypes binding, bring results back, compare with the CPU oracle."""
from __future__ import annotations

import numpy as np
import torch

from oracle import scan_oracle as so
from paper_2411_17887_b200 import binding as B

GUARD = 1024          # sentinel elements placed before and after the output
SENT_I = -0x5A5A5A5B
SENT_F = -1.2345e30


def to_device(x: np.ndarray, dtype: str) -> torch.Tensor:
    if dtype == "i8":
        return torch.from_numpy(np.ascontiguousarray(x, dtype=np.int8)).cuda()
    if dtype == "f16":
        return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float16)).cuda()
    if dtype == "bf16":
        return torch.from_numpy(np.ascontiguousarray(x, dtype=np.uint16).view(np.int16)).cuda().view(torch.bfloat16)
    raise ValueError(dtype)


class Runner:
    """Owns a workspace and calls the library; checks guard regions and device status."""

    def __init__(self, max_rows: int, max_cols: int, ws_bytes: int = None):
        self.ws_bytes = ws_bytes if ws_bytes is not None else B.tcu_scan_workspace_bytes(max_rows, max_cols, 0, 16)
        self.ws = torch.empty(self.ws_bytes + 256, dtype=torch.uint8, device="cuda")
        self.ws_ptr = self.ws.data_ptr() + (-self.ws.data_ptr()) % 256
        B.check(B.tcu_scan_workspace_init(self.ws_ptr, self.ws_bytes, 0))
        torch.cuda.synchronize()

    def run(self, x: np.ndarray, dtype: str, s: int, exclusive: bool = False, level0: bool = False,
            d_in: torch.Tensor = None, **options) -> np.ndarray:
        """`options` are the keywords of binding.tcu_scan_ex (variant, upper_level_path, max_ctas, ...); the
        call's statistics are left in self.stats."""
        rows, cols = (1, x.size) if x.ndim == 1 else x.shape
        d_in = to_device(x, dtype) if d_in is None else d_in
        n = rows * cols
        is_int = dtype == "i8"
        out = torch.full((n + 2 * GUARD,), SENT_I if is_int else SENT_F,
                         dtype=torch.int32 if is_int else torch.float32, device="cuda")
        d_out = out[GUARD:GUARD + n]
        assert d_out.data_ptr() % 16 == 0
        stream = torch.cuda.current_stream().cuda_stream
        dt = B.DTYPES[dtype]
        self.stats = {}
        if options:
            rc = B.tcu_scan_ex(d_in, d_out, rows, cols, dt, s, self.ws_ptr, self.ws_bytes, stream,
                               exclusive=int(exclusive), stats=self.stats, **options)
        elif level0:
            rc = B.tcu_scan_level0_debug(d_in, d_out, n, dt, s, self.ws_ptr, self.ws_bytes, stream)
        elif x.ndim == 1:
            fn = B.tcu_scan_exclusive if exclusive else B.tcu_scan_inclusive
            rc = fn(d_in, d_out, n, dt, s, self.ws_ptr, self.ws_bytes, stream)
        else:
            rc = B.tcu_scan_batched(d_in, d_out, rows, cols, dt, s, int(exclusive), self.ws_ptr, self.ws_bytes, stream)
        B.check(rc)
        if not options:
            self.stats = B.tcu_scan_last_stats()
        B.check(B.tcu_scan_device_status(self.ws_ptr, stream))
        host = out.cpu().numpy()
        sent = np.int32(SENT_I) if is_int else np.float32(SENT_F)
        assert (host[:GUARD] == sent).all() and (host[GUARD + n:] == sent).all(), "write outside the output"
        return host[GUARD:GUARD + n].reshape(x.shape)


def assert_int_equal(got: np.ndarray, x: np.ndarray, exclusive: bool):
    want = so.scan(x, "i8", exclusive)["y32"]
    if not np.array_equal(got, want):
        bad = np.flatnonzero(got.reshape(-1) != want.reshape(-1))
        raise AssertionError(f"{bad.size} mismatches, first at {bad[0]}: got {got.reshape(-1)[bad[0]]} want {want.reshape(-1)[bad[0]]}")


def assert_float_close(got: np.ndarray, x: np.ndarray, dtype: str, exclusive: bool):
    r = so.scan(x, dtype, exclusive)
    err = np.abs(got.astype(np.float64) - r["y"])
    tol = so.float_tolerance(r["a"])          # 1e-5 * sum|x| + 1e-6
    if not (err <= tol).all():
        bad = np.flatnonzero((err > tol).reshape(-1))
        i = bad[0]
        raise AssertionError(f"{bad.size} out of tolerance, first at {i}: got {got.reshape(-1)[i]} want {r['y'].reshape(-1)[i]} tol {tol.reshape(-1)[i]}")
    return float((err / tol).max())


def check(runner: Runner, x: np.ndarray, dtype: str, s: int, exclusive: bool = False, **options):
    got = runner.run(x, dtype, s, exclusive, **options)
    if dtype == "i8":
        assert_int_equal(got, x, exclusive)
    else:
        assert_float_close(got, x, dtype, exclusive)
    return got
