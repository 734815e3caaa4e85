"""Convenience layer for PyTorch callers: allocates the output and the workspace with
torch (plumbing) and calls the C-ABI entry points.  No arithmetic happens here."""
from __future__ import annotations

import torch

from . import binding as B

_TORCH_IN = {"i8": torch.int8, "f16": torch.float16, "bf16": torch.bfloat16}


class Workspace:
    """Device workspace for the cross-tile carry scan, cleared once at creation."""

    def __init__(self, rows: int, cols: int, dtype: str = "i8", s: int = 16, device="cuda"):
        self.bytes = B.tcu_scan_workspace_bytes(rows, cols, B.DTYPES[dtype], s)
        self.buf = torch.empty(self.bytes + 256, dtype=torch.uint8, device=device)
        off = (-self.buf.data_ptr()) % 256
        self.ptr = self.buf.data_ptr() + off
        B.check(B.tcu_scan_workspace_init(self.ptr, self.bytes, torch.cuda.current_stream().cuda_stream))

    def status(self) -> int:
        return B.tcu_scan_device_status(self.ptr, torch.cuda.current_stream().cuda_stream)


def dtype_name(t: torch.Tensor) -> str:
    for k, v in _TORCH_IN.items():
        if t.dtype == v:
            return k
    raise TypeError(f"unsupported input dtype {t.dtype}")


def scan(x: torch.Tensor, s: int = 16, exclusive: bool = False, out: torch.Tensor = None,
         ws: Workspace = None) -> torch.Tensor:
    """Scan a contiguous 1-D CUDA tensor (or the rows of a 2-D one); returns int32 / fp32."""
    assert x.is_cuda and x.is_contiguous()
    dn = dtype_name(x)
    rows, cols = (1, x.numel()) if x.dim() == 1 else (x.shape[0], x.shape[1])
    if out is None:
        out = torch.empty(x.shape, dtype=torch.int32 if dn == "i8" else torch.float32, device=x.device)
    if ws is None:
        ws = Workspace(rows, cols, dn, s, x.device)
    stream = torch.cuda.current_stream().cuda_stream
    if x.dim() == 1:
        fn = B.tcu_scan_exclusive if exclusive else B.tcu_scan_inclusive
        B.check(fn(x, out, cols, B.DTYPES[dn], s, ws.ptr, ws.bytes, stream))
    else:
        B.check(B.tcu_scan_batched(x, out, rows, cols, B.DTYPES[dn], s, int(exclusive), ws.ptr, ws.bytes, stream))
    return out


def segmented_scan(x: torch.Tensor, offsets: torch.Tensor, s: int = 16, exclusive: bool = False,
                   out: torch.Tensor = None) -> torch.Tensor:
    """Scan every segment x[offsets[k]:offsets[k+1]] of a contiguous 1-D CUDA tensor on its own.  `offsets` is an
    int64 CUDA tensor, non-decreasing, from 0 to len(x)."""
    assert x.is_cuda and x.is_contiguous() and x.dim() == 1
    assert offsets.is_cuda and offsets.dtype == torch.int64 and offsets.is_contiguous() and offsets.numel() >= 1
    dn = dtype_name(x)
    n = x.numel()
    if out is None:
        out = torch.empty(n, dtype=torch.int32 if dn == "i8" else torch.float32, device=x.device)
    ws_bytes = B.tcu_scan_segmented_workspace_bytes(n, B.DTYPES[dn], s)
    buf = torch.zeros(ws_bytes + 256, dtype=torch.uint8, device=x.device)
    ptr = buf.data_ptr() + (-buf.data_ptr()) % 256
    stream = torch.cuda.current_stream().cuda_stream
    B.check(B.tcu_scan_segmented(x, out, n, offsets, offsets.numel() - 1, B.DTYPES[dn], s, int(exclusive), ptr, ws_bytes, stream))
    B.check(B.tcu_scan_device_status(ptr, stream))
    return out
