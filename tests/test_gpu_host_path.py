"""tcu_scan_host: host buffers in, host buffers out.  Long inclusive scans go through the pipelined
path (pieces of 2^24 elements, each continuing from the last output of the previous piece)."""
import numpy as np
import pytest
import torch

from oracle import scan_oracle as so
from paper_2411_17887_b200 import binding as B
from paper_2411_17887_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,n,exclusive", [("i8", 5000, False), ("i8", 3 * (1 << 24) + 777, False),
                                               ("f16", 2 * (1 << 24) + 16384 + 5, False),
                                               ("i8", 3 * (1 << 24) + 777, True), ("bf16", (1 << 24) + 3, True)])
def test_host_buffers(dtype, n, exclusive):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    if dtype == "i8":
        x = inputs.int8_uniform(n, -127, 127, 61)
        h_in = torch.from_numpy(x).pin_memory()
    elif dtype == "f16":
        x = inputs.f16_uniform(n, -1.0, 1.0, 62)
        h_in = torch.from_numpy(x).pin_memory()
    else:
        x = inputs.bf16_normal(n, 63)
        h_in = torch.from_numpy(x.view(np.int16)).pin_memory()
    out_dtype = torch.int32 if dtype == "i8" else torch.float32
    h_out = torch.empty(n, dtype=out_dtype).pin_memory()
    d_in = torch.empty(n, dtype=h_in.dtype, device="cuda")
    d_out = torch.empty(n, dtype=out_dtype, device="cuda")
    dt = B.DTYPES[dtype]
    ws_bytes = B.tcu_scan_workspace_bytes(1, n, dt, 16)
    ws = torch.empty(ws_bytes + 256, dtype=torch.uint8, device="cuda")
    ptr = ws.data_ptr() + (-ws.data_ptr()) % 256
    B.check(B.tcu_scan_workspace_init(ptr, ws_bytes, 0))
    stream = torch.cuda.current_stream().cuda_stream
    for _ in range(2):                                     # twice: the internal streams are reused
        h_out.fill_(-3)
        B.check(B.tcu_scan_host(h_in, h_out, n, dt, 16, int(exclusive), d_in, d_out, ptr, ws_bytes, stream))
        torch.cuda.current_stream().synchronize()
        B.check(B.tcu_scan_device_status(ptr, stream))
        got = h_out.numpy()
        ref = so.scan(x, dtype, exclusive)
        if dtype == "i8":
            assert np.array_equal(got, ref["y32"])
        else:
            assert (np.abs(got.astype(np.float64) - ref["y"]) <= so.float_tolerance(ref["a"])).all()
