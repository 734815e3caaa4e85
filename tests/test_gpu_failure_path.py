"""The device-side waits are bounded: a wait that nothing satisfies runs out, the kernel returns,
the host reads TCU_ERR_TIMEOUT, and the library keeps working afterwards."""
import numpy as np
import pytest
import torch

from paper_2411_17887_b200 import binding as B
from paper_2411_17887_b200 import inputs

pytestmark = pytest.mark.gpu


def test_bounded_wait_reports_timeout_and_recovers():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from oracle import scan_oracle as so
    n = 3 * 16384 + 5
    ws_bytes = B.tcu_scan_workspace_bytes(1, n, 0, 16)
    ws = torch.empty(ws_bytes + 256, dtype=torch.uint8, device="cuda")
    ptr = ws.data_ptr() + (-ws.data_ptr()) % 256
    B.check(B.tcu_scan_workspace_init(ptr, ws_bytes, 0))
    assert B.tcu_scan_device_status(ptr, 0) == B.TCU_OK
    assert B.tcu_scan_selftest_timeout(ptr, ws_bytes, 0, 0) == B.TCU_ERR_INVALID_ARG
    B.check(B.tcu_scan_selftest_timeout(ptr, ws_bytes, 20, 0))      # 20 ms wait on a flag nothing sets
    assert B.tcu_scan_device_status(ptr, 0) == B.TCU_ERR_TIMEOUT
    # the context is intact: clear the workspace and scan with it
    B.check(B.tcu_scan_workspace_init(ptr, ws_bytes, 0))
    assert B.tcu_scan_device_status(ptr, 0) == B.TCU_OK
    x = inputs.int8_uniform(n, -127, 127, 77)
    d_in = torch.from_numpy(x).cuda()
    d_out = torch.empty(n, dtype=torch.int32, device="cuda")
    B.check(B.tcu_scan_inclusive(d_in, d_out, n, B.TCU_I8_I32, 16, ptr, ws_bytes, 0))
    assert B.tcu_scan_device_status(ptr, 0) == B.TCU_OK
    assert np.array_equal(d_out.cpu().numpy(), so.scan(x, "i8")["y32"])
