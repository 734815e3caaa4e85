"""The device-side waits are bounded.  The ordinary scan kernel is launched with the records of one tile
never published and a short limit on every wait: the tiles behind it wait in vain, the kernel records the
time-out, every role leaves its loop, copies in flight are drained, tensor memory is freed, the kernel
returns, the host reads TCU_ERR_TIMEOUT, and the library keeps working afterwards.  Nothing faults."""
import numpy as np
import pytest
import torch

from paper_2411_17887_b200 import binding as B
from paper_2411_17887_b200 import inputs

pytestmark = pytest.mark.gpu
TILE = 128 * 128


# (input type, s, tiles, silent tile, upper_level_path, down_sweep_path): the ordinary path with the silent tile first,
# inside the first wave and in the second wave; then the optional tensor-core branches, in which the four totals warps
# and the four warps of a store group meet at barriers inside their loops and have to give up together
CASES = [("i8", 16, 40, 3, 0, 0), ("f16", 128, 12, 0, 0, 0), ("i8", 64, 400, 150, 0, 0),
         ("i8", 16, 40, 3, 1, 0), ("f16", 16, 200, 160, 1, 0), ("f16", 128, 40, 3, 0, 1), ("f16", 128, 300, 149, 1, 1),
         ("i8", 16, 40, 3, 2, 0), ("f16", 64, 200, 155, 2, 0), ("f16", 16, 200, 151, 2, 1)]


@pytest.mark.parametrize("dtype,s,tiles,skip,upper,down", CASES)
def test_real_kernel_wait_runs_out_and_recovers(dtype, s, tiles, skip, upper, down):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from oracle import scan_oracle as so
    n = tiles * TILE
    dt = B.DTYPES[dtype]
    ws_bytes = B.tcu_scan_workspace_bytes(1, n, dt, s)
    ws = torch.empty(ws_bytes + 256, dtype=torch.uint8, device="cuda")
    ptr = ws.data_ptr() + (-ws.data_ptr()) % 256
    B.check(B.tcu_scan_workspace_init(ptr, ws_bytes, 0))
    assert B.tcu_scan_device_status(ptr, 0) == B.TCU_OK
    x = inputs.int8_uniform(n, -127, 127, 77) if dtype == "i8" else inputs.f16_uniform(n, -1.0, 1.0, 78)
    d_in = torch.from_numpy(x).cuda()
    d_out = torch.empty(n, dtype=torch.int32 if dtype == "i8" else torch.float32, device="cuda")
    # argument checks of the self-test itself
    assert B.tcu_scan_selftest_timeout(d_in, d_out, n, dt, s, skip, 0, ptr, ws_bytes, 0) == B.TCU_ERR_INVALID_ARG
    assert B.tcu_scan_selftest_timeout(d_in, d_out, n, dt, s, tiles, 20, ptr, ws_bytes, 0) == B.TCU_ERR_INVALID_ARG
    # tile `skip` never publishes; every wait gives up after 20 ms
    B.check(B.tcu_scan_selftest_timeout(d_in, d_out, n, dt, s, skip, 20, ptr, ws_bytes, 0, upper_level_path=upper,
                                        down_sweep_path=down))
    assert B.tcu_scan_device_status(ptr, 0) == B.TCU_ERR_TIMEOUT
    assert B.tcu_scan_last_stats()["upper_level_path"] == upper and B.tcu_scan_last_stats()["down_sweep_path"] == down
    # the tiles before the silent one were not affected
    ref = so.scan(x, dtype)
    got = d_out.cpu().numpy()
    if dtype == "i8":
        assert np.array_equal(got[:skip * TILE], ref["y32"][:skip * TILE])
    # the context is intact: clear the workspace and scan with it
    B.check(B.tcu_scan_workspace_init(ptr, ws_bytes, 0))
    assert B.tcu_scan_device_status(ptr, 0) == B.TCU_OK
    d_out.fill_(0)
    B.check(B.tcu_scan_inclusive(d_in, d_out, n, dt, s, ptr, ws_bytes, 0))
    assert B.tcu_scan_device_status(ptr, 0) == B.TCU_OK
    got = d_out.cpu().numpy()
    if dtype == "i8":
        assert np.array_equal(got, ref["y32"])
    else:
        assert (np.abs(got.astype(np.float64) - ref["y"]) <= so.float_tolerance(ref["a"])).all()
