"""Radix sort by one-bit splits built on the exclusive scan: keys must come out exactly as a
library sort orders them."""
import numpy as np
import pytest
import torch

from paper_2411_17887_b200 import binding as B
from paper_2411_17887_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n", [1, 2, 127, 1000, 16384, 3 * 16384 + 77, (1 << 21) + 12345])
def test_sort_matches_numpy(n):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    g = inputs.rng(500 + n % 101)
    keys = g.integers(0, 1 << 32, size=n, dtype=np.uint64).astype(np.uint32)
    if n > 100:
        keys[: n // 3] = keys[n // 3: 2 * (n // 3)]            # plenty of duplicates
        keys[-5:] = [0, 0xFFFFFFFF, 0x80000000, 0x7FFFFFFF, 1]
    d_in = torch.from_numpy(keys.view(np.int32)).cuda()
    d_out = torch.empty_like(d_in)
    tmp_bytes = B.tcu_sort_tmp_bytes(n)
    tmp = torch.empty(tmp_bytes + 256, dtype=torch.uint8, device="cuda")
    tmp_ptr = tmp.data_ptr() + (-tmp.data_ptr()) % 256
    ws_bytes = B.tcu_scan_workspace_bytes(1, n, B.TCU_I8_I32, 16)
    ws = torch.empty(ws_bytes + 256, dtype=torch.uint8, device="cuda")
    ws_ptr = ws.data_ptr() + (-ws.data_ptr()) % 256
    B.check(B.tcu_scan_workspace_init(ws_ptr, ws_bytes, 0))
    B.check(B.tcu_sort_u32(d_in, d_out, n, tmp_ptr, tmp_bytes, ws_ptr, ws_bytes, 0))
    B.check(B.tcu_scan_device_status(ws_ptr, 0))
    got = d_out.cpu().numpy().view(np.uint32)
    assert np.array_equal(got, np.sort(keys))
    assert np.array_equal(d_in.cpu().numpy().view(np.uint32), keys)      # the input is left alone
