"""tcu_scan_inclusive_noalloc: the scan for callers that cannot pass a workspace (say, code that
runs inside a host program which handed out all device memory at start-up and allows no further
cudaMalloc).  Its carry records live in an array inside the library, so the only thing to check is
that it computes what the ordinary entry point computes - also when the array still holds the
records of an earlier call.  Collected last on purpose: a failure here cannot hide another test."""
import numpy as np
import pytest
import torch

from paper_2411_17887_b200 import binding as B
from paper_2411_17887_b200 import inputs

pytestmark = pytest.mark.gpu
TILE = 128 * 128


def _reference(d_in, n, dt, s):
    """The existing entry point, with a caller-allocated workspace."""
    out = torch.empty(n, dtype=torch.int32 if dt == B.TCU_I8_I32 else torch.float32, device="cuda")
    ws_bytes = B.tcu_scan_workspace_bytes(1, n, dt, s)
    ws = torch.empty(ws_bytes + 256, dtype=torch.uint8, device="cuda")
    ptr = ws.data_ptr() + (-ws.data_ptr()) % 256
    B.check(B.tcu_scan_workspace_init(ptr, ws_bytes, 0))
    B.check(B.tcu_scan_inclusive(d_in, out, n, dt, s, ptr, ws_bytes, 0))
    B.check(B.tcu_scan_device_status(ptr, 0))
    return out


def test_noalloc_matches_the_workspace_entry_point_twice_in_a_row():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from oracle import scan_oracle as so
    stream = torch.cuda.current_stream().cuda_stream
    # two calls back to back, the second smaller than the first, so that it finds the first call's
    # records (and some it does not overwrite) in the shared array
    cases = [("i8", 300 * TILE + 77, 16), ("i8", 9 * TILE + 128 * 3 + 1, 128),
             ("f16", 200 * TILE + 5, 64), ("f16", 3 * TILE, 16)]
    for dtype, n, s in cases:
        x = inputs.int8_uniform(n, -127, 127, n % 97) if dtype == "i8" else inputs.f16_uniform(n, -1.0, 1.0, n % 89)
        d_in = torch.from_numpy(x).cuda()
        dt = B.DTYPES[dtype]
        want = _reference(d_in, n, dt, s)
        got = torch.full((n,), -7, dtype=want.dtype, device="cuda")
        B.check(B.tcu_scan_inclusive_noalloc(d_in, got, n, dt, s, stream))
        torch.cuda.synchronize()
        if dtype == "i8":
            assert torch.equal(got, want)
        else:
            a = so.scan(x, "f16")["a"]
            tol = torch.from_numpy(2 * so.float_tolerance(a)).cuda()      # each side is within 1e-5*sum|x|+1e-6 of the oracle
            assert bool(((got.double() - want.double()).abs() <= tol).all())


def test_noalloc_rejects_what_does_not_fit():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    d_in = torch.zeros(256, dtype=torch.int8, device="cuda")
    d_out = torch.zeros(256, dtype=torch.int32, device="cuda")
    too_many = B.TCU_SCAN_NOALLOC_MAX_ELEMENTS + 1
    assert B.tcu_scan_inclusive_noalloc(d_in, d_out, too_many, B.TCU_I8_I32, 16, 0) == B.TCU_ERR_TOO_LARGE
    assert "scratch" in B.tcu_status_string(B.TCU_ERR_TOO_LARGE)
    assert B.tcu_scan_inclusive_noalloc(d_in, d_out, 0, B.TCU_I8_I32, 16, 0) == B.TCU_OK
    torch.cuda.synchronize()
    assert int(d_out.abs().sum()) == 0                                   # nothing was launched, nothing written
