"""tcu_scan_inclusive_noalloc: the scan for callers that cannot pass a workspace (say, code that
runs inside a host program which handed out all device memory at start-up and allows no further
cudaMalloc).  Its carry records live in an array inside the library, so what has to be checked is
that it computes what the ordinary entry point computes - also when the array still holds the
records of an earlier call - that both agree with the CPU oracle, and that the caller can ask
whether a wait gave up.  Collected last on purpose: a failure here cannot hide another test."""
import numpy as np
import pytest
import torch

from paper_2411_17887_b200 import binding as B
from paper_2411_17887_b200 import inputs

pytestmark = pytest.mark.gpu
TILE = 128 * 128


def _with_workspace(d_in, n, dt, s):
    """The existing entry point, with a caller-allocated workspace."""
    out = torch.empty(n, dtype=torch.int32 if dt == B.TCU_I8_I32 else torch.float32, device="cuda")
    ws_bytes = B.tcu_scan_workspace_bytes(1, n, dt, s)
    ws = torch.empty(ws_bytes + 256, dtype=torch.uint8, device="cuda")
    ptr = ws.data_ptr() + (-ws.data_ptr()) % 256
    B.check(B.tcu_scan_workspace_init(ptr, ws_bytes, 0))
    B.check(B.tcu_scan_inclusive(d_in, out, n, dt, s, ptr, ws_bytes, 0))
    B.check(B.tcu_scan_device_status(ptr, 0))
    return out


def test_noalloc_matches_the_workspace_entry_point_and_the_oracle_twice_in_a_row():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from oracle import scan_oracle as so
    stream = torch.cuda.current_stream().cuda_stream
    # calls back to back, each smaller than the one before, so that each finds its predecessor's
    # records (and some it does not overwrite) in the shared array; the first one uses the array to
    # its last record (n = the stated maximum)
    cases = [("i8", B.TCU_SCAN_NOALLOC_MAX_ELEMENTS, 16), ("i8", 300 * TILE + 77, 16), ("i8", 9 * TILE + 128 * 3 + 1, 128),
             ("f16", 200 * TILE + 5, 64), ("f16", 3 * TILE, 16)]
    for dtype, n, s in cases:
        x = inputs.int8_uniform(n, -127, 127, n % 97) if dtype == "i8" else inputs.f16_uniform(n, -1.0, 1.0, n % 89)
        d_in = torch.from_numpy(x).cuda()
        dt = B.DTYPES[dtype]
        want = _with_workspace(d_in, n, dt, s)
        got = torch.full((n,), -7, dtype=want.dtype, device="cuda")
        B.check(B.tcu_scan_inclusive_noalloc(d_in, got, n, dt, s, stream))
        assert B.tcu_scan_noalloc_status(stream) == B.TCU_OK
        ref = so.scan(x, dtype)
        if dtype == "i8":
            assert torch.equal(got, want)
            assert np.array_equal(got.cpu().numpy(), ref["y32"])
        else:
            tol = so.float_tolerance(ref["a"])                 # 1e-5 * sum|x| + 1e-6, the bar of every float test
            assert (np.abs(got.cpu().numpy().astype(np.float64) - ref["y"]) <= tol).all()
            assert (np.abs(want.cpu().numpy().astype(np.float64) - ref["y"]) <= tol).all()
        del want, got, d_in


def test_noalloc_rejects_what_does_not_fit_or_is_malformed_before_touching_the_stream():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    d_in = torch.zeros(256, dtype=torch.int8, device="cuda")
    d_out = torch.zeros(256, dtype=torch.int32, device="cuda")
    too_many = B.TCU_SCAN_NOALLOC_MAX_ELEMENTS + 1
    assert B.tcu_scan_inclusive_noalloc(d_in, d_out, too_many, B.TCU_I8_I32, 16, 0) == B.TCU_ERR_TOO_LARGE
    assert "scratch" in B.tcu_status_string(B.TCU_ERR_TOO_LARGE)
    assert B.tcu_scan_inclusive_noalloc(d_in, d_out, 0, B.TCU_I8_I32, 16, 0) == B.TCU_OK
    # the same answers as the workspace entry point gives for the same mistakes
    assert B.tcu_scan_inclusive_noalloc(d_in, d_out, 0, 7, 16, 0) == B.TCU_ERR_INVALID_ARG          # dtype, even for n = 0
    assert B.tcu_scan_inclusive_noalloc(d_in, d_out, 256, B.TCU_I8_I32, 32, 0) == B.TCU_ERR_UNSUPPORTED
    assert B.tcu_scan_inclusive_noalloc(None, d_out, 256, B.TCU_I8_I32, 16, 0) == B.TCU_ERR_INVALID_ARG
    assert B.tcu_scan_inclusive_noalloc(d_in.data_ptr() + 4, d_out, 128, B.TCU_I8_I32, 16, 0) == B.TCU_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert int(d_out.abs().sum()) == 0                                   # nothing was launched, nothing written
