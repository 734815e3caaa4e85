"""Host-only checks of the C-ABI library: it loads without a GPU, exports every symbol the
header declares, sizes workspaces as documented and rejects bad arguments before any launch."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2411_17887_b200 import build
    build.build()
    from paper_2411_17887_b200 import binding
    return binding


def declared_functions():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names += re.findall(r"\b(tcu_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def test_every_declared_symbol_is_exported(B):
    lib = ctypes.CDLL(B.LIB_PATH)
    names = declared_functions()
    assert {"tcu_scan_inclusive", "tcu_scan_exclusive", "tcu_scan_batched", "tcu_scan_workspace_bytes"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
        assert hasattr(B, n), f"binding lacks {n}"


def test_status_strings(B):
    assert B.tcu_status_string(B.TCU_OK) == "ok"
    codes = [B.TCU_OK, B.TCU_ERR_INVALID_ARG, B.TCU_ERR_UNSUPPORTED, B.TCU_ERR_WORKSPACE, B.TCU_ERR_CUDA,
             B.TCU_ERR_TIMEOUT, B.TCU_ERR_TOO_LARGE]
    assert codes == list(range(7))
    seen = {B.tcu_status_string(i) for i in codes}
    assert len(seen) == 7 and "unknown status" not in seen      # every status of the header has its own text
    assert B.tcu_status_string(7) == "unknown status"
    assert B.tcu_status_string(99) == "unknown status"


def test_workspace_bytes(B):
    tile = 128 * 128
    base = B.tcu_scan_workspace_bytes(1, 0, 0, 16)
    assert base >= 256
    # single arrays: 16 bytes of record per tile, plus room for the two-sweep variant's scan of the tile totals by the
    # library itself (four term arrays, their four scans, the inner scans' own records): a few dozen bytes per tile
    one = B.tcu_scan_workspace_bytes(1, tile, 0, 16)
    assert base < one <= base + 4096
    assert one <= B.tcu_scan_workspace_bytes(1, tile + 128, 1, 64) <= one + 4096
    big = B.tcu_scan_workspace_bytes(1, 1 << 28, 0, 16)
    assert 16 * (1 << 14) < big <= 48 * (1 << 14)
    assert big % 256 == 0 and one % 256 == 0
    # dense rows: records only
    assert B.tcu_scan_workspace_bytes(4096, 65536, 2, 16) == 256 + 16 + 16 * 4096 * 4


def test_argument_checks_return_before_any_launch(B):
    ws = 1 << 20
    ok_in, ok_out, ok_ws = 0x10000, 0x800000, 0x4000000   # never dereferenced: every call below fails a host check
    assert B.tcu_scan_inclusive(None, None, 0, 0, 16, None, 0) == B.TCU_OK                 # empty: nothing to do
    assert B.tcu_scan_inclusive(None, ok_out, 10, 0, 16, ok_ws, ws) == B.TCU_ERR_INVALID_ARG
    assert B.tcu_scan_inclusive(ok_in, None, 10, 0, 16, ok_ws, ws) == B.TCU_ERR_INVALID_ARG
    assert B.tcu_scan_inclusive(ok_in + 4, ok_out, 10, 0, 16, ok_ws, ws) == B.TCU_ERR_INVALID_ARG   # misaligned
    assert B.tcu_scan_inclusive(ok_in, ok_out + 8, 10, 0, 16, ok_ws, ws) == B.TCU_ERR_INVALID_ARG
    assert B.tcu_scan_inclusive(ok_in, ok_out, 10, 0, 32, ok_ws, ws) == B.TCU_ERR_UNSUPPORTED       # s not offered
    assert B.tcu_scan_inclusive(ok_in, ok_out, 10, 5, 16, ok_ws, ws) == B.TCU_ERR_INVALID_ARG       # dtype
    assert B.tcu_scan_exclusive(ok_in, ok_out, 10, 0, 16, None, 0) == B.TCU_ERR_WORKSPACE
    assert B.tcu_scan_exclusive(ok_in, ok_out, 1 << 20, 0, 16, ok_ws, 64) == B.TCU_ERR_WORKSPACE    # too small
    assert B.tcu_scan_inclusive(ok_in, ok_in + 64, 1 << 10, 0, 16, ok_ws, ws) == B.TCU_ERR_INVALID_ARG  # overlap
    assert B.tcu_scan_batched(ok_in, ok_out, 4, (1 << 40) + 16, 0, 16, 0, ok_ws, ws) == B.TCU_ERR_UNSUPPORTED   # too large
    # one scan holds at most 2^37 elements (2^30 rows of 128 under a signed 32-bit row coordinate)
    far_in, far_out = 0x10000, 0x7000_0000_0000
    assert B.tcu_scan_inclusive(far_in, far_out, (1 << 37) + 128, 0, 16, ok_ws, ws) == B.TCU_ERR_UNSUPPORTED
    assert B.tcu_scan_inclusive(far_in, far_out, 1 << 37, 0, 16, ok_ws, ws) == B.TCU_ERR_WORKSPACE       # the size itself is accepted
    # the general call: malformed options are refused, carries belong to single arrays only
    assert B.tcu_scan_ex(ok_in, ok_out, 1, 10, 0, 16, ok_ws, ws, variant=2) == B.TCU_ERR_INVALID_ARG
    assert B.tcu_scan_ex(ok_in, ok_out, 1, 10, 0, 16, ok_ws, ws, upper_level_path=3) == B.TCU_ERR_INVALID_ARG
    assert B.tcu_scan_ex(ok_in, ok_out, 2, 16, 0, 16, ok_ws, ws, d_carry_in=0x9000) == B.TCU_ERR_INVALID_ARG
    assert B.tcu_scan_ex(ok_in, ok_out, 1, 16, 0, 16, ok_ws, ws, d_carry_in=0x9004) == B.TCU_ERR_INVALID_ARG  # 8-byte aligned
    assert B.tcu_scan_ex(ok_in, ok_out, 1, 16, 0, 16, ok_ws, ws, variant=1, d_carry_in=0x9000) == B.TCU_ERR_UNSUPPORTED
    assert B.tcu_scan_selftest_timeout(ok_in, ok_out, 128, 0, 16, 0, 0, ok_ws, ws) == B.TCU_ERR_INVALID_ARG
    assert B.tcu_scan_selftest_timeout(ok_in, ok_out, 100, 0, 16, 0, 20, ok_ws, ws) == B.TCU_ERR_INVALID_ARG
    assert B.tcu_reduce_total(ok_in, 100, 0, None, ok_ws, ws) == B.TCU_ERR_INVALID_ARG
    assert B.tcu_reduce_total(ok_in + 1, 100, 0, 0x9000, ok_ws, ws) == B.TCU_ERR_INVALID_ARG
    assert B.tcu_reduce_total(ok_in, 1 << 30, 0, 0x9000, ok_ws, 64) == B.TCU_ERR_WORKSPACE
    assert B.tcu_carry_exclusive_prefix(0x9000, 4, 5, 0, 0xA000) == B.TCU_ERR_INVALID_ARG          # index > count
    assert B.tcu_carry_exclusive_prefix(0x9000, 4, 2, 9, 0xA000) == B.TCU_ERR_INVALID_ARG          # dtype
    assert B.tcu_scan_inclusive_noalloc(ok_in, ok_out, (1 << 26) + 1, 0, 16) == B.TCU_ERR_TOO_LARGE
    assert B.tcu_scan_inclusive_noalloc(ok_in, ok_out, 0, 9, 16) == B.TCU_ERR_INVALID_ARG
    assert B.tcu_scan_inclusive_noalloc(ok_in + 2, ok_out, 64, 0, 16) == B.TCU_ERR_INVALID_ARG
    assert B.tcu_scan_level0_debug(ok_in, ok_out, 100, 0, 16, ok_ws, ws) == B.TCU_ERR_UNSUPPORTED
    assert B.tcu_scan_workspace_init(None, 1024, 0) == B.TCU_ERR_WORKSPACE
    assert B.tcu_scan_device_status(None, 0) == B.TCU_ERR_WORKSPACE
