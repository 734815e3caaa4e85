"""GPU parity at the full sizes of the five build configurations (plus the fp16 run of the
headline size), in the launch configuration the benchmark times.  The oracle is evaluated
piecewise (carry handed from piece to piece) so that host memory stays bounded."""
import numpy as np
import pytest
import torch

from oracle import scan_oracle as so
from paper_2411_17887_b200 import binding as B
from paper_2411_17887_b200 import inputs

pytestmark = pytest.mark.gpu
PIECE = 1 << 24


@pytest.fixture(scope="module")
def runner():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from tests.gpu_util import Runner
    return Runner(4096, 1 << 28)


def compare_piecewise(got: np.ndarray, x: np.ndarray, dtype: str, exclusive: bool):
    """1-D arrays: oracle on pieces of 2^24 elements with the running carry passed along."""
    carry, acarry = 0, 0.0
    worst = 0.0
    for lo in range(0, x.size, PIECE):
        xs = x[lo:lo + PIECE]
        g = got[lo:lo + PIECE]
        if dtype == "i8":
            y = so.scan_i8(xs, exclusive, init=carry)
            carry = int(y[-1]) + (int(xs[-1]) if exclusive else 0)
            assert np.array_equal(g, so.wrap_int32(y)), f"mismatch in piece at {lo}"
        else:
            x64 = so.widen(xs, dtype)
            y, a = so.scan_f64(x64, exclusive, init=carry)
            a = a + acarry
            carry = float(y[-1]) + (float(x64[-1]) if exclusive else 0.0)
            acarry = float(a[-1]) + (abs(float(x64[-1])) if exclusive else 0.0)
            err = np.abs(g.astype(np.float64) - y)
            tol = so.float_tolerance(a)
            assert (err <= tol).all(), f"out of tolerance in piece at {lo}: worst ratio {(err / tol).max()}"
            worst = max(worst, float((err / tol).max()))
    return worst


@pytest.mark.parametrize("name", ["C1", "C2", "C3", "C5", "C3h"])
def test_single_array_configs(runner, name):
    cfg = inputs.CONFIGS[name]
    x = inputs.make(cfg)
    from tests.gpu_util import to_device
    d_in = to_device(x, cfg.dtype)
    for s in cfg.s:
        for exclusive in cfg.exclusive:
            got = runner.run(x, cfg.dtype, s, exclusive, d_in=d_in)
            compare_piecewise(got, x, cfg.dtype, exclusive)
            if cfg.dtype == "i8":                      # integer results are identical from run to run
                again = runner.run(x, cfg.dtype, s, exclusive, d_in=d_in)
                assert np.array_equal(got, again)
            st = B.tcu_scan_last_stats()
            assert st["sxs_products"] == x.size // (s * s)        # the n / s^2 level-0 products
            assert st["levels_used"] <= max(st["depth_bound"], 5)


def test_batched_config_C4(runner):
    cfg = inputs.CONFIGS["C4"]
    x = inputs.make(cfg)
    got = runner.run(x, cfg.dtype, 16, False)
    block = 256
    for r0 in range(0, x.shape[0], block):
        xs = x[r0:r0 + block]
        y, a = so.scan_f64(so.widen(xs, cfg.dtype))
        err = np.abs(got[r0:r0 + block].astype(np.float64) - y)
        assert (err <= so.float_tolerance(a)).all(), f"rows {r0}.."


def test_beyond_four_gigabytes_of_output():
    # n = 2^30 + 12345 int8: the output is larger than 4 GiB, so every 32-bit index or byte offset would show
    from tests.gpu_util import Runner
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    n = (1 << 30) + 12345
    x = inputs.int8_uniform(n, -127, 127, 31)
    big = Runner(1, n)
    got = big.run(x, "i8", 16)
    compare_piecewise(got, x, "i8", False)
    got = big.run(x, "i8", 128, exclusive=True)
    compare_piecewise(got, x, "i8", True)


def test_two_sweep_with_scanned_totals_beyond_one_inner_tile():
    # more than 128 x 128 tile totals: the inner scans over the terms of the totals have tiles and a tail of their own
    from tests.gpu_util import Runner
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    n = (16384 + 300) * 16384 + 5
    x = inputs.int8_uniform(n, -127, 127, 41)
    big = Runner(1, n)
    got = big.run(x, "i8", 16, variant=1, upper_level_path=1)
    compare_piecewise(got, x, "i8", False)
    assert big.stats["variant"] == 1 and big.stats["upper_level_path"] == 1 and big.stats["tiles"] == 16384 + 300


def test_segmented_at_the_headline_size():
    # n = 2^28 int8 cut at random points (mean segment 2^12, some empty segments), in the launch configuration the
    # benchmark times; every output compared with the oracle's per-segment loop
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    n = 1 << 28
    x = inputs.make(inputs.CONFIGS["C3"])
    g = inputs.rng(77)
    cuts = np.sort(g.integers(0, n + 1, size=n >> 12))
    off = np.concatenate([[0, 0], cuts, cuts[::1000], [n]]).astype(np.int64)
    off.sort()
    d_in = torch.from_numpy(x).cuda()
    d_out = torch.empty(n, dtype=torch.int32, device="cuda")
    d_off = torch.from_numpy(off).cuda()
    ws_bytes = B.tcu_scan_segmented_workspace_bytes(n, B.TCU_I8_I32, 16)
    ws = torch.empty(ws_bytes + 256, dtype=torch.uint8, device="cuda")
    ptr = ws.data_ptr() + (-ws.data_ptr()) % 256
    B.check(B.tcu_scan_workspace_init(ptr, ws_bytes, 0))
    B.check(B.tcu_scan_segmented(d_in, d_out, n, d_off, off.size - 1, B.TCU_I8_I32, 16, 0, ptr, ws_bytes, 0))
    B.check(B.tcu_scan_device_status(ptr, 0))
    got = d_out.cpu().numpy()
    want = so.scan_segments(x, "i8", off)["y32"]
    assert np.array_equal(got, want)


def test_batched_rows_of_odd_length_at_size():
    # 4099 rows of 65521 bf16 values (neither a multiple of 16): rows become segments of one 2^28-sized array
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from tests.gpu_util import Runner
    rows, cols = 4099, 65521
    x = inputs.bf16_normal((rows, cols), 41)
    runner = Runner(rows, cols)
    got = runner.run(x, "bf16", 16, False)
    assert runner.stats["segments_path"] == 1
    block = 512
    for r0 in range(0, rows, block):
        y, a = so.scan_f64(so.widen(x[r0:r0 + block], "bf16"))
        err = np.abs(got[r0:r0 + block].astype(np.float64) - y)
        assert (err <= so.float_tolerance(a)).all(), f"rows {r0}.."
