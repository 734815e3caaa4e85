"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element.

Integers must match bit for bit; fp32 outputs must satisfy
|y - y_ref| <= 1e-5 * sum_{j<=i}|x_j| + 1e-6 with y_ref the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import scan_oracle as so
from oracle import tcu_model as tm
from paper_2411_17887_b200 import inputs

pytestmark = pytest.mark.gpu

TILE = 128 * 128


@pytest.fixture(scope="module")
def runner():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from tests.gpu_util import Runner
    return Runner(64, 1 << 22)


def gen(dtype, shape, seed):
    if dtype == "i8":
        return inputs.int8_uniform(shape, -127, 127, seed)
    if dtype == "f16":
        return inputs.f16_uniform(shape, -1.0, 1.0, seed)
    return inputs.bf16_normal(shape, seed)


@pytest.mark.parametrize("dtype", ["i8", "f16", "bf16"])
@pytest.mark.parametrize("s", [16, 64, 128])
def test_level0_is_upsweep_round_0(runner, dtype, s):
    # After up-sweep round t = 0 of Algorithm 1 every chunk of s elements holds its own scan:
    # compare with the model's BatchMatMul(x, L_s) on three tiles.
    n = 3 * TILE
    x = gen(dtype, n, 40 + s)
    got = runner.run(x, dtype, s, level0=True)
    if dtype == "i8":
        want = tm.batch_matmul(x.astype(np.int64), tm.L_matrix(s))
        assert np.array_equal(got.astype(np.int64), want)
    else:
        x64 = so.widen(x, dtype)
        want = tm.batch_matmul(x64, tm.L_matrix(s, np.float64))
        bound = 1e-5 * tm.batch_matmul(np.abs(x64), tm.L_matrix(s, np.float64)) + 1e-6
        assert (np.abs(got - want) <= bound).all()


EDGE_SIZES = [1, 2, 15, 16, 17, 127, 128, 129, 255, 256, 257, 16 * 16 + 1, TILE - 1, TILE, TILE + 1,
              TILE + 128, 3 * TILE + 5, 5 * TILE - 128]


@pytest.mark.parametrize("dtype", ["i8", "f16", "bf16"])
@pytest.mark.parametrize("exclusive", [False, True])
def test_edge_sizes(runner, dtype, exclusive):
    from tests.gpu_util import check
    for s in (16, 64, 128):
        for n in EDGE_SIZES:
            x = gen(dtype, n, 1000 + n % 977 + s)
            check(runner, x, dtype, s, exclusive)


@pytest.mark.parametrize("dtype,s", [("i8", 16), ("i8", 128), ("f16", 16), ("bf16", 64)])
def test_around_one_wave_of_tiles(runner, dtype, s):
    # one tile per SM, one less, one more, and a ragged tail: exercises the persistent schedule
    from tests.gpu_util import check
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    for n in (sms * TILE - 1, sms * TILE, sms * TILE + 1, (sms + 1) * TILE + 77, (2 * sms + 3) * TILE + 128 * 9 + 3):
        for exclusive in (False, True):
            check(runner, gen(dtype, n, n % 1013), dtype, s, exclusive)


def test_all_ones_fp16_is_exact(runner):
    # every partial sum is an integer <= 2^22, exactly representable in fp32 whatever the association:
    # a layout or carry bug that the tolerance would hide shows up here
    n = 1 << 22
    x = np.ones(n, np.float16)
    for s in (16, 64, 128):
        got = runner.run(x, "f16", s)
        assert np.array_equal(got, np.arange(1, n + 1, dtype=np.float32))
        got = runner.run(x, "f16", s, exclusive=True)
        assert np.array_equal(got, np.arange(0, n, dtype=np.float32))


def test_int_position_sensitivity(runner):
    # distinct weights per position: a permuted row / chunk inside a tile cannot cancel out
    n = 4 * TILE + 128 * 3
    x = ((np.arange(n) * 37 + (np.arange(n) // 128) * 11) % 251 - 125).astype(np.int8)
    from tests.gpu_util import check
    for s in (16, 64, 128):
        check(runner, x, "i8", s)
        check(runner, x, "i8", s, True)


def test_int_wraps_modulo_2_32():
    # sums that leave the int32 range: 2^26 elements of 127 reach 8.5e9 (past 2^32, wrapping twice), 2^25
    # elements of -128 reach -4.3e9 (past -2^31); the device must hold the exact sum modulo 2^32 throughout
    from tests.gpu_util import Runner, check
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    big = Runner(1, 1 << 26)
    n = 1 << 26
    got = check(big, np.full(n, 127, np.int8), "i8", 16)
    assert int(got[-1]) == ((127 * n + 2**31) % 2**32) - 2**31 and 127 * n > 2**32
    assert int((got[1:] < got[:-1]).sum()) == 2          # the int32 view jumps down twice: at 2^31 and at 2^31 + 2^32
    n = 1 << 25
    got = check(big, np.full(n, -128, np.int8), "i8", 128, True)
    assert int(got[-1]) == ((-128 * (n - 1) + 2**31) % 2**32) - 2**31 and -128 * (n - 1) < -2**31


@pytest.mark.parametrize("dtype", ["i8", "bf16", "f16"])
def test_batched_rows(runner, dtype):
    from tests.gpu_util import check
    for rows, cols in [(1, 128), (3, 128), (5, TILE), (4, 2 * TILE + 128 * 5), (64, 65536), (7, 128 * 129),
                       (6, 16), (9, 112), (5, 128 + 16), (3, TILE + 128 * 3 + 48), (33, 2 * TILE - 16)]:
        for s in (16, 128):
            check(runner, gen(dtype, (rows, cols), rows * 7 + cols % 101), dtype, s, False)
        check(runner, gen(dtype, (rows, cols), rows * 7 + cols % 103), dtype, 64, True)


def test_repeatable_and_workspace_reuse(runner):
    # the same workspace serves different shapes back to back; integer results never change between runs
    from tests.gpu_util import check
    x = gen("i8", 200 * TILE + 9, 5)
    a = check(runner, x, "i8", 16)
    y = gen("f16", 3 * TILE, 6)
    check(runner, y, "f16", 64)
    b = check(runner, x, "i8", 16)
    assert np.array_equal(a, b)


def test_stats_report(runner):
    from paper_2411_17887_b200 import binding as B
    n = 1 << 20
    runner.run(gen("f16", n, 3), "f16", 64)
    st = B.tcu_scan_last_stats()
    assert st["tiles"] == n // TILE and st["s"] == 64 and st["sxs_products"] == n // (64 * 64)
    assert st["depth_bound"] == 2 * 3 and st["levels_used"] == 5 and st["variant"] == 0 and st["upper_level_path"] == 0
    assert st["mma_instructions"] == st["tiles"] * (2 * 4 + 8)      # U_64 products + row-total products


@pytest.mark.parametrize("dtype", ["i8", "f16", "bf16"])
def test_two_sweep_variant_matches_oracle(runner, dtype):
    # the reduce-then-scan structure (input read twice) must satisfy the same parity bars
    from paper_2411_17887_b200 import binding as B
    from tests.gpu_util import to_device, assert_int_equal, assert_float_close
    for n, s in [(TILE, 16), (37 * TILE + 128 * 5 + 9, 64), (1500 * TILE + 77, 16)]:
        x = gen(dtype, n, 4000 + n % 911)
        d_in = to_device(x, dtype)
        out = torch.empty(n, dtype=torch.int32 if dtype == "i8" else torch.float32, device="cuda")
        B.check(B.tcu_scan_ex(d_in, out, 1, n, B.DTYPES[dtype], s, runner.ws_ptr, runner.ws_bytes, 0, variant=1))
        B.check(B.tcu_scan_device_status(runner.ws_ptr, 0))
        assert B.tcu_scan_last_stats()["variant"] == 1
        got = out.cpu().numpy()
        if dtype == "i8":
            assert_int_equal(got, x, False)
        else:
            assert_float_close(got, x, dtype, False)
    # and the single-pass path still works on the same workspace afterwards
    from tests.gpu_util import check
    check(runner, gen(dtype, 5 * TILE + 3, 17), dtype, 16)


@pytest.mark.parametrize("dtype", ["i8", "f16", "bf16"])
def test_two_sweep_with_the_totals_scanned_by_the_library_itself(runner, dtype):
    # Section 2.2 step 3 literally: the tile totals, split into exact narrow terms, go through the tensor-core scan again
    # (one inner scan per term) and are recombined; integers stay bit-exact, floats within the tolerance
    from tests.gpu_util import check
    cases = [(TILE, 16, 1), (37 * TILE + 128 * 5 + 9, 64, 1), (128 * TILE, 16, 2), (1500 * TILE + 77, 16, 1),
             (1500 * TILE + 77, 128, 2), (130 * TILE + 1, 64, 2)]
    for n, s, path in cases:
        for exclusive in (False, True):
            check(runner, gen(dtype, n, 5000 + n % 907), dtype, s, exclusive, variant=1, upper_level_path=path)
            st = runner.stats
            assert st["variant"] == 1 and st["upper_level_path"] == path
    if dtype == "i8":
        # tile totals of +-2 080 768 (digits of both signs, carries between the digits), prefix sums that wrap twice
        for value in (127, -127, -128):
            x = np.full(1 << 26, value, dtype=np.int8)
            check(runner, x, "i8", 16, variant=1, upper_level_path=1)
    else:
        # all-ones input: every total and every prefix is an integer below 2^24, so the result must be exact
        n = 900 * TILE + 128 * 3 + 5
        got = runner.run(inputs_ones(dtype, n), dtype, 16, variant=1, upper_level_path=1)
        assert np.array_equal(got, np.arange(1, n + 1, dtype=np.float32))
    # the single-pass path still works on the same workspace afterwards
    check(runner, gen(dtype, 5 * TILE + 3, 17), dtype, 16)


def inputs_ones(dtype, n):
    if dtype == "f16":
        return np.ones(n, dtype=np.float16)
    return np.full(n, 0x3F80, dtype=np.uint16)          # bf16 1.0


def test_result_does_not_depend_on_the_number_of_ctas(runner):
    # the p of the paper's p-TCU bound: any number of persistent CTAs gives the same integers
    from paper_2411_17887_b200 import binding as B
    from tests.gpu_util import check
    x = gen("i8", 200 * TILE + 128 * 7 + 3, 99)
    for p in (1, 3, 32):
        check(runner, x, "i8", 16, max_ctas=p)
        assert runner.stats["grid"] == p


def test_row_total_scan_on_tensor_cores_gives_the_same_integers(runner):
    # upper level as a triangular product on 8-bit limbs instead of warp shuffles (int8 input)
    from paper_2411_17887_b200 import binding as B
    from tests.gpu_util import check
    for n, s in [(TILE, 16), (9 * TILE + 128 * 3 + 5, 64), (700 * TILE + 77, 16), (300 * TILE, 128)]:
        x = gen("i8", n, 7000 + n % 313)
        check(runner, x, "i8", s, upper_level_path=1)
        check(runner, x, "i8", s, True, upper_level_path=1)
        assert runner.stats["upper_level_path"] == 1
    extreme = np.full(5 * TILE, -128, np.int8)          # row totals of -2^14: the limb split at its limit
    check(runner, extreme, "i8", 16, upper_level_path=1)
    check(runner, np.full(5 * TILE, 127, np.int8), "i8", 16, upper_level_path=1)
    d = torch.zeros(256, dtype=torch.int8, device="cuda")
    o = torch.zeros(256, dtype=torch.int32, device="cuda")
    assert B.tcu_scan_ex(d, o, 1, 256, 0, 16, runner.ws_ptr, runner.ws_bytes, 0, upper_level_path=3) == B.TCU_ERR_INVALID_ARG


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_row_total_scan_on_tensor_cores_floating_point(runner, dtype):
    # the same upper level for fp32 totals: each split exactly into three bf16 terms, one triangular kind::f16
    # product, three fp32 additions to recombine; same tolerance, and exact on input whose sums are small integers
    from tests.gpu_util import check
    for n, s in [(TILE, 16), (9 * TILE + 128 * 3 + 5, 64), (400 * TILE + 77, 16), (150 * TILE, 128)]:
        x = gen(dtype, n, 7100 + n % 313)
        check(runner, x, dtype, s, upper_level_path=1)
        check(runner, x, dtype, s, True, upper_level_path=1)
        assert runner.stats["upper_level_path"] == 1
        assert runner.stats["mma_instructions"] == runner.stats["tiles"] * ((128 // max(s, 16)) * (max(s, 16) // 16) + 8 + 8)
    got = runner.run(np.ones(1 << 22, np.float16), "f16", 16, upper_level_path=1)
    assert np.array_equal(got, np.arange(1, (1 << 22) + 1, dtype=np.float32))
    check(runner, gen(dtype, 7 * TILE + 3, 5), dtype, 128, upper_level_path=1, down_sweep_path=1)   # both products at once
    assert runner.stats["upper_level_path"] == 1 and runner.stats["down_sweep_path"] == 1


@pytest.mark.parametrize("dtype", ["i8", "f16", "bf16"])
def test_chunk_level_on_tensor_cores(runner, dtype):
    # upper_level_path = 2: besides the scan over the row totals, the carries of the 128 / s chunks of a row are a product
    # of the chunk totals (two 8-bit limbs / three bf16 terms) with a strictly upper triangular ones matrix
    from tests.gpu_util import check
    per_tile = {"i8": {16: 4 + 4 + 4 + 1, 64: 4 + 4 + 4 + 1}, "f": {16: 8 + 8 + 8 + 2, 64: 8 + 8 + 8 + 2}}["i8" if dtype == "i8" else "f"]
    for n, s in [(TILE, 16), (9 * TILE + 128 * 3 + 5, 64), (500 * TILE + 77, 16), (300 * TILE, 64)]:
        x = gen(dtype, n, 7300 + n % 313)
        check(runner, x, dtype, s, upper_level_path=2)
        check(runner, x, dtype, s, True, upper_level_path=2)
        assert runner.stats["upper_level_path"] == 2
        assert runner.stats["mma_instructions"] == runner.stats["tiles"] * per_tile[s]
    if dtype == "i8":
        check(runner, np.full(5 * TILE, -128, np.int8), "i8", 64, upper_level_path=2)     # chunk totals of -2^13: the limb split at its limit
        check(runner, np.full(5 * TILE, 127, np.int8), "i8", 64, upper_level_path=2)
        x = ((np.arange(4 * TILE) * 37 + (np.arange(4 * TILE) // 16) * 11) % 251 - 125).astype(np.int8)   # every chunk different
        check(runner, x, "i8", 16, upper_level_path=2)
    else:
        for s in (16, 64):
            got = runner.run(np.ones(1 << 22, np.float16), "f16", s, upper_level_path=2)
            assert np.array_equal(got, np.arange(1, (1 << 22) + 1, dtype=np.float32))
    check(runner, gen(dtype, 3 * TILE + 9, 5), dtype, 128, upper_level_path=2)     # a row of s = 128 is one chunk: same as 1
    assert runner.stats["upper_level_path"] == 2
    check(runner, gen(dtype, 64 * 65536, 6).reshape(64, 65536), dtype, 16, upper_level_path=2)   # batched rows too


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_down_sweep_as_a_tensor_core_product(runner, dtype):
    # the carry of every row added by accumulator += C * ones (C = carry in three bf16 terms) instead of vector adds
    from paper_2411_17887_b200 import binding as B
    from tests.gpu_util import check
    for n in (TILE, 9 * TILE + 128 * 3 + 5, 400 * TILE + 77):
        for exclusive in (False, True):
            check(runner, gen(dtype, n, 8000 + n % 211), dtype, 128, exclusive, down_sweep_path=1)
            assert runner.stats["down_sweep_path"] == 1
    got = runner.run(np.ones(1 << 22, np.float16), "f16", 128, down_sweep_path=1)   # integers up to 2^22: must stay exact
    assert np.array_equal(got, np.arange(1, (1 << 22) + 1, dtype=np.float32))
    check(runner, gen(dtype, 5 * TILE, 3), dtype, 16, down_sweep_path=1)        # other tile sizes ignore the choice
    assert runner.stats["down_sweep_path"] == 0
    check(runner, gen("i8", 5 * TILE, 4), "i8", 128, down_sweep_path=1)
    assert runner.stats["down_sweep_path"] == 0


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_down_sweep_as_a_product_per_chunk(runner, dtype):
    # s < 128: every chunk's carry (row base + what the earlier chunks of the row add up to) is added to the chunk's
    # elements by one product with a 0 / 1 selector matrix, the paper's B_s; needs the chunk totals as a product
    # (upper_level_path = 2), from which the carries come
    from tests.gpu_util import check
    for n, s in [(TILE, 16), (9 * TILE + 128 * 3 + 5, 64), (400 * TILE + 77, 16), (300 * TILE, 64)]:
        for exclusive in (False, True):
            check(runner, gen(dtype, n, 9100 + n % 127), dtype, s, exclusive, upper_level_path=2, down_sweep_path=1)
            st = runner.stats
            assert st["down_sweep_path"] == 1 and st["upper_level_path"] == 2
            assert st["mma_instructions"] == st["tiles"] * (8 + 8 + 8 + 2 + (2 if s == 16 else 1))
    for s in (16, 64):
        got = runner.run(np.ones(1 << 22, np.float16), "f16", s, upper_level_path=2, down_sweep_path=1)   # must stay exact
        assert np.array_equal(got, np.arange(1, (1 << 22) + 1, dtype=np.float32))
    check(runner, gen(dtype, 32 * 65536, 6).reshape(32, 65536), dtype, 16, upper_level_path=2, down_sweep_path=1)   # batched rows
    check(runner, gen("i8", 5 * TILE, 4), "i8", 16, upper_level_path=2, down_sweep_path=1)      # integers: no such product
    assert runner.stats["down_sweep_path"] == 0


def test_widening_copy_measuring_aid():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2411_17887_b200 import binding as B
    from tests.gpu_util import to_device
    from oracle import scan_oracle as so
    for dtype in ("i8", "f16", "bf16"):
        for n in (5 * TILE + 16, 4, 2048, 2052, 3 * 2048 - 4):       # whole blocks, a ragged last block, one piece
            x = gen(dtype, n, 77)
            d_in = to_device(x, dtype)
            d_out = torch.full((n + 8,), 7, dtype=torch.int32 if dtype == "i8" else torch.float32, device="cuda")
            B.check(B.tcu_widen_copy(d_in, d_out, n, B.DTYPES[dtype], 0))
            got = d_out.cpu().numpy()
            want = x.astype(np.int32) if dtype == "i8" else so.widen(x, dtype).astype(np.float32)
            assert np.array_equal(got[:n], want) and (got[n:] == 7).all()
    d_in = torch.zeros(64, dtype=torch.int8, device="cuda")
    d_out = torch.zeros(64, dtype=torch.int32, device="cuda")
    assert B.tcu_widen_copy(d_in, d_out, 17, 0, 0) == B.TCU_ERR_INVALID_ARG
    assert B.tcu_widen_copy(d_in, d_out, 16, 5, 0) == B.TCU_ERR_INVALID_ARG
    assert B.tcu_widen_copy(d_in[1:], d_out, 16, 0, 0) == B.TCU_ERR_INVALID_ARG
    assert B.tcu_widen_copy(d_in, d_out, 0, 0, 0) == B.TCU_OK


def test_two_streams_at_the_same_time_with_a_workspace_each():
    # two persistent launches share the SMs: neither may depend on CTAs of its own grid that are not resident yet
    # (tiles are claimed by running CTAs only), and each keeps its carries in its own workspace
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2411_17887_b200 import binding as B
    from oracle import scan_oracle as so
    n_max = 600 * TILE + 77
    x = gen("i8", n_max, 31)
    want = so.scan(x, "i8")["y32"]
    d_in = torch.from_numpy(x).cuda()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    spaces = []
    for _ in streams:
        ws_bytes = B.tcu_scan_workspace_bytes(1, n_max, 0, 16)
        ws = torch.empty(ws_bytes + 256, dtype=torch.uint8, device="cuda")
        ptr = ws.data_ptr() + (-ws.data_ptr()) % 256
        B.check(B.tcu_scan_workspace_init(ptr, ws_bytes, 0))
        spaces.append((ws, ptr, ws_bytes))
    torch.cuda.synchronize()
    results = []
    for n, s in [(n_max, 16), (148 * TILE, 64), (100 * TILE + 5, 128), (n_max, 64), (TILE, 16), (300 * TILE, 16)]:
        for strm, (ws, ptr, ws_bytes) in zip(streams, spaces):
            with torch.cuda.stream(strm):
                out = torch.empty(n, dtype=torch.int32, device="cuda")
                B.check(B.tcu_scan_inclusive(d_in, out, n, 0, s, ptr, ws_bytes, strm.cuda_stream))
                results.append((n, out))
    torch.cuda.synchronize()
    for ws, ptr, ws_bytes in spaces:
        assert B.tcu_scan_device_status(ptr, 0) == B.TCU_OK
    for n, out in results:
        assert np.array_equal(out.cpu().numpy(), want[:n])


def test_scans_replayed_from_a_cuda_graph(runner):
    # the workspace entry points only queue work on the given stream (kernels, and memsets for the segmented path), so a
    # sequence of scans can be captured once and replayed; every replay must give the same integers as the oracle
    from paper_2411_17887_b200 import binding as B
    from oracle import scan_oracle as so
    sizes = [(1 << 16, 16), (37 * TILE + 128 * 5 + 9, 64), (300 * TILE + 77, 16)]
    xs = [gen("i8", n, 600 + i) for i, (n, s) in enumerate(sizes)]
    d_ins = [torch.from_numpy(x).cuda() for x in xs]
    outs = [torch.zeros(x.size, dtype=torch.int32, device="cuda") for x in xs]
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        cap = torch.cuda.current_stream().cuda_stream
        for (n, s), d_in, out in zip(sizes, d_ins, outs):
            B.check(B.tcu_scan_inclusive(d_in, out, n, 0, s, runner.ws_ptr, runner.ws_bytes, cap))
    for replay in range(3):
        for out in outs:
            out.fill_(-1)
        graph.replay()
        torch.cuda.synchronize()
        B.check(B.tcu_scan_device_status(runner.ws_ptr, 0))
        for x, out in zip(xs, outs):
            assert np.array_equal(out.cpu().numpy(), so.scan(x, "i8")["y32"]), f"replay {replay}"
    del graph


def test_many_back_to_back_launches_agree(runner):
    # consecutive launches overlap their set-up with the previous kernel's tail and reuse one workspace:
    # every one of them must reproduce the integers of the first, whatever the number of CTAs
    from paper_2411_17887_b200 import binding as B
    from oracle import scan_oracle as so
    from tests.gpu_util import to_device
    n = 600 * TILE + 77
    x = gen("i8", n, 123)
    ref = torch.from_numpy(so.scan(x, "i8")["y32"]).cuda()
    d_in = to_device(x, "i8")
    outs = [torch.empty(n, dtype=torch.int32, device="cuda") for _ in range(4)]
    for it in range(120):
        out = outs[it % 4]
        B.check(B.tcu_scan_ex(d_in, out, 1, n, B.TCU_I8_I32, 16, runner.ws_ptr, runner.ws_bytes, 0,
                              max_ctas=[0, 5, 77, 148][it // 30]))
        if it % 4 == 3:
            for o in outs:
                assert torch.equal(o, ref)
                o.fill_(-1)
    B.check(B.tcu_scan_device_status(runner.ws_ptr, 0))
