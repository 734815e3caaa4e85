"""GPU parity of the segmented scan (caller-given segments inside one array) and of batched rows whose
length is not a multiple of 16 (which take the same path), against the CPU oracle's per-segment loop.
Integers bit for bit; fp32 within 1e-5 * (sum of |x| over the element's own segment so far) + 1e-6."""
import numpy as np
import pytest
import torch

from oracle import scan_oracle as so
from paper_2411_17887_b200 import binding as B
from paper_2411_17887_b200 import inputs

pytestmark = pytest.mark.gpu
TILE = 128 * 128
GUARD = 512


def gen(dtype, n, seed):
    if dtype == "i8":
        return inputs.int8_uniform(n, -127, 127, seed)
    if dtype == "f16":
        return inputs.f16_uniform(n, -1.0, 1.0, seed)
    return inputs.bf16_normal(n, seed)


def run_segmented(x, dtype, offsets, s, exclusive):
    from tests.gpu_util import to_device
    n = x.size
    dt = B.DTYPES[dtype]
    is_int = dtype == "i8"
    sent = -0x5A5A5A5B if is_int else -1.2345e30
    d_in = to_device(x, dtype)
    out = torch.full((n + 2 * GUARD,), sent, dtype=torch.int32 if is_int else torch.float32, device="cuda")
    d_out = out[GUARD:GUARD + n]
    d_off = torch.from_numpy(np.asarray(offsets, dtype=np.int64)).cuda()
    ws_bytes = B.tcu_scan_segmented_workspace_bytes(n, dt, s)
    ws = torch.empty(ws_bytes + 256, dtype=torch.uint8, device="cuda")
    ptr = ws.data_ptr() + (-ws.data_ptr()) % 256
    B.check(B.tcu_scan_workspace_init(ptr, ws_bytes, 0))
    for _ in range(2):                           # twice on the same workspace: stale row notes must not matter
        d_out.fill_(7)
        B.check(B.tcu_scan_segmented(d_in, d_out, n, d_off, len(offsets) - 1, dt, s, int(exclusive), ptr, ws_bytes, 0))
        B.check(B.tcu_scan_device_status(ptr, 0))
    assert B.tcu_scan_last_stats()["segments_path"] == 1
    host = out.cpu().numpy()
    ref_sent = np.int32(sent) if is_int else np.float32(sent)
    assert (host[:GUARD] == ref_sent).all() and (host[GUARD + n:] == ref_sent).all(), "write outside the output"
    return host[GUARD:GUARD + n]


def compare(got, x, dtype, offsets, exclusive):
    ref = so.scan_segments(x, dtype, offsets, exclusive)
    if dtype == "i8":
        if not np.array_equal(got, ref["y32"]):
            bad = np.flatnonzero(got != ref["y32"])
            raise AssertionError(f"{bad.size} mismatches, first at {bad[0]} (row {bad[0] // 128}, col {bad[0] % 128}): "
                                 f"got {got[bad[0]]} want {ref['y32'][bad[0]]}")
    else:
        err = np.abs(got.astype(np.float64) - ref["y"])
        tol = so.float_tolerance(ref["a"])
        if not (err <= tol).all():
            i = int(np.flatnonzero(err > tol)[0])
            raise AssertionError(f"out of tolerance at {i} (row {i // 128}, col {i % 128}): got {got[i]} want {ref['y'][i]}")


def random_offsets(n, mean_len, seed, extra=()):
    """Sorted cut points: geometric-ish lengths around mean_len, plus duplicates (empty segments) and `extra`."""
    g = inputs.rng(seed)
    cuts = np.unique(g.integers(0, n + 1, size=max(1, n // mean_len)))
    dup = cuts[g.integers(0, cuts.size, size=max(1, cuts.size // 10))]
    allc = np.sort(np.concatenate([cuts, dup, np.asarray(extra, dtype=np.int64)]))
    allc = allc[(allc >= 0) & (allc <= n)]
    return np.concatenate([[0], allc, [n]]).astype(np.int64)


@pytest.mark.parametrize("dtype", ["i8", "f16", "bf16"])
@pytest.mark.parametrize("exclusive", [False, True])
def test_random_segments(dtype, exclusive):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    for n, mean_len, s in [(5 * TILE + 128 * 7 + 19, 50, 16), (9 * TILE, 1000, 64), (300 * TILE + 77, 1 << 14, 128),
                           (40 * TILE + 5, 7, 16), (3 * TILE + 127, 1 << 16, 16)]:
        # cut points on tile edges, on row edges, one element apart, at both ends, and inside the incomplete last row
        extra = [TILE, 2 * TILE, 2 * TILE + 1, 128, 256, 129, TILE - 1, n - 1, n, n - (n % 128), 0, 1]
        off = random_offsets(n, mean_len, n % 1009 + mean_len, extra)
        x = gen(dtype, n, 300 + mean_len)
        compare(run_segmented(x, dtype, off, s, exclusive), x, dtype, off, exclusive)


@pytest.mark.parametrize("dtype", ["i8", "f16"])
def test_degenerate_segmentations(dtype):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    n = 2 * TILE + 128 * 3 + 50
    x = gen(dtype, n, 77)
    cases = {
        "one segment (the plain scan)": [0, n],
        "every element its own segment": list(range(n + 1)),
        "only empty segments around one": [0, 0, 0, n, n, n],
        "segments shorter than s": list(range(0, n, 5)) + [n],
        "a start in every row at column 127": [0] + list(range(127, n, 128)) + [n],
        "a start at every row boundary": list(range(0, n, 128)) + [n],
        "tile-sized segments": [0, TILE, 2 * TILE, n],
    }
    for name, off in cases.items():
        for exclusive in (False, True):
            try:
                compare(run_segmented(x, dtype, off, 16, exclusive), x, dtype, off, exclusive)
            except AssertionError as e:
                raise AssertionError(f"{name}, exclusive={exclusive}: {e}")
    # arrays shorter than one row never reach the tile kernel
    for m in (1, 5, 127):
        xs = gen(dtype, m, m)
        off = [0, m // 2, m]
        for exclusive in (False, True):
            compare(run_segmented(xs, dtype, off, 16, exclusive), xs, dtype, off, exclusive)


@pytest.mark.parametrize("dtype", ["i8", "bf16", "f16"])
def test_batched_rows_of_any_length(dtype):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from tests.gpu_util import Runner, check
    runner = Runner(1, 1, ws_bytes=max(B.tcu_scan_workspace_bytes(r, c, 0, 16) for r, c in [(4096, 1001), (5, 3 * TILE + 1)]))
    for rows, cols in [(7, 100), (33, 129), (5, TILE + 1), (1000, 37), (3, 1), (2, 15), (64, 127), (9, 1000), (4096, 1001),
                       (5, 3 * TILE + 1)]:
        for s, exclusive in [(16, False), (128, True)]:
            x = gen(dtype, rows * cols, rows + cols).reshape(rows, cols)
            check(runner, x, dtype, s, exclusive)
            assert runner.stats["segments_path"] == 1 and runner.stats["rows"] == rows and runner.stats["cols"] == cols
    check(runner, gen(dtype, 8 * 160, 1).reshape(8, 160), dtype, 16)       # multiples of 16 keep the dense-row path
    assert runner.stats["segments_path"] == 0


def test_segmented_argument_checks():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    d = torch.zeros(1024, dtype=torch.int8, device="cuda")
    o = torch.zeros(1024, dtype=torch.int32, device="cuda")
    off = torch.tensor([0, 1024], dtype=torch.int64, device="cuda")
    ws_bytes = B.tcu_scan_segmented_workspace_bytes(1024, 0, 16)
    # beside the tile records: one flag byte and one 4-byte value per row of 128 elements
    assert B.tcu_scan_segmented_workspace_bytes(1 << 24, 0, 16) >= 256 + 5 * ((1 << 24) // 128) + 16 * ((1 << 24) // TILE)
    ws = torch.zeros(ws_bytes + 256, dtype=torch.uint8, device="cuda")
    ptr = ws.data_ptr() + (-ws.data_ptr()) % 256
    assert B.tcu_scan_segmented(d, o, 1024, None, 1, 0, 16, 0, ptr, ws_bytes, 0) == B.TCU_ERR_INVALID_ARG
    assert B.tcu_scan_segmented(d, o, 1024, off, 0, 0, 16, 0, ptr, ws_bytes, 0) == B.TCU_ERR_INVALID_ARG
    assert B.tcu_scan_segmented(d, o, 1024, off, 1, 0, 16, 0, ptr, ws_bytes - 64, 0) == B.TCU_ERR_WORKSPACE
    assert B.tcu_scan_segmented(d, o, 0, off, 0, 0, 16, 0, ptr, ws_bytes, 0) == B.TCU_OK
    assert B.tcu_scan_segmented(d, o, 1024, off, 1, 0, 48, 0, ptr, ws_bytes, 0) == B.TCU_ERR_UNSUPPORTED


def test_row_notes_of_a_small_segmented_scan_never_read_as_records_of_a_later_larger_scan():
    # One workspace, sized for the larger problem, is used by a small segmented scan and then by a large plain scan.  The
    # row notes of the first lie where the second keeps its tile records.  The notes are chosen so that, read as records,
    # they would carry the epoch of the second launch and the status "inclusive": rows 4i hand on 4 * 2 + 2 = 10 (one
    # start at column 118 of an all-ones row), rows 4i + 1 hold no start, rows 4i + 2 hand on 28.  The library wipes its
    # notes before it returns the workspace, so the large scan must come out right.
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    n_small, n_big = 64 * TILE, 3000 * TILE + 77
    ws_bytes = max(B.tcu_scan_workspace_bytes(1, n_big, 0, 16), B.tcu_scan_segmented_workspace_bytes(n_small, 0, 16))
    ws = torch.empty(ws_bytes + 256, dtype=torch.uint8, device="cuda")
    ptr = ws.data_ptr() + (-ws.data_ptr()) % 256
    big = inputs.int8_uniform(n_big, -127, 127, 5)
    d_big = torch.from_numpy(big).cuda()
    want = so.scan(big, "i8")["y32"]
    rows = n_small // 128
    starts = np.concatenate([np.arange(0, rows, 4) * 128 + 118, np.arange(2, rows, 4) * 128 + 100])
    offsets = np.concatenate([[0], np.sort(starts), [n_small]]).astype(np.int64)
    ones = np.ones(n_small, dtype=np.int8)
    d_ones = torch.from_numpy(ones).cuda()
    d_off = torch.from_numpy(offsets).cuda()
    for trial in range(3):
        B.check(B.tcu_scan_workspace_init(ptr, ws_bytes, 0))              # epoch 0: the next two launches use epochs 1 and 2
        o_small = torch.empty(n_small, dtype=torch.int32, device="cuda")
        B.check(B.tcu_scan_segmented(d_ones, o_small, n_small, d_off, len(offsets) - 1, 0, 16, 0, ptr, ws_bytes, 0))
        o_big = torch.empty(n_big, dtype=torch.int32, device="cuda")
        B.check(B.tcu_scan_inclusive(d_big, o_big, n_big, 0, 16, ptr, ws_bytes, 0))
        B.check(B.tcu_scan_device_status(ptr, 0))
        compare(o_small.cpu().numpy(), ones, "i8", offsets, False)
        got = o_big.cpu().numpy()
        assert np.array_equal(got, want), f"trial {trial}: first mismatch at {int(np.flatnonzero(got != want)[0])}"


def test_one_workspace_shared_by_calls_of_every_kind_and_size():
    # scans of different kinds leave different things in the workspace (records, row notes, the scratch of the two-sweep
    # variant); whatever order they come in, on one workspace sized for the largest, every result must be right
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from tests.gpu_util import to_device
    g = inputs.rng(99)
    n_max = 700 * TILE + 55
    ws_bytes = max(B.tcu_scan_workspace_bytes(1, n_max, 0, 16), B.tcu_scan_segmented_workspace_bytes(n_max, 0, 16))
    ws = torch.empty(ws_bytes + 256, dtype=torch.uint8, device="cuda")
    ptr = ws.data_ptr() + (-ws.data_ptr()) % 256
    B.check(B.tcu_scan_workspace_init(ptr, ws_bytes, 0))
    for it in range(48):
        kind = ["plain", "segmented", "two_sweep_scanned_totals", "plain", "two_sweep"][it % 5]
        n = int(g.integers(1, n_max)) if it % 3 else int(g.choice([n_max, 148 * TILE, 3 * TILE + 1, 127]))
        dtype = ["i8", "f16", "bf16"][int(g.integers(0, 3))]
        s = int(g.choice([16, 64, 128]))
        exclusive = bool(g.integers(0, 2))
        x = gen(dtype, n, 1000 + it)
        d_in = to_device(x, dtype)
        out = torch.empty(n, dtype=torch.int32 if dtype == "i8" else torch.float32, device="cuda")
        dt = B.DTYPES[dtype]
        if kind == "segmented":
            off = random_offsets(n, int(g.choice([5, 300, 20000])), it)
            B.check(B.tcu_scan_segmented(d_in, out, n, torch.from_numpy(off).cuda(), len(off) - 1, dt, s, int(exclusive), ptr, ws_bytes, 0))
        else:
            off = np.array([0, n], dtype=np.int64)
            opts = {"two_sweep": dict(variant=1), "two_sweep_scanned_totals": dict(variant=1, upper_level_path=1)}.get(kind, {})
            B.check(B.tcu_scan_ex(d_in, out, 1, n, dt, s, ptr, ws_bytes, 0, exclusive=int(exclusive), **opts))
        B.check(B.tcu_scan_device_status(ptr, 0))
        try:
            compare(out.cpu().numpy(), x, dtype, off, exclusive)
        except AssertionError as e:
            raise AssertionError(f"call {it} ({kind}, n={n}, {dtype}, s={s}, exclusive={exclusive}): {e}")
