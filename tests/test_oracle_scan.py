"""Pins for the result oracle (oracle/scan_oracle.*): things fixed by the
mathematics, not by the oracle itself."""
import itertools

import numpy as np
import pytest
import torch

from oracle import scan_oracle as so
from paper_2411_17887_b200 import inputs


def brute_inclusive(x):
    """O(n^2) double loop straight from y_i = sum_{j<=i} x_j, Python ints / floats."""
    out = []
    for i in range(len(x)):
        acc = 0
        for j in range(i + 1):
            acc = acc + x[j]
        out.append(acc)
    return out


@pytest.mark.parametrize("n", [1, 2, 3, 15, 16, 17, 63, 64])
def test_int_brute_force(n):
    x = inputs.int8_uniform(n, -127, 127, 100 + n)
    want = brute_inclusive([int(v) for v in x])
    got = so.scan_i8(x)
    assert got.tolist() == want
    # exclusive = inclusive shifted right by one with the identity 0 in front
    ex = so.scan_i8(x, exclusive=True)
    assert ex.tolist() == [0] + want[:-1]


@pytest.mark.parametrize("n", [1, 2, 5, 33, 64])
def test_float_brute_force(n):
    x = inputs.f16_uniform(n, -1.0, 1.0, 200 + n)
    xs = [float(v) for v in x]                 # fp16 -> Python float (fp64) is exact
    want = brute_inclusive(xs)                 # same left-to-right order => identical bits
    y, a = so.scan_f64(so.widen(x, "f16"))
    assert y.tolist() == want
    assert a.tolist() == brute_inclusive([abs(v) for v in xs])
    yex, aex = so.scan_f64(so.widen(x, "f16"), exclusive=True)
    assert yex.tolist() == [0.0] + want[:-1]
    assert aex.tolist() == [0.0] + a.tolist()[:-1]


@pytest.mark.parametrize("dtype", ["i8", "f16", "bf16"])
def test_all_ones_gives_i_plus_1(dtype):
    n = 5000
    if dtype == "i8":
        x = np.ones(n, np.int8)
    elif dtype == "f16":
        x = np.ones(n, np.float16)
    else:
        x = np.full(n, 0x3F80, np.uint16)      # 1.0 in bfloat16
    r = so.scan(x, dtype)
    assert np.array_equal(r["y"], np.arange(1, n + 1))
    rex = so.scan(x, dtype, exclusive=True)
    assert np.array_equal(rex["y"], np.arange(0, n))


def test_last_element_is_total_and_matches_library_cumsum():
    x = inputs.int8_uniform(100_003, -127, 127, 7)
    y = so.scan_i8(x)
    assert int(y[-1]) == int(x.astype(np.int64).sum())
    assert np.array_equal(y, np.cumsum(x.astype(np.int64)))
    xf = inputs.f16_uniform(100_003, -1.0, 1.0, 8)
    yf, a = so.scan_f64(so.widen(xf, "f16"))
    # numpy's cumsum is the same sequential recurrence in fp64
    assert np.array_equal(yf, np.cumsum(xf.astype(np.float64)))
    assert np.array_equal(a, np.cumsum(np.abs(xf.astype(np.float64))))
    # the total agrees with an exactly rounded sum to fp64 accuracy
    import math
    assert abs(yf[-1] - math.fsum(float(v) for v in xf)) <= 1e-9


def test_init_carries_over_chunks():
    x = inputs.int8_uniform(1000, -8, 8, 9)
    whole = so.scan_i8(x)
    first = so.scan_i8(x[:400])
    second = so.scan_i8(x[400:], init=int(first[-1]))
    assert np.array_equal(np.concatenate([first, second]), whole)


def test_rows_are_independent():
    x = inputs.int8_uniform((7, 129), -8, 8, 10)
    y = so.scan_i8(x)
    for r in range(7):
        assert np.array_equal(y[r], np.cumsum(x[r].astype(np.int64)))
    xb = inputs.bf16_normal((5, 77), 11)
    wide = so.bf16_bits_to_f64(xb)
    yb, ab = so.scan_f64(so.widen(xb, "bf16"))
    for r in range(5):
        assert np.array_equal(yb[r], np.cumsum(wide[r]))
        # the running sum of |x| that scales the tolerance restarts with every row as well
        assert np.array_equal(ab[r], np.cumsum(np.abs(wide[r])))
        assert ab[r][0] == abs(wide[r][0]) and (np.diff(ab[r]) >= 0).all()
    yex, aex = so.scan_f64(so.widen(xb, "bf16"), exclusive=True)
    for r in range(5):
        assert yex[r].tolist() == [0.0] + np.cumsum(wide[r]).tolist()[:-1]
        assert aex[r].tolist() == [0.0] + np.cumsum(np.abs(wide[r])).tolist()[:-1]


def test_float_init_carries_over_pieces():
    # scanning two halves, the second started from the first half's last value, reproduces the whole
    # scan bit for bit (the additions happen in the same order); `a` never includes init
    x = so.widen(inputs.f16_uniform(1000, -1.0, 1.0, 12), "f16")
    whole, a_whole = so.scan_f64(x)
    first, a_first = so.scan_f64(x[:400])
    second, a_second = so.scan_f64(x[400:], init=float(first[-1]))
    assert np.array_equal(np.concatenate([first, second]), whole)
    assert np.array_equal(a_second, np.cumsum(np.abs(x[400:])))
    assert np.allclose(np.concatenate([a_first, a_second + a_first[-1]]), a_whole, rtol=1e-14, atol=0)
    # exclusive form: y[0] is init itself, and the chain continues from init + x[0]
    ex, a_ex = so.scan_f64(x[400:], exclusive=True, init=float(first[-1]))
    assert ex[0] == first[-1] and ex[1] == first[-1] + x[400] and a_ex[0] == 0.0
    assert np.array_equal(ex[1:], second[:-1])
    # a closed form: constant input 0.5 from init 10 is exactly 10 + (i + 1) / 2
    y, a = so.scan_f64(np.full(64, 0.5), init=10.0)
    assert y.tolist() == [10.0 + (i + 1) / 2 for i in range(64)] and a.tolist() == [(i + 1) / 2 for i in range(64)]


def _segments_by_definition(x, offsets, exclusive):
    """Every output computed on its own: the sum over the part of its segment before it (brute force)."""
    out = [0] * len(x)
    for k in range(len(offsets) - 1):
        lo, hi = int(offsets[k]), int(offsets[k + 1])
        for i in range(lo, hi):
            acc = 0
            for j in range(lo, i if exclusive else i + 1):
                acc = acc + x[j]
            out[i] = acc
    return out


@pytest.mark.parametrize("exclusive", [False, True])
def test_segmented_scan_brute_force(exclusive):
    # empty segments, segments of one element, a long one; integer and floating point
    offsets = [0, 0, 1, 1, 4, 20, 20, 21, 64]
    x = inputs.int8_uniform(64, -127, 127, 13)
    r = so.scan_segments(x, "i8", offsets, exclusive)
    assert r["y"].tolist() == _segments_by_definition([int(v) for v in x], offsets, exclusive)
    xf = inputs.f16_uniform(64, -1.0, 1.0, 14)
    rf = so.scan_segments(xf, "f16", offsets, exclusive)
    vals = [float(v) for v in xf]
    assert rf["y"].tolist() == _segments_by_definition(vals, offsets, exclusive)
    assert rf["a"].tolist() == _segments_by_definition([abs(v) for v in vals], offsets, exclusive)
    # one segment is the plain scan; one segment per element gives x itself (inclusive) or zeros (exclusive)
    assert np.array_equal(so.scan_segments(x, "i8", [0, 64], exclusive)["y"], so.scan_i8(x, exclusive))
    single = so.scan_segments(x, "i8", list(range(65)), exclusive)["y"]
    assert np.array_equal(single, np.zeros(64, np.int64) if exclusive else x.astype(np.int64))
    # dense rows are the special case of equal segments
    rows = so.scan_segments(x, "i8", [0, 16, 32, 48, 64], exclusive)["y"]
    assert np.array_equal(rows.reshape(4, 16), so.scan_i8(x.reshape(4, 16), exclusive))


def test_int32_wrap():
    # 2^31 - 1 + 1 wraps to -2^31; sums beyond 32 bits keep only the low word
    y64 = np.array([2**31 - 1, 2**31, 2**32 + 5, -1, -(2**31) - 1], dtype=np.int64)
    assert so.wrap_int32(y64).tolist() == [2**31 - 1, -(2**31), 5, -1, 2**31 - 1]
    # a scan long enough to wrap: 127 * 2^25 > 2^31
    n = 1 << 25
    x = np.full(n, 127, np.int8)
    y = so.scan_i8(x)
    assert int(y[-1]) == 127 * n
    w = so.wrap_int32(y)
    assert int(w[-1]) == ((127 * n + 2**31) % 2**32) - 2**31


def test_bf16_widening_and_rounding_match_torch():
    g = np.random.default_rng(5)
    f = g.standard_normal(10000).astype(np.float32)
    f[:6] = [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.0e38]   # includes exact ties
    bits = inputs.f32_to_bf16_bits(f)
    t = torch.from_numpy(f).bfloat16()
    assert np.array_equal(bits, t.view(torch.int16).numpy().view(np.uint16))
    assert np.array_equal(so.bf16_bits_to_f64(bits), t.double().numpy())


def test_generators_are_seeded_and_in_range():
    a = inputs.make(inputs.CONFIGS["C1"])
    b = inputs.make(inputs.CONFIGS["C1"])
    assert np.array_equal(a, b) and a.min() == -8 and a.max() == 8 and a.dtype == np.int8
    c = inputs.make(inputs.CONFIGS["C3"], (1 << 16,))
    assert c.min() == -127 and c.max() == 127
    d = inputs.make(inputs.CONFIGS["C5"], (1 << 16,))
    assert d.dtype == np.float16 and d.min() >= 0 and d.max() <= 1
    e = inputs.make(inputs.CONFIGS["C2"], (1 << 16,))
    assert e.min() >= -1 and e.max() <= 1 and abs(float(e.astype(np.float64).mean())) < 0.02
    f = so.bf16_bits_to_f64(inputs.make(inputs.CONFIGS["C4"], (64, 1024)))
    assert abs(f.mean()) < 0.02 and abs(f.std() - 1) < 0.02
