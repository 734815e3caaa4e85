"""Pins for the instrumented model of the paper's matrix recursion
(oracle/tcu_model.py): the worked example the paper prints, closed forms,
bounds of Lemma 1 / Theorem 1 / Corollary 1, and invariants from the
correctness proof."""
import math
import os

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

from oracle import tcu_model as tm

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def fig1a_rows():
    rows = []
    with open(os.path.join(GOLDEN, "fig1a_s4.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                rows.append([int(v) for v in line.split()])
    return rows


def test_constant_matrices():
    # L_s w is the prefix sum of w; B_s [alpha; q] = [alpha; q + alpha]  (Section 2)
    w = np.array([3, -1, 4, 1, -5])
    assert (tm.L_matrix(5) @ w).tolist() == [3, 2, 6, 7, 2]
    assert (tm.B_matrix(5) @ w).tolist() == [3, 2, 7, 4, -2]
    assert tm.B_matrix(4).tolist() == [[1, 0, 0, 0], [1, 1, 0, 0], [1, 0, 1, 0], [1, 0, 0, 1]]
    # for s = 2 the two coincide (the Brent-Kung special case)
    assert np.array_equal(tm.B_matrix(2), tm.L_matrix(2))


def test_figure_1a_every_round():
    rows = fig1a_rows()
    trace = []
    c = tm.Counters(4)
    out = tm.matmul_scan(np.array(rows[0]), 4, c, trace)
    assert [t.tolist() for t in trace] == rows[1:]
    assert out.tolist() == rows[3]
    assert c.rounds == 3 and c.matmuls == [1, 1, 1]


def test_batch_matmul_with_L2_pairs():
    # With s = 2 every column of a chunk is a pair (a, b) and L_2 (a, b) = (a, a + b):
    # the situation of the paper's Figure 2 (y = 1..16, A = L_2), worked by hand.
    y = np.arange(1, 17)
    z = tm.batch_matmul(y, tm.L_matrix(2))
    want = y.copy()
    want[1::2] = y[0::2] + y[1::2]
    assert z.tolist() == want.tolist()
    assert z.tolist() == [1, 3, 3, 7, 5, 11, 7, 15, 9, 19, 11, 23, 13, 27, 15, 31]


def test_batch_matmul_is_columnwise_and_drops_padding():
    # chunk view: consecutive runs of s entries are the columns; L_s scans each run
    s = 3
    y = np.array([5, 1, 2, 7, 7, 7, 1, 0, -1, 4, 4])          # m = 11: pads to 18, 2 products
    c = tm.Counters(s)
    z = tm.batch_matmul(y, tm.L_matrix(s), c)
    assert z.tolist() == [5, 6, 8, 7, 14, 21, 1, 1, 0, 4, 8]
    assert c.matmuls == [2] and c.stacked_cols == [4]
    # a non-symmetric, non-triangular matrix catches a transposed operand or a row-major view
    A = np.array([[0, 1, 0], [0, 0, 1], [2, 0, 0]])
    z2 = tm.batch_matmul(np.arange(1, 10), A)
    assert z2.tolist() == [2, 3, 2, 5, 6, 8, 8, 9, 14]


@pytest.mark.parametrize("s,k", [(2, 1), (2, 4), (2, 7), (3, 3), (4, 2), (4, 4), (5, 3), (16, 2), (16, 3)])
def test_lemma1_depth_and_products(s, k):
    n = s ** k
    rng = np.random.default_rng(s * 100 + k)
    x = rng.integers(-50, 50, size=n)
    c = tm.Counters(s)
    out = tm.matmul_scan(x, s, c)
    assert np.array_equal(out, np.cumsum(x))
    assert c.rounds == 2 * k - 1                                    # Lemma 1: depth 2k - 1
    closed = 2 * (s ** (k - 1) - 1) // (s - 1) + 1                  # telescoped sum of ceil(n/s^(t+2))...
    assert c.total_matmuls == closed
    assert c.total_matmuls <= tm.lemma1_matmul_bound(n, s)          # Lemma 1 bound
    # work: ceil(n(1 + s/2)) + O(s^3 log_s n)
    assert c.useful_adds <= math.ceil(n * (1 + s / 2)) + s ** 3 * max(k, 1)
    # Theorem 1: time O(n + l k): with the stacked view every round costs s ceil(m/s) + l
    lat = 1000
    assert c.tcu_time(lat) == c.tcu_time(0) + lat * (2 * k - 1)
    assert c.tcu_time(0) <= 4 * n + 2 * s * k


@pytest.mark.parametrize("s,k", [(3, 1), (3, 4), (4, 3), (5, 3), (7, 2), (16, 2), (16, 3)])
def test_exact_work_of_both_sweeps(s, k):
    # Additions on real data, counted from the structure of Algorithm 1 (proof of Lemma 1) for n = s^k.
    # Up-sweep round t scans n / s^(t+1) full groups of s entries, s(s-1)/2 additions each: in total
    # (s-1)/2 * (n + n/s + ... + s) = s (n - 1) / 2.  Down-sweep round t works on the block ends of size
    # s^(t-1) from position s^t - 1 on, s^(k-t+1) - s + 1 of them: s^(k-t) - 1 full groups, in each of which
    # B_s adds the leading prefix to the other s - 1 entries, and one entry left over.  Summed over
    # t = 1 .. k-1: (s-1) * sum_j (s^j - 1) = n - s - (k-1)(s-1).
    n = s ** k
    c_up, c_all = tm.Counters(s), tm.Counters(s)
    tm.matmul_scan(np.ones(n, dtype=np.int64), s, c_up, up_sweep_only=True)
    tm.matmul_scan(np.ones(n, dtype=np.int64), s, c_all)
    assert c_up.useful_adds == s * (n - 1) // 2
    assert c_all.useful_adds - c_up.useful_adds == n - s - (k - 1) * (s - 1)      # the B_s rounds alone, exactly
    # a scan needs at least n - 1 additions, and the lemma's bound holds
    assert n - 1 <= c_all.useful_adds <= math.ceil(n * (1 + s / 2)) + s ** 3 * k


def test_constant_matrices_entry_by_entry():
    for s in (2, 3, 5, 16):
        L, Bm = tm.L_matrix(s), tm.B_matrix(s)
        for i in range(s):
            for j in range(s):
                assert L[i, j] == (1 if j <= i else 0)
                assert Bm[i, j] == (1 if (j == i or j == 0) else 0)


@pytest.mark.parametrize("k", range(1, 11))
def test_s2_work_equals_brent_kung(k):
    # Table 1: Brent-Kung performs 2n - log2(n) - 2 additions, and Algorithm 1 with s = 2 is Brent-Kung
    n = 2 ** k
    c = tm.Counters(2)
    tm.matmul_scan(np.ones(n, dtype=np.int64), 2, c)
    assert c.useful_adds == 2 * n - k - 2
    assert c.rounds == 2 * k - 1                                    # Table 1: depth 2 log2 n - 1


@pytest.mark.parametrize("k", range(1, 6))
def test_s4_depth_table1(k):
    n = 4 ** k
    c = tm.Counters(4)
    tm.matmul_scan(np.ones(n, dtype=np.int64), 4, c)
    assert c.rounds == int(math.log2(n)) - 1                        # Table 1: depth log2 n - 1
    assert c.useful_adds <= 3 * n + 64 * k                          # Table 1: work 3n + O(log n)


@pytest.mark.parametrize("s,k", [(2, 5), (3, 3), (4, 3), (16, 2)])
def test_up_sweep_invariant(s, k):
    # From the correctness proof: after up-sweep round t every position p with
    # (p + 1) % s^(t+1) == 0 holds the sum of its aligned block of s^(t+1) entries, and
    # after the whole up-sweep the last entry is the grand total.
    n = s ** k
    x = np.random.default_rng(1).integers(-9, 9, size=n)
    trace = []
    tm.matmul_scan(x, s, None, trace)
    for t in range(k):
        blk = s ** (t + 1)
        state = trace[t]
        for p in range(blk - 1, n, blk):
            assert state[p] == x[p - blk + 1: p + 1].sum()
    assert trace[k - 1][-1] == x.sum()


@pytest.mark.parametrize("s,k", [(2, 6), (3, 4), (4, 3), (16, 2)])
def test_algorithm2_agrees_with_algorithm1(s, k):
    n = s ** k
    x = np.random.default_rng(2).integers(-100, 100, size=n)
    c1, c2 = tm.Counters(s), tm.Counters(s)
    a = tm.matmul_scan(x, s, c1)
    b = tm.matmul_scan_recursive(x, s, c2)
    assert np.array_equal(a, b) and np.array_equal(a, np.cumsum(x))
    assert c1.total_matmuls == c2.total_matmuls
    assert c1.useful_adds == c2.useful_adds


def test_float_model_matches_definition_closely():
    x = np.random.default_rng(3).uniform(-1, 1, size=4 ** 5)
    out = tm.matmul_scan(x, 4)
    ref = np.cumsum(x)
    assert np.max(np.abs(out - ref)) <= 1e-12 * np.cumsum(np.abs(x))[-1]


def test_base_s_segments():
    assert tm.base_s_segments(2 ** 26, 16) == [16 ** 6] * 4
    assert tm.base_s_segments(2 ** 26, 128) == [128 ** 3] * 32
    assert tm.base_s_segments(27, 4) == [16, 4, 4, 1, 1, 1]
    assert tm.base_s_segments(5, 16) == [1] * 5


@settings(max_examples=60, deadline=None)
@given(st.integers(2, 9), st.integers(1, 700), st.integers(0, 2 ** 31))
def test_general_length_scan(s, n, seed):
    x = np.random.default_rng(seed).integers(-1000, 1000, size=n)
    c = tm.Counters(s)
    y, rep = tm.matmul_scan_general(x, s, c)
    assert np.array_equal(y, np.cumsum(x))
    counts = tm.model_counts(n, s)
    assert counts.total_matmuls == rep.total_matmuls == c.total_matmuls
    assert counts.depth == rep.depth == c.rounds
    # Corollary 1: depth <= 2 floor(log_s n) whenever the scan of the totals fits beside the
    # down-sweep (2q <= k_1); O(n/s^2) products with the constants of Section 2.2
    if len(rep.segments) > 1 and 2 * rep.q <= rep.k1:
        assert rep.depth <= tm.corollary1_depth_bound(n, s)
    k1 = max(rep.k1, 1)
    assert rep.total_matmuls <= math.ceil(4 * n / (s * (s - 1))) + 4 * s * k1 * k1 + 4


def test_counts_at_build_sizes():
    # n = s^k: depth 2k-1, products 2(s^(k-1)-1)/(s-1)+1, within Lemma 1's bound
    for k, bound in [(4, 553), (6, 139821), (7, 2236975)]:
        n = 16 ** k
        r = tm.model_counts(n, 16)
        assert r.depth == 2 * k - 1
        assert r.total_matmuls == 2 * (16 ** (k - 1) - 1) // 15 + 1
        assert tm.lemma1_matmul_bound(n, 16) == bound and r.total_matmuls <= bound
        assert r.total_matmuls >= n // 256                        # at least the n/s^2 level-0 products
    # n = 2^26 through Section 2.2: mu segments of s^k1, one product for their totals, and
    # ceil(s^k1 / (s(s-1))) products per carried segment
    n = 2 ** 26
    for s, k1, mu in [(16, 6, 4), (64, 4, 4), (128, 3, 32)]:
        r = tm.model_counts(n, s)
        per_seg = 2 * (s ** (k1 - 1) - 1) // (s - 1) + 1
        carry = -(-(s ** k1) // (s * (s - 1)))
        assert r.segments == [s ** k1] * mu and r.q == 1
        assert r.total_matmuls == mu * per_seg + 1 + (mu - 1) * carry
        assert r.depth == 2 * k1 == tm.corollary1_depth_bound(n, s)   # Corollary 1 met with equality
        assert r.total_matmuls <= math.ceil(4 * n / (s * (s - 1))) + s * k1 * k1
        assert r.total_matmuls < 4 * n // (s * s)                  # O(n/s^2) with a small constant
    assert tm.model_counts(n, 16).total_matmuls == 768963
    assert tm.model_counts(n, 64).total_matmuls == 45779
    assert tm.model_counts(n, 128).total_matmuls == 12319
