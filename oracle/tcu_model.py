"""Instrumented CPU model of the paper's matrix-multiplication scan.

TEST INFRASTRUCTURE ONLY.  It shares no code with the CUDA library.

The model follows the paper's algorithms step by step, in the paper's order
and notation, with literal dense s x s matrix products (``numpy.matmul`` is the
one library primitive used, as the tensor-unit step), and counts

* ``rounds``            - depth: batched-product rounds on the critical path,
* ``matmuls``           - s x s products, one list entry per executed round,
* ``useful_adds``       - scalar additions whose operands are both real data
                          (padding zeros and structural zeros of the constant
                          matrices excluded), the quantity Lemma 1 calls work,
* ``tcu_time(l)``       - model time with the stacked s x ceil(m/s) view of
                          Theorem 1: every round costs s*ceil(m/s) + l.

Passages followed:

* BatchMatMul          - Algorithm 1, second procedure, and the paragraph after
                         Figure 2 (chunks of s*s entries, each viewed as an
                         s x s matrix in column-major layout, pre-multiplied by
                         the constant matrix, flattened back the same way).
* MatMulScan           - Algorithm 1, first procedure (up-sweep with L_s on the
                         slices x[s^t-1 :: s^t], down-sweep with B_s on the
                         slices x[s^t-1 :: s^(t-1)]).
* MatMulScanRecursive  - Algorithm 2 (appendix).
* arbitrary length     - Section 2.2, steps 1-4.

Readings taken where the text leaves a choice (each is also listed in the
design notes of the repository):

* The constant matrix multiplies from the left (Section 2 describes the local
  prefix sum as L_s applied to a column vector w).
* Slice lengths are the true lengths ceil((n - start)/step); the floor
  expressions in the proof of Lemma 1 are one short for some t, which does not
  affect the lemma's bounds.
* Products are counted with the tensor view, ceil(m/s^2) per round (Lemma 1);
  latency is counted with the stacked view, one invocation per round
  (Theorem 1).
* Section 2.2 step 2 asks for the largest value of each segment; the value meant
  is the last entry of the segment after its up-sweep, i.e. the segment total
  (a literal maximum would be wrong for signed input).
* Section 2.2 step 3: q is the smallest integer with (actual number of
  segments) <= s^q, rather than the worst case k_1 (s-1) <= s^q.
* Section 2.2 step 4: a segment of length m that receives a carry is viewed as
  (s-1) x ceil(m/(s-1)) column-major with the carry prepended as row 0, which
  costs ceil(m / (s (s-1))) products; the first segment receives no carry.
* Depth of the general case: the scan of the segment totals (2q-1 rounds)
  starts after the up-sweep of the largest segments (k_1 rounds) and runs
  beside their down-sweep (k_1-1 rounds); step 4 adds one round.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np


# --------------------------------------------------------------------------- constants
def L_matrix(s: int, dtype=np.int64) -> np.ndarray:
    """L_s: entry (i, j) is 1 when j <= i, else 0 (Section 1, notation): L_s w is the
    inclusive prefix sum of a column vector w."""
    i, j = np.indices((s, s))
    return (j <= i).astype(dtype)


def B_matrix(s: int, dtype=np.int64) -> np.ndarray:
    """B_s: entry (i, j) is 1 on the diagonal and in column 0, else 0 (displayed equation
    of Section 2): B_s [alpha; q] = [alpha; q + alpha 1], the scalar/vector add."""
    i, j = np.indices((s, s))
    return ((j == i) | (j == 0)).astype(dtype)


# --------------------------------------------------------------------------- counters
@dataclass
class Counters:
    s: int
    rounds: int = 0
    matmuls: List[int] = field(default_factory=list)      # per executed BatchMatMul call
    stacked_cols: List[int] = field(default_factory=list)  # ceil(m/s) per call (Theorem 1 view)
    useful_adds: int = 0

    @property
    def total_matmuls(self) -> int:
        return int(sum(self.matmuls))

    def tcu_time(self, latency: int) -> int:
        """Sum over calls of s*ceil(m/s) + latency (proof of Theorem 1)."""
        return int(sum(self.s * c + latency for c in self.stacked_cols))


def _is_L(A: np.ndarray) -> bool:
    return bool(np.array_equal(A, L_matrix(A.shape[0], A.dtype)))


# --------------------------------------------------------------------------- BatchMatMul
def batch_matmul(y: np.ndarray, A: np.ndarray, counters: Optional[Counters] = None) -> np.ndarray:
    """BatchMatMul(y, A_s) of Algorithm 1.

    m = len(y); zero-pad to s^2 * ceil(m/s^2); chunk c becomes the matrix T_c
    whose column j is y[c s^2 + j s : c s^2 + (j+1) s]; W_c = A T_c; the result
    is W flattened with the same column-major rule, padding dropped.
    """
    s = A.shape[0]
    m = int(len(y))
    if m == 0:
        return np.array(y, copy=True)
    chunks = -(-m // (s * s))
    padded = np.zeros(chunks * s * s, dtype=np.result_type(y.dtype, A.dtype))
    padded[:m] = y
    # T[c, i, j] = padded[c s^2 + j s + i]   (column-major chunk view)
    T = np.empty((chunks, s, s), dtype=padded.dtype)
    for c in range(chunks):
        for j in range(s):
            T[c, :, j] = padded[c * s * s + j * s: c * s * s + (j + 1) * s]
    W = np.matmul(A, T)                     # one s x s product per chunk
    z = np.empty_like(padded)
    for c in range(chunks):
        for j in range(s):
            z[c * s * s + j * s: c * s * s + (j + 1) * s] = W[c, :, j]
    if counters is not None:
        counters.matmuls.append(chunks)
        counters.stacked_cols.append(-(-m // s))
        # additions on real data only: a column holding v real entries costs
        # v(v-1)/2 with L_s (prefix sums) and v-1 with B_s (alpha added to the rest)
        full_cols, rem = divmod(m, s)
        if _is_L(A):
            counters.useful_adds += full_cols * (s * (s - 1) // 2) + rem * (rem - 1) // 2
        else:
            counters.useful_adds += full_cols * (s - 1) + max(rem - 1, 0)
    return z[:m]


# --------------------------------------------------------------------------- Algorithm 1
def exact_log(n: int, s: int) -> Optional[int]:
    """k with s**k == n, or None."""
    k, p = 0, 1
    while p < n:
        p *= s
        k += 1
    return k if p == n else None


@dataclass(frozen=True)
class Round:
    """One batched-product round of Algorithm 1: the sub-vector x[first::stride] is replaced by
    BatchMatMul(sub-vector, operand), operand being "L" (up-sweep) or "B" (down-sweep)."""
    first: int
    stride: int
    operand: str


def algorithm1_rounds(k: int, s: int) -> List[Round]:
    """The schedule of Algorithm 1 for n = s^k.  Up-sweep, level t = 0 .. k-1: the entries that end a
    block of s^t elements (positions s^t - 1, 2 s^t - 1, ...) are scanned in groups of s.  Down-sweep,
    level t = k-1 .. 1: starting at the end of the first block of s^t elements, the entries that end a
    block of s^(t-1) elements are taken; every group of s begins with a finished prefix, which B_s adds
    to the s - 1 block ends behind it."""
    up = [Round(s ** t - 1, s ** t, "L") for t in range(k)]
    down = [Round(s ** t - 1, s ** (t - 1), "B") for t in range(k - 1, 0, -1)]
    return up + down


def matmul_scan(x: np.ndarray, s: int, counters: Optional[Counters] = None,
                trace: Optional[list] = None, up_sweep_only: bool = False,
                count_rounds: bool = True) -> np.ndarray:
    """MatMulScan(x, s) of Algorithm 1 for len(x) = s^k.  Returns a new array.

    ``trace`` (a list) receives a copy of x after every round.
    """
    state = np.array(x, copy=True)
    k = exact_log(len(state), s)
    if k is None:
        raise ValueError(f"Algorithm 1 needs len(x) = s^k, got n={len(state)}, s={s}")
    operands = {"L": L_matrix(s, state.dtype), "B": B_matrix(s, state.dtype)}
    for rnd in algorithm1_rounds(k, s):
        if up_sweep_only and rnd.operand == "B":
            break
        picked = slice(rnd.first, None, rnd.stride)
        state[picked] = batch_matmul(state[picked], operands[rnd.operand], counters)
        if counters is not None and count_rounds:
            counters.rounds += 1
        if trace is not None:
            trace.append(state.copy())
    return state


# --------------------------------------------------------------------------- Algorithm 2
def matmul_scan_recursive(x: np.ndarray, s: int, counters: Optional[Counters] = None) -> np.ndarray:
    """MatMulScanRecursive(x, s) of Algorithm 2: local scans of all chunks first, then the recursive
    procedure on the result.  Rounds are not counted here (the recursion interleaves them); products
    and additions are."""
    x = np.asarray(x)
    local = batch_matmul(np.array(x, copy=True), L_matrix(s, x.dtype), counters)
    return _finish_from_chunk_scans(local, s, counters)


def _finish_from_chunk_scans(v: np.ndarray, s: int, counters: Optional[Counters]) -> np.ndarray:
    """Algorithm 2's recursive procedure.  On entry every chunk of s entries of v holds its own scan,
    so the chunk totals sit at positions s-1, 2s-1, ...  A vector of at most s entries is already done.
    Otherwise: scan the chunk totals (their own chunk scans by one product, the rest by recursion),
    write them back, and let B_s add each finished total to the s - 1 entries that follow it."""
    if len(v) <= s:
        return v
    ends = slice(s - 1, None, s)
    totals = batch_matmul(v[ends], L_matrix(s, v.dtype), counters)
    v[ends] = _finish_from_chunk_scans(totals, s, counters)
    v[s - 1:] = batch_matmul(v[s - 1:], B_matrix(s, v.dtype), counters)
    return v


# --------------------------------------------------------------------------- Section 2.2
def base_s_segments(n: int, s: int) -> List[int]:
    """Segment lengths of Section 2.2: n = sum_i mu_i s^{k_i}, largest power first,
    mu_i segments of length s^{k_i} each, laid out left to right."""
    segs: List[int] = []
    k1 = 0
    while s ** (k1 + 1) <= n:
        k1 += 1
    rest = n
    for k in range(k1, -1, -1):
        mu, rest = divmod(rest, s ** k)
        segs.extend([s ** k] * mu)
    assert sum(segs) == n
    return segs


@dataclass
class GeneralReport:
    segments: List[int]
    k1: int
    q: int
    depth: int
    matmuls_step1: int
    matmuls_step3: int
    matmuls_step4: int

    @property
    def total_matmuls(self) -> int:
        return self.matmuls_step1 + self.matmuls_step3 + self.matmuls_step4


def matmul_scan_general(x: np.ndarray, s: int, counters: Optional[Counters] = None):
    """Scan of arbitrary length by the four steps of Section 2.2.

    Returns (result, GeneralReport).  For len(x) = s^k this is Algorithm 1.
    """
    x = np.array(x, copy=True)
    n = len(x)
    if n == 0:
        return x, GeneralReport([], 0, 0, 0, 0, 0, 0)
    segs = base_s_segments(n, s)
    k1 = exact_log(segs[0], s)
    own = counters if counters is not None else Counters(s)
    before = own.total_matmuls

    if len(segs) == 1:
        out = matmul_scan(x, s, own, count_rounds=False)
        depth = max(2 * k1 - 1, 0)
        own.rounds += depth
        return out, GeneralReport(segs, k1, 0, depth, own.total_matmuls - before, 0, 0)

    # step 1: Algorithm 1 on every segment (in parallel in the model: depth = the largest)
    bounds = np.concatenate(([0], np.cumsum(segs)))
    w = np.zeros(len(segs), dtype=x.dtype)
    for i, m in enumerate(segs):
        lo, hi = int(bounds[i]), int(bounds[i + 1])
        # step 2: the segment total is the last entry once the segment's up-sweep is done
        after_up = matmul_scan(x[lo:hi], s, None, up_sweep_only=True)
        w[i] = after_up[-1]
        x[lo:hi] = matmul_scan(x[lo:hi], s, own, count_rounds=False)
    m1 = own.total_matmuls - before

    # step 3: scan the totals, zero-padded to s^q
    q = 1
    while s ** q < len(segs):
        q += 1
    wpad = np.zeros(s ** q, dtype=x.dtype)
    wpad[:len(segs)] = w
    wscan = matmul_scan(wpad, s, own, count_rounds=False)[:len(segs)]
    m3 = own.total_matmuls - before - m1

    # step 4: broadcast-add w_i onto segment i+1 with B_s, carry prepended as row 0
    Bs = B_matrix(s, x.dtype)
    m4 = 0
    for i in range(len(segs) - 1):
        lo, hi = int(bounds[i + 1]), int(bounds[i + 2])
        seg = x[lo:hi]
        m = len(seg)
        cols = -(-m // (s - 1))
        y = np.zeros(cols * s, dtype=x.dtype)
        for c in range(cols):
            piece = seg[c * (s - 1):(c + 1) * (s - 1)]
            y[c * s] = wscan[i]
            y[c * s + 1: c * s + 1 + len(piece)] = piece
        z = batch_matmul(y, Bs, None)
        for c in range(cols):
            piece_len = min(s - 1, m - c * (s - 1))
            seg[c * (s - 1): c * (s - 1) + piece_len] = z[c * s + 1: c * s + 1 + piece_len]
        prods = -(-cols // s)
        m4 += prods
        own.matmuls.append(prods)
        own.stacked_cols.append(cols)
        own.useful_adds += m
    depth = k1 + max(k1 - 1, 2 * q - 1) + 1
    own.rounds += depth
    return x, GeneralReport(segs, k1, q, depth, m1, m3, m4)


# --------------------------------------------------------------------------- closed forms
def lemma1_matmul_bound(n: int, s: int) -> int:
    """ceil(2n / (s(s-1))) + 2k - 2 of Lemma 1, for n = s^k."""
    k = exact_log(n, s)
    return -(-2 * n // (s * (s - 1))) + 2 * k - 2


def corollary1_depth_bound(n: int, s: int) -> int:
    """2 floor(log_s n) of Corollary 1."""
    k1 = 0
    while s ** (k1 + 1) <= n:
        k1 += 1
    return 2 * k1


# --------------------------------------------------------------------------- counts without data
def _alg1_call_lengths(n: int, s: int) -> List[int]:
    """Lengths m of the vectors handed to BatchMatMul by Algorithm 1, in order (the number of
    positions first, first + stride, ... below n)."""
    return [-(-(n - rnd.first) // rnd.stride) for rnd in algorithm1_rounds(exact_log(n, s), s)]


def model_counts(n: int, s: int) -> GeneralReport:
    """Depth and product counts of the model for length n, walking the same
    rounds as ``matmul_scan_general`` but with vector lengths only (no data), so
    that the counts can be evaluated at sizes the data-carrying model cannot
    reach.  Tests check that the two agree wherever both run."""
    segs = base_s_segments(n, s)
    k1 = exact_log(segs[0], s)

    def alg1_products(m: int) -> int:
        return sum(-(-l // (s * s)) for l in _alg1_call_lengths(m, s))

    if len(segs) == 1:
        return GeneralReport(segs, k1, 0, max(2 * k1 - 1, 0), alg1_products(n), 0, 0)
    m1 = sum(alg1_products(m) for m in segs)
    q = 1
    while s ** q < len(segs):
        q += 1
    m3 = alg1_products(s ** q)
    m4 = sum(-(-(-(-m // (s - 1))) // s) for m in segs[1:])
    depth = k1 + max(k1 - 1, 2 * q - 1) + 1
    return GeneralReport(segs, k1, q, depth, m1, m3, m4)
