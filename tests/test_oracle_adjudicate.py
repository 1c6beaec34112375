"""Pins for the oracle's timing adjudication (CPU only).

The paper names an "adjudicated latency" (Algorithm 1) and shows that timing
tails reorder close candidates (Appendix, Relative Variability Metrics) but
prints no statistic.  The reading: per-candidate median and IQR by the linear
(type-7) quantile, and pairwise doubled Mann-Whitney win counts.  Pins: a
hand-checkable example, scipy's mannwhitneyu, numpy.percentile, brute force in
Python integers, and the identities the statistic must satisfy.
"""
import itertools
from fractions import Fraction

import numpy as np
import pytest
from scipy import stats

import oracle


def test_worked_example():
    t = np.array([[1, 2, 3, 4], [2, 2, 5, 0.5], [1, 2, 3, 4], [3, 3, 3, 3]], dtype=np.float32)
    med, iqr, W = oracle.adjudicate(t)
    # a vs b = [2,2,5,.5]: a_i<b_j pairs: 1<{2,2,5}=3, 2<{5}=1, 3<{5}=1, 4<{5}=1 -> 6; ties 2=={2,2} -> 2
    assert W.tolist() == [[16, 14, 16, 20], [18, 16, 18, 24], [16, 14, 16, 20], [12, 8, 12, 16]]
    assert med.tolist() == [2.5, 2.0, 2.5, 3.0]
    assert iqr.tolist() == [1.5, 1.125, 1.5, 0.0]
    q, srt = oracle.quantiles(t[1])
    assert q.tolist() == [1.625, 2.0, 2.75, 1.125] and srt.tolist() == [0.5, 2.0, 2.0, 5.0]


@pytest.mark.parametrize("S", [1, 2, 3, 5, 9, 20])
def test_wins_equal_scipy_mann_whitney(S):
    """scipy's U for (a, b) counts a_i > b_j plus half the ties, so W = 2*S*S - 2*U."""
    rng = np.random.default_rng(S)
    for trial in range(6):
        a = np.round(rng.lognormal(0, 0.2, S), 1 if trial % 2 else 6).astype(np.float32)
        b = np.round(rng.lognormal(0, 0.2, S), 1 if trial % 2 else 6).astype(np.float32)
        U = stats.mannwhitneyu(a.astype(np.float64), b.astype(np.float64),
                               alternative="two-sided", method="asymptotic").statistic
        assert oracle.wins_pair(a, b) == round(2 * S * S - 2 * U)


def test_wins_bruteforce_small_alphabet():
    vals = [0.5, 1.0, 1.0, 2.0]
    for a in itertools.product(vals, repeat=3):
        for b in itertools.product(vals[:3], repeat=3):
            want = sum(2 * (x < y) + (x == y) for x in a for y in b)
            assert oracle.wins_pair(np.float32(a), np.float32(b)) == want


def test_win_direction_smaller_time_wins():
    fast, slow = np.float32([1, 1, 1]), np.float32([2, 2, 2])
    assert oracle.wins_pair(fast, slow) == 18 and oracle.wins_pair(slow, fast) == 0


def test_signed_zero_timings_tie():
    assert oracle.wins_pair(np.float32([0.0]), np.float32([-0.0])) == 1


@pytest.mark.parametrize("K,S", [(5, 7), (3, 32), (8, 33), (4, 100)])
def test_win_matrix_identities(K, S):
    rng = np.random.default_rng(K * 100 + S)
    t = np.round(rng.lognormal(0, 0.1, (K, S)), 2).astype(np.float32)     # many ties
    _, _, W = oracle.adjudicate(t)
    W = W.astype(np.int64)
    assert (W + W.T == 2 * S * S).all()              # U_ab + U_ba = S_a * S_b, doubled
    assert (np.diag(W) == S * S).all()
    # samples within a row may come in any order
    t2 = np.stack([rng.permutation(row) for row in t])
    assert (oracle.adjudicate(t2)[2] == W).all()
    # a strictly increasing map of all timings changes no comparison
    t3 = np.exp(t.astype(np.float64)).astype(np.float32)
    assert len(np.unique(t3)) == len(np.unique(t))
    assert (oracle.adjudicate(t3)[2] == W).all()
    # all-equal timings
    med, iqr, We = oracle.adjudicate(np.full((K, S), 1.25, dtype=np.float32))
    assert (We == S * S).all() and (iqr == 0).all() and (med == 1.25).all()


def test_wins_rows_and_threads_agree_with_full():
    rng = np.random.default_rng(8)
    t = rng.lognormal(0, 0.1, (11, 13)).astype(np.float32)
    W = oracle.adjudicate(t)[2]
    assert (oracle.adjudicate(t, threads=3)[2] == W).all()
    assert (oracle.wins_rows(t, 4, 9) == W[4:9]).all()


@pytest.mark.parametrize("S", [1, 2, 3, 4, 5, 6, 7, 8, 9, 31, 32, 33, 64, 100, 200, 2000])
def test_quantiles_against_numpy_percentile(S):
    rng = np.random.default_rng(S)
    # small integers: every intermediate is exact, so the match must be exact
    row = rng.integers(0, 64, S).astype(np.float32)
    q, srt = oracle.quantiles(row)
    want = np.percentile(row.astype(np.float64), [25, 50, 75])
    assert q[0] == want[0] and q[1] == want[1] and q[2] == want[2] and q[3] == want[2] - want[0]
    assert (srt == np.sort(row)).all()
    # general values: within one binary32 ulp of the float64 evaluation
    row = rng.lognormal(0, 0.3, S).astype(np.float32)
    q, _ = oracle.quantiles(row)
    want = np.percentile(row.astype(np.float64), [25, 50, 75])
    for g, w in zip(q[:3], want):
        assert abs(float(g) - w) <= np.spacing(np.float32(w))


def test_quantile_operation_order_exact():
    """x_lo + (rem/4)*(x_hi - x_lo) with each step rounded, checked in exact arithmetic."""
    from tests import exact32 as E
    rng = np.random.default_rng(77)
    for S in [2, 3, 6, 11, 50]:
        row = rng.lognormal(0, 1.0, S).astype(np.float32)
        q, srt = oracle.quantiles(row)
        x = [E.from_float(float(v)) for v in np.sort(row)]
        got = []
        for j in (1, 2, 3):
            pos = j * (S - 1)
            lo, rem = divmod(pos, 4)
            hi = min(lo + 1, S - 1)
            if rem == 0:
                got.append(x[lo])
            else:
                w = Fraction(rem, 4)
                got.append(E.add(x[lo], E.mul(w, E.sub(x[hi], x[lo]))))
        assert [E.to_bits(g) for g in got] == [int(np.float32(v).view(np.uint32)) for v in q[:3]]
        assert E.to_bits(E.sub(got[2], got[0])) == int(np.float32(q[3]).view(np.uint32))


def test_median_is_middle_or_midpoint():
    assert oracle.quantiles(np.float32([5, 1, 3]))[0][1] == 3
    assert oracle.quantiles(np.float32([5, 1, 3, 4]))[0][1] == 3.5
    assert oracle.quantiles(np.float32([7]))[0].tolist() == [7, 7, 7, 0]


def test_signed_zeros_sort_negative_first_and_fix_the_sign_of_zero_quantiles():
    """A row that mixes -0 and +0: the sorted row is unique (value, then -0 before +0), so the
    sign of a quantile that is zero is fixed.  The expected signs are worked out by hand."""
    def bits(v):
        return [int(x) for x in np.asarray(v, dtype=np.float32).view(np.uint32)]
    NZ, PZ = 0x80000000, 0x00000000
    # S = 5: positions 1, 2, 3 hit samples exactly (rem = 0).
    q, srt = oracle.quantiles(np.float32([0.0, -0.0, 0.0, -0.0, -0.0]))
    assert bits(srt) == [NZ, NZ, NZ, PZ, PZ]
    # Q1 = x1 = -0, median = x2 = -0, Q3 = x3 = +0, IQR = (+0) - (-0) = +0
    assert bits(q) == [NZ, NZ, PZ, PZ]
    q, srt = oracle.quantiles(np.float32([0.0, 0.0, -0.0, 0.0, 0.0]))
    assert bits(srt) == [NZ, PZ, PZ, PZ, PZ]
    # Q1 = +0, median = +0, Q3 = +0, IQR = (+0) - (+0) = +0
    assert bits(q) == [PZ, PZ, PZ, PZ]
    # S = 2, row {+0, -0} -> sorted {-0, +0}: Q_j = -0 + (j/4)*((+0) - (-0)) = -0 + (+0) = +0
    q, srt = oracle.quantiles(np.float32([0.0, -0.0]))
    assert bits(srt) == [NZ, PZ] and bits(q) == [PZ, PZ, PZ, PZ]
    # S = 2, row {-0, -0}: Q_j = -0 + (j/4)*((-0) - (-0)) = -0 + (j/4)*(+0) = -0 + +0 = +0
    q, srt = oracle.quantiles(np.float32([-0.0, -0.0]))
    assert bits(srt) == [NZ, NZ] and bits(q) == [PZ, PZ, PZ, PZ]
    # S = 1: every quantile is the sample itself; IQR = (-0) - (-0) = +0
    q, _ = oracle.quantiles(np.float32([-0.0]))
    assert bits(q) == [NZ, NZ, NZ, PZ]
    # zeros among other values: [-1, +0, -0, 2, -0] sorts to [-1, -0, -0, +0, 2]
    q, srt = oracle.quantiles(np.float32([-1.0, 0.0, -0.0, 2.0, -0.0]))
    assert bits(srt) == [0xBF800000, NZ, NZ, PZ, 0x40000000]
    assert bits(q) == [NZ, NZ, PZ, PZ]
    # the order of the input does not matter
    rng = np.random.default_rng(5)
    row = np.float32([0.0, -0.0, 0.0, -0.0, 1.0, -1.0, -0.0, 0.0, 0.0])
    want = bits(oracle.quantiles(row)[1])
    assert want == [0xBF800000, NZ, NZ, NZ, PZ, PZ, PZ, PZ, 0x3F800000]
    for _ in range(20):
        assert bits(oracle.quantiles(rng.permutation(row))[1]) == want


def test_nonfinite_timing_is_an_error():
    t = np.ones((3, 4), dtype=np.float32)
    for bad in (np.nan, np.inf, -np.inf):
        t2 = t.copy()
        t2[1, 2] = bad
        with pytest.raises(oracle.NonFiniteTiming):
            oracle.adjudicate(t2)
        with pytest.raises(oracle.NonFiniteTiming):
            oracle.quantiles(t2[1])


# ---- rows of different lengths --------------------------------------------------------------

def test_ragged_wins_equal_scipy_and_sum_to_twice_the_product():
    """U_ab + U_ba = S_a * S_b (doubled here), for unequal sample counts."""
    rng = np.random.default_rng(31)
    rows = [np.round(rng.lognormal(0, 0.2, n), 1).astype(np.float32) for n in (1, 4, 7, 16, 60, 3)]
    med, iqr, W = oracle.adjudicate_ragged(rows)
    K = len(rows)
    for a in range(K):
        q, _ = oracle.quantiles(rows[a])
        assert med[a] == q[1] and iqr[a] == q[3]
        assert W[a, a] == rows[a].size ** 2
        for b in range(K):
            assert int(W[a, b]) + int(W[b, a]) == 2 * rows[a].size * rows[b].size
            if a != b:
                U = stats.mannwhitneyu(rows[a].astype(np.float64), rows[b].astype(np.float64),
                                       alternative="two-sided", method="asymptotic").statistic
                assert int(W[a, b]) == round(2 * rows[a].size * rows[b].size - 2 * U)


def test_ragged_with_equal_lengths_is_the_rectangular_case():
    rng = np.random.default_rng(32)
    t = np.round(rng.lognormal(0, 0.1, (6, 9)), 2).astype(np.float32)
    m1, i1, w1 = oracle.adjudicate(t)
    m2, i2, w2 = oracle.adjudicate_ragged(list(t))
    assert (m1 == m2).all() and (i1 == i2).all() and (w1 == w2).all()
    with pytest.raises(oracle.NonFiniteTiming):
        oracle.adjudicate_ragged([np.float32([1, 2]), np.float32([np.inf])])
