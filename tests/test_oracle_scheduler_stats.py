"""Pins for the oracle's scheduler-side statistics (CPU only): the runtime score of Eq. 2 and
promotion by it, the tail ratios of the appendix, and Copeland counts from the win matrix."""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from tests import exact32 as E

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def consts():
    out = {}
    for ln in open(os.path.join(GOLD, "paper_score_constants.txt")):
        if ln.strip() and not ln.startswith("#"):
            key, *vals = ln.split()
            out[key] = [float(v) for v in vals]
    return out


# ---- runtime score (Sec. 3.1, Eq. 2) ---------------------------------------------------

def test_score_of_the_papers_sample_run():
    """The sample run ends at rung 2 (60 timed iterations) with best score 384.36
    (Sec. 4, Observed Run Trajectory): gamma = 0.02*2 + 0.01*60 = 0.64, so the latency
    behind it is 1e6 / 383.72 us; the score of that latency must print as 384.36."""
    c = consts()
    alpha, beta, b2 = c["alpha"][0], c["beta"][0], int(c["iterations"][2])
    latency_ms = 1e6 / (384.36 - (alpha * 2 + beta * b2)) / 1000.0
    s = oracle.score(latency_ms, 2, b2, alpha, beta)
    assert f"{float(s):.2f}" == "384.36"


def test_score_closed_forms():
    assert oracle.score(1.0, 0, 0, 0.02, 0.01) == np.float32(1000.0)          # 1 ms = 1000 us
    assert oracle.score(0.0005, 0, 0, 0.02, 0.01) == np.float32(1e6)          # below 1 us: max(1, .)
    assert oracle.score(0.001, 3, 0, 0.5, 0.0) == np.float32(1e6 + 1.5)
    # later rungs weigh more at the same latency
    assert oracle.score(2.0, 2, 60, 0.02, 0.01) > oracle.score(2.0, 1, 16, 0.02, 0.01) > \
        oracle.score(2.0, 0, 4, 0.02, 0.01)


def test_score_operation_order_exact():
    rng = np.random.default_rng(3)
    for _ in range(200):
        med = np.float32(rng.lognormal(0, 2))
        r, b = int(rng.integers(0, 4)), int(rng.integers(1, 100))
        alpha, beta = np.float32(0.02), np.float32(0.01)
        l_us = E.mul(E.from_float(float(med)), E.from_float(1000.0))
        m = l_us if l_us > 1 else Fraction(1)
        base = E.div(E.from_float(1e6), m)
        gamma = E.add(E.mul(E.from_float(float(alpha)), Fraction(r)), E.mul(E.from_float(float(beta)), Fraction(b)))
        want = E.to_bits(E.add(base, gamma))
        assert int(oracle.score(med, r, b, alpha, beta).view(np.uint32)) == want


def records(passed):
    rec = np.zeros(len(passed), dtype=oracle.RESULT_DTYPE)
    rec["pass"] = passed
    return rec


@pytest.mark.parametrize("K,budget", [(1, 1), (9, 4), (40, 40), (30, 50)])
def test_select_by_score_against_python_sorted(K, budget):
    rng = np.random.default_rng(K + budget)
    for trial in range(6):
        passed = (rng.random(K) < 0.7).astype(np.uint32)
        med = rng.choice(np.float32([0.0004, 0.0009, 0.9, 1.0, 1.0, 1.1]), K) if trial % 2 else \
            rng.lognormal(0, 0.3, K).astype(np.float32)
        sc, surv, n = oracle.select_by_score(records(passed), med, 1, 16, 0.02, 0.01, budget)
        for k in range(K):
            assert sc[k] == oracle.score(med[k], 1, 16, 0.02, 0.01)
        want = sorted([k for k in range(K) if passed[k]], key=lambda k: (-float(sc[k]), k))[:budget]
        assert n == len(want) and surv[:n].tolist() == want and (surv[n:] == -1).all()


def test_sub_microsecond_latencies_tie_and_fall_back_to_the_index():
    med = np.float32([0.0009, 0.0002, 0.0005, 0.002])       # three below 1 us: same score 1e6 + gamma
    sc, surv, n = oracle.select_by_score(records([1, 1, 1, 1]), med, 0, 4, 0.02, 0.01, 4)
    assert sc[0] == sc[1] == sc[2] > sc[3]
    assert surv.tolist() == [0, 1, 2, 3]


# ---- tail ratios (Appendix, Relative Variability Metrics) ---------------------------------

@pytest.mark.parametrize("S", [1, 2, 3, 5, 16, 60, 101, 200, 2000])
def test_tail_ratios_against_numpy_percentile(S):
    rng = np.random.default_rng(S)
    t = rng.lognormal(0, 0.1, (3, S)).astype(np.float32)
    got = oracle.tail_ratios(t)
    for k in range(3):
        p = np.percentile(t[k].astype(np.float64), [50, 90, 95, 99])
        for j in range(3):
            want = p[j + 1] / p[0]
            assert abs(float(got[k, j]) - want) <= 4 * np.spacing(np.float32(want)), (S, k, j)
    assert (got[:, 0] <= got[:, 1]).all() and (got[:, 1] <= got[:, 2]).all() and (got >= 1).all()


def test_tail_ratio_operation_order_exact():
    rng = np.random.default_rng(42)
    for S in [7, 33, 101, 250]:
        row = rng.lognormal(0, 0.5, S).astype(np.float32)
        got = oracle.tail_ratios(row)[0]
        x = [E.from_float(float(v)) for v in np.sort(row)]
        p = []
        for q in (50, 90, 95, 99):
            lo, rem = divmod(q * (S - 1), 100)
            hi = min(lo + 1, S - 1)
            if rem == 0:
                p.append(x[lo])
            else:
                w = E.div(Fraction(rem), Fraction(100))
                p.append(E.add(x[lo], E.mul(w, E.sub(x[hi], x[lo]))))
        want = [E.to_bits(E.div(p[j], p[0])) for j in (1, 2, 3)]
        assert [int(np.float32(v).view(np.uint32)) for v in got] == want


def test_tail_ratios_closed_forms():
    assert oracle.tail_ratios(np.full((1, 50), 2.5, np.float32)).tolist() == [[1.0, 1.0, 1.0]]
    # 0..100: the q-th percentile of 101 equally spaced samples is q itself
    assert oracle.tail_ratios(np.arange(101, dtype=np.float32)).tolist() == \
        [[np.float32(90) / np.float32(50), np.float32(95) / np.float32(50), np.float32(99) / np.float32(50)]]
    # lognormal noise: p_q / p50 -> exp(z_q * sigma)
    t = np.random.default_rng(0).lognormal(0, 0.05, (1, 200000)).astype(np.float32)
    r = oracle.tail_ratios(t)[0]
    for got, z in zip(r, (1.2816, 1.6449, 2.3263)):
        assert abs(float(got) - math.exp(z * 0.05)) < 2e-3
    with pytest.raises(oracle.NonFiniteTiming):
        oracle.tail_ratios(np.float32([1, np.nan, 2]))


def test_paper_tail_ratios_are_ordered_like_ours():
    """Every row of the paper's table satisfies 1 <= p90/p50 <= p95/p50 <= p99/p50, the
    ordering the statistic has by construction."""
    for ln in open(os.path.join(GOLD, "paper_tail_ratios.txt")):
        if ln.strip() and not ln.startswith("#"):
            a, b, c = (float(v) for v in ln.split()[2:5])
            assert 1.0 <= a <= b <= c


# ---- Copeland counts ------------------------------------------------------------------------

def test_copeland_bruteforce_and_identities():
    rng = np.random.default_rng(8)
    for K, S in [(2, 3), (5, 4), (9, 16), (12, 5)]:
        t = np.round(rng.lognormal(0, 0.2, (K, S)), 1).astype(np.float32)
        t[K - 1] = t[0]                                            # an exact tie between two candidates
        W = oracle.adjudicate(t)[2]
        beats, ties = oracle.copeland(W, S)
        for a in range(K):
            assert beats[a] == sum(1 for b in range(K) if b != a and int(W[a, b]) > S * S)
            assert ties[a] == sum(1 for b in range(K) if b != a and int(W[a, b]) == S * S)
        # every unordered pair is a win for one side or a tie for both
        assert int(beats.sum()) + int(ties.sum()) // 2 == K * (K - 1) // 2
        assert ties[0] >= 1 and ties[K - 1] >= 1


def test_copeland_separated_candidates_rank_by_speed():
    t = np.float32([[3, 3.1, 3.2], [1, 1.1, 1.2], [2, 2.1, 2.2], [4, 4.1, 4.2]])
    beats, ties = oracle.copeland(oracle.adjudicate(t)[2], 3)
    assert beats.tolist() == [1, 3, 2, 0] and ties.tolist() == [0, 0, 0, 0]


# ---- re-measure and confirm --------------------------------------------------------------

def test_confirm_truth_table():
    prev = np.float32([100, 100, 100, 100, 100])
    s1 = np.float32([104, 120, 120, 90, 105.0001])
    s2 = np.float32([50, 118, 103, 300, 200])
    st, sc = oracle.confirm(s1, s2, prev, 0.05)
    # +4%: below the threshold, taken as is.  +20% re-measured at +18%: confirmed, the lower
    # of the two.  +20% re-measured at +3%: reverted to the incumbent.  A regression is never
    # flagged.  Just above the bar and confirmed.
    assert st.tolist() == [0, 1, 2, 0, 1]
    assert sc.tolist() == [104.0, 118.0, 100.0, 90.0, np.float32(105.0001)]


def test_confirm_boundary_is_strict_and_in_binary32():
    from fractions import Fraction
    rng = np.random.default_rng(5)
    prev = rng.lognormal(5, 1, 500).astype(np.float32)
    s1 = (prev * rng.choice(np.float32([1.0, 1.05, 1.0500001, 1.2]), 500)).astype(np.float32)
    s2 = (prev * rng.choice(np.float32([0.9, 1.05, 1.06, 1.3]), 500)).astype(np.float32)
    thr = np.float32(0.05)
    st, sc = oracle.confirm(s1, s2, prev, thr)
    for k in range(500):
        bar = E.mul(E.from_float(float(thr)), E.from_float(float(prev[k])))
        f = E.sub(E.from_float(float(s1[k])), E.from_float(float(prev[k]))) > bar
        c = E.sub(E.from_float(float(s2[k])), E.from_float(float(prev[k]))) > bar
        want = 0 if not f else (1 if c else 2)
        assert st[k] == want
        assert sc[k] == (s1[k] if want == 0 else min(s1[k], s2[k]) if want == 1 else prev[k])
