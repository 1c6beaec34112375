"""Pins for the oracle's promotion decision (CPU only).

Sec. 3.4 (Adaptive Resource Allocation): candidates are ranked "with
deterministic tie-breaking", the top part is promoted, the rest pruned;
failed candidates never advance (Sec. 3.2 policy check; Sec. 3.4 Verifier).
Pins: Python's sorted() on tuple keys, the funnel counts of the paper's sample
run, and the runtime score of Eq. 2 (ranking by median latency ascending is
ranking by score descending inside one rung).
"""
import os

import numpy as np
import pytest

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def records(passed, rel):
    rec = np.zeros(len(passed), dtype=oracle.RESULT_DTYPE)
    rec["pass"] = passed
    rec["mismatch_count"] = 1 - np.asarray(passed)
    rec["max_rel_err"] = rel
    return rec


@pytest.mark.parametrize("policy", [0, 1])
@pytest.mark.parametrize("K,budget", [(1, 1), (7, 3), (33, 8), (64, 64), (40, 100)])
def test_against_python_sorted(policy, K, budget):
    rng = np.random.default_rng(K * 7 + budget + policy)
    for trial in range(5):
        passed = (rng.random(K) < 0.7).astype(np.uint32)
        rel = rng.choice(np.float32([0.0, 2.0 ** -7, 2.0 ** -8, 0.01, np.inf]), K)   # heavy ties
        med = rng.choice(np.float32([0.9, 1.0, 1.0, 1.1, 1.25]), K) if trial % 2 else \
            rng.lognormal(0, 0.1, K).astype(np.float32)
        elig = [k for k in range(K) if passed[k]]
        if policy == 0:
            want = sorted(elig, key=lambda k: (float(rel[k]), float(med[k]), k))
        else:
            want = sorted(elig, key=lambda k: (float(med[k]), k))
        want = want[:budget]
        surv, n = oracle.select(records(passed, rel), med, policy, budget)
        assert n == len(want)
        assert surv[:n].tolist() == want
        assert (surv[n:] == -1).all()


def test_no_eligible_candidate():
    surv, n = oracle.select(records([0, 0, 0], np.float32([0, 0, 0])), np.float32([1, 2, 3]), 0, 2)
    assert n == 0 and surv.tolist() == [-1, -1]


def test_lower_index_wins_full_ties():
    surv, n = oracle.select(records([1, 1, 1, 1], np.float32([0.5] * 4)), np.float32([1.0] * 4), 0, 3)
    assert surv.tolist() == [0, 1, 2]


def test_error_key_dominates_time_key():
    rec = records([1, 1, 1], np.float32([0.2, 0.1, 0.1]))
    surv, _ = oracle.select(rec, np.float32([0.5, 2.0, 1.0]), 0, 3)
    assert surv.tolist() == [2, 1, 0]
    surv, _ = oracle.select(rec, np.float32([0.5, 2.0, 1.0]), 1, 3)
    assert surv.tolist() == [0, 2, 1]


def test_paper_sample_run_funnel():
    """21 enter rung 0, 5 fail, 7 are promoted; of those 2 fail, 3 are promoted; all 3 pass."""
    rows = [tuple(map(int, ln.split())) for ln in open(os.path.join(GOLD, "paper_run_trajectory.txt"))
            if ln.strip() and not ln.startswith("#")]
    rng = np.random.default_rng(4)
    pool = np.arange(rows[0][1])
    for rung, entered, n_pass, n_fail, promoted in rows:
        assert len(pool) == entered and n_pass + n_fail == entered
        passed = np.ones(entered, dtype=np.uint32)
        passed[rng.choice(entered, n_fail, replace=False)] = 0
        med = rng.lognormal(0, 0.3, entered).astype(np.float32)
        budget = max(1, promoted)
        surv, n = oracle.select(records(passed, np.zeros(entered, np.float32)), med, 1, budget)
        if promoted:
            assert n == promoted                      # enough passing candidates to fill the budget
            assert all(passed[s] == 1 for s in surv[:n])
            # nobody left behind is both passing and faster than a survivor
            worst = max(med[s] for s in surv[:n])
            left = [k for k in range(entered) if passed[k] and k not in set(surv[:n].tolist())]
            assert all(med[k] >= worst for k in left)
            pool = pool[surv[:n]]
        else:
            assert int(passed.sum()) == n_pass


def test_time_policy_orders_by_runtime_score():
    """Eq. 2: S = 1e6/max(1, latency_us) + alpha*r + beta*b_r.  Inside one rung gamma is a
    constant, so descending score is ascending latency (for latencies above 1 us)."""
    consts = {}
    for ln in open(os.path.join(GOLD, "paper_score_constants.txt")):
        if ln.strip() and not ln.startswith("#"):
            key, *vals = ln.split()
            consts[key] = [float(v) for v in vals]
    alpha, beta = consts["alpha"][0], consts["beta"][0]
    rng = np.random.default_rng(9)
    K = 25
    med_ms = rng.lognormal(0, 0.4, K).astype(np.float32)
    assert len(np.unique(med_ms)) == K
    for rung, b_r in enumerate(consts["iterations"]):
        score = 1e6 / np.maximum(1.0, med_ms.astype(np.float64) * 1e3) + alpha * rung + beta * b_r
        want = list(np.argsort(-score, kind="stable"))
        surv, n = oracle.select(records(np.ones(K, np.uint32), np.zeros(K, np.float32)), med_ms, 1, K)
        assert n == K and surv.tolist() == want


def test_rejects_bad_arguments():
    with pytest.raises(ValueError):
        oracle.select(records([1], np.float32([0])), np.float32([1]), 2, 1)
