"""Pins for the oracle's merge of range records (CPU only): the gate over a range split into
consecutive parts, merged, must be the gate over the whole range -- checked against the oracle's
own whole-range gate (already pinned in test_oracle_screen.py) on inputs built so that every
clause of the merge decides something, and on a hand-made case."""
import numpy as np
import pytest

import oracle

F32, F16, BF16 = oracle.F32, oracle.F16, oracle.BF16
FIELDS = ("mismatch_count", "nan_count", "inf_count", "argmax_idx", "pass")


def same(a, b):
    for f in FIELDS:
        assert (a[f] == b[f]).all(), f
    for f in ("max_abs_err", "max_rel_err"):
        assert (a[f].view(np.uint32) == b[f].view(np.uint32)).all(), f


def screen_parts(ref, cands, cuts, atol, rtol, dtype=F32):
    first = [0] + list(cuts)
    last = list(cuts) + [ref.size]
    parts = [oracle.screen(ref[a:b], [c[a:b] for c in cands], dtype, atol, rtol) for a, b in zip(first, last)]
    return parts, first


def test_hand_made_case():
    # two parts of four elements; |c - r| by element: part 0: 0, .5, .25, nan ; part 1: .5, 0, 1, inf-inf
    ref = np.array([1, 2, 4, 1, 8, 1, 16, np.inf], dtype=np.float32)
    cand = np.array([1, 2.5, 4.25, np.nan, 8.5, 1, 17, np.inf], dtype=np.float32)
    parts, first = screen_parts(ref, [cand], [4], 0.3, 0.0)
    assert parts[0]["argmax_idx"][0] == 1 and parts[1]["argmax_idx"][0] == 2       # local indices
    m = oracle.merge_ranges(parts, first)
    assert m["mismatch_count"][0] == 4            # .5, nan, .5, 1 exceed atol = .3 (Inf == Inf matches)
    assert m["nan_count"][0] == 1 and m["inf_count"][0] == 1
    assert m["argmax_idx"][0] == 6 and m["max_abs_err"][0] == 1.0                  # global index 4 + 2
    assert m["max_rel_err"][0] == np.float32(0.25)                                 # .5 / 2 in part 0
    assert m["pass"][0] == 0
    same(m, oracle.screen(ref, [cand], F32, 0.3, 0.0))


def test_the_earlier_part_keeps_a_tied_maximum_and_an_empty_handed_part_is_skipped():
    ref = np.zeros(12, dtype=np.float32)
    c0 = ref.copy(); c0[[2, 5, 9]] = 0.5              # the same largest error in all three parts
    c1 = ref.copy(); c1[:4] = np.nan; c1[7] = 0.25    # part 0 has no finite difference at all
    c2 = np.full(12, np.nan, dtype=np.float32)        # no part has one
    parts, first = screen_parts(ref, [c0, c1, c2], [4, 8], 1.0, 0.0)
    m = oracle.merge_ranges(parts, first)
    assert list(m["argmax_idx"]) == [2, 7, -1]
    assert list(m["max_abs_err"]) == [0.5, 0.25, 0.0]
    assert list(m["nan_count"]) == [0, 4, 12] and list(m["pass"]) == [1, 0, 0]
    same(m, oracle.screen(ref, [c0, c1, c2], F32, 1.0, 0.0))


@pytest.mark.parametrize("dtype,np_dt", [(F32, np.float32), (F16, np.float16)])
@pytest.mark.parametrize("cuts", [[1], [4096], [5, 6, 7], [1000, 5000, 9000], [4096, 8192]])
def test_merged_parts_equal_the_whole_range(dtype, np_dt, cuts):
    rng = np.random.default_rng(len(cuts) * 100 + cuts[0] + dtype)
    N = 10000
    ref = rng.standard_normal(N).astype(np_dt)
    cands = []
    for k in range(6):
        c = ref.copy()
        idx = rng.integers(0, N, 40)
        c[idx] = (c[idx].astype(np.float64) * (1 + 2.0 ** -(k + 3))).astype(np_dt)   # many equal relative errors
        if k % 2:
            c[rng.integers(0, N, 3)] = np.nan
            c[rng.integers(0, N, 2)] = np.inf
        if k == 4:                                  # the same absolute error on both sides of every cut
            for cut in cuts:
                c[cut - 1] = ref[cut - 1] = np_dt(1.0)
                c[cut] = ref[cut] = np_dt(1.0)
                c[cut - 1] += np_dt(0.5)
                c[cut] += np_dt(0.5)
        cands.append(c)
    arr = (lambda a: a) if dtype == F32 else (lambda a: a.view(np.uint16))
    whole = oracle.screen(arr(ref), [arr(c) for c in cands], dtype, 1e-3, 1e-2)
    first = [0] + cuts
    last = cuts + [N]
    parts = [oracle.screen(arr(ref[a:b]), [arr(c[a:b]) for c in cands], dtype, 1e-3, 1e-2)
             for a, b in zip(first, last)]
    same(oracle.merge_ranges(parts, first), whole)


def test_bad_arguments():
    rec = oracle.screen(np.zeros(4, np.float32), [np.zeros(4, np.float32)], F32, 0.0, 0.0)
    with pytest.raises(ValueError):
        oracle.merge_ranges([rec, rec], [4, 4])        # the parts' first indices must ascend
