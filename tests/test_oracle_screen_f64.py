"""Pins for the oracle's double-precision gate (CPU only).

Same gate as the binary32 one (Sec. 3.1 K(p); Sec. 3.4 Verifier), every operation in
binary64.  Pins: a hand-checkable example, an exact-rational brute force over awkward
binary64 values, numpy.isclose, agreement with the binary32 gate where both are exact,
closed forms for constructed perturbations, and invariants.
"""
import itertools
from fractions import Fraction

import numpy as np
import pytest

import oracle
from tests import exact64 as E


def f64(x):
    return np.asarray(x, dtype=np.float64)


def bits64(x) -> int:
    return int(np.float64(x).view(np.uint64))


def _arr(bits):
    return np.asarray(bits, dtype=np.uint64).view(np.float64)


def one(ref, cand, atol, rtol, mask=None):
    return oracle.screen_f64(f64(ref), [f64(cand)], atol, rtol, mask)[0]


def test_worked_example():
    # dyadic values: every step below is exact and can be checked by hand
    ref = f64([0, 1, -2, 0.5, 64, np.inf, np.nan, 3, 0, -np.inf, 4, 1])
    cand = f64([0, 1.25, -2.5, 0.75, 65, np.inf, np.nan, np.nan, 0.125, np.inf, np.inf, 1])
    r = one(ref, cand, 0.25, 0.0078125)        # atol = 1/4, rtol = 1/128
    # tol: i=1 0.2578125 (d=.25 ok), i=2 0.265625 (d=.5 no), i=3 0.25390625 (d=.25 ok),
    # i=4 0.75 (d=1 no), i=8 0.25 (d=.125 ok); non-finite: 5 equal, 6 7 9 10 mismatch
    assert r["mismatch_count"] == 6
    assert r["nan_count"] == 2 and r["inf_count"] == 3
    assert r["argmax_idx"] == 4 and r["max_abs_err"] == 1.0
    assert r["max_rel_err"] == 0.5             # i = 3: 0.25 / 0.5
    assert r["pass"] == 0 and r["reserved"] == 0


def model_screen(ref_bits, cand_bits, atol_bits, rtol_bits, selected=None):
    atol, rtol = E.from_bits(atol_bits), E.from_bits(rtol_bits)
    mism = nans = infs = 0
    have = False
    max_abs = Fraction(0)
    max_rel = Fraction(0)
    arg = -1
    for i, (rb, cb) in enumerate(zip(ref_bits, cand_bits)):
        if selected is not None and not selected(i):
            continue
        r, c = E.from_bits(rb), E.from_bits(cb)
        d = E.fabs(E.sub(c, r))
        tol = E.add(atol, E.mul(rtol, E.fabs(r)))
        match = E.eq(c, r) or (E.is_finite(d) and E.le(d, tol))
        mism += not match
        nans += E.is_nan(c)
        infs += E.is_inf(c)
        if E.is_finite(d):
            if not have or d > max_abs:
                max_abs, arg, have = d, i, True
            if E.is_finite(r) and r != 0:
                q = E.div(d, E.fabs(r))
                if E.is_inf(q) or (not E.is_inf(max_rel) and q > max_rel):
                    max_rel = q
    return dict(mismatch_count=mism, nan_count=nans, inf_count=infs, argmax_idx=arg,
                max_abs_bits=E.to_bits(max_abs), max_rel_bits=E.to_bits(max_rel),
                passed=int(mism == 0))


ALPHABET = [
    0x0000000000000000, 0x8000000000000000,          # +0, -0
    0x3FF0000000000000, 0xBFF0000000000000,          # +-1
    0x3FF0000000000001,                              # 1 + ulp
    0x3FEFFFFFFFFFFFFF,                              # 1 - ulp/2
    0x0000000000000001, 0x8000000000000001,          # smallest subnormals
    0x0010000000000000,                              # smallest normal
    0x7FEFFFFFFFFFFFFF, 0xFFEFFFFFFFFFFFFF,          # +-DBL_MAX
    0x7FF0000000000000, 0xFFF0000000000000,          # +-Inf
    0x7FF8000000000000, 0xFFF8000000000001,          # NaNs
    0x3F50624DD2F1A9FC,                              # 1e-3
    0x4008000000000000, 0xC000000000000000,          # 3, -2
    0x3FB999999999999A,                              # 0.1
    0x7E37E43C8800759C,                              # 1e300
    0x01A56E1FC2F8F359,                              # 1e-300
    0x4059000000000000, 0x4059033333333333,          # 100, 100.05
    0x3FF0000010000000,                              # 1 + 2^-24: invisible in binary32
]

TOLS = [
    (0x0000000000000000, 0x0000000000000000),        # exact equality only
    (0x3EE4F8B588E368F1, 0x3F50624DD2F1A9FC),        # 1e-5, 1e-3
    (0x3E45798EE2308C3A, 0x3E112E0BE826D695),        # 1e-8, 1e-9
    (0x7FE0000000000000, 0x4000000000000000),        # huge atol, rtol = 2: tol overflows
    (0x0000000000000001, 0x3FF0000000000000),        # subnormal atol, rtol = 1
]


def _check(got, want, ctx=""):
    assert got["mismatch_count"] == want["mismatch_count"], ctx
    assert got["nan_count"] == want["nan_count"], ctx
    assert got["inf_count"] == want["inf_count"], ctx
    assert got["argmax_idx"] == want["argmax_idx"], ctx
    assert bits64(got["max_abs_err"]) == want["max_abs_bits"], ctx
    assert bits64(got["max_rel_err"]) == want["max_rel_bits"], ctx
    assert got["pass"] == want["passed"], ctx


@pytest.mark.parametrize("tol", TOLS)
def test_bruteforce_single_elements(tol):
    ab, rb = tol
    atol, rtol = float(_arr([ab])[0]), float(_arr([rb])[0])
    for r_bits, c_bits in itertools.product(ALPHABET, ALPHABET):
        want = model_screen([r_bits], [c_bits], ab, rb)
        got = one(_arr([r_bits]), _arr([c_bits]), atol, rtol)
        _check(got, want, f"r={r_bits:#x} c={c_bits:#x} tol={tol}")


@pytest.mark.parametrize("tol", TOLS[:3])
def test_bruteforce_whole_vector_and_masks(tol):
    ab, rb = tol
    atol, rtol = float(_arr([ab])[0]), float(_arr([rb])[0])
    pairs = list(itertools.product(ALPHABET, ALPHABET))
    rng = np.random.default_rng(6)
    for trial in range(3):
        order = rng.permutation(len(pairs))
        rbits = [pairs[i][0] for i in order]
        cbits = [pairs[i][1] for i in order]
        _check(one(_arr(rbits), _arr(cbits), atol, rtol), model_screen(rbits, cbits, ab, rb))
        for log2_tile, stride, phase in [(0, 3, 1), (3, 5, 4), (6, 2, 1)]:
            want = model_screen(rbits, cbits, ab, rb,
                                selected=lambda i: ((i >> log2_tile) % stride) == phase)
            got = one(_arr(rbits), _arr(cbits), atol, rtol, ("strided", log2_tile, stride, phase))
            _check(got, want)


@pytest.mark.parametrize("atol,rtol", [(1e-8, 1e-9), (0.0, 1e-12), (1e-12, 0.0)])
def test_mismatch_count_equals_numpy_isclose(atol, rtol):
    rng = np.random.default_rng(17)
    ref = rng.standard_normal(5000) * np.exp(rng.normal(0, 3, 5000))
    cand = ref * (1 + rng.choice([0, 1e-13, 1e-10, 1e-8, -1e-9], 5000)) + rng.choice([0, 1e-12, 1e-7], 5000)
    got = one(ref, cand, atol, rtol)
    assert got["mismatch_count"] == int((~np.isclose(cand, ref, rtol=rtol, atol=atol)).sum())
    d = np.abs(cand - ref)
    assert got["argmax_idx"] == int(np.argmax(d)) and got["max_abs_err"] == d.max()
    assert got["max_rel_err"] == (d / np.abs(ref)).max()


def test_agrees_with_the_binary32_gate_where_both_are_exact():
    """Small dyadic values and dyadic tolerances: no operation rounds in either precision."""
    rng = np.random.default_rng(23)
    ref = rng.integers(-64, 64, 4000) / 16.0
    ref[ref == 0] = 0.5
    cand = ref + rng.integers(-4, 5, 4000) / 32.0
    for atol, rtol in [(0.0625, 0.0), (0.03125, 0.015625), (0.0, 0.0)]:
        a = one(ref, cand, atol, rtol)
        b = oracle.screen_one(ref.astype(np.float32), cand.astype(np.float32), oracle.F32, atol, rtol)
        for f in ("mismatch_count", "nan_count", "inf_count", "argmax_idx", "pass"):
            assert a[f] == b[f]
        assert a["max_abs_err"] == float(b["max_abs_err"])
    # relative errors of power-of-two references are exact quotients in both
    ref = np.ldexp(1.0, rng.integers(-6, 6, 1000))
    cand = ref * (1 + rng.integers(-8, 9, 1000) / 64.0)
    a = one(ref, cand, 0.0, 0.03125)
    b = oracle.screen_one(ref.astype(np.float32), cand.astype(np.float32), oracle.F32, 0.0, 0.03125)
    assert a["max_rel_err"] == float(b["max_rel_err"]) and a["mismatch_count"] == b["mismatch_count"]


def test_sees_differences_below_binary32_resolution():
    ref = np.ones(100)
    cand = ref.copy()
    cand[37] = 1 + 2.0 ** -40
    r = one(ref, cand, 0.0, 2.0 ** -45)
    assert r["mismatch_count"] == 1 and r["argmax_idx"] == 37
    assert r["max_abs_err"] == 2.0 ** -40 and r["max_rel_err"] == 2.0 ** -40
    assert one(ref, cand, 0.0, 2.0 ** -40)["pass"] == 1          # d <= tol: equality passes


def test_one_ulp_flip_closed_forms():
    for k in (-300, -1, 0, 7, 500):
        r = np.ldexp(1.0, k)
        c = np.nextafter(r, np.inf)
        got = one([r], [c], 0.0, 0.0)
        assert got["max_abs_err"] == np.ldexp(1.0, k - 52) and got["max_rel_err"] == 2.0 ** -52
        assert got["mismatch_count"] == 1
        assert one([r], [c], 0.0, 2.0 ** -52)["pass"] == 1


def test_special_values_and_ties():
    nan, inf = np.nan, np.inf
    assert one([nan], [nan], 1e300, 1e300)["mismatch_count"] == 1           # NaN never matches
    r = one([inf, -inf, 0.0, -0.0], [inf, -inf, -0.0, 0.0], 0.0, 0.0)
    assert r["pass"] == 1 and r["inf_count"] == 2 and r["argmax_idx"] == 2  # first finite d (0)
    r = one([1.0, 2.0, 3.0], [1.5, 2.5, 3.25], 0.0, 0.0)
    assert r["argmax_idx"] == 0 and r["max_abs_err"] == 0.5                 # first index wins ties
    assert one([inf, nan], [1.0, 1.0], 0.0, 0.0)["argmax_idx"] == -1        # no finite difference
    r = one([0.0, 4.0], [0.5, 5.0], 1.0, 0.0)
    assert r["max_rel_err"] == 0.25 and r["pass"] == 1                      # r = 0 judged, not in rel
    # the reference is on the right of the tolerance, and the divisor of the relative error
    assert one([100.0], [1.0], 0.0, 0.99)["pass"] == 1 and one([1.0], [100.0], 0.0, 0.99)["pass"] == 0
    assert one([4.0], [1.0], 0.0, 0.0)["max_rel_err"] == 0.75


def test_disjoint_masks_combine():
    rng = np.random.default_rng(4)
    ref = rng.standard_normal(3000)
    cand = ref + rng.choice([0, 1e-9, 1e-3], 3000) * rng.standard_normal(3000)
    full = one(ref, cand, 1e-8, 1e-8)
    parts = [one(ref, cand, 1e-8, 1e-8, ("strided", 4, 3, ph)) for ph in range(3)]
    assert sum(int(p["mismatch_count"]) for p in parts) == full["mismatch_count"]
    assert max(p["max_abs_err"] for p in parts) == full["max_abs_err"]
    assert max(p["max_rel_err"] for p in parts) == full["max_rel_err"]
    best = max(parts, key=lambda p: (p["max_abs_err"], -int(p["argmax_idx"])))
    assert best["argmax_idx"] == full["argmax_idx"]
    words = np.array([~np.uint64(0)] * 2, dtype=np.uint64)
    again = one(ref, cand, 1e-8, 1e-8, ("bitmap", 5, words))
    assert again == full
