"""Pins for the oracle's correctness gate (CPU only).

The paper states the gate in words only (Sec. 3.1 K(p) "passes task and
numerical tests"; Sec. 3.4 Verifier "checks output correctness against the
reference"), so the pins are: a hand-checkable worked example, an exact
rational-arithmetic brute force over a small alphabet of awkward values,
library special cases (numpy.isclose, numpy/torch half decoders), closed forms
for constructed perturbations, and invariants.
"""
import itertools
import struct
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from tests import exact32 as E

F32, F16, BF16 = oracle.F32, oracle.F16, oracle.BF16


def f32(x):
    return np.asarray(x, dtype=np.float32)


def bits32(x) -> int:
    return int(np.float32(x).view(np.uint32))


# --------------------------------------------------------------------------
# worked example: every value below can be checked with pencil and paper
# --------------------------------------------------------------------------

def test_worked_example_fp32():
    ref = f32([0, 1, -2, 1e-3, 100, np.inf, np.nan, 3, 0, -np.inf, 4, 1])
    cand = f32([0, 1.0005, -2.01, 1.2e-3, 100.05, np.inf, np.nan, np.nan, 1e-6, np.inf, np.inf, 1])
    r = oracle.screen_one(ref, cand, F32, 1e-5, 1e-3)
    # matches: i=0 (equal), 1 (5e-4 <= 1.01e-3), 4 (0.05 <= 0.10001), 5 (Inf == Inf),
    #          8 (1e-6 <= 1e-5 at r = 0), 11 (equal).  Mismatches: 2, 3, 6, 7, 9, 10.
    assert r["mismatch_count"] == 6
    assert r["nan_count"] == 2          # i = 6, 7
    assert r["inf_count"] == 3          # i = 5, 9, 10
    assert r["argmax_idx"] == 4         # 100.05f - 100f = 0.05000305... is the largest finite d
    assert bits32(r["max_abs_err"]) == 0x3D4CD000
    assert bits32(r["max_rel_err"]) == 0x3E4CCCCD   # 0.2 from i = 3: (1.2e-3 - 1e-3)/1e-3
    assert r["pass"] == 0 and r["reserved"] == 0


# --------------------------------------------------------------------------
# exact-arithmetic brute force over a small alphabet
# --------------------------------------------------------------------------

def model_screen(ref_bits, cand_bits, atol_bits, rtol_bits, selected=None):
    """The seven steps of the gate evaluated with exact rationals + explicit rounding."""
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
    0x00000000, 0x80000000,              # +0, -0
    0x3F800000, 0xBF800000,              # +-1
    0x3F800001,                          # 1 + ulp
    0x3F7FFFFF,                          # 1 - ulp/2
    0x00000001, 0x80000001,              # smallest subnormals
    0x00800000,                          # smallest normal
    0x7F7FFFFF, 0xFF7FFFFF,              # +-FLT_MAX
    0x7F800000, 0xFF800000,              # +-Inf
    0x7FC00000, 0xFFC00001,              # NaNs
    0x3A83126F,                          # 1e-3
    0x40400000, 0xC0000000,              # 3, -2
    0x3DCCCCCD,                          # 0.1
    0x7E967699,                          # 1e38
    0x0DA24260,                          # 1e-30
    0x42C80000, 0x42C8199A,              # 100, 100.05
]

TOLS = [
    (0x00000000, 0x00000000),            # exact equality only
    (0x3727C5AC, 0x3A83126F),            # 1e-5, 1e-3
    (0x3C23D70A, 0x3C83126F),            # 1e-2, 1.6e-2
    (0x7F000000, 0x40000000),            # huge atol, rtol = 2: tol overflows to +Inf
    (0x00000001, 0x3F800000),            # subnormal atol, rtol = 1
]


def _arr(bits):
    return np.asarray(bits, dtype=np.uint32).view(np.float32)


@pytest.mark.parametrize("tol", TOLS)
def test_bruteforce_single_elements(tol):
    """Every (r, c) pair of the alphabet as its own one-element tensor."""
    ab, rb = tol
    atol, rtol = _arr([ab])[0], _arr([rb])[0]
    for r_bits, c_bits in itertools.product(ALPHABET, ALPHABET):
        want = model_screen([r_bits], [c_bits], ab, rb)
        got = oracle.screen_one(_arr([r_bits]), _arr([c_bits]), F32, atol, rtol)
        ctx = f"r={r_bits:#x} c={c_bits:#x} tol={tol}"
        assert got["mismatch_count"] == want["mismatch_count"], ctx
        assert got["nan_count"] == want["nan_count"], ctx
        assert got["inf_count"] == want["inf_count"], ctx
        assert got["argmax_idx"] == want["argmax_idx"], ctx
        assert bits32(got["max_abs_err"]) == want["max_abs_bits"], ctx
        assert bits32(got["max_rel_err"]) == want["max_rel_bits"], ctx
        assert got["pass"] == want["passed"], ctx


@pytest.mark.parametrize("tol", TOLS[:3])
def test_bruteforce_whole_vector(tol):
    """All pairs as one tensor: exercises accumulation, first-index ties, running maxima."""
    ab, rb = tol
    pairs = list(itertools.product(ALPHABET, ALPHABET))
    rng = np.random.default_rng(5)
    for trial in range(4):
        order = rng.permutation(len(pairs))
        rbits = [pairs[i][0] for i in order]
        cbits = [pairs[i][1] for i in order]
        want = model_screen(rbits, cbits, ab, rb)
        got = oracle.screen_one(_arr(rbits), _arr(cbits), F32, _arr([ab])[0], _arr([rb])[0])
        assert got["mismatch_count"] == want["mismatch_count"]
        assert got["nan_count"] == want["nan_count"]
        assert got["inf_count"] == want["inf_count"]
        assert got["argmax_idx"] == want["argmax_idx"]
        assert bits32(got["max_abs_err"]) == want["max_abs_bits"]
        assert bits32(got["max_rel_err"]) == want["max_rel_bits"]


def test_bruteforce_masks():
    pairs = list(itertools.product(ALPHABET[:12], ALPHABET[:12]))
    rbits = [p[0] for p in pairs]
    cbits = [p[1] for p in pairs]
    ab, rb = TOLS[1]
    n = len(pairs)
    for log2_tile, stride, phase in [(0, 3, 1), (2, 2, 0), (3, 5, 4), (4, 1, 0), (6, 2, 1)]:
        sel = lambda i: ((i >> log2_tile) % stride) == phase
        want = model_screen(rbits, cbits, ab, rb, sel)
        got = oracle.screen_one(_arr(rbits), _arr(cbits), F32, _arr([ab])[0], _arr([rb])[0],
                                mask=("strided", log2_tile, stride, phase))
        assert got["mismatch_count"] == want["mismatch_count"]
        assert got["argmax_idx"] == want["argmax_idx"]
        assert bits32(got["max_abs_err"]) == want["max_abs_bits"]
        assert bits32(got["max_rel_err"]) == want["max_rel_bits"]
        # the same selection as a bitmap
        ntiles = (n + (1 << log2_tile) - 1) >> log2_tile
        words = np.zeros((ntiles + 63) // 64, dtype=np.uint64)
        for t in range(ntiles):
            if t % stride == phase:
                words[t >> 6] |= np.uint64(1) << np.uint64(t & 63)
        got2 = oracle.screen_one(_arr(rbits), _arr(cbits), F32, _arr([ab])[0], _arr([rb])[0],
                                 mask=("bitmap", log2_tile, words))
        assert got2 == got


# --------------------------------------------------------------------------
# library special cases
# --------------------------------------------------------------------------

def test_decoders_against_numpy_and_torch():
    """All 65536 patterns of both 16-bit formats."""
    pat = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    want16 = pat.view(np.float16).astype(np.float32).view(np.uint32)
    wantbf = torch.from_numpy(pat.view(np.int16)).view(torch.bfloat16).to(torch.float32) \
        .numpy().view(np.uint32)
    L = oracle.lib()
    for p in range(65536):
        g16 = struct.unpack("<I", struct.pack("<f", L.kbo_decode_f16(p)))[0]
        gbf = struct.unpack("<I", struct.pack("<f", L.kbo_decode_bf16(p)))[0]
        if (want16[p] & 0x7FFFFFFF) > 0x7F800000:          # NaN: payload may be quieted en route
            assert (g16 & 0x7FFFFFFF) > 0x7F800000
        else:
            assert g16 == want16[p], hex(p)
        if (wantbf[p] & 0x7FFFFFFF) > 0x7F800000:
            assert (gbf & 0x7FFFFFFF) > 0x7F800000
        else:
            assert gbf == wantbf[p], hex(p)


@pytest.mark.parametrize("atol,rtol", [(1e-5, 1e-3), (1e-2, 1.6e-2), (0.0, 1e-2), (1e-6, 0.0)])
def test_mismatch_count_equals_numpy_isclose(atol, rtol):
    """For finite float32 inputs numpy.isclose(c, r) evaluates |c-r| <= atol + rtol*|r|
    in float32 -- the reference on the right, exactly the gate's predicate."""
    rng = np.random.default_rng(11)
    n = 20000
    r = (rng.standard_normal(n) * np.exp(3 * rng.standard_normal(n))).astype(np.float32)
    c = r.copy()
    pick = rng.random(n) < 0.5
    c[pick] = (r[pick] * (1 + rng.standard_normal(pick.sum()) * rtol)).astype(np.float32)
    c[rng.random(n) < 0.05] += np.float32(atol)
    want = int((~np.isclose(c, r, rtol=np.float32(rtol), atol=np.float32(atol))).sum())
    got = oracle.screen_one(r, c, F32, atol, rtol)
    assert got["mismatch_count"] == want
    assert got["nan_count"] == 0 and got["inf_count"] == 0


def test_float64_evaluation_agrees():
    """Each binary32 operation equals the float64 operation rounded once (p = 53 >=
    2*24 + 2 makes the double rounding innocuous for +, -, *, /)."""
    rng = np.random.default_rng(12)
    n = 50000
    r = (rng.standard_normal(n) * np.exp(2 * rng.standard_normal(n))).astype(np.float32)
    c = (r * (1 + 1e-3 * rng.standard_normal(n))).astype(np.float32)
    r[::97] = 0.0
    got = oracle.screen_one(r, c, F32, 1e-5, 1e-3)
    r64, c64 = r.astype(np.float64), c.astype(np.float64)
    d = np.abs((c64 - r64).astype(np.float32)).astype(np.float64)
    prod = (np.float64(np.float32(1e-3)) * np.abs(r64)).astype(np.float32).astype(np.float64)
    tol = (np.float64(np.float32(1e-5)) + prod).astype(np.float32).astype(np.float64)
    assert got["mismatch_count"] == int((~((c64 == r64) | (d <= tol))).sum())
    assert got["max_abs_err"] == np.float32(d.max())
    assert got["argmax_idx"] == int(np.argmax(d))
    nz = r64 != 0
    assert got["max_rel_err"] == (d[nz] / np.abs(r64[nz])).astype(np.float32).max()


# --------------------------------------------------------------------------
# closed forms for constructed candidates
# --------------------------------------------------------------------------

@pytest.mark.parametrize("dtype,np_view", [(F32, None), (F16, np.float16), (BF16, "bf16")])
def test_identical_candidate(dtype, np_view):
    rng = np.random.default_rng(1)
    x = rng.standard_normal(5000).astype(np.float32)
    if dtype == F32:
        a = x
    elif dtype == F16:
        a = x.astype(np.float16).view(np.uint16)
    else:
        a = (x.view(np.uint32) >> 16).astype(np.uint16)
    r = oracle.screen_one(a, a.copy(), dtype, 0.0, 0.0)
    assert (r["mismatch_count"], r["nan_count"], r["inf_count"]) == (0, 0, 0)
    assert r["max_abs_err"] == 0 and r["max_rel_err"] == 0
    assert r["argmax_idx"] == 0 and r["pass"] == 1
    # under a mask the first SELECTED index is reported, as a flat index of the full tensor
    r = oracle.screen_one(a, a.copy(), dtype, 0.0, 0.0, mask=("strided", 4, 7, 3))
    assert r["argmax_idx"] == 3 * 16 and r["pass"] == 1


def test_injected_nan_inf_counts_are_recovered():
    rng = np.random.default_rng(2)
    ref = rng.standard_normal(4096).astype(np.float32)
    for n_nan, n_inf in [(0, 1), (3, 1), (5, 0), (7, 8)]:
        c = ref.copy()
        idx = rng.choice(ref.size, size=n_nan + n_inf, replace=False)
        c[idx[:n_nan]] = np.nan
        c[idx[n_nan:]] = np.where(rng.random(n_inf) < 0.5, np.inf, -np.inf)
        r = oracle.screen_one(ref, c, F32, 1e-5, 1e-3)
        assert r["nan_count"] == n_nan and r["inf_count"] == n_inf
        assert r["mismatch_count"] == n_nan + n_inf
        assert r["max_abs_err"] == 0 and r["max_rel_err"] == 0 and r["pass"] == 0
        assert r["argmax_idx"] == (0 if 0 not in idx else int(np.setdiff1d(np.arange(9), idx)[0]))


def test_only_nonfinite_differences_gives_no_argmax():
    ref = f32([1, 2, 3])
    cand = f32([np.nan, np.inf, -np.inf])
    r = oracle.screen_one(ref, cand, F32, 1.0, 1.0)
    assert r["argmax_idx"] == -1 and r["max_abs_err"] == 0 and r["max_rel_err"] == 0
    assert r["mismatch_count"] == 3 and r["nan_count"] == 1 and r["inf_count"] == 2


def test_burst_max_abs_error_is_largest_injected_perturbation():
    rng = np.random.default_rng(3)
    ref = rng.standard_normal(10000).astype(np.float32)
    c = ref.copy()
    start, length = 1234, 100
    delta = np.float32(0.01)
    c[start:start + length] = ref[start:start + length] + delta       # fp32 add
    # the injected perturbation, measured element by element in exact arithmetic
    exact = [abs(Fraction(float(c[i])) - Fraction(float(ref[i]))) for i in range(start, start + length)]
    biggest = max(exact)
    first = start + exact.index(biggest)
    r = oracle.screen_one(ref, c, F32, 1e-5, 1e-3)
    assert Fraction(float(r["max_abs_err"])) == biggest      # c - r is exact here (Sterbenz-like range)
    assert r["argmax_idx"] == first
    assert r["mismatch_count"] == length


def test_one_ulp_flip_of_power_of_two_gives_rel_2_pow_minus_7_bf16():
    ref = np.array([0x3F80, 0x4000, 0x4049, 0xC080], dtype=np.uint16)    # 1, 2, 3.14, -4
    c = ref.copy()
    c[1] += 1                                                            # 2 -> 2 + 2^-6
    r = oracle.screen_one(ref, c, BF16, 1e-2, 1.6e-2)
    assert r["max_rel_err"] == np.float32(2.0 ** -7) and r["max_abs_err"] == np.float32(2.0 ** -6)
    assert r["argmax_idx"] == 1 and r["pass"] == 1
    c = ref.copy()
    c[1] -= 1                                                            # 2 -> 2 - 2^-7
    r = oracle.screen_one(ref, c, BF16, 1e-2, 1.6e-2)
    assert r["max_rel_err"] == np.float32(2.0 ** -8)


def test_ulp_flip_bounds_fp16_fp32():
    rng = np.random.default_rng(4)
    x = (rng.standard_normal(20000) * 2).astype(np.float16)
    x = x[np.abs(x) >= 6.2e-5]                                           # normal range only
    bits = x.view(np.uint16)
    step = rng.integers(-1, 2, size=bits.size)
    c = (bits.astype(np.int32) + step).astype(np.uint16)
    r = oracle.screen_one(bits, c, F16, 1e-3, 1e-2)
    assert r["max_rel_err"] <= np.float32(2.0 ** -10) and r["mismatch_count"] == 0
    y = rng.standard_normal(20000).astype(np.float32)
    yb = y.view(np.uint32)
    c32 = (yb.astype(np.int64) + rng.integers(-1, 2, size=yb.size)).astype(np.uint32).view(np.float32)
    r = oracle.screen_one(y, c32, F32, 1e-6, 1e-3)
    assert r["max_rel_err"] <= np.float32(2.0 ** -23) and r["mismatch_count"] == 0


# --------------------------------------------------------------------------
# invariants and orientation
# --------------------------------------------------------------------------

def test_reference_is_on_the_right_of_the_tolerance():
    """tol uses |r|, not |c| and not max(|r|,|c|)."""
    a, b = f32([100.0]), f32([101.005])
    assert oracle.screen_one(a, b, F32, 0.0, 1e-2)["mismatch_count"] == 1   # tol = 1.0  < d
    assert oracle.screen_one(b, a, F32, 0.0, 1e-2)["mismatch_count"] == 0   # tol = 1.01 >= d


def test_rel_error_divides_by_reference_not_candidate():
    r = oracle.screen_one(f32([2.0]), f32([4.0]), F32, 0.0, 0.0)
    assert r["max_rel_err"] == 1.0 and r["max_abs_err"] == 2.0              # 2/|2|, not 2/|4|


def test_zero_reference_is_excluded_from_rel_error_but_still_judged():
    r = oracle.screen_one(f32([0.0, -0.0, 1.0]), f32([0.5, 1e-7, 1.0]), F32, 1e-6, 1e-3)
    assert r["max_rel_err"] == 0 and r["mismatch_count"] == 1 and r["max_abs_err"] == 0.5


def test_nan_never_matches_even_nan():
    r = oracle.screen_one(f32([np.nan]), f32([np.nan]), F32, 1.0, 1.0)
    assert r["mismatch_count"] == 1 and r["nan_count"] == 1 and r["argmax_idx"] == -1


def test_signed_zeros_and_same_sign_infinities_match():
    r = oracle.screen_one(f32([0.0, np.inf, -np.inf]), f32([-0.0, np.inf, -np.inf]), F32, 0.0, 0.0)
    assert r["mismatch_count"] == 0 and r["inf_count"] == 2 and r["pass"] == 1
    assert r["argmax_idx"] == 0 and r["max_abs_err"] == 0


def test_first_index_wins_ties_and_first_finite_initialises():
    r = oracle.screen_one(f32([np.nan, 1, 1, 1, 1]), f32([0, 1, 3, 3, 1]), F32, 0.0, 0.0)
    assert r["argmax_idx"] == 2 and r["max_abs_err"] == 2
    r = oracle.screen_one(f32([np.nan, 1, 1]), f32([0, 1, 1]), F32, 0.0, 0.0)
    assert r["argmax_idx"] == 1 and r["max_abs_err"] == 0


def test_disjoint_masks_combine_and_full_mask_equals_none():
    rng = np.random.default_rng(6)
    n = 5000
    ref = rng.standard_normal(n).astype(np.float32)
    c = (ref * (1 + 2e-3 * rng.standard_normal(n))).astype(np.float32)
    c[rng.choice(n, 20, replace=False)] = np.nan
    whole = oracle.screen_one(ref, c, F32, 1e-5, 1e-3)
    assert oracle.screen_one(ref, c, F32, 1e-5, 1e-3, mask=("strided", 5, 1, 0)) == whole
    parts = [oracle.screen_one(ref, c, F32, 1e-5, 1e-3, mask=("strided", 5, 3, p)) for p in range(3)]
    assert sum(p["mismatch_count"] for p in parts) == whole["mismatch_count"]
    assert sum(p["nan_count"] for p in parts) == whole["nan_count"]
    assert max(p["max_rel_err"] for p in parts) == whole["max_rel_err"]
    best = max(parts, key=lambda p: (p["max_abs_err"], -p["argmax_idx"]))
    assert best["max_abs_err"] == whole["max_abs_err"] and best["argmax_idx"] == whole["argmax_idx"]


def test_rejects_bad_arguments():
    a = f32([1, 2, 3])
    with pytest.raises(ValueError):
        oracle.screen_one(a, f32([1, 2]), F32, 0, 0)
    with pytest.raises(TypeError):
        oracle.screen_one(a.astype(np.float64), a, F32, 0, 0)
    with pytest.raises(ValueError):
        oracle.screen_one(a, a, F32, 0, 0, mask=("strided", 0, 2, 2))


# --------------------------------------------------------------------------
# 8-bit float formats
# --------------------------------------------------------------------------

def test_fp8_decoders_against_torch():
    """All 256 patterns of both formats against torch's float8 -> float32 conversion."""
    pat = torch.arange(256, dtype=torch.uint8)
    L = oracle.lib()
    for name, fn in (("float8_e4m3fn", L.kbo_decode_f8e4m3), ("float8_e5m2", L.kbo_decode_f8e5m2)):
        want = pat.view(getattr(torch, name)).to(torch.float32).numpy().view(np.uint32)
        for p in range(256):
            g = struct.unpack("<I", struct.pack("<f", fn(p)))[0]
            if (want[p] & 0x7FFFFFFF) > 0x7F800000:
                assert (g & 0x7FFFFFFF) > 0x7F800000, (name, hex(p))
            else:
                assert g == want[p], (name, hex(p))
    assert L.kbo_decode_f8e4m3(0x7E) == 448.0 and L.kbo_decode_f8e5m2(0x7B) == 57344.0
    assert np.isinf(L.kbo_decode_f8e5m2(0x7C)) and np.isnan(L.kbo_decode_f8e4m3(0xFF))


@pytest.mark.parametrize("code,name", [(oracle.F8E4M3, "float8_e4m3fn"), (oracle.F8E5M2, "float8_e5m2")])
def test_fp8_screen_equals_fp32_screen_of_the_decoded_values(code, name):
    """Decoding is exact, so screening fp8 tensors must equal screening their fp32 images."""
    rng = np.random.default_rng(code)
    r8 = rng.integers(0, 256, 5000).astype(np.uint8)
    c8 = r8.copy()
    flip = rng.random(5000) < 0.3
    c8[flip] = (c8[flip].astype(np.int32) + rng.integers(-2, 3, flip.sum())).astype(np.uint8)
    to32 = lambda a: torch.from_numpy(a).view(getattr(torch, name)).to(torch.float32).numpy()
    got = oracle.screen_one(r8, c8, code, 1e-2, 6e-2)
    want = oracle.screen_one(to32(r8), to32(c8), F32, 1e-2, 6e-2)
    assert got == want
    assert got["nan_count"] > 0 and got["mismatch_count"] > 0
