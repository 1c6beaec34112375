"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle.

Everything is compared bit for bit: counts, flags, indices, the bit patterns of
max_abs_err / max_rel_err / median / IQR, the win counts and the survivor
order.  Sizes span several 4096-element tiles plus ragged tails, all three
dtypes, masks finer and coarser than a kernel tile, candidate counts around
the chunk size of the streaming kernel, and several forced grid sizes (the
result must not depend on the launch shape).
"""
import json
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2608_02611_b200 import synth

pytestmark = pytest.mark.gpu

GOLD = os.path.join(os.path.dirname(__file__), "golden")
FIELDS = ["mismatch_count", "nan_count", "inf_count", "argmax_idx", "pass", "reserved"]


@pytest.fixture(scope="module")
def kb():
    from paper_2608_02611_b200 import binding
    return binding


@pytest.fixture(scope="module")
def ctx(kb):
    c = kb.Context(0)
    yield c
    c.close()


def fbits(a):
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


def assert_records_equal(got, want, label=""):
    for f in FIELDS:
        bad = np.nonzero(got[f] != want[f])[0]
        assert bad.size == 0, f"{label} field {f} differs at candidates {bad[:8]}: " \
                              f"got {got[f][bad[:8]]} want {want[f][bad[:8]]}"
    for f in ("max_abs_err", "max_rel_err"):
        bad = np.nonzero(fbits(got[f]) != fbits(want[f]))[0]
        assert bad.size == 0, f"{label} field {f} differs at candidates {bad[:8]}: " \
                              f"got {got[f][bad[:8]]} want {want[f][bad[:8]]}"


def oracle_screen(case_dtype, ref_t, cand_ts, atol, rtol, mask_spec=None, threads=None):
    threads = threads or max(1, len(os.sched_getaffinity(0)))
    ref = synth.to_oracle_array(ref_t, case_dtype)
    cands = [synth.to_oracle_array(c, case_dtype) for c in cand_ts]
    return oracle.screen(ref, cands, case_dtype, atol, rtol, mask_spec, threads=threads)


def awkward(n, dtype_code, rng, device):
    """Random values with zeros, subnormals, huge values, NaN and Inf mixed in."""
    x = rng.standard_normal(n) * np.exp(3 * rng.standard_normal(n))
    x[rng.random(n) < 0.02] = 0.0
    t = torch.from_numpy(x).to(synth.TORCH_DTYPE[dtype_code])
    bits = synth._bits(t, dtype_code)
    u = torch.from_numpy(rng.random(n))
    inf_mag = synth._INF_MAG[dtype_code]
    sign = synth._SIGN_BIT[dtype_code]
    specials = [1, 2, inf_mag - 1, inf_mag, inf_mag | 1, sign | inf_mag, sign | 1, sign]
    for j, pat in enumerate(specials):
        bits = torch.where((u >= 0.004 * j) & (u < 0.004 * (j + 1)), torch.full_like(bits, pat), bits)
    return synth._from_bits(bits, dtype_code).to(device)


def perturbed(ref, dtype_code, rng, device, p_flip=0.3, p_big=0.01, p_special=0.003):
    n = ref.numel()
    step = torch.from_numpy(rng.integers(-2, 3, n)) * torch.from_numpy(rng.random(n) < p_flip)
    c = synth.ulp_step(ref.cpu(), dtype_code, step.to(torch.int64))
    big = torch.from_numpy(rng.random(n) < p_big)
    c = torch.where(big, (c.float() * 1.5 + 0.25).to(c.dtype), c)
    u = torch.from_numpy(rng.random(n))
    bits = synth._bits(c.contiguous(), dtype_code)
    inf_mag, sign = synth._INF_MAG[dtype_code], synth._SIGN_BIT[dtype_code]
    nan_pat = inf_mag | 1 if dtype_code != synth.F8E4M3 else inf_mag      # e4m3fn: 0x7F is its NaN
    bits = torch.where(u < p_special, torch.full_like(bits, nan_pat), bits)
    bits = torch.where((u >= p_special) & (u < 2 * p_special), torch.full_like(bits, inf_mag), bits)
    bits = torch.where((u >= 2 * p_special) & (u < 3 * p_special), torch.full_like(bits, sign | inf_mag), bits)
    c = synth._from_bits(bits, dtype_code)
    return c.contiguous().to(device)


def run_screen(ctx, kb, ref, cands, atol, rtol, mask_spec=None, N=None):
    mask = None
    if mask_spec is not None:
        N = ref.numel()
        if mask_spec[0] == "strided":
            mask = ctx.mask_strided(N, mask_spec[1], mask_spec[2], mask_spec[3])
        else:
            mask = ctx.mask_bitmap(N, mask_spec[1], mask_spec[2])
    # both dispatch paths: the general (streaming) one and, where the size allows it, the
    # single-launch kernel for small problems; they must agree byte for byte
    # (and the general path with the streaming kernel launched in plain stream order instead of
    # as a programmatic dependent of the lead kernel)
    try:
        ctx.set_small_path(False)
        rec = kb.records(ctx.screen(ref, cands, atol, rtol, mask))
        ctx.set_dependent_launch(False)
        rec_plain = kb.records(ctx.screen(ref, cands, atol, rtol, mask))
        ctx.set_dependent_launch(True)
        for mode in (2, 3):                 # the sharp and the by-definition instantiation
            ctx.set_filter(mode)
            rec_mode = kb.records(ctx.screen(ref, cands, atol, rtol, mask))
            assert rec.tobytes() == rec_mode.tobytes(), f"filter mode {mode}"
    finally:
        ctx.set_small_path(True)
        ctx.set_dependent_launch(True)
        ctx.set_filter(0)
    rec_small = kb.records(ctx.screen(ref, cands, atol, rtol, mask))
    assert ctx.poll() == 0
    assert rec.tobytes() == rec_small.tobytes()
    assert rec.tobytes() == rec_plain.tobytes()
    if mask is not None:
        mask.close()
    return rec


# --------------------------------------------------------------------------
# stored + live oracle on the small seeded configurations
# --------------------------------------------------------------------------

def _golden():
    with open(os.path.join(GOLD, "oracle_small_cases.json")) as f:
        return json.load(f)


def _check_against_stored(rec, med, iqr, wins, surv, n, stored):
    for k, s in enumerate(stored["screen"]):
        assert int(rec["mismatch_count"][k]) == s["mismatch_count"]
        assert int(rec["nan_count"][k]) == s["nan_count"]
        assert int(rec["inf_count"][k]) == s["inf_count"]
        assert int(rec["argmax_idx"][k]) == s["argmax_idx"]
        assert int(fbits(rec["max_abs_err"])[k]) == s["max_abs_err_bits"]
        assert int(fbits(rec["max_rel_err"])[k]) == s["max_rel_err_bits"]
        assert int(rec["pass"][k]) == s["passed"]
    assert fbits(med).tolist() == stored["median_bits"]
    assert fbits(iqr).tolist() == stored["iqr_bits"]
    assert wins.astype(np.int64).tolist() == stored["wins"]
    assert surv.tolist() == stored["survivors"] and n == stored["n_survivors"]


SMALL = {
    "config1": lambda dev: synth.config1(dev),
    "config2_side512_K16": lambda dev: synth.config2(dev, side=512, K=16, n_bad=3),
    "config3_small": lambda dev: synth.config3(dev, B=1, H=2, S=64, D=128, K=12, n_nan=2,
                                               n_transposed=2, S_t=50),
    "config4_small": lambda dev: synth.config4(dev, N=1 << 14, K=40, S_t=16),
}


@pytest.mark.parametrize("name", list(SMALL))
def test_small_configs_whole_path(ctx, kb, name):
    # inputs are built on the host so that the bytes are the ones the stored values came from
    case, timings = SMALL[name]("cpu")
    stored = _golden()[name]
    dev = torch.device("cuda", 0)
    ref = case.ref.to(dev)
    cands_cpu = case.cands()
    cands = [c.to(dev) for c in cands_cpu]
    out = ctx.screen(ref, cands, case.atol, case.rtol)
    t = torch.from_numpy(timings).to(dev)
    med, iqr, wins = ctx.adjudicate(t)
    surv, n = ctx.select(out, med, stored["policy"], stored["budget"])
    assert ctx.poll() == 0
    rec = kb.records(out)
    want = oracle_screen(case.dtype, case.ref, cands_cpu, case.atol, case.rtol)
    assert_records_equal(rec, want, name)
    _check_against_stored(rec, med.cpu().numpy(), iqr.cpu().numpy(),
                          wins.cpu().numpy().view(np.uint32), surv.cpu().numpy(), int(n.item()), stored)


def test_config5_small_two_tier(ctx, kb):
    c5 = synth.config5("cpu", N=1 << 20, K=32, budget=4, S1=20, S2=40)
    case = c5["case"]
    stored = _golden()["config5_small_tier1"]
    dev = torch.device("cuda", 0)
    ref = case.ref.to(dev)
    cands_cpu = case.cands()
    cands = [c.to(dev) for c in cands_cpu]
    _, log2_tile, stride, phase = case.mask
    mask = ctx.mask_strided(case.N, log2_tile, stride, phase)
    assert mask.n_selected == case.N // stride
    out1 = ctx.screen(ref, cands, case.atol, case.rtol, mask)
    med1, iqr1, wins1 = ctx.adjudicate(torch.from_numpy(c5["timings1"]).to(dev))
    surv, n = ctx.select(out1, med1, kb.KB_SELECT_ERR_THEN_TIME, c5["budget"])
    assert ctx.poll() == 0
    rec1 = kb.records(out1)
    _check_against_stored(rec1, med1.cpu().numpy(), iqr1.cpu().numpy(),
                          wins1.cpu().numpy().view(np.uint32), surv.cpu().numpy(), int(n.item()), stored)
    # tier 2: the survivors on every element, chained from the device-side survivor list
    s = surv.cpu().numpy()[: int(n.item())].tolist()
    out2 = ctx.screen(ref, [cands[k] for k in s], case.atol, case.rtol)
    rec2 = kb.records(out2)
    want2 = oracle_screen(case.dtype, case.ref, [cands_cpu[k] for k in s], case.atol, case.rtol)
    assert_records_equal(rec2, want2, "tier2")
    t2 = c5["make_timings2"](s)
    med2, iqr2, wins2 = ctx.adjudicate(torch.from_numpy(t2).to(dev))
    omed, oiqr, owins = oracle.adjudicate(t2)
    assert (fbits(med2.cpu().numpy()) == fbits(omed)).all()
    assert (fbits(iqr2.cpu().numpy()) == fbits(oiqr)).all()
    assert (wins2.cpu().numpy().view(np.uint32) == owins).all()
    mask.close()


# --------------------------------------------------------------------------
# awkward values, ragged sizes, chunk boundaries, grid independence
# --------------------------------------------------------------------------

@pytest.mark.parametrize("dtype_code", [synth.F32, synth.F16, synth.BF16, synth.F8E4M3, synth.F8E5M2])
@pytest.mark.parametrize("N", [1, 7, 8, 9, 15, 16, 17, 4095, 4096, 4097, 3 * 4096 + 5, 20 * 4096 + 123])
def test_awkward_values_and_ragged_sizes(ctx, kb, dtype_code, N):
    rng = np.random.default_rng(N * 3 + dtype_code)
    dev = torch.device("cuda", 0)
    ref = awkward(N, dtype_code, rng, dev)
    cands = [ref.clone(), perturbed(ref, dtype_code, rng, dev), awkward(N, dtype_code, rng, dev),
             perturbed(ref, dtype_code, rng, dev, p_flip=0.01, p_big=0.0, p_special=0.0)]
    for atol, rtol in [(1e-5, 1e-3), (0.0, 0.0), (1e-2, 1.6e-2)]:
        got = run_screen(ctx, kb, ref, cands, atol, rtol)
        want = oracle_screen(dtype_code, ref, cands, atol, rtol)
        assert_records_equal(got, want, f"N={N} dtype={dtype_code} tol=({atol},{rtol})")


@pytest.mark.parametrize("dtype_code", [synth.F32, synth.F16, synth.BF16])
@pytest.mark.parametrize("atol,rtol", [(1e-3, 0.0), (0.0, 1e-2), (1e-2, 1e-7), (0.0, 3e-3), (1e30, 0.0),
                                       (1e-4, 5e-4), (0.0, 1.0), (6e-8, 9.5367431640625e-07)])
def test_tolerance_regimes_on_dense_small_differences(ctx, kb, dtype_code, atol, rtol):
    """Differences of a unit or two in the last place on a third of the elements, values near zero
    included (their relative error is large, so they pass by atol or not at all): relative error
    below, around and above rtol; rtol too small for the filter's shortcut; atol only; rtol only."""
    rng = np.random.default_rng(int(atol * 1e9) + int(rtol * 1e9) + dtype_code)
    dev = torch.device("cuda", 0)
    N = 48 * 4096 + 77
    x = rng.standard_normal(N) * np.exp(2 * rng.standard_normal(N))
    x[rng.random(N) < 0.05] *= 1e-6
    x[rng.random(N) < 0.01] = 0.0
    ref = torch.from_numpy(x).to(synth.TORCH_DTYPE[dtype_code]).to(dev)
    cands = [perturbed(ref, dtype_code, rng, dev, p_flip=0.33, p_big=0.0, p_special=0.0) for _ in range(5)]
    cands.append(perturbed(ref, dtype_code, rng, dev, p_flip=0.33, p_big=0.001, p_special=0.0))
    cands.append(perturbed(ref, dtype_code, rng, dev, p_flip=0.33, p_big=0.0, p_special=0.0005))
    cands.append(ref.clone())
    got = run_screen(ctx, kb, ref, cands, atol, rtol)
    want = oracle_screen(dtype_code, ref, cands, atol, rtol)
    assert_records_equal(got, want, f"dtype={dtype_code} tol=({atol},{rtol})")


def test_many_quotients_within_units_in_the_last_place_of_the_max_rel_err(ctx, kb):
    """Relative errors packed within a few units in the last place of each other: the running
    maximum is challenged from both sides of every rounding boundary.  fp32: c = r*(1 + q0*(1+u)),
    |u| < 2^-21.  bf16 / fp16: one-ulp differences everywhere except on the powers of two, so that
    the largest quotient (1/129, 1/1025) is inexact and shared by a whole significand class."""
    rng = np.random.default_rng(99)
    dev = torch.device("cuda", 0)
    N = 64 * 4096 + 333
    r64 = rng.standard_normal(N) * np.exp(rng.standard_normal(N))
    r32 = r64.astype(np.float32)
    cands = []
    for q0 in (0.01, 0.0123456, 2.0 ** -7 * 1.5, 0.3):
        u = rng.uniform(-2.0 ** -21, 2.0 ** -21, N)
        cands.append(torch.from_numpy((r32.astype(np.float64) * (1 + q0 * (1 + u))).astype(np.float32)).to(dev))
    ref = torch.from_numpy(r32).to(dev)
    for atol, rtol in [(1e-2, 1.6e-2), (0.0, 0.5), (1e-3, 1e-3)]:
        got = run_screen(ctx, kb, ref, cands, atol, rtol)
        want = oracle_screen(synth.F32, ref, cands, atol, rtol)
        assert_records_equal(got, want, f"fp32 near ties tol=({atol},{rtol})")
    for code in (synth.BF16, synth.F16):
        tdt = synth.TORCH_DTYPE[code]
        ref = torch.from_numpy(r64).to(tdt).to(dev)
        eps = 2.0 ** -8 if code == synth.BF16 else 2.0 ** -11
        cands = []
        for k in range(6):
            flip = torch.from_numpy(rng.random(N) < (0.25 if k < 4 else 0.01)).to(dev)
            cands.append(torch.where(flip, (ref.float() * (1 + eps)).to(tdt), ref))   # ties-to-even spares 2^k
        got = run_screen(ctx, kb, ref, cands, 1e-2, 1.6e-2)
        want = oracle_screen(code, ref, cands, 1e-2, 1.6e-2)
        assert_records_equal(got, want, f"dtype={code} shared inexact maximum")


@pytest.mark.parametrize("K", [1, 3, 33, 127, 128, 129, 300])
def test_candidate_counts_around_chunk_size(ctx, kb, K):
    rng = np.random.default_rng(K)
    dev = torch.device("cuda", 0)
    N = 6 * 4096 + 17
    ref = awkward(N, synth.BF16, rng, dev)
    base = [perturbed(ref, synth.BF16, rng, dev) for _ in range(5)]
    cands = []
    for k in range(K):
        c = base[k % 5].clone()
        c[(k * 977) % N] = float(k)            # make every candidate different
        cands.append(c)
    got = run_screen(ctx, kb, ref, cands, 1e-2, 1.6e-2)
    want = oracle_screen(synth.BF16, ref, cands, 1e-2, 1.6e-2)
    assert_records_equal(got, want, f"K={K}")


def test_prepared_candidate_set_is_the_same_call(ctx, kb):
    rng = np.random.default_rng(4242)
    dev = torch.device("cuda", 0)
    N = 5 * 4096 + 3
    ref = awkward(N, synth.BF16, rng, dev)
    cands = [perturbed(ref, synth.BF16, rng, dev) for _ in range(9)]
    held = kb.Candidates(cands)
    assert len(held) == 9
    want = oracle_screen(synth.BF16, ref, cands, 1e-2, 1.6e-2)
    for _ in range(3):                                          # the same object serves every call
        got = kb.records(ctx.screen(ref, held, 1e-2, 1.6e-2))
        assert_records_equal(got, want, "prepared candidate set")
    m = ctx.mask_strided(N, 12, 2, 1)
    assert torch.equal(ctx.screen(ref, held, 1e-2, 1.6e-2, m), ctx.screen(ref, cands, 1e-2, 1.6e-2, m))
    m.close()
    with pytest.raises(kb.KbError):                             # made for another element count
        ctx.screen(ref[:4096].contiguous(), held, 1e-2, 1.6e-2)
    with pytest.raises(kb.KbError):
        kb.Candidates([cands[0], cands[1].float()])


@pytest.mark.parametrize("grid", [1, 2, 5, 37, 0])
def test_result_does_not_depend_on_grid(ctx, kb, grid):
    rng = np.random.default_rng(99)
    dev = torch.device("cuda", 0)
    N = 41 * 4096 + 1000
    ref = awkward(N, synth.F16, rng, dev)
    cands = [perturbed(ref, synth.F16, rng, dev) for _ in range(9)] + [ref.clone()]
    want = oracle_screen(synth.F16, ref, cands, 1e-3, 1e-2)
    try:
        ctx.set_grid(grid)
        got = run_screen(ctx, kb, ref, cands, 1e-3, 1e-2)
    finally:
        ctx.set_grid(0)
    assert_records_equal(got, want, f"grid={grid}")


def test_ties_on_max_abs_err_pick_lowest_index(ctx, kb):
    dev = torch.device("cuda", 0)
    N = 30 * 4096
    ref = torch.zeros(N, dtype=torch.float32, device=dev)
    c = ref.clone()
    hits = [29 * 4096 + 5, 17 * 4096 + 4000, 3 * 4096 + 77, 3 * 4096 + 78]
    c[hits] = 0.5                                  # equal errors in several tiles and threads
    for grid in (0, 1, 3):
        ctx.set_grid(grid)
        rec = run_screen(ctx, kb, ref, [c, ref.clone()], 0.0, 0.0)
        ctx.set_grid(0)
        assert rec["argmax_idx"].tolist() == [3 * 4096 + 77, 0]
        assert rec["max_abs_err"].tolist() == [0.5, 0.0]
        assert rec["mismatch_count"].tolist() == [4, 0]
        assert rec["max_rel_err"].tolist() == [0.0, 0.0]       # reference is zero everywhere


MASKS = [("strided", 0, 3, 1), ("strided", 3, 2, 0), ("strided", 7, 5, 4), ("strided", 11, 2, 1),
         ("strided", 12, 2, 1), ("strided", 12, 16, 5), ("strided", 13, 3, 0), ("strided", 14, 1, 0),
         ("strided", 20, 1, 0)]


@pytest.mark.parametrize("mask_spec", MASKS)
@pytest.mark.parametrize("N", [50 * 4096, 50 * 4096 + 999])
def test_masks(ctx, kb, mask_spec, N):
    rng = np.random.default_rng(N + mask_spec[1])
    dev = torch.device("cuda", 0)
    ref = awkward(N, synth.BF16, rng, dev)
    cands = [perturbed(ref, synth.BF16, rng, dev) for _ in range(3)] + [ref.clone()]
    got = run_screen(ctx, kb, ref, cands, 1e-2, 1.6e-2, mask_spec)
    want = oracle_screen(synth.BF16, ref, cands, 1e-2, 1.6e-2, mask_spec)
    assert_records_equal(got, want, f"mask={mask_spec} N={N}")


@pytest.mark.parametrize("log2_tile", [2, 9, 12, 13])
def test_bitmap_masks_and_empty_selection(ctx, kb, log2_tile):
    rng = np.random.default_rng(log2_tile)
    dev = torch.device("cuda", 0)
    N = 33 * 4096 + 77
    nt = (N + (1 << log2_tile) - 1) >> log2_tile
    ref = awkward(N, synth.F32, rng, dev)
    cands = [perturbed(ref, synth.F32, rng, dev) for _ in range(3)]
    for density in (0.0, 0.3, 1.0):
        words = np.zeros((nt + 63) // 64, dtype=np.uint64)
        for t in np.nonzero(rng.random(nt) < density)[0] if density < 1.0 else range(nt):
            words[int(t) >> 6] |= np.uint64(1) << np.uint64(int(t) & 63)
        spec = ("bitmap", log2_tile, words)
        got = run_screen(ctx, kb, ref, cands, 1e-5, 1e-3, spec)
        want = oracle_screen(synth.F32, ref, cands, 1e-5, 1e-3, spec)
        assert_records_equal(got, want, f"bitmap log2_tile={log2_tile} density={density}")
        if density == 0.0:
            assert (got["argmax_idx"] == -1).all() and (got["pass"] == 1).all()


def test_extreme_reference_magnitudes(ctx, kb):
    """Tiny and huge |r| where the filter's products could underflow or overflow."""
    dev = torch.device("cuda", 0)
    vals = np.float32([1e-38, 3e-39, 1e-45, 2e-44, 1e38, 3e38, 1e-31, 1e31, 1.0, 0.0])
    N = 5 * 4096
    rng = np.random.default_rng(3)
    ref_np = rng.choice(vals, N).astype(np.float32)
    ref = torch.from_numpy(ref_np).to(dev)
    cands = []
    for scale in (1.0000001, 1.5, 0.5, 3.0):
        c = (ref_np.astype(np.float64) * scale).astype(np.float32)
        same = rng.random(N) < 0.5
        c[same] = ref_np[same]
        cands.append(torch.from_numpy(c).to(dev))
    cands.append(torch.from_numpy(np.nextafter(ref_np, np.float32(np.inf))).to(dev))
    got = run_screen(ctx, kb, ref, cands, 0.0, 1e-3)
    want = oracle_screen(synth.F32, ref, cands, 0.0, 1e-3)
    assert_records_equal(got, want, "extreme")


# --------------------------------------------------------------------------
# argument errors leave outputs untouched and never reach the device
# --------------------------------------------------------------------------

def test_argument_errors(ctx, kb):
    dev = torch.device("cuda", 0)
    ref = torch.zeros(64, dtype=torch.float32, device=dev)
    out = torch.full((1, 48), 0xAB, dtype=torch.uint8, device=dev)
    for atol, rtol in [(-1.0, 0.0), (0.0, float("inf")), (float("nan"), 0.0)]:
        with pytest.raises(kb.KbError) as e:
            ctx.screen(ref, [ref.clone()], atol, rtol, out=out)
        assert e.value.status == 1
    with pytest.raises(kb.KbError) as e:
        ctx.screen(ref, [], 0.0, 0.0)
    assert e.value.status == 1
    with pytest.raises(kb.KbError) as e:                       # misaligned candidate view
        big = torch.zeros(65, dtype=torch.float32, device=dev)
        ctx.screen(ref, [big[1:]], 0.0, 0.0, out=out)
    assert e.value.status == 2
    with pytest.raises(kb.KbError) as e:                       # dtype constraint of the policy check
        ctx.screen(ref.double(), [ref.double()], 0.0, 0.0, out=out)
    assert e.value.status == 3
    with pytest.raises(kb.KbError):
        ctx.mask_strided(64, 3, 2, 2)
    m = ctx.mask_strided(128, 3, 2, 1)
    with pytest.raises(kb.KbError):                            # mask made for another N
        ctx.screen(ref, [ref.clone()], 0.0, 0.0, m, out=out)
    m.close()
    assert (out.cpu() == 0xAB).all()
    t = torch.ones((3, 4), dtype=torch.float32, device=dev)
    with pytest.raises(kb.KbError):
        ctx.select(out, t[0], 7, 1)
    assert ctx.poll() == 0


# --------------------------------------------------------------------------
# adjudication and selection
# --------------------------------------------------------------------------

@pytest.mark.parametrize("K,S", [(1, 1), (2, 2), (3, 3), (4, 4), (5, 5), (21, 4), (21, 16), (21, 60),
                                 (8, 31), (9, 32), (17, 33), (33, 64), (16, 100), (24, 200), (7, 256),
                                 (6, 257), (5, 300), (12, 1000), (4, 2000), (3, 2049)])
def test_adjudicate_matches_oracle(ctx, kb, K, S):
    """Both win-count algorithms (direct comparison of all sample pairs; binary search on
    the sorted rows) give the oracle's integers."""
    rng = np.random.default_rng(K * 10007 + S)
    dev = torch.device("cuda", 0)
    for ties in (False, True):
        t = rng.lognormal(0, 0.1, (K, S))
        if ties:
            t = np.round(t, 2)
        t = t.astype(np.float32)
        omed, oiqr, owins = oracle.adjudicate(t)
        for algo in (1, 2, 3, 0):
            if algo == 3 and S > 1024:
                continue
            try:
                ctx.set_wins_algo(algo)
                med, iqr, wins = ctx.adjudicate(torch.from_numpy(t).to(dev))
            finally:
                ctx.set_wins_algo(0)
            assert ctx.poll() == 0
            assert (fbits(med.cpu().numpy()) == fbits(omed)).all()
            assert (fbits(iqr.cpu().numpy()) == fbits(oiqr)).all()
            w = wins.cpu().numpy().view(np.uint32)
            assert (w == owins).all(), (algo, np.argwhere(w != owins)[:5])


def test_adjudicate_long_rows_use_direct_comparison(ctx, kb):
    """S > 4096: a block of sorted rows no longer fits shared memory."""
    rng = np.random.default_rng(4097)
    dev = torch.device("cuda", 0)
    t = np.round(rng.lognormal(0, 0.1, (3, 4100)), 3).astype(np.float32)
    med, iqr, wins = ctx.adjudicate(torch.from_numpy(t).to(dev))
    omed, oiqr, owins = oracle.adjudicate(t)
    assert (fbits(med.cpu().numpy()) == fbits(omed)).all()
    assert (wins.cpu().numpy().view(np.uint32) == owins).all()
    ctx.set_wins_algo(2)
    try:
        with pytest.raises(kb.KbError):
            ctx.adjudicate(torch.from_numpy(t).to(dev))
    finally:
        ctx.set_wins_algo(0)


def test_adjudicate_negative_and_zero_timings(ctx, kb):
    """Zeros of both signs: the sorted row is unique (-0 before +0), so medians and IQRs are
    compared as bit patterns, signs of zeros included."""
    dev = torch.device("cuda", 0)
    t = np.float32([[0.0, -1.0, 2.0, -0.0, 1.0], [1.0, 0.0, -2.0, 5.0, 1.0], [3.0, 3.0, 3.0, 3.0, 3.0],
                    [0.0, -0.0, 0.0, -0.0, -0.0], [-0.0, 0.0, 0.0, 0.0, 0.0], [-0.0, -0.0, -0.0, -0.0, -0.0]])
    omed, oiqr, owins = oracle.adjudicate(t)
    assert fbits(omed).tolist()[3:] == [0x80000000, 0, 0x80000000]
    for algo in (1, 2, 3):
        ctx.set_wins_algo(algo)
        med, iqr, wins = ctx.adjudicate(torch.from_numpy(t).to(dev))
        ctx.set_wins_algo(0)
        assert (fbits(med.cpu().numpy()) == fbits(omed)).all()
        assert (fbits(iqr.cpu().numpy()) == fbits(oiqr)).all()
        assert (wins.cpu().numpy().view(np.uint32) == owins).all()
    rng = np.random.default_rng(18)
    for S in (2, 7, 32, 33, 100, 257):
        t = rng.choice(np.float32([0.0, -0.0, 0.0, -0.0, 1.0, -1.0]), (9, S)).astype(np.float32)
        omed, oiqr, owins = oracle.adjudicate(t)
        med, iqr, wins = ctx.adjudicate(torch.from_numpy(t).to(dev))
        assert (fbits(med.cpu().numpy()) == fbits(omed)).all(), S
        assert (fbits(iqr.cpu().numpy()) == fbits(oiqr)).all(), S
        assert (wins.cpu().numpy().view(np.uint32) == owins).all()
        rat = ctx.tail_ratios(torch.from_numpy(np.abs(t) + np.float32(1.0)).to(dev))
        assert (fbits(rat.cpu().numpy()) == fbits(oracle.tail_ratios(np.abs(t) + np.float32(1.0)))).all()


def test_adjudicate_flags_nonfinite(ctx, kb):
    dev = torch.device("cuda", 0)
    for bad in (float("nan"), float("inf"), float("-inf")):
        t = torch.ones((5, 40), dtype=torch.float32, device=dev)
        t[3, 17] = bad
        ctx.adjudicate(t)
        assert ctx.poll() == 6          # KB_ERR_NONFINITE
        assert ctx.poll() == 0          # the status word is cleared by the read


def test_adjudicate_flags_nonfinite_with_many_candidates(ctx, kb):
    """The lane-per-row merge (K >= 225) stages its rows with non-finite samples replaced, so
    that its walk stays inside the rows; the call is flagged and the other rows' medians hold."""
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(3)
    base = rng.lognormal(0, 0.1, (300, 50)).astype(np.float32)
    omed = oracle.adjudicate(base, want_wins=False)[0]
    for bad in (float("nan"), float("inf"), float("-inf")):
        t = torch.from_numpy(base).to(dev)
        t[7, 3] = bad
        t[250, 49] = bad
        med, iqr, wins = ctx.adjudicate(t)
        assert ctx.poll() == 6          # KB_ERR_NONFINITE
        keep = np.ones(300, dtype=bool)
        keep[[7, 250]] = False
        assert (med.cpu().numpy()[keep] == omed[keep]).all()


@pytest.mark.parametrize("policy", [0, 1])
@pytest.mark.parametrize("K,budget", [(1, 1), (7, 3), (33, 8), (64, 64), (40, 100), (300, 32), (1000, 7)])
def test_select_matches_oracle(ctx, kb, policy, K, budget):
    rng = np.random.default_rng(K * 31 + budget + policy)
    dev = torch.device("cuda", 0)
    rec = np.zeros(K, dtype=oracle.RESULT_DTYPE)
    rec["pass"] = rng.random(K) < 0.6
    rec["mismatch_count"] = 1 - rec["pass"]
    rec["max_rel_err"] = rng.choice(np.float32([0.0, 2.0 ** -7, 2.0 ** -8, 0.01, np.inf]), K)
    med = rng.choice(np.float32([0.9, 1.0, 1.0, 1.1, 0.0, -0.0]), K).astype(np.float32)
    d_rec = torch.from_numpy(rec.view(np.uint8).reshape(K, 48).copy()).to(dev)
    surv, n = ctx.select(d_rec, torch.from_numpy(med).to(dev), policy, budget)
    osurv, on = oracle.select(rec, med, policy, budget)
    assert int(n.item()) == on
    assert surv.cpu().numpy().tolist() == osurv.tolist()


def test_screen_host_matches_screen(ctx, kb):
    """kb_screen_host (host buffers, batched copies) gives the records of kb_screen."""
    case, _ = synth.config2("cpu", side=256, K=9, n_bad=2, block=64)
    N = case.N - 77
    ref = case.ref[:N].clone()
    cands = [case.make_cand(k)[:N].clone() for k in range(case.K)]
    got = ctx.screen_host(ref, cands, case.atol, case.rtol)
    dev = torch.device("cuda", 0)
    want = kb.records(ctx.screen(ref.to(dev), [c.to(dev) for c in cands], case.atol, case.rtol))
    assert got.tobytes() == want.tobytes()
    oracle_rec = oracle_screen(case.dtype, ref, cands, case.atol, case.rtol)
    assert_records_equal(got, oracle_rec, "screen_host")


# --------------------------------------------------------------------------
# scheduler-side statistics: runtime score, tail ratios, Copeland counts
# --------------------------------------------------------------------------

@pytest.mark.parametrize("K,budget", [(1, 1), (9, 4), (64, 32), (300, 50), (1000, 1000)])
def test_select_by_score_matches_oracle(ctx, kb, K, budget):
    rng = np.random.default_rng(K + budget)
    dev = torch.device("cuda", 0)
    for rung, b_r in [(0, 4), (1, 16), (2, 60)]:
        rec = np.zeros(K, dtype=oracle.RESULT_DTYPE)
        rec["pass"] = rng.random(K) < 0.7
        med = rng.lognormal(0, 1.0, K).astype(np.float32)
        med[rng.random(K) < 0.2] = np.float32(0.0005)             # below 1 us: scores tie
        med[rng.random(K) < 0.2] = np.float32(1.0)
        d_rec = torch.from_numpy(rec.view(np.uint8).reshape(K, 48).copy()).to(dev)
        score, surv, n = ctx.select_by_score(d_rec, torch.from_numpy(med).to(dev), rung, b_r, 0.02, 0.01, budget)
        osc, osurv, on = oracle.select_by_score(rec, med, rung, b_r, 0.02, 0.01, budget)
        assert (fbits(score.cpu().numpy()) == fbits(osc)).all()
        assert int(n.item()) == on and surv.cpu().numpy().tolist() == osurv.tolist()


@pytest.mark.parametrize("K,S", [(1, 1), (3, 2), (21, 4), (21, 16), (21, 60), (7, 101), (64, 100),
                                 (5, 2000), (2, 5000)])
def test_tail_ratios_match_oracle(ctx, kb, K, S):
    rng = np.random.default_rng(K * 77 + S)
    dev = torch.device("cuda", 0)
    t = rng.lognormal(0, 0.1, (K, S)).astype(np.float32)
    got = ctx.tail_ratios(torch.from_numpy(t).to(dev)).cpu().numpy()
    assert ctx.poll() == 0
    want = oracle.tail_ratios(t)
    assert (fbits(got) == fbits(want)).all()


@pytest.mark.parametrize("K,S", [(1, 3), (2, 3), (9, 16), (64, 100), (130, 20)])
def test_copeland_matches_oracle(ctx, kb, K, S):
    rng = np.random.default_rng(K + S)
    dev = torch.device("cuda", 0)
    t = np.round(rng.lognormal(0, 0.1, (K, S)), 2).astype(np.float32)
    if K > 1:
        t[K - 1] = t[0]
    med, iqr, wins = ctx.adjudicate(torch.from_numpy(t).to(dev))
    beats, ties = ctx.copeland(wins, S)
    ob, ot = oracle.copeland(oracle.adjudicate(t)[2], S)
    assert (beats.cpu().numpy().view(np.uint32) == ob).all()
    assert (ties.cpu().numpy().view(np.uint32) == ot).all()


def test_confirm_matches_oracle(ctx, kb):
    rng = np.random.default_rng(21)
    dev = torch.device("cuda", 0)
    K = 3000
    prev = rng.lognormal(5, 1, K).astype(np.float32)
    s1 = (prev * rng.choice(np.float32([0.9, 1.0, 1.05, 1.0500001, 1.2]), K)).astype(np.float32)
    s2 = (prev * rng.choice(np.float32([0.9, 1.05, 1.06, 1.3]), K)).astype(np.float32)
    st, sc = ctx.confirm(torch.from_numpy(s1).to(dev), torch.from_numpy(s2).to(dev),
                         torch.from_numpy(prev).to(dev), 0.05)
    ost, osc = oracle.confirm(s1, s2, prev, 0.05)
    assert (st.cpu().numpy().view(np.uint32) == ost).all()
    assert (fbits(sc.cpu().numpy()) == fbits(osc)).all()
    assert set(ost.tolist()) == {0, 1, 2}


# --------------------------------------------------------------------------
# device-resident tier chaining: select -> screen_indexed, no host round trip
# --------------------------------------------------------------------------

def _tier_setup(dev):
    c5 = synth.config5("cpu", N=(1 << 20) + 333, K=32, budget=4, S1=20, S2=40)
    case = c5["case"]
    ref = case.ref.to(dev)
    cands_cpu = case.cands()
    cands = [c.to(dev) for c in cands_cpu]
    return c5, case, ref, cands_cpu, cands


@pytest.mark.parametrize("budget", [4, 30])
def test_screen_indexed_chain(ctx, kb, budget):
    dev = torch.device("cuda", 0)
    c5, case, ref, cands_cpu, cands = _tier_setup(dev)
    _, log2_tile, stride, phase = case.mask
    mask = ctx.mask_strided(case.N, log2_tile, stride, phase)
    table = ctx.pointer_table(cands)
    out1 = ctx.screen(ref, cands, case.atol, case.rtol, mask)
    med1, _, _ = ctx.adjudicate(torch.from_numpy(c5["timings1"]).to(dev))
    surv, n = ctx.select(out1, med1, kb.KB_SELECT_ERR_THEN_TIME, budget)
    out2 = ctx.screen_indexed(ref, table, surv, n, case.atol, case.rtol)      # nothing came to the host yet
    assert ctx.poll() == 0
    s = surv.cpu().numpy()
    nn = int(n.item())
    assert nn == min(budget, 16) and (s[nn:] == -1).all()
    rec2 = kb.records(out2)
    want = oracle_screen(case.dtype, case.ref, [cands_cpu[k] for k in s[:nn]], case.atol, case.rtol)
    assert_records_equal(rec2[:nn], want, "indexed tier 2")
    for j in range(nn, budget):                                            # empty slots
        r = rec2[j]
        assert (r["mismatch_count"], r["nan_count"], r["inf_count"], r["argmax_idx"], r["pass"]) == (0, 0, 0, -1, 0)
    # the same through the host-driven call
    rec_host = kb.records(ctx.screen(ref, [cands[k] for k in s[:nn]], case.atol, case.rtol))
    assert rec_host.tobytes() == rec2[:nn].tobytes()
    mask.close()


def test_screen_indexed_rejects_bad_selections_on_the_device(ctx, kb):
    dev = torch.device("cuda", 0)
    N = 3 * 4096 + 5
    ref = torch.zeros(N, dtype=torch.float32, device=dev)
    big = torch.zeros(N + 1, dtype=torch.float32, device=dev)
    good = ref.clone()                                                     # must outlive the table
    table = ctx.pointer_table([good, big[1:]])                             # entry 1 is misaligned
    one = torch.tensor([1], dtype=torch.int32, device=dev)
    cases = [(torch.tensor([0, 7], dtype=torch.int32, device=dev), torch.tensor([2], dtype=torch.int32, device=dev), 1),
             (torch.tensor([0, 1], dtype=torch.int32, device=dev), torch.tensor([2], dtype=torch.int32, device=dev), 2),
             (torch.tensor([0, 0], dtype=torch.int32, device=dev), torch.tensor([3], dtype=torch.int32, device=dev), 1)]
    for index, count, status in cases:
        out = ctx.screen_indexed(ref, table, index, count, 0.0, 0.0)
        assert ctx.poll() == status
        rec = kb.records(out)
        assert (rec["pass"] == 0).all() and (rec["argmax_idx"] == -1).all()
    out = ctx.screen_indexed(ref, table, torch.tensor([0, 1], dtype=torch.int32, device=dev), one, 0.0, 0.0)
    assert ctx.poll() == 0                                                  # the bad entry is beyond the count
    rec = kb.records(out)
    assert rec["pass"].tolist() == [1, 0] and rec["argmax_idx"].tolist() == [0, -1]


def test_two_tier_chain_in_one_cuda_graph(ctx, kb):
    dev = torch.device("cuda", 0)
    c5, case, ref, cands_cpu, cands = _tier_setup(dev)
    _, log2_tile, stride, phase = case.mask
    mask = ctx.mask_strided(case.N, log2_tile, stride, phase)
    table = ctx.pointer_table(cands)
    t1 = torch.from_numpy(c5["timings1"]).to(dev)
    budget = 4
    out1 = torch.empty((case.K, kb.RESULT_BYTES), dtype=torch.uint8, device=dev)
    out2 = torch.empty((budget, kb.RESULT_BYTES), dtype=torch.uint8, device=dev)

    def chain():
        ctx.screen(ref, cands, case.atol, case.rtol, mask, out=out1)
        med, iqr, wins = ctx.adjudicate(t1)
        surv, n = ctx.select(out1, med, kb.KB_SELECT_ERR_THEN_TIME, budget)
        ctx.screen_indexed(ref, table, surv, n, case.atol, case.rtol, out=out2)
        return surv, n

    surv, n = chain()                      # warm-up: grows every workspace before the capture
    torch.cuda.synchronize()
    want1, want2 = kb.records(out1).tobytes(), kb.records(out2).tobytes()
    want_s = surv.cpu().numpy().tolist()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            g_surv, g_n = chain()
    for _ in range(2):
        out1.fill_(0xEE)
        out2.fill_(0xEE)
        graph.replay()
        torch.cuda.synchronize()
        assert kb.records(out1).tobytes() == want1 and kb.records(out2).tobytes() == want2
        assert g_surv.cpu().numpy().tolist() == want_s
    assert ctx.poll() == 0
    mask.close()


@pytest.mark.parametrize("K,smax", [(1, 5), (6, 60), (21, 60), (40, 300), (9, 4096)])
def test_adjudicate_ragged_matches_oracle(ctx, kb, K, smax):
    rng = np.random.default_rng(K * 13 + smax)
    dev = torch.device("cuda", 0)
    lens = rng.integers(1, smax + 1, K)
    lens[0] = smax
    rows = [np.round(rng.lognormal(0, 0.1, int(n)), 2).astype(np.float32) for n in lens]
    off = np.zeros(K + 1, dtype=np.int32)
    off[1:] = np.cumsum(lens)
    flat = torch.from_numpy(np.concatenate(rows)).to(dev)
    med, iqr, wins = ctx.adjudicate_ragged(flat, torch.from_numpy(off).to(dev), smax)
    assert ctx.poll() == 0
    omed, oiqr, owins = oracle.adjudicate_ragged(rows)
    assert (fbits(med.cpu().numpy()) == fbits(omed)).all()
    assert (fbits(iqr.cpu().numpy()) == fbits(oiqr)).all()
    assert (wins.cpu().numpy().view(np.uint32) == owins).all()


def test_adjudicate_ragged_flags_a_row_longer_than_the_bound(ctx, kb):
    dev = torch.device("cuda", 0)
    flat = torch.ones(30, dtype=torch.float32, device=dev)
    off = torch.tensor([0, 10, 30], dtype=torch.int32, device=dev)       # second row has 20 > 16
    ctx.adjudicate_ragged(flat, off, 16)
    assert ctx.poll() == 1


@pytest.mark.parametrize("dtype_code", [synth.F32, synth.BF16, synth.F8E4M3])
def test_screen_multi_shapes_in_one_launch(ctx, kb, dtype_code):
    """Three output shapes of one benchmark (512, 1024, 2048 elements, as the mat-vec sweep of
    the paper's appendix) plus an awkward one, 21 candidates each, one launch."""
    rng = np.random.default_rng(7 + dtype_code)
    dev = torch.device("cuda", 0)
    groups, want = [], []
    for N in (512, 1024, 2048, 3 * 4096 + 17):
        ref = awkward(N, dtype_code, rng, dev)
        cands = [ref.clone()] + [perturbed(ref, dtype_code, rng, dev) for _ in range(20)]
        groups.append((ref, cands))
        want.append(oracle_screen(dtype_code, ref, cands, 1e-2, 1.6e-2))
    launches0 = ctx.launch_count
    for _ in range(2):                                    # twice: the tickets reset themselves
        out = ctx.screen_multi(groups, 1e-2, 1.6e-2)
        got = kb.records(out)
        assert_records_equal(got, np.concatenate(want), "multi")
    assert ctx.launch_count - launches0 == 2
    assert ctx.poll() == 0
    # a job that is too large is refused with a pointer to kb_screen
    big = torch.zeros(4096 * 30, dtype=torch.uint8, device=dev).view(torch.int8).to(torch.float32).to(synth.TORCH_DTYPE[dtype_code]) \
        if dtype_code == synth.F8E4M3 else torch.zeros(4096 * 30, dtype=synth.TORCH_DTYPE[dtype_code], device=dev)
    with pytest.raises(kb.KbError) as e:
        ctx.screen_multi([(big, [big] * 100)], 0.0, 0.0)
    assert e.value.status == 3


@pytest.mark.parametrize("dtype_code", [synth.F8E4M3, synth.F8E5M2])
def test_fp8_large_with_masks_and_grids(ctx, kb, dtype_code):
    """8-bit formats through the streaming kernel: many tiles, a ragged tail, a coarse mask."""
    rng = np.random.default_rng(100 + dtype_code)
    dev = torch.device("cuda", 0)
    N = 300 * 4096 + 77
    ref = awkward(N, dtype_code, rng, dev)
    cands = [perturbed(ref, dtype_code, rng, dev, p_flip=0.01, p_big=0.0, p_special=0.0) for _ in range(6)]
    cands += [perturbed(ref, dtype_code, rng, dev), ref.clone()]
    for mask_spec in (None, ("strided", 12, 4, 1)):
        want = oracle_screen(dtype_code, ref, cands, 1e-2, 7e-2, mask_spec)
        for grid in (0, 3):
            ctx.set_grid(grid)
            got = run_screen(ctx, kb, ref, cands, 1e-2, 7e-2, mask_spec)
            ctx.set_grid(0)
            assert_records_equal(got, want, f"fp8 {dtype_code} mask={mask_spec} grid={grid}")


def test_alu_probe_reports_a_rate(ctx, kb):
    rate = ctx.alu_probe(2000)
    assert 1e11 < rate < 1e14          # sample pairs per second; 148 SMs x 64 lanes x 2 GHz / 2 = 9.3e12
    assert ctx.poll() == 0


@pytest.mark.parametrize("dtype_code", [synth.F8E4M3, synth.F8E5M2])
def test_fp8_every_byte_pair_behind_established_maxima(ctx, kb, dtype_code):
    """Every (reference byte, candidate byte) combination of an 8-bit format, each ALONE in the
    512 bytes a warp of the e4m3 kernel looks at in one step (everything around it identical in
    reference and candidate), scanned after a leading block has established a large absolute
    error and a chosen relative error.  The e4m3 kernel declares a warp clean from its packed
    half-precision pre-filter alone, so here that decision rests on one pair at a time: a pair
    wrongly declared clean (a subtraction that rounds in binary16, a product that rounds to zero,
    a tie with a running maximum, NaN patterns, zeros) loses a count or a maximum.  Candidates
    keep different subsets of the pairs, so that they stay lean or not and establish different
    maxima; tolerances lie on both sides of the pre-filter's bound of 1/2."""
    dev = torch.device("cuda", 0)
    tdt = synth.TORCH_DTYPE[dtype_code]
    val = torch.arange(256, dtype=torch.uint8).view(tdt).float()               # value of every byte
    rb = torch.arange(256, dtype=torch.int64).repeat_interleave(256)          # reference byte
    cb = torch.arange(256, dtype=torch.int64).repeat(256)                     # candidate byte
    one = {synth.F8E4M3: 0x38, synth.F8E5M2: 0x3C}[dtype_code]                # the byte of 1.0
    lead = 8 * 4096                                                           # the scouted tiles
    rng = np.random.default_rng(8 + dtype_code)
    perm = torch.from_numpy(rng.permutation(65536))
    rb, cb = rb[perm], cb[perm]
    # pair p sits in tile p // 4, in the first 512-byte region of warp p % 4, at a varying offset
    pos = lead + (torch.arange(65536) // 4) * 4096 + (torch.arange(65536) % 4) * 512 + \
        (torch.arange(65536) * 37) % 512
    N = lead + 16384 * 4096
    fill = torch.from_numpy(rng.integers(0, 0x78, N)).to(torch.int64)          # finite positive fillers
    fill[:lead] = one
    ref_bytes = fill.clone()
    ref_bytes[pos] = rb
    d = (val[cb] - val[rb]).abs()
    ratio = d / val[rb].abs()
    keep_sets = [torch.ones(65536, dtype=torch.bool), ratio <= 0.3, ratio <= 0.14, d <= 1.0,
                 (rb - cb).abs() <= 1, (ratio <= 0.126) & (d <= 0.5), (d <= 2.0) & (ratio <= 0.5)]
    two = one + 8 if dtype_code == synth.F8E4M3 else one + 4                   # the byte of 2.0
    leads = [(0x7E, one + 1), (0x50, one + 2), (one + 1, one + 1), (0x7E, one), (0x60, one + 4), (0x30, one + 1),
             (two, one + 1)]                                                   # (established error 1.0: pairs above it follow)
    to_t = lambda b: b.to(torch.uint8).to(dev).view(tdt)
    ref = to_t(ref_bytes)
    cts = []
    for keep, (big, small) in zip(keep_sets, leads):
        c = ref_bytes.clone()
        c[pos[keep]] = cb[keep]
        c[5] = big            # a large absolute error at a low index
        c[9000] = small       # a relative error of a few units in the last place
        cts.append(to_t(c))
    for atol, rtol in ((1e-2, 0.13), (0.0, 0.26), (1e-3, 0.5), (1e-2, 0.75), (0.0, 0.0), (1.0, 0.04)):
        want = oracle_screen(dtype_code, ref, cts, atol, rtol)
        for grid in (0, 5):
            ctx.set_grid(grid)
            try:
                ctx.set_small_path(False)
                got = kb.records(ctx.screen(ref, cts, atol, rtol))
            finally:
                ctx.set_small_path(True)
                ctx.set_grid(0)
            assert ctx.poll() == 0
            assert_records_equal(got, want, f"fp8 {dtype_code} atol={atol} rtol={rtol} grid={grid}")


# --------------------------------------------------------------------------
# records of a range from the records of its parts (element-range sharding)
# --------------------------------------------------------------------------

@pytest.mark.parametrize("dtype_code", [synth.F32, synth.BF16, synth.F16])
@pytest.mark.parametrize("cuts", [[], [4096], [4096, 8192, 12288], [8192, 36864]])
def test_merge_ranges_gives_the_whole_range(ctx, kb, dtype_code, cuts):
    rng = np.random.default_rng(31 + dtype_code + len(cuts))
    dev = torch.device("cuda", 0)
    N = 10 * 4096 + 333
    ref = awkward(N, dtype_code, rng, dev)
    cands = [perturbed(ref, dtype_code, rng, dev) for _ in range(5)]
    same_err = ref.clone()                          # the same largest error on both sides of every cut
    ref[0] = 1.0
    same_err[0] = 1.0
    for cut in cuts:
        for i in (cut - 1, cut):
            ref[i] = 1.0
            same_err[i] = 3.0
    for c in cands:
        for i in [0] + [j for cut in cuts for j in (cut - 1, cut)]:
            c[i] = ref[i]
    all_nan_first_part = ref.clone()                # a part without any finite difference
    all_nan_first_part[: (cuts[0] if cuts else N)] = float("nan")
    cands += [same_err, all_nan_first_part]
    want = oracle_screen(dtype_code, ref, cands, 1e-2, 1.6e-2)
    first = [0] + cuts
    last = cuts + [N]
    parts = torch.stack([ctx.screen(ref[a:b], [c[a:b] for c in cands], 1e-2, 1.6e-2) for a, b in zip(first, last)])
    got = kb.records(ctx.merge_ranges(parts, first))
    assert_records_equal(got, want, f"dtype={dtype_code} cuts={cuts}")
    # ... and the oracle's own merge of the oracle's own part records says the same
    oparts = [oracle_screen(dtype_code, ref[a:b], [c[a:b] for c in cands], 1e-2, 1.6e-2) for a, b in zip(first, last)]
    assert_records_equal(got, oracle.merge_ranges(oparts, first), "oracle merge")
    assert ctx.poll() == 0


def test_merge_ranges_argument_errors(ctx, kb):
    dev = torch.device("cuda", 0)
    parts = torch.zeros((2, 3, 48), dtype=torch.uint8, device=dev)
    with pytest.raises(kb.KbError):
        ctx.merge_ranges(parts, [4096, 4096])                     # must ascend
    with pytest.raises(kb.KbError):
        ctx.merge_ranges(parts, [0])                              # one index per part
    with pytest.raises(kb.KbError):
        ctx.merge_ranges(torch.zeros((65, 1, 48), dtype=torch.uint8, device=dev), list(range(0, 65 * 4096, 4096)))
    assert ctx.poll() == 0
