"""GPU parity of the double-precision gate (kb_screen_f64) against the CPU oracle, bit for bit.

Seeded synthetic float64 tensors: a reference with a wide magnitude spread, candidates that
differ by a few binary64 ulps on part of the elements, a few large errors, NaN / Inf
injections, zeros, subnormals and huge values.  Sizes span several 4096-element tiles, both
halves of a tile and ragged tails; candidate counts sit around the chunk size; masks are
coarser and finer than a kernel tile; forced grids show that the launch shape is immaterial.
"""
import os

import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu

FIELDS = ["mismatch_count", "nan_count", "inf_count", "argmax_idx", "pass", "reserved"]
THREADS = max(1, len(os.sched_getaffinity(0)))


@pytest.fixture(scope="module")
def kb():
    from paper_2608_02611_b200 import binding
    return binding


@pytest.fixture(scope="module")
def ctx(kb):
    c = kb.Context(0)
    yield c
    c.close()


def make_ref(n, rng, awkward=True):
    x = rng.standard_normal(n) * np.exp(3 * rng.standard_normal(n))
    if awkward:
        u = rng.random(n)
        x[u < 0.02] = 0.0
        specials = [5e-324, -5e-324, 2.2250738585072014e-308, 1.7976931348623157e308, np.inf, -np.inf,
                    np.nan, -0.0, 1e-300, -1e-295]
        for j, v in enumerate(specials):
            x[(u >= 0.02 + 0.002 * j) & (u < 0.02 + 0.002 * (j + 1))] = v
    return x


def perturb(ref, rng, p_flip=0.3, p_big=0.01, p_special=0.002, max_step=2):
    n = ref.size
    bits = ref.view(np.int64).copy()
    step = rng.integers(-max_step, max_step + 1, n) * (rng.random(n) < p_flip)
    mag = bits & np.int64(0x7FFFFFFFFFFFFFFF)
    finite = mag < np.int64(0x7FF0000000000000)
    newmag = np.clip(mag + step, 0, np.int64(0x7FEFFFFFFFFFFFFF))
    bits = np.where(finite, (bits & np.int64(-0x8000000000000000)) | newmag, bits)
    c = bits.view(np.float64).copy()
    big = rng.random(n) < p_big
    with np.errstate(all="ignore"):
        c[big] = c[big] * 1.5 + 0.25
    u = rng.random(n)
    c[u < p_special] = np.nan
    c[(u >= p_special) & (u < 2 * p_special)] = np.inf
    c[(u >= 2 * p_special) & (u < 3 * p_special)] = -np.inf
    return c


def run(ctx, kb, ref, cands, atol, rtol, mask_spec=None):
    dev = torch.device("cuda:0")
    ref_t = torch.from_numpy(ref).to(dev)
    cand_t = [torch.from_numpy(c).to(dev) for c in cands]
    mask = None
    if mask_spec is not None:
        if mask_spec[0] == "strided":
            mask = ctx.mask_strided(ref.size, mask_spec[1], mask_spec[2], mask_spec[3])
        else:
            mask = ctx.mask_bitmap(ref.size, mask_spec[1], mask_spec[2])
    got = kb.records_f64(ctx.screen_f64(ref_t, cand_t, atol, rtol, mask))
    assert ctx.poll() == 0
    if mask is not None:
        mask.close()
    return got


def check(got, want, label=""):
    for f in FIELDS:
        bad = np.nonzero(got[f] != want[f])[0]
        assert bad.size == 0, f"{label} {f} differs at {bad[:8]}: got {got[f][bad[:8]]} want {want[f][bad[:8]]}"
    for f in ("max_abs_err", "max_rel_err"):
        g = np.ascontiguousarray(got[f]).view(np.uint64)
        w = np.ascontiguousarray(want[f]).view(np.uint64)
        bad = np.nonzero(g != w)[0]
        assert bad.size == 0, f"{label} {f} differs at {bad[:8]}: got {got[f][bad[:8]]} want {want[f][bad[:8]]}"


def both(ctx, kb, ref, cands, atol, rtol, mask_spec=None, label=""):
    got = run(ctx, kb, ref, cands, atol, rtol, mask_spec)
    want = oracle.screen_f64(ref, cands, atol, rtol, mask_spec, threads=THREADS)
    check(got, want, label)
    return got


@pytest.mark.parametrize("N", [1, 100, 2048, 4096, 4096 + 17, 5 * 4096 + 2047, 40 * 4096 + 333,
                               300 * 4096 + 2049])
def test_sizes_and_tails(ctx, kb, N):
    rng = np.random.default_rng(N)
    ref = make_ref(N, rng)
    cands = [perturb(ref, rng, p_flip=0.1 * (k % 4), p_big=0.0 if k % 3 else 0.01) for k in range(9)]
    cands.append(ref.copy())
    both(ctx, kb, ref, cands, 1e-12, 1e-15, label=f"N={N}")
    both(ctx, kb, ref, cands, 0.0, 0.0, label=f"N={N} exact")


@pytest.mark.parametrize("K", [1, 7, 63, 64, 65, 130])
def test_candidate_counts_around_chunk_size(ctx, kb, K):
    rng = np.random.default_rng(100 + K)
    N = 24 * 4096 + 1000
    ref = make_ref(N, rng, awkward=False)
    cands = [perturb(ref, rng, p_flip=0.2, p_big=0.001 * (k % 5), p_special=0.0 if k % 7 else 0.001)
             for k in range(K)]
    both(ctx, kb, ref, cands, 1e-13, 3e-16, label=f"K={K}")


@pytest.mark.parametrize("grid", [1, 3, 37])
def test_result_does_not_depend_on_grid(ctx, kb, grid):
    rng = np.random.default_rng(7)
    N = 64 * 4096 + 5
    ref = make_ref(N, rng)
    cands = [perturb(ref, rng) for _ in range(20)]
    try:
        ctx.set_grid(grid)
        both(ctx, kb, ref, cands, 1e-10, 1e-15, label=f"grid={grid}")
    finally:
        ctx.set_grid(0)


@pytest.mark.parametrize("mask_spec", [("strided", 12, 3, 1), ("strided", 13, 2, 0), ("strided", 5, 4, 3),
                                       ("strided", 0, 7, 2), ("strided", 12, 1000, 999)])
def test_masks(ctx, kb, mask_spec):
    rng = np.random.default_rng(11)
    N = 50 * 4096 + 777
    ref = make_ref(N, rng)
    cands = [perturb(ref, rng) for _ in range(6)]
    both(ctx, kb, ref, cands, 1e-12, 1e-15, mask_spec, label=str(mask_spec))


def test_bitmap_masks_and_empty_selection(ctx, kb):
    rng = np.random.default_rng(12)
    N = 40 * 4096 + 50
    ref = make_ref(N, rng)
    cands = [perturb(ref, rng) for _ in range(5)]
    for log2_tile in (12, 6):
        ntiles = (N + (1 << log2_tile) - 1) >> log2_tile
        words = rng.integers(0, 2 ** 63, (ntiles + 63) // 64, dtype=np.int64).astype(np.uint64)
        both(ctx, kb, ref, cands, 1e-12, 1e-15, ("bitmap", log2_tile, words), label=f"bitmap {log2_tile}")
        empty = np.zeros((ntiles + 63) // 64, dtype=np.uint64)
        got = both(ctx, kb, ref, cands, 1e-12, 1e-15, ("bitmap", log2_tile, empty))
        assert (got["argmax_idx"] == -1).all() and (got["pass"] == 1).all()


def test_identical_candidates_and_ties_pick_the_lowest_index(ctx, kb):
    rng = np.random.default_rng(13)
    N = 30 * 4096
    ref = np.ldexp(rng.integers(1, 1 << 20, N).astype(np.float64), -10)     # dyadic
    same = ref.copy()
    ties = ref.copy()
    pos = np.sort(rng.choice(N, 40, replace=False))
    ties[pos] += 0.5                                   # the same error at 40 places
    late = ref.copy()
    late[pos[-1]] += 0.5
    late[pos[5]] += 0.25
    got = both(ctx, kb, ref, [same, ties, late, same], 0.0, 0.0)
    assert got["argmax_idx"][0] == 0 and got["max_abs_err"][0] == 0.0 and got["pass"][0] == 1
    assert got["argmax_idx"][1] == pos[0] and got["argmax_idx"][2] == pos[-1]


def test_extreme_reference_magnitudes(ctx, kb):
    rng = np.random.default_rng(14)
    N = 12 * 4096 + 100
    expo = rng.integers(-1074, -940, N)
    ref = np.ldexp(1.0 + rng.random(N), expo) * rng.choice([-1.0, 1.0], N)
    cands = [perturb(ref, rng, p_flip=0.5, max_step=3) for _ in range(6)]
    both(ctx, kb, ref, cands, 0.0, 1e-15, label="tiny")
    ref = np.ldexp(1.0 + rng.random(N), rng.integers(1000, 1024, N)) * rng.choice([-1.0, 1.0], N)
    cands = [perturb(ref, rng, p_flip=0.5, max_step=3) for _ in range(6)]
    both(ctx, kb, ref, cands, 1e300, 1e-15, label="huge")


def test_sees_differences_below_binary32_resolution(ctx, kb):
    N = 8 * 4096
    ref = np.ones(N)
    cand = ref.copy()
    cand[20000] = 1 + 2.0 ** -40
    got = both(ctx, kb, ref, [cand], 0.0, 2.0 ** -45)
    assert got["mismatch_count"][0] == 1 and got["argmax_idx"][0] == 20000
    assert got["max_abs_err"][0] == 2.0 ** -40


def test_argument_errors(ctx, kb):
    dev = torch.device("cuda:0")
    ref = torch.zeros(4096, dtype=torch.float64, device=dev)
    with pytest.raises(kb.KbError):
        ctx.screen_f64(ref, [ref.float()], 0.0, 0.0)
    with pytest.raises(kb.KbError):
        ctx.screen_f64(ref, [ref], -1.0, 0.0)
    with pytest.raises(kb.KbError):
        ctx.screen_f64(ref, [ref], 0.0, float("inf"))
    with pytest.raises(kb.KbError):
        ctx.screen_f64(ref, [], 0.0, 0.0)
    with pytest.raises(kb.KbError):
        ctx.screen_f64(ref, [ref[1:4095].clone()[1:]], 0.0, 0.0)
    big = torch.zeros(4098, dtype=torch.float64, device=dev)
    with pytest.raises(kb.KbError) as e:
        ctx.screen_f64(big[1:4097], [ref], 0.0, 0.0)          # 8-byte aligned only
    assert e.value.status == 2
    assert ctx.poll() == 0


def test_large(ctx, kb):
    """2^24 elements, 12 candidates: the launch configuration of a full-size call."""
    rng = np.random.default_rng(15)
    N = (1 << 24) + 4096 + 5
    ref = make_ref(N, rng, awkward=False)
    cands = []
    for k in range(12):
        c = ref.copy()
        m = rng.random(N) < 0.25
        c[m] = c[m] * (1 + rng.choice([-1, 1], int(m.sum())) * 2.0 ** -52)
        if k % 4 == 3:
            c[rng.integers(0, N, 50)] *= 1.01
        if k == 5:
            c[rng.integers(0, N, 3)] = np.nan
        cands.append(c)
    both(ctx, kb, ref, cands, 1e-14, 3e-16, label="large")
