"""Randomised GPU parity: seeded random dtypes, sizes, candidate counts, data shapes (quantised
values with many ties, standard normal, wide dynamic range), perturbations, tolerances, masks,
forced grids and dispatch paths, each compared bit for bit with the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_02611_b200 import synth

pytestmark = pytest.mark.gpu

FIELDS = ["mismatch_count", "nan_count", "inf_count", "argmax_idx", "pass", "reserved"]
TOLS = [(1e-2, 1.6e-2), (0.0, 0.0), (1e-3, 0.0), (0.0, 1e-2), (1e-5, 1e-7), (0.5, 0.5), (1e-4, 2e-3)]
F64 = 99


@pytest.fixture(scope="module")
def kb():
    from paper_2608_02611_b200 import binding
    return binding


@pytest.fixture(scope="module")
def ctx(kb):
    c = kb.Context(0)
    yield c
    c.close()


def same(got, want):
    bad = [f for f in FIELDS if (got[f] != want[f]).any()]
    for f in ("max_abs_err", "max_rel_err"):
        g, w = np.ascontiguousarray(got[f]), np.ascontiguousarray(want[f])
        v = np.uint64 if g.dtype == np.float64 else np.uint32
        if (g.view(v) != w.view(v)).any():
            bad.append(f)
    return bad


def one_case(ctx, kb, seed, log2_lo, log2_hi):
    rng = np.random.default_rng(seed)
    dev = torch.device("cuda", 0)
    code = int(rng.choice([synth.F32, synth.F16, synth.BF16, synth.F8E4M3, synth.F8E5M2, F64]))
    N = int(2 ** rng.uniform(log2_lo, log2_hi))
    K = int(rng.choice([1, 2, 3, 5, 7, 8, 9, 13, 16, 21, 33, 64, 65, 100, 130]))
    if N * K > 2 ** 26:
        K = max(1, 2 ** 26 // N)
    kind = rng.choice(["quant", "normal", "wide"])
    if kind == "quant":
        x = rng.integers(-8, 9, N) / rng.choice([1, 4, 16]) + 0.0
    elif kind == "normal":
        x = rng.standard_normal(N)
    else:
        x = rng.standard_normal(N) * np.exp(3 * rng.standard_normal(N))
    x[rng.random(N) < 0.01] = 0.0
    atol, rtol = TOLS[int(rng.integers(0, len(TOLS)))]
    mask_spec = None
    m = int(rng.integers(0, 5))
    if m in (1, 2):
        stride = int(rng.integers(1, 6))
        log2_tile = int(rng.choice([12, 13])) if m == 1 else int(rng.integers(0, 12))
        mask_spec = ("strided", log2_tile, stride, int(rng.integers(0, stride)))
    elif m == 3:
        log2_tile = int(rng.choice([12, 8, 14]))
        nt = (N + (1 << log2_tile) - 1) >> log2_tile
        mask_spec = ("bitmap", log2_tile, rng.integers(0, 2 ** 63, (nt + 63) // 64, dtype=np.int64).astype(np.uint64))
    grid = int(rng.choice([0, 0, 1, 3, 17, 50]))
    small = bool(rng.integers(0, 2))

    def make_mask():
        if mask_spec is None:
            return None
        if mask_spec[0] == "strided":
            return ctx.mask_strided(N, *mask_spec[1:])
        return ctx.mask_bitmap(N, mask_spec[1], mask_spec[2])

    if code == F64:
        ref = x.astype(np.float64)
        cands = []
        for _ in range(K):
            c = ref.copy()
            mode = int(rng.integers(0, 4))
            f = rng.random(N) < rng.choice([0.01, 0.3])
            if mode == 0:
                c[f] = np.nextafter(c[f], np.inf)
            elif mode == 1:
                c[f] = c[f] + rng.choice([0.5, 0.25, 1.0])
            elif mode == 2:
                c[f] = c[f] * (1 + 1e-9)
            if rng.random() < 0.2:
                c[int(rng.integers(0, N))] = np.nan
            cands.append(c)
        mk = make_mask()
        try:
            ctx.set_grid(grid)
            got = kb.records_f64(ctx.screen_f64(torch.from_numpy(ref).to(dev),
                                                [torch.from_numpy(c).to(dev) for c in cands], atol, rtol, mk))
        finally:
            ctx.set_grid(0)
        want = oracle.screen_f64(ref, cands, atol, rtol, mask_spec, threads=8)
    else:
        tdt = synth.TORCH_DTYPE[code]
        ref = torch.from_numpy(x).to(tdt)
        cands = []
        for _ in range(K):
            mode = int(rng.integers(0, 4))
            f = torch.from_numpy(rng.random(N) < rng.choice([0.01, 0.3]))
            if mode == 0:
                step = torch.from_numpy(rng.integers(-2, 3, N)) * f
                c = synth.ulp_step(ref, code, step.to(torch.int64))
            elif mode == 1:
                c = torch.where(f, (ref.float() + float(rng.choice([0.5, 0.25, 1.0]))).to(tdt), ref)
            elif mode == 2:
                c = torch.where(f, (ref.float() * 1.01).to(tdt), ref)
            else:
                c = ref.clone()
            cands.append(c.contiguous())
        mk = make_mask()
        try:
            ctx.set_grid(grid)
            ctx.set_small_path(small)
            ctx.set_filter(int(rng.integers(0, 4)))      # automatic, plain, sharp or by definition
            got = kb.records(ctx.screen(ref.to(dev), [c.to(dev) for c in cands], atol, rtol, mk))
        finally:
            ctx.set_grid(0)
            ctx.set_small_path(True)
            ctx.set_filter(0)
        want = oracle.screen(synth.to_oracle_array(ref, code), [synth.to_oracle_array(c, code) for c in cands],
                             code, atol, rtol, mask_spec, threads=8)
    assert ctx.poll() == 0
    if mk is not None:
        mk.close()
    bad = same(got, want)
    assert not bad, (f"seed={seed} dtype={code} N={N} K={K} data={kind} tol=({atol},{rtol}) "
                     f"mask={mask_spec[:2] if mask_spec else None} grid={grid} small={small}: {bad} differ")


@pytest.mark.parametrize("block", range(8))
def test_random_small_and_medium(ctx, kb, block):
    for i in range(40):
        one_case(ctx, kb, 7_000_000 + block * 1000 + i, 0, 21)


@pytest.mark.parametrize("block", range(4))
def test_random_large(ctx, kb, block):
    for i in range(5):
        one_case(ctx, kb, 9_000_000 + block * 1000 + i, 20, 24)


@pytest.mark.parametrize("block", range(4))
def test_random_tiny_magnitudes(ctx, kb, block):
    """References and candidates whose magnitudes go from ordinary down through 2^-100, the
    smallest normals and the subnormals to zero, under tolerances from nothing to generous, through
    the plain, the sharp and the by-definition instantiation: where products underflow and
    quotients are undefined is where a filter would go wrong first."""
    rng = np.random.default_rng(31_000 + block)
    dev = torch.device("cuda", 0)
    ctx.set_small_path(False)
    try:
        for _ in range(25):
            code = int(rng.choice([synth.F32, synth.BF16]))
            tdt = synth.TORCH_DTYPE[code]
            N = int(rng.integers(3, 40)) * 4096 + int(rng.integers(0, 4096))
            K = int(rng.choice([1, 3, 8]))
            e = rng.choice([0, -60, -90, -105, -115, -124, -130, -140, -149], size=N,
                           p=[.4, .05, .05, .1, .1, .1, .1, .05, .05])
            x = rng.standard_normal(N) * np.exp2(e.astype(np.float64))
            x[rng.random(N) < 0.05] = 0.0
            ref = torch.from_numpy(x).to(torch.float32).to(tdt)
            cands = []
            for _k in range(K):
                kind = int(rng.integers(0, 4))
                if kind == 0:
                    c = torch.from_numpy(x * (1 + rng.standard_normal(N) * 1e-3)).to(torch.float32).to(tdt)
                elif kind == 1:
                    step = torch.from_numpy(rng.integers(-2, 3, N) * (rng.random(N) < 0.3)).to(torch.int64)
                    c = synth.ulp_step(ref, code, step)
                elif kind == 2:
                    c = torch.where(torch.from_numpy(rng.random(N) < 0.2), torch.zeros_like(ref), ref)
                else:
                    c = torch.where(torch.from_numpy(rng.random(N) < 0.2), ref * 2, ref)
                cands.append(c.contiguous())
            atol = float(rng.choice([0.0, 1e-45, 1e-38, 1e-30, 1e-6]))
            rtol = float(rng.choice([0.0, 1e-7, 1e-3, 1.6e-2, 0.5]))
            want = oracle.screen(synth.to_oracle_array(ref, code), [synth.to_oracle_array(c, code) for c in cands],
                                 code, atol, rtol, threads=8)
            d_ref, d_cands = ref.to(dev), [c.to(dev) for c in cands]
            for mode in (3, 1, 2):
                ctx.set_filter(mode)
                got = kb.records(ctx.screen(d_ref, d_cands, atol, rtol))
                assert not same(got, want), f"mode={mode} dtype={code} N={N} K={K} tol=({atol},{rtol})"
    finally:
        ctx.set_filter(0)
        ctx.set_small_path(True)
    assert ctx.poll() == 0


def fbits(a):
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


@pytest.mark.parametrize("block", range(4))
def test_random_adjudicate_and_select(ctx, kb, block):
    """Random [K][S] timings (log-normal, rounded to create ties, with zero and negative values
    now and then), both win-count algorithms, then selection by both policies and by score."""
    dev = torch.device("cuda", 0)
    for i in range(12):
        rng = np.random.default_rng(11_000_000 + block * 1000 + i)
        K = int(rng.choice([1, 2, 3, 7, 8, 9, 21, 40, 64, 100, 257]))
        S = int(rng.choice([1, 2, 3, 4, 5, 16, 31, 32, 33, 60, 100, 200, 257, 700]))
        t = rng.lognormal(0, rng.choice([0.02, 0.3]), (K, S)) * np.exp(rng.normal(0, 0.2, (K, 1)))
        if rng.random() < 0.5:
            t = np.round(t, int(rng.choice([1, 2])))
        if rng.random() < 0.2:
            t[rng.random((K, S)) < 0.05] = 0.0
            t[(t == 0.0) & (rng.random((K, S)) < 0.5)] = -0.0       # zeros of both signs
        if rng.random() < 0.1:
            t = t - 1.0
        t = t.astype(np.float32)
        omed, oiqr, owins = oracle.adjudicate(t, threads=8)
        for algo in (1, 2, 3):
            try:
                ctx.set_wins_algo(algo)
                med, iqr, wins = ctx.adjudicate(torch.from_numpy(t).to(dev))
            finally:
                ctx.set_wins_algo(0)
            assert ctx.poll() == 0
            label = f"seed block={block} i={i} K={K} S={S} algo={algo}"
            assert (fbits(med.cpu().numpy()) == fbits(omed)).all(), label   # bit patterns: the sorted
            assert (fbits(iqr.cpu().numpy()) == fbits(oiqr)).all(), label   # row is unique (-0 before +0)
            assert (wins.cpu().numpy().view(np.uint32) == owins).all(), label
        rec = np.zeros(K, dtype=oracle.RESULT_DTYPE)
        rec["pass"] = rng.random(K) < 0.7
        rec["mismatch_count"] = 1 - rec["pass"]
        rec["max_rel_err"] = rng.choice(np.float32([0.0, 2.0 ** -7, 2.0 ** -8, 0.01]), K)
        d_rec = torch.from_numpy(rec.view(np.uint8).reshape(K, 48).copy()).to(dev)
        budget = int(rng.integers(1, K + 3))
        for policy in (0, 1):
            surv, n = ctx.select(d_rec, med, policy, budget)
            osurv, on = oracle.select(rec, omed, policy, budget)
            assert int(n.item()) == on and surv.cpu().numpy().tolist() == osurv.tolist()
        if (omed > 0).all():
            sc, surv, n = ctx.select_by_score(d_rec, med, 1, 16, 0.02, 0.01, budget)
            osc, osurv, on = oracle.select_by_score(rec, omed, 1, 16, 0.02, 0.01, budget)
            assert (fbits(sc.cpu().numpy()) == fbits(osc)).all()
            assert int(n.item()) == on and surv.cpu().numpy().tolist() == osurv.tolist()
