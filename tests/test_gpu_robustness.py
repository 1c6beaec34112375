"""Failure paths and out-of-bounds checks on the GPU, none of which faults, traps or hangs it.

* a bounded device-side wait that runs out (a stand-alone warp waiting on a barrier nothing
  completes, with no copy in flight) is reported through kb_ctx_poll and leaves the context
  usable;
* a workspace allocation that fails (refused by a hook, the device's memory is not touched)
  leaves the context with its old, valid buffers;
* guard bands: every caller-owned output sits between two bands of a canary pattern that must
  be intact after the call, and the library's own device buffers carry the same bands
  (kb_ctx_check_guards) -- the stand-in for a memory checker;
* reads: every input sits between halos of NaN patterns, so that an element read from outside
  a tensor changes the records (NaN count, mismatch count, non-finite timing).
"""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2608_02611_b200 import synth

pytestmark = pytest.mark.gpu

THREADS = max(1, len(os.sched_getaffinity(0)))
CANARY = 0xA5
BAND = 256


@pytest.fixture(scope="module")
def kb():
    from paper_2608_02611_b200 import binding
    return binding


@pytest.fixture()
def ctx(kb):
    c = kb.Context(0)
    yield c
    c.close()


def fbits(a):
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


def same_records(got, want):
    for f in want.dtype.names:
        a, b = got[f], want[f]
        if a.dtype.kind == "f":
            a, b = a.view(np.uint32 if a.dtype.itemsize == 4 else np.uint64), \
                b.view(np.uint32 if b.dtype.itemsize == 4 else np.uint64)
        assert (a == b).all(), f


class Guarded:
    """A device tensor of `shape`/`dtype` placed between two canary bands."""

    def __init__(self, shape, dtype, dev):
        n = int(np.prod(shape)) * torch.empty(0, dtype=dtype).element_size()
        self.nbytes = n
        self.raw = torch.full((n + 2 * BAND,), CANARY, dtype=torch.uint8, device=dev)
        self.t = self.raw[BAND:BAND + n].view(dtype).view(shape)

    def intact(self):
        torch.cuda.synchronize()
        return bool((self.raw[:BAND] == CANARY).all()) and bool((self.raw[BAND + self.nbytes:] == CANARY).all())


def oracle_records(case_dtype, ref, cands, atol, rtol, mask=None):
    return oracle.screen(synth.to_oracle_array(ref, case_dtype),
                         [synth.to_oracle_array(c, case_dtype) for c in cands],
                         case_dtype, atol, rtol, mask, threads=THREADS)


# ---------------------------------------------------------------------------------------------

def test_bounded_wait_runs_out_and_the_context_stays_usable(ctx, kb):
    dev = torch.device("cuda", 0)
    case, _ = synth.config2(dev, side=768, K=12, n_bad=3)          # K*N > 2^22: the streaming gate
    cands = case.cands()
    want = oracle_records(case.dtype, case.ref, cands, case.atol, case.rtol)
    same_records(kb.records(ctx.screen(case.ref, cands, case.atol, case.rtol)), want)
    assert ctx.poll() == 0
    ctx.selftest_wait(1_000_000)                   # one warp, 1 ms limit, nothing arrives
    assert ctx.poll() == 7                         # KB_ERR_DEVICE_TIMEOUT
    assert ctx.poll() == 0                         # cleared by the read
    # the next call on the same context is exact, and the status stays clear
    same_records(kb.records(ctx.screen(case.ref, cands, case.atol, case.rtol)), want)
    assert ctx.poll() == 0
    with pytest.raises(kb.KbError):
        ctx.selftest_wait(10)                      # limits outside [1 us, 100 ms] are refused
    with pytest.raises(kb.KbError):
        ctx.selftest_wait(10_000_000_000)


def test_failed_workspace_growth_keeps_the_old_workspace(ctx, kb):
    dev = torch.device("cuda", 0)
    ctx.set_small_path(False)                      # the general path uses the growing workspace
    rng = np.random.default_rng(11)
    ref = torch.from_numpy(rng.standard_normal(5000).astype(np.float32)).to(dev)
    cands = [ref.clone() for _ in range(40)]
    cands[7][123] += 1.0
    want = oracle_records(synth.F32, ref, cands, 1e-5, 1e-3)
    same_records(kb.records(ctx.screen(ref, cands, 1e-5, 1e-3)), want)       # workspace for 40 (x2)
    many = [ref] * 3000                            # needs a larger workspace
    out = torch.full((3000, kb.RESULT_BYTES), 0xAB, dtype=torch.uint8, device=dev)
    ctx.fail_next_allocs(1)
    with pytest.raises(kb.KbError) as e:
        ctx.screen(ref, many, 1e-5, 1e-3, out=out)
    assert e.value.status == 4                     # KB_ERR_WORKSPACE
    assert (out.cpu() == 0xAB).all()               # nothing was launched
    # the old workspace is still there and still right
    same_records(kb.records(ctx.screen(ref, cands, 1e-5, 1e-3)), want)
    # and with the hook spent the large call goes through
    rec = kb.records(ctx.screen(ref, many, 1e-5, 1e-3, out=out))
    assert (rec["pass"] == 1).all()
    assert ctx.poll() == 0

    # sorted-timings buffer of kb_adjudicate
    t_small = np.round(rng.lognormal(0, 0.1, (16, 40)), 2).astype(np.float32)
    t_big = np.round(rng.lognormal(0, 0.1, (64, 200)), 2).astype(np.float32)
    ctx.set_wins_algo(2)
    med, iqr, wins = ctx.adjudicate(torch.from_numpy(t_small).to(dev))
    ow = oracle.adjudicate(t_small)[2]
    assert (wins.cpu().numpy().view(np.uint32) == ow).all()
    ctx.fail_next_allocs(1)
    with pytest.raises(kb.KbError) as e:
        ctx.adjudicate(torch.from_numpy(t_big).to(dev))
    assert e.value.status == 4
    med, iqr, wins = ctx.adjudicate(torch.from_numpy(t_small).to(dev))      # old buffer, still valid
    assert (wins.cpu().numpy().view(np.uint32) == ow).all()
    ctx.set_wins_algo(0)
    ctx.fail_next_allocs(1)                        # automatic choice: falls back to direct comparison
    med, iqr, wins = ctx.adjudicate(torch.from_numpy(t_big).to(dev))
    assert (wins.cpu().numpy().view(np.uint32) == oracle.adjudicate(t_big, threads=THREADS)[2]).all()
    assert ctx.poll() == 0

    # host-buffer path: the SECOND of its two batch buffers fails to grow
    h_ref = ref.cpu()
    h_cands = [c.cpu() for c in cands]
    same_records(ctx.screen_host(h_ref, h_cands, 1e-5, 1e-3), want)
    big_ref = torch.from_numpy(rng.standard_normal(300000).astype(np.float32))
    big_cands = [big_ref.clone() for _ in range(3)]
    big_cands[1][299999] = float("nan")
    ctx.fail_next_allocs(1, skip=2)                # reference staging, first batch buffer pass
    with pytest.raises(kb.KbError) as e:
        ctx.screen_host(big_ref, big_cands, 1e-5, 1e-3)
    assert e.value.status == 4
    same_records(ctx.screen_host(h_ref, h_cands, 1e-5, 1e-3), want)          # small call still right
    rec = ctx.screen_host(big_ref, big_cands, 1e-5, 1e-3)
    assert rec["pass"].tolist() == [1, 0, 1] and rec["nan_count"].tolist() == [0, 1, 0]
    nb, bad = ctx.check_guards()
    assert nb >= 6 and bad == 0


@pytest.mark.parametrize("dtype", [synth.F32, synth.F16, synth.BF16])
def test_guard_bands_around_screen_outputs(ctx, kb, dtype):
    """kb_screen on every dispatch path writes K records and nothing else."""
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(100 + dtype)
    N = 5 * 4096 + 37                              # full tiles plus a ragged tail
    tdt = synth.TORCH_DTYPE[dtype]
    ref = torch.from_numpy(rng.standard_normal(N).astype(np.float32)).to(tdt).to(dev)
    K = 13
    cands = []
    for k in range(K):
        c = ref.clone()
        if k % 3 == 1:
            c[rng.integers(0, N, 5)] = 2.5
        if k == 4:
            c[N - 1] = float("nan")
        cands.append(c)
    want = oracle_records(dtype, ref, cands, 1e-3, 1e-2)
    spec = ("strided", 5, 3, 1)
    want_fine = oracle_records(dtype, ref, cands, 1e-3, 1e-2, spec)
    spec_c = ("strided", 12, 2, 1)
    want_coarse = oracle_records(dtype, ref, cands, 1e-3, 1e-2, spec_c)
    fine = ctx.mask_strided(N, 5, 3, 1)
    coarse = ctx.mask_strided(N, 12, 2, 1)
    for small in (True, False):
        ctx.set_small_path(small)
        for grid in (0, 1, 5):
            ctx.set_grid(grid)
            for mask, w in ((None, want), (fine, want_fine), (coarse, want_coarse)):
                g = Guarded((K, kb.RESULT_BYTES), torch.uint8, dev)
                ctx.screen(ref, cands, 1e-3, 1e-2, mask, out=g.t)
                assert g.intact(), (small, grid)
                same_records(kb.records(g.t), w)
    ctx.set_grid(0)
    ctx.set_small_path(True)
    fine.close()
    coarse.close()
    # several shapes in one launch
    groups = [(ref[:n].clone(), [c[:n].clone() for c in cands[:kk]]) for n, kk in ((700, 3), (4096, 5), (9001, 2))]
    g = Guarded((10, kb.RESULT_BYTES), torch.uint8, dev)
    ctx.screen_multi(groups, 1e-3, 1e-2, out=g.t)
    assert g.intact()
    got = kb.records(g.t)
    o = 0
    for r, cs in groups:
        same_records(got[o:o + len(cs)], oracle_records(dtype, r, cs, 1e-3, 1e-2))
        o += len(cs)
    # a selection that lives on the device, with fewer survivors than slots
    table = ctx.pointer_table(cands)
    index = torch.tensor([4, 0, 9, 1, 1, 1], dtype=torch.int32, device=dev)
    count = torch.tensor([3], dtype=torch.int32, device=dev)
    g = Guarded((6, kb.RESULT_BYTES), torch.uint8, dev)
    ctx.screen_indexed(ref, table, index, count, 1e-3, 1e-2, out=g.t)
    assert g.intact()
    got = kb.records(g.t)
    same_records(got[:3], want[[4, 0, 9]])
    assert (got["pass"][3:] == 0).all() and (got["argmax_idx"][3:] == -1).all()
    assert ctx.poll() == 0
    nb, bad = ctx.check_guards()
    assert nb >= 3 and bad == 0                    # status words, single-launch workspace, accumulators


def test_guard_bands_around_the_double_precision_gate(ctx, kb):
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(64)
    N = 9 * 4096 + 5
    ref = torch.from_numpy(rng.standard_normal(N)).to(dev)
    cands = [ref.clone() for _ in range(5)]
    cands[2][N - 1] += 1e-3
    cands[3][4096] = float("inf")
    g = Guarded((5, kb.RESULT_F64_BYTES), torch.uint8, dev)
    ctx.screen_f64(ref, cands, 1e-12, 1e-9, out=g.t)
    assert g.intact()
    want = oracle.screen_f64(ref.cpu().numpy(), [c.cpu().numpy() for c in cands], 1e-12, 1e-9)
    same_records(kb.records_f64(g.t), want)
    assert ctx.poll() == 0
    assert ctx.check_guards()[1] == 0


@pytest.mark.parametrize("K,S", [(3, 5), (13, 33), (37, 100), (230, 17), (9, 4100)])
def test_guard_bands_around_adjudication_and_selection_outputs(ctx, kb, K, S):
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(K * 1000 + S)
    t = np.round(rng.lognormal(0, 0.1, (K, S)), 2).astype(np.float32)
    omed, oiqr, owins = oracle.adjudicate(t, threads=THREADS)
    d_t = torch.from_numpy(t).to(dev)
    for algo in (0, 1, 2, 3):
        if (algo == 2 and S > 4096) or (algo == 3 and S > 1024):
            continue
        ctx.set_wins_algo(algo)
        gm, gi = Guarded((K,), torch.float32, dev), Guarded((K,), torch.float32, dev)
        gw = Guarded((K, K), torch.int32, dev)
        ctx.adjudicate(d_t, out=(gm.t, gi.t, gw.t))
        assert gm.intact() and gi.intact() and gw.intact(), algo
        assert (fbits(gm.t.cpu().numpy()) == fbits(omed)).all()
        assert (fbits(gi.t.cpu().numpy()) == fbits(oiqr)).all()
        assert (gw.t.cpu().numpy().view(np.uint32) == owins).all()
    ctx.set_wins_algo(0)
    rec = np.zeros(K, dtype=oracle.RESULT_DTYPE)
    rec["pass"] = rng.random(K) < 0.7
    rec["mismatch_count"] = 1 - rec["pass"]
    rec["max_rel_err"] = rng.choice(np.float32([0.0, 2.0 ** -7, 0.01]), K)
    d_rec = torch.from_numpy(rec.view(np.uint8).reshape(K, 48).copy()).to(dev)
    for budget in (1, K, K + 5):
        gs, gn = Guarded((budget,), torch.int32, dev), Guarded((1,), torch.int32, dev)
        ctx.select(d_rec, gm.t, 0, budget, out=(gs.t, gn.t))
        assert gs.intact() and gn.intact()
        osurv, on = oracle.select(rec, omed, 0, budget)
        assert int(gn.t.item()) == on and gs.t.cpu().numpy().tolist() == osurv.tolist()
    assert ctx.poll() == 0
    assert ctx.check_guards()[1] == 0


def test_static_scratch_is_untouched_beyond_the_part_a_call_uses(kb):
    """kb_screen_static with K candidates uses the status words, K accumulators of either set and
    K table entries of its fixed array; every byte beyond them keeps its value."""
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(9)
    N = 3 * 4096 + 11
    ref = torch.from_numpy(rng.standard_normal(N).astype(np.float32)).to(dev)
    K = 37
    cands = [ref.clone() for _ in range(K)]
    cands[5][100] = 7.0
    out = torch.empty((K, kb.RESULT_BYTES), dtype=torch.uint8, device=dev)
    kb.screen_static(ref, cands[:3], 1e-5, 1e-3, out=out[:3])      # set-up call
    before = kb.static_scratch_read()
    kb.screen_static(ref, cands, 1e-5, 1e-3, out=out)
    after = kb.static_scratch_read()
    # [status words and counters 256 B | accumulators, set 0 | accumulators, set 1 | pointer table]
    set_bytes = 1024 * 48
    tab0 = 256 + 2 * set_bytes
    assert (after[tab0 + K * 8:] == before[tab0 + K * 8:]).all()
    for s0 in (256, 256 + set_bytes):
        assert (after[s0 + K * 48:s0 + set_bytes] == 0).all()
    same_records(kb.records(out), oracle_records(synth.F32, ref, cands, 1e-5, 1e-3))


def test_general_path_takes_two_launches_and_leaves_its_scratch_clean(ctx, kb):
    """Up to 480 candidates the streaming gate is two launches (lead: scouted tiles, ragged tail,
    pointer table, zeroing of the accumulator set the next call uses; streaming kernel, whose
    last CTA writes the records).  Calls of different sizes, dtypes and precisions follow one
    another on one context, larger after smaller, so that stale accumulators would show."""
    dev = torch.device("cuda", 0)
    ctx.set_small_path(False)
    rng = np.random.default_rng(21)

    def make(N, K, dtype):
        tdt = synth.TORCH_DTYPE[dtype]
        ref = torch.from_numpy(rng.standard_normal(N).astype(np.float32)).to(tdt).to(dev)
        cands = []
        for k in range(K):
            c = ref.clone()
            if k % 2:
                idx = torch.from_numpy(rng.integers(0, N, 3)).to(dev)
                c[idx] = 1.75
            cands.append(c)
        return ref, cands

    def run(N, K, dtype, expect_launches):
        ref, cands = make(N, K, dtype)
        n0 = ctx.launch_count
        got = kb.records(ctx.screen(ref, cands, 1e-3, 1e-2))
        assert ctx.launch_count - n0 == expect_launches, (N, K, ctx.launch_count - n0)
        same_records(got, oracle_records(dtype, ref, cands, 1e-3, 1e-2))

    run(40 * 4096 + 5, 30, synth.BF16, 2)          # scout + tail | stream
    run(40 * 4096, 7, synth.F16, 2)                # scout | stream
    run(4096, 3, synth.F32, 2)                     # one tile, nothing to scout, no tail: housekeeping | stream
    run(4096 + 1, 100, synth.F32, 2)               # tail | stream
    run(12 * 4096 + 100, 481, synth.BF16, 4)       # pointer table: 2 x prep | lead | stream
    run(300, 5, synth.F32, 2)                      # no full tile: lead (tail) | finalize
    run(40 * 4096 + 5, 30, synth.BF16, 2)
    # the double-precision gate uses the same workspace with another layout
    ref64 = torch.from_numpy(rng.standard_normal(9000)).to(dev)
    c64 = [ref64.clone(), ref64 + 1e-3]
    got = kb.records_f64(ctx.screen_f64(ref64, c64, 1e-12, 1e-9))
    same_records(got, oracle.screen_f64(ref64.cpu().numpy(), [c.cpu().numpy() for c in c64], 1e-12, 1e-9))
    run(40 * 4096 + 5, 30, synth.BF16, 2)
    run(40 * 4096 + 5, 200, synth.BF16, 2)         # more candidates than either set has seen cleaned
    run(40 * 4096 + 5, 9, synth.F16, 2)
    run(40 * 4096 + 5, 200, synth.BF16, 2)
    run(9 * 4096, 190, synth.F32, 2)
    assert ctx.poll() == 0
    assert ctx.check_guards()[1] == 0


def test_sharp_filter_is_chosen_for_dense_rounded_down_quotients_and_changes_nothing(ctx, kb):
    """One-ulp differences on many elements, none of them a power of two: the largest quotient
    (1/129 in bf16) is inexact and rounded down, and every element of its significand class
    fails the plain filter without being a new maximum.  After a few calls the context switches
    to the streaming kernel's sharp instantiation; the records are the oracle's either way, and
    sparse differences never make it switch."""
    dev = torch.device("cuda", 0)
    ctx.set_small_path(False)
    g = torch.Generator(device=dev)
    g.manual_seed(3)
    N = 200 * 4096 + 77
    ref = (torch.randn(N, device=dev, generator=g) * 4).to(torch.bfloat16)
    bits = ref.view(torch.int16)

    def flipped(frac, K):
        out = []
        for _ in range(K):
            f = (torch.rand(N, device=dev, generator=g) < frac) & ((bits & 0x7F) != 0)
            out.append(torch.where(f, (bits + 1).view(torch.bfloat16), ref))
        return out

    dense = flipped(0.5, 10)
    sparse = flipped(0.001, 10)
    want_dense = oracle_records(synth.BF16, ref, dense, 1e-2, 1.6e-2)
    want_sparse = oracle_records(synth.BF16, ref, sparse, 1e-2, 1.6e-2)
    assert (want_dense["pass"] == 1).all() and (fbits(want_dense["max_rel_err"]) == fbits(np.float32(1.0) / np.float32(129.0))).all()
    for mode in (1, 2):                               # forced plain, forced sharp
        ctx.set_filter(mode)
        same_records(kb.records(ctx.screen(ref, dense, 1e-2, 1.6e-2)), want_dense)
        assert ctx.last_filter_mode == (1 if mode == 2 else 0)
        same_records(kb.records(ctx.screen(ref, sparse, 1e-2, 1.6e-2)), want_sparse)
    ctx.set_filter(0)                                 # automatic
    seen = []
    for _ in range(8):
        same_records(kb.records(ctx.screen(ref, dense, 1e-2, 1.6e-2)), want_dense)    # (synchronises)
        seen.append(ctx.last_filter_mode)
    assert seen[0] == 0 and seen[-1] == 1, seen       # plain first, sharp once the reports are in
    ctx.set_filter(0)                                 # forget
    for _ in range(8):
        same_records(kb.records(ctx.screen(ref, sparse, 1e-2, 1.6e-2)), want_sparse)
        assert not ctx.last_filter_sharp
    assert ctx.poll() == 0


@pytest.mark.parametrize("dtype", [synth.BF16, synth.F16, synth.F32])
def test_by_definition_filter_is_chosen_for_absolute_noise_and_changes_nothing(ctx, kb, dtype):
    """Candidates that differ from the reference by absolute noise: where the reference is near
    zero the relative error is far above rtol and the element passes by atol alone.  The plain
    filter then sends nearly every step to a fruitless second look; after a few calls the
    context switches to the instantiation that tests such steps by the definition.  Same
    records in every mode, for passing and for failing candidates."""
    dev = torch.device("cuda", 0)
    ctx.set_small_path(False)
    g = torch.Generator(device=dev)
    g.manual_seed(17 + dtype)
    tdt = synth.TORCH_DTYPE[dtype]
    N = 150 * 4096 + 901
    base = torch.randn(N, device=dev, generator=g) * 4
    ref = base.to(tdt)
    sigma, atol, rtol = {synth.BF16: (1e-3, 1e-2, 1.6e-2), synth.F16: (1e-4, 1e-3, 1e-2),
                         synth.F32: (1e-6, 1e-5, 1e-6)}[dtype]
    noisy = [(base + torch.randn(N, device=dev, generator=g) * sigma).to(tdt) for _ in range(6)]
    failing = [(base + torch.randn(N, device=dev, generator=g) * (30 * sigma)).to(tdt) for _ in range(3)]
    failing[1][5] = float("nan")
    failing[2][N - 1] = float("inf")
    want = oracle_records(dtype, ref, noisy, atol, rtol)
    want_fail = oracle_records(dtype, ref, failing, atol, rtol)
    assert (want["pass"] == 1).all() and (want["max_rel_err"] > rtol).all()
    assert (want_fail["pass"] == 0).all()
    for mode in (1, 2, 3):                            # forced plain, sharp, by definition
        ctx.set_filter(mode)
        same_records(kb.records(ctx.screen(ref, noisy, atol, rtol)), want)
        assert ctx.last_filter_mode == {1: 0, 2: 1, 3: 3}[mode]
        same_records(kb.records(ctx.screen(ref, failing, atol, rtol)), want_fail)
        same_records(kb.records(ctx.screen(ref, noisy + failing, atol, rtol)), np.concatenate([want, want_fail]))
    ctx.set_filter(0)                                 # automatic
    seen = []
    for _ in range(8):
        same_records(kb.records(ctx.screen(ref, noisy, atol, rtol)), want)
        seen.append(ctx.last_filter_mode)
    assert seen[0] == 0 and seen[-1] == 3, seen       # plain first, by definition once the reports are in
    ctx.set_filter(0)
    ctx.set_small_path(True)
    assert ctx.poll() == 0


def test_by_definition_filter_is_chosen_for_nonzero_candidates_under_zero_references(ctx, kb):
    """A rectified reference (half of it exactly zero) and candidates that are tiny but not zero
    there: such elements have no quotient, the relative test cannot pass them, and in the plain
    instantiation every step ends in an exact path that changes nothing.  Those are reported and
    the context moves to the by-definition instantiation; one candidate is too large under a
    zero reference and must be counted out exactly as the oracle says, in every mode."""
    dev = torch.device("cuda", 0)
    ctx.set_small_path(False)
    g = torch.Generator(device=dev)
    g.manual_seed(99)
    N = 120 * 4096 + 13
    ref = torch.relu(torch.randn(N, device=dev, generator=g) * 4).to(torch.bfloat16)
    cands = []
    for k in range(5):
        tiny = (torch.rand(N, device=dev, generator=g) * (3e-2 if k == 4 else 1e-4)).to(torch.bfloat16)
        cands.append(torch.where(ref == 0, tiny, ref))
    want = oracle_records(synth.BF16, ref, cands, 1e-2, 1.6e-2)
    assert list(want["pass"]) == [1, 1, 1, 1, 0] and want["mismatch_count"][4] > 1000
    assert (want["max_rel_err"] == 0).all()               # no element with a non-zero reference differs
    for mode in (1, 2, 3):
        ctx.set_filter(mode)
        same_records(kb.records(ctx.screen(ref, cands, 1e-2, 1.6e-2)), want)
    ctx.set_filter(0)
    seen = []
    for _ in range(8):
        same_records(kb.records(ctx.screen(ref, cands[:4], 1e-2, 1.6e-2)), want[:4])
        seen.append(ctx.last_filter_mode)
    assert seen[0] == 0 and seen[-1] == 3, seen
    ctx.set_filter(0)
    ctx.set_small_path(True)
    assert ctx.poll() == 0


@pytest.mark.parametrize("dtype", [synth.F32, synth.BF16])
def test_outputs_with_long_tails_of_tiny_values(ctx, kb, dtype):
    """A softmax over widely spread logits: thousands of outputs below 2^-100, some subnormal,
    some zero.  Threads that hold such values leave the filter in the plain instantiation; the
    by-definition one judges the danger per step from the running maximum.  Same records in
    every mode; tiny values are exactly where a missed maximum of the relative error would hide."""
    dev = torch.device("cuda", 0)
    ctx.set_small_path(False)
    g = torch.Generator(device=dev)
    g.manual_seed(41 + dtype)
    tdt = synth.TORCH_DTYPE[dtype]
    rows, cols = 48, 8192
    atol, rtol = (1e-6, 1e-3) if dtype == synth.F32 else (1e-3, 1.6e-2)
    cands, refs = [], None
    for spread in (10.0, 25.0):
        logits = torch.randn(rows, cols, device=dev, generator=g) * spread
        ref = torch.softmax(logits, dim=1).reshape(-1).to(tdt)
        assert int(((ref.float() > 0) & (ref.float() < 7.8e-31)).sum()) > 200
        cs = [torch.softmax(logits + torch.randn(rows, cols, device=dev, generator=g) * 1e-4, dim=1).reshape(-1).to(tdt)
              for _ in range(4)]
        cs.append(torch.where(ref.float() < 1e-33, ref * 2, ref))            # tiny values doubled: quotient 1
        cs.append(torch.where(ref.float() < 1e-36, torch.zeros_like(ref), ref))   # ... flushed to zero
        want = oracle_records(dtype, ref, cs, atol, rtol)
        for mode in (1, 2, 3, 0, 0, 0, 0, 0, 0):
            ctx.set_filter(mode) if mode else None
            same_records(kb.records(ctx.screen(ref, cs, atol, rtol)), want)
        ctx.set_filter(0)
    ctx.set_small_path(True)
    assert ctx.poll() == 0


def test_by_definition_filter_at_the_edge_of_the_tolerance(ctx, kb):
    """Beyond the lean bound the by-definition instantiation tests |d| <= tol by a sufficient
    condition with a margin of 2^-20: elements whose error EQUALS the tolerance, or misses it by
    one unit in the last place either way, must come out as the definition says."""
    dev = torch.device("cuda", 0)
    ctx.set_small_path(False)
    rng = np.random.default_rng(2025)
    N = 40 * 4096 + 5
    atol, rtol = np.float32(2.0 ** -10), np.float32(2.0 ** -6)
    r = (rng.integers(1, 1 << 12, N).astype(np.float32) / np.float32(256.0))        # multiples of 2^-8 below 16
    r[::7] = np.float32(2.0 ** -12)                       # tiny references ...
    tol = (atol + (rtol * np.abs(r)).astype(np.float32)).astype(np.float32)          # exact here: dyadic values
    cands = []
    for shift in (0, 1, -1):                              # error = tol, one ulp above, one ulp below
        c = (r + tol).astype(np.float32)
        assert ((c - r).astype(np.float32) == tol).all()
        if shift:
            c = np.nextafter(c, np.float32(np.inf if shift > 0 else -np.inf), dtype=np.float32)
        c[::7] = r[::7] + np.float32(2.0 ** -11)          # ... whose error passes by atol with a quotient of 2
        cands.append(c)
    ref_t = torch.from_numpy(r).to(dev)
    cand_t = [torch.from_numpy(c).to(dev) for c in cands]
    want = oracle.screen(r, cands, oracle.F32, float(atol), float(rtol), threads=THREADS)
    assert want["pass"][0] == 1 and want["pass"][2] == 1 and want["pass"][1] == 0
    assert want["mismatch_count"][1] == N - len(r[::7]) and (want["max_rel_err"] == 2.0).all()
    for mode in (1, 2, 3, 0):
        ctx.set_filter(mode)
        for _ in range(3):
            same_records(kb.records(ctx.screen(ref_t, cand_t, float(atol), float(rtol))), want)
    ctx.set_filter(0)
    ctx.set_small_path(True)
    assert ctx.poll() == 0


# ---------------------------------------------------------------------------------------------
# out-of-range READS: every input tensor sits between two halos of NaN patterns (all-ones bytes
# are NaN in all six storage types).  An element read from outside [0, N) as a candidate would
# be counted as NaN, as a reference it would count a mismatch: either differs from the oracle,
# which only ever sees the tensor itself.
# ---------------------------------------------------------------------------------------------

HALO = 32768       # bytes on either side: a whole kernel tile of any type (and a multiple of 256)


def between_nan_halos(values: torch.Tensor) -> torch.Tensor:
    n = values.numel() * values.element_size()
    raw = torch.full((n + 2 * HALO,), 0xFF, dtype=torch.uint8, device=values.device)
    raw[HALO:HALO + n] = values.contiguous().view(torch.uint8).reshape(-1)
    return raw[HALO:HALO + n].view(values.dtype)


@pytest.mark.parametrize("dtype", [synth.F32, synth.F16, synth.BF16, synth.F8E4M3, synth.F8E5M2])
def test_inputs_between_nan_halos_are_read_inside_their_bounds_only(ctx, kb, dtype):
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(900 + dtype)
    tdt = synth.TORCH_DTYPE[dtype]
    rtol = 0.3 if dtype in (synth.F8E4M3, synth.F8E5M2) else 1.6e-2
    for N in (1, 7, 16, 4095, 4096, 4097, 3 * 4096 + 1000, 70000):
        base = torch.from_numpy(rng.standard_normal(N).astype(np.float32)).to(dev)
        ref = between_nan_halos(base.to(tdt))
        cands = []
        for k in range(3):
            c = base.clone()
            if k:                                   # a few real differences, first and last element among them
                c[[0, N - 1]] += 0.5 * k
                c[rng.integers(0, N, 3)] *= 1.01
            cands.append(between_nan_halos(c.to(tdt)))
        want = oracle_records(dtype, ref, cands, 1e-2, rtol)
        assert (want["nan_count"] == 0).all()
        masks = [(None, want)]
        if N >= 4096:
            spec = ("strided", 12, 2, 0)
            masks.append((ctx.mask_strided(N, 12, 2, 0), oracle_records(dtype, ref, cands, 1e-2, rtol, spec)))
        for small in (True, False):
            ctx.set_small_path(small)
            for mask, w in masks:
                same_records(kb.records(ctx.screen(ref, cands, 1e-2, rtol, mask)), w)
        ctx.set_small_path(True)
        for m, _ in masks[1:]:
            m.close()
    assert ctx.poll() == 0


def test_double_precision_inputs_between_nan_halos(ctx, kb):
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(977)
    for N in (1, 9, 2047, 2048, 2049, 4097, 3 * 4096 + 1000):
        base = torch.from_numpy(rng.standard_normal(N)).to(dev)
        ref = between_nan_halos(base)
        cands = [between_nan_halos(base * (1.0 + 1e-9 * k)) for k in range(3)]
        want = oracle.screen_f64(ref.cpu().numpy(), [c.cpu().numpy() for c in cands], 1e-12, 1e-8)
        got = kb.records_f64(ctx.screen_f64(ref, cands, 1e-12, 1e-8))
        same_records(got, want)
        assert (got["nan_count"] == 0).all()
    assert ctx.poll() == 0


@pytest.mark.parametrize("K,S", [(1, 1), (3, 5), (13, 33), (37, 100), (230, 17), (5, 2100)])
def test_timings_between_nan_halos(ctx, kb, K, S):
    """A timing read from outside [0, K*S) would be NaN: the call would report a non-finite
    timing, or the medians and win counts would differ from the oracle's."""
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(K * 1000 + S)
    t = (1.0 + rng.random((K, S))).astype(np.float32)
    d_t = between_nan_halos(torch.from_numpy(t).to(dev).reshape(-1)).view(K, S)
    want_med, want_iqr, want_wins = oracle.adjudicate(t)
    for algo in (0, 1, 2, 3):
        if algo == 3 and S > 1024:                  # the merge win count's row limit
            continue
        ctx.set_wins_algo(algo)
        med, iqr, wins = ctx.adjudicate(d_t)
        assert ctx.poll() == 0, algo
        assert (fbits(med.cpu().numpy()) == fbits(want_med)).all(), algo
        assert (fbits(iqr.cpu().numpy()) == fbits(want_iqr)).all(), algo
        assert (wins.cpu().numpy() == want_wins).all(), algo
    ctx.set_wins_algo(0)
    ratios = ctx.tail_ratios(d_t)
    assert torch.isfinite(ratios).all() and ctx.poll() == 0


def test_kernel_timers_record_a_subset_of_a_sequence_of_calls(ctx, kb):
    dev = torch.device("cuda", 0)
    ref = torch.zeros(64 * 4096, dtype=torch.bfloat16, device=dev)
    cands = kb.Candidates([ref.clone() for _ in range(4)])
    ctx.set_small_path(False)
    for i in range(9):                              # timers on for calls 0, 4 and 8
        if i % 4 == 0:
            ctx.enable_timing(True, keep=i > 0)
        elif i % 4 == 1:
            ctx.enable_timing(False)
        ctx.screen(ref, cands, 0.0, 0.0)
    ms = ctx.read_timer(kb.KB_TIMER_SCREEN_STREAM)
    assert len(ms) == 3 and (ms > 0).all()
    assert len(ctx.read_timer(kb.KB_TIMER_SCREEN_STREAM)) == 0      # a read clears the record
    ctx.enable_timing(True)                                          # a plain "on" starts afresh
    ctx.screen(ref, cands, 0.0, 0.0)
    assert len(ctx.read_timer(kb.KB_TIMER_SCREEN_STREAM)) == 1
    ctx.enable_timing(False)
    ctx.set_small_path(True)
    assert ctx.poll() == 0
