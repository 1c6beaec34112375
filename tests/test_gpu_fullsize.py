"""GPU parity at the full sizes of the five configurations, in the launch
configuration the benchmark times.

Every candidate of every configuration is compared bit for bit with the oracle,
which reads the very bytes the GPU screened (copied back from the device; under
config 5's first-tier mask only the selected tiles are copied, into a host
array whose other tiles hold NaN patterns the oracle must never touch).  The
closed-form consequences of how each candidate was built are asserted as well.
A last case exercises the largest tensor the boundary accepts (N = 2^32).
"""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2608_02611_b200 import synth

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


def fbits(a):
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


def same_record(got, want):
    for f in FIELDS:
        if got[f] != want[f]:
            return False
    return fbits(got["max_abs_err"]) == fbits(want["max_abs_err"]) and \
        fbits(got["max_rel_err"]) == fbits(want["max_rel_err"])


def oracle_for(case, ref_np, cand_t, mask="case"):
    m = case.mask if mask == "case" else mask
    return oracle.screen_one(ref_np, synth.to_oracle_array(cand_t, case.dtype), case.dtype,
                             case.atol, case.rtol, m)


def check_adjudicate(ctx, timings, sample_rows=None):
    dev = torch.device("cuda", 0)
    med, iqr, wins = ctx.adjudicate(torch.from_numpy(timings).to(dev))
    assert ctx.poll() == 0
    K = timings.shape[0]
    omed, oiqr, _ = oracle.adjudicate(timings, want_wins=False)
    assert (fbits(med.cpu().numpy()) == fbits(omed)).all()
    assert (fbits(iqr.cpu().numpy()) == fbits(oiqr)).all()
    w = wins.cpu().numpy().view(np.uint32)
    S = timings.shape[1]
    assert ((w.astype(np.int64) + w.T.astype(np.int64)) == 2 * S * S).all()
    if sample_rows is None:
        _, _, ow = oracle.adjudicate(timings, threads=THREADS)
        assert (w == ow).all()
    else:
        for a in sample_rows:
            assert (w[a] == oracle.wins_rows(timings, a, a + 1)[0]).all(), a
    return med, omed


def test_config2_full(ctx, kb):
    dev = torch.device("cuda", 0)
    case, timings = synth.config2(dev)
    assert case.N == 4096 * 4096 and case.K == 64
    cands = case.cands()
    out = ctx.screen(case.ref, cands, case.atol, case.rtol)
    got = kb.records(out)
    assert ctx.poll() == 0
    ref_np = synth.to_oracle_array(case.ref, case.dtype)
    cands_np = [synth.to_oracle_array(c, case.dtype) for c in cands]
    want = oracle.screen(ref_np, cands_np, case.dtype, case.atol, case.rtol, threads=THREADS)
    for k in range(case.K):
        assert same_record(got[k], want[k]), (k, got[k], want[k])
        assert bool(got[k]["pass"]) == case.truth[k]["passes"]
    assert int(got["pass"].sum()) == 54
    # the same batch through every instantiation of the streaming kernel, and in plain stream order
    for mode, dependent in ((1, True), (2, True), (3, True), (1, False), (3, False)):
        ctx.set_filter(mode)
        ctx.set_dependent_launch(dependent)
        again = kb.records(ctx.screen(case.ref, cands, case.atol, case.rtol))
        assert again.tobytes() == got.tobytes(), (mode, dependent)
    ctx.set_filter(0)
    ctx.set_dependent_launch(True)
    med, omed = check_adjudicate(ctx, timings)
    surv, n = ctx.select(out, med, kb.KB_SELECT_ERR_THEN_TIME, 32)
    osurv, on = oracle.select(want, omed, 0, 32)
    assert int(n.item()) == on and surv.cpu().numpy().tolist() == osurv.tolist()


def test_config4_full(ctx, kb):
    dev = torch.device("cuda", 0)
    case, timings = synth.config4(dev)
    assert case.N == 1 << 20 and case.K == 1024 and timings.shape == (1024, 64)
    cands = case.cands()
    out = ctx.screen(case.ref, cands, case.atol, case.rtol)
    got = kb.records(out)
    assert ctx.poll() == 0
    ref_np = synth.to_oracle_array(case.ref, case.dtype)
    want = oracle.screen(ref_np, [synth.to_oracle_array(c, case.dtype) for c in cands], case.dtype,
                         case.atol, case.rtol, threads=THREADS)
    for k in range(case.K):
        assert same_record(got[k], want[k]), (k, case.truth[k], got[k], want[k])
        assert bool(got[k]["pass"]) == case.truth[k]["passes"]
    med, omed = check_adjudicate(ctx, timings)          # many exact ties (1 us grid)
    surv, n = ctx.select(out, med, kb.KB_SELECT_TIME, 100)
    osurv, on = oracle.select(want, omed, 1, 100)
    assert int(n.item()) == on and surv.cpu().numpy().tolist() == osurv.tolist()


def oracle_all(case, ref_np, cands, mask="case"):
    """The oracle's record of every candidate in `cands` (device tensors), copied back one by
    one on the worker threads."""
    from concurrent.futures import ThreadPoolExecutor
    want = np.zeros(len(cands), dtype=oracle.RESULT_DTYPE)

    def one(j):
        want[j] = oracle_for(case, ref_np, cands[j], mask)

    with ThreadPoolExecutor(max_workers=THREADS) as ex:
        list(ex.map(one, range(len(cands))))
    return want


def test_config3_full(ctx, kb):
    dev = torch.device("cuda", 0)
    case, timings = synth.config3(dev)
    assert case.N == 8 * 32 * 2048 * 128 and case.K == 256
    cands = case.cands()                                 # 32 GiB of fp16 on the device
    out = ctx.screen(case.ref, cands, case.atol, case.rtol)
    got = kb.records(out)
    assert ctx.poll() == 0
    assert sum(case.truth[k]["kind"] != "ulp_noise" for k in range(case.K)) == 26
    ref_np = synth.to_oracle_array(case.ref, case.dtype)
    want = oracle_all(case, ref_np, cands)               # all 256 candidates
    for k in range(case.K):
        assert same_record(got[k], want[k]), (k, case.truth[k], got[k], want[k])
    # and by construction
    for k in range(case.K):
        tr = case.truth[k]
        assert bool(got[k]["pass"]) == tr["passes"], (k, tr, got[k])
        if tr["kind"] == "nan_row":
            assert got[k]["nan_count"] == 128 and got[k]["mismatch_count"] >= 128
        elif tr["kind"] == "transposed_head":
            assert got[k]["nan_count"] == 0 and got[k]["mismatch_count"] > 0.5 * 2048 * 128
            blk = int(got[k]["argmax_idx"]) // (2048 * 128)
            assert blk == tr["head"]
        else:
            assert got[k]["mismatch_count"] == 0 and got[k]["nan_count"] == 0
            assert 0 < got[k]["max_abs_err"] <= 2.0 ** -9          # one fp16 ulp below |x| < 4
    del cands
    torch.cuda.empty_cache()
    med, omed = check_adjudicate(ctx, timings)           # the whole win matrix
    surv, n = ctx.select(out, med, kb.KB_SELECT_ERR_THEN_TIME, 64)
    osurv, on = oracle.select(want, omed, 0, 64)
    assert int(n.item()) == on and surv.cpu().numpy().tolist() == osurv.tolist()


def test_config5_full_two_tier(ctx, kb):
    from concurrent.futures import ThreadPoolExecutor
    dev = torch.device("cuda", 0)
    c5 = synth.config5(dev)
    case = c5["case"]
    assert case.N == 1 << 28 and case.K == 512
    _, log2_tile, stride, phase = case.mask
    assert log2_tile == 12
    mask = ctx.mask_strided(case.N, log2_tile, stride, phase)
    assert mask.n_selected == 1 << 24
    ref_np = synth.to_oracle_array(case.ref, case.dtype)
    labels = c5["labels"]
    out1 = torch.empty((case.K, kb.RESULT_BYTES), dtype=torch.uint8, device=dev)
    want1 = np.zeros(case.K, dtype=oracle.RESULT_DTYPE)

    # Host images for the oracle: full-size arrays in which only the tiles the mask selects are
    # ever written (from the device); all other tiles keep a NaN pattern, so an oracle that read
    # an unselected element would report NaNs the GPU does not.
    import queue
    pool = queue.Queue()
    for _ in range(THREADS):
        pool.put(np.full(case.N, 0x7FC0, dtype=np.uint16))

    def one(k, sel_tiles):
        img = pool.get()
        try:
            img.reshape(-1, stride, 1 << log2_tile)[:, phase, :] = sel_tiles
            want1[k] = oracle.screen_one(ref_np, img, case.dtype, case.atol, case.rtol, case.mask)
        finally:
            pool.put(img)

    B = 64                                               # 32 GiB of candidates per batch
    with ThreadPoolExecutor(max_workers=THREADS) as ex:
        jobs = []
        for k0 in range(0, case.K, B):
            batch = [case.make_cand(k) for k in range(k0, k0 + B)]
            ctx.screen(case.ref, batch, case.atol, case.rtol, mask, out=out1[k0:k0 + B])
            torch.cuda.synchronize()
            for jb in jobs:                              # at most two batches of tiles on the host
                jb.result()
            jobs = []
            for j, c in enumerate(batch):
                tiles = c.view(torch.int16).view(-1, stride, 1 << log2_tile)[:, phase, :].contiguous()
                jobs.append(ex.submit(one, k0 + j, tiles.cpu().numpy().view(np.uint16)))
            del batch
        for jb in jobs:
            jb.result()
    assert ctx.poll() == 0
    rec1 = kb.records(out1)
    for k in range(case.K):                              # all 512 candidates, bit for bit
        assert same_record(rec1[k], want1[k]), (k, labels[k], rec1[k], want1[k])
    for k in range(case.K):
        assert bool(rec1[k]["pass"]) == case.truth[k]["tier1_pass"], (k, case.truth[k], rec1[k])
        if labels[k] == "nan_inf":
            assert rec1[k]["nan_count"] == case.truth[k]["nan"] and rec1[k]["inf_count"] == case.truth[k]["inf"]
    assert int(rec1["pass"].sum()) == 256

    med1, omed1 = check_adjudicate(ctx, c5["timings1"])
    surv, n = ctx.select(out1, med1, kb.KB_SELECT_ERR_THEN_TIME, c5["budget"])
    osurv, on = oracle.select(want1, omed1, 0, c5["budget"])      # the oracle's own records
    assert int(n.item()) == on == 32 and surv.cpu().numpy().tolist() == osurv.tolist()

    # tier 2: the 32 survivors on every element (16 GiB), regenerated from their seeds
    s = osurv[:on].tolist()
    cands2 = [case.make_cand(k) for k in s]
    out2 = ctx.screen(case.ref, cands2, case.atol, case.rtol)
    rec2 = kb.records(out2)
    assert ctx.poll() == 0
    want2 = oracle_all(case, ref_np, cands2, mask=None)   # all 32 survivors
    for j, k in enumerate(s):
        assert same_record(rec2[j], want2[j]), (k, labels[k], rec2[j], want2[j])
        assert bool(rec2[j]["pass"]) == case.truth[k]["tier2_pass"], (k, case.truth[k], rec2[j])
    hidden = [j for j, k in enumerate(s) if labels[k] == "hidden_burst"]
    cleanj = [j for j, k in enumerate(s) if labels[k] == "clean"]
    assert hidden and cleanj                             # the second tier has something to catch
    del cands2
    torch.cuda.empty_cache()
    check_adjudicate(ctx, c5["make_timings2"](s))
    mask.close()


def test_largest_tensor_two_pow_32(ctx, kb):
    """N = 2^32 bf16 elements (8 GiB per tensor): index arithmetic at the top of the range.
    Expected values follow in closed form from where the perturbations were written."""
    dev = torch.device("cuda", 0)
    N = 1 << 32
    ref = torch.empty(N, dtype=torch.bfloat16, device=dev)
    g = torch.Generator(device=dev)
    g.manual_seed(5)
    for s in range(0, N, 1 << 28):
        ref[s:s + (1 << 28)].normal_(0.0, 4.0, generator=g)
    ref[N - 1] = 1.5
    ref[(1 << 31) + 5] = 2.0
    ref[12345] = 1.0
    c0 = ref.clone()
    c0[N - 1] = float("nan")                      # last element of the range
    c0[(1 << 31) + 5] = 3.0                       # error 1.0 above index 2^31
    c0[12345] = 2.0                               # the same error at a low index: wins the tie
    c1 = ref.clone()
    c1[N - 1] = 1.75                              # error 0.25 at the very last index
    rec = kb.records(ctx.screen(ref, [c0, c1], 1e-2, 1.6e-2))
    assert ctx.poll() == 0
    assert rec["mismatch_count"].tolist() == [3, 1]
    assert rec["nan_count"].tolist() == [1, 0] and rec["inf_count"].tolist() == [0, 0]
    assert rec["argmax_idx"].tolist() == [12345, N - 1]
    assert rec["max_abs_err"].tolist() == [1.0, 0.25]
    assert rec["max_rel_err"][0] == 1.0 and rec["max_rel_err"][1] == np.float32(0.25 / 1.5)
    # under a coarse mask that keeps only the last 2^20-element tile
    m = ctx.mask_strided(N, 20, 4096, 4095)
    rec = kb.records(ctx.screen(ref, [c0, c1], 1e-2, 1.6e-2, m))
    assert rec["mismatch_count"].tolist() == [1, 1] and rec["nan_count"].tolist() == [1, 0]
    assert rec["argmax_idx"].tolist() == [N - (1 << 20), N - 1]
    m.close()
