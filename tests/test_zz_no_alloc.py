"""kb_screen_static: the gate for hosts that cannot let a library allocate.

A serving process that forbids allocation after start-up, or a framework that
has already handed all device memory to its own allocator, cannot afford a
cudaMalloc inside a library call.  kb_screen_static keeps its scratch in a fixed
array inside the library instead.  Here it is called through the C ABI twice in
a row (the array keeps the previous call's contents, so the second call proves
that what must start at zero is cleared) and compared, bit for bit, with
kb_screen on the same inputs and with the CPU oracle; the device's free memory
is read around the calls to see that nothing was allocated.  The file sorts
last on purpose.
"""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2608_02611_b200 import synth

pytestmark = pytest.mark.gpu


def _bits(rec):
    return rec.view(np.uint8).reshape(-1)


def test_static_entry_point_matches_kb_screen_twice_in_a_row():
    from paper_2608_02611_b200 import binding
    dev = torch.device("cuda", 0)
    ctx = binding.Context(0)
    try:
        # call 1: bf16, several tiles plus a ragged tail, failures of every kind
        case, _ = synth.config2(dev, side=512, K=16, n_bad=3)
        N1 = case.N - 123
        ref1 = case.ref[:N1].clone()
        cands1 = [case.make_cand(k)[:N1].clone() for k in range(case.K)]
        cands1[5][777] = float("nan")
        cands1[6][N1 - 1] = float("inf")
        out_static = torch.full((len(cands1), binding.RESULT_BYTES), 0xCD, dtype=torch.uint8, device=dev)
        binding.screen_static(ref1, cands1, case.atol, case.rtol, out=out_static)
        want1 = binding.records(ctx.screen(ref1, cands1, case.atol, case.rtol))
        got1 = binding.records(out_static)
        assert (_bits(got1) == _bits(want1)).all()
        assert got1["nan_count"][5] == 1 and got1["inf_count"][6] == 1 and got1["pass"][0] == 1

        # call 2 straight after, other dtype, other K, mostly clean candidates: stale counts
        # or maxima from call 1 would show
        case2, _ = synth.config4(dev, N=(1 << 15) + 5, K=24, S_t=8)
        cands2 = [case2.make_cand(k) for k in range(case2.K)]
        got2 = binding.records(binding.screen_static(case2.ref, cands2, case2.atol, case2.rtol))
        want2 = binding.records(ctx.screen(case2.ref, cands2, case2.atol, case2.rtol))
        assert (_bits(got2) == _bits(want2)).all()

        # and call 1 again gives call 1's answer again
        got1b = binding.records(binding.screen_static(ref1, cands1, case.atol, case.rtol))
        assert (_bits(got1b) == _bits(want1)).all()
        assert ctx.poll() == 0

        # against the oracle directly, not only against the other entry point
        threads = max(1, len(os.sched_getaffinity(0)))
        o1 = oracle.screen(synth.to_oracle_array(ref1, case.dtype),
                           [synth.to_oracle_array(c, case.dtype) for c in cands1],
                           case.dtype, case.atol, case.rtol, threads=threads)
        assert (_bits(got1) == _bits(o1)).all()
        o2 = oracle.screen(synth.to_oracle_array(case2.ref, case2.dtype),
                           [synth.to_oracle_array(c, case2.dtype) for c in cands2],
                           case2.dtype, case2.atol, case2.rtol, threads=threads)
        assert (_bits(got2) == _bits(o2)).all()
    finally:
        ctx.close()


def test_static_entry_point_allocates_nothing():
    """With the output pre-allocated by the caller, the device's free memory is the same before
    and after a run of calls (the first call on the device, which looks up the array's address,
    has been made before)."""
    from paper_2608_02611_b200 import binding
    dev = torch.device("cuda", 0)
    case, _ = synth.config2(dev, side=640, K=24, n_bad=4)          # K*N = 9.8e6: streaming kernels
    cands = case.cands()
    out = torch.empty((case.K, binding.RESULT_BYTES), dtype=torch.uint8, device=dev)
    small = [c[:5000] for c in cands[:5]]
    binding.screen_static(case.ref, cands, case.atol, case.rtol, out=out)     # set-up call
    torch.cuda.synchronize()
    free0, total0 = torch.cuda.mem_get_info(dev)
    for _ in range(5):
        binding.screen_static(case.ref, cands, case.atol, case.rtol, out=out)
        binding.screen_static(case.ref[:5000], small, case.atol, case.rtol, out=out[:5])
        binding.screen_static(case.ref, cands[:7], case.atol, case.rtol, out=out[:7])
    torch.cuda.synchronize()
    free1, total1 = torch.cuda.mem_get_info(dev)
    assert (free1, total1) == (free0, total0)
    binding.screen_static(case.ref, cands, case.atol, case.rtol, out=out)
    want = oracle.screen(synth.to_oracle_array(case.ref, case.dtype),
                         [synth.to_oracle_array(c, case.dtype) for c in cands],
                         case.dtype, case.atol, case.rtol, threads=max(1, len(os.sched_getaffinity(0))))
    assert (_bits(binding.records(out)) == _bits(want)).all()


def test_static_entry_point_refuses_more_candidates_than_its_scratch_holds():
    from paper_2608_02611_b200 import binding
    dev = torch.device("cuda", 0)
    ref = torch.zeros(64, dtype=torch.float32, device=dev)
    out = torch.full((binding.KB_STATIC_MAX_K + 1, binding.RESULT_BYTES), 0xAB, dtype=torch.uint8, device=dev)
    with pytest.raises(binding.KbError) as e:
        binding.screen_static(ref, [ref] * (binding.KB_STATIC_MAX_K + 1), 0.0, 0.0, out=out)
    assert e.value.status == 4                      # KB_ERR_WORKSPACE
    assert "exceeds" in str(e.value)
    assert (out.cpu() == 0xAB).all()                # nothing was launched
    # the largest allowed K works
    got = binding.records(binding.screen_static(ref, [ref] * binding.KB_STATIC_MAX_K, 0.0, 0.0))
    assert (got["pass"] == 1).all() and (got["argmax_idx"] == 0).all()
