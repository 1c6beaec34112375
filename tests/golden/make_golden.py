"""Writes tests/golden/oracle_small_cases.json from the CPU oracle alone.

Run from the repository root:  python tests/golden/make_golden.py
The file stores the oracle's results on small seeded inputs (bit patterns for
floats) so that (a) a change in the oracle's arithmetic shows up as a diff and
(b) the GPU parity tests have a second, stored copy of the expected values.
Nothing here touches the CUDA library.
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2608_02611_b200 import synth  # noqa: E402

OUT = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_small_cases.json")


def fbits(x) -> int:
    return int(np.float32(x).view(np.uint32))


def rec_to_json(r):
    return dict(mismatch_count=int(r["mismatch_count"]), nan_count=int(r["nan_count"]),
                inf_count=int(r["inf_count"]), argmax_idx=int(r["argmax_idx"]),
                max_abs_err_bits=fbits(r["max_abs_err"]), max_rel_err_bits=fbits(r["max_rel_err"]),
                passed=int(r["pass"]))


def run_case(case, timings, budget, policy, mask="case"):
    ref = synth.to_oracle_array(case.ref, case.dtype)
    m = case.mask if mask == "case" else mask
    recs = oracle.screen(ref, [synth.to_oracle_array(case.make_cand(k), case.dtype)
                               for k in range(case.K)], case.dtype, case.atol, case.rtol, m)
    med, iqr, wins = oracle.adjudicate(timings)
    surv, n = oracle.select(recs, med, policy, budget)
    return dict(
        screen=[rec_to_json(r) for r in recs],
        median_bits=[fbits(v) for v in med], iqr_bits=[fbits(v) for v in iqr],
        wins=wins.astype(np.int64).tolist(), survivors=surv.tolist(), n_survivors=n,
        budget=budget, policy=policy,
    )


def build():
    out = {}
    case, timings = synth.config1()
    out["config1"] = run_case(case, timings, 2, 0)
    case, timings = synth.config2(side=512, K=16, n_bad=3)
    out["config2_side512_K16"] = run_case(case, timings, 4, 0)
    case, timings = synth.config3(B=1, H=2, S=64, D=128, K=12, n_nan=2, n_transposed=2, S_t=50)
    out["config3_small"] = run_case(case, timings, 5, 0)
    case, timings = synth.config4(N=1 << 14, K=40, S_t=16)
    out["config4_small"] = run_case(case, timings, 8, 1)
    c5 = synth.config5(N=1 << 20, K=32, budget=4, S1=20, S2=40)
    out["config5_small_tier1"] = run_case(c5["case"], c5["timings1"], 4, 0)
    return out


if __name__ == "__main__":
    with open(OUT, "w") as f:
        json.dump(build(), f, indent=0, sort_keys=True)
        f.write("\n")
    print("wrote", OUT)
