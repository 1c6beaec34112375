"""Benchmark of the whole hot path on synthetic config 2.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

A step is one pass of the path over one batch: kb_screen of K=64 bf16
candidates of 4096x4096 against one reference, kb_adjudicate of timings
[64][100], kb_select of the top 32.  Inputs are resident in HBM before the
timed region; they total 2.18 GB per step, far above the 126 MB L2, so no cache
flush is needed between steps.  One JSON line is printed by rank 0.

With N > 1 (torchrun, one process per GPU) the candidates are independent, so
every rank screens its own 64 candidates against its own replica of the
reference (weak scaling, no data-path collective); the time is the maximum
over ranks.

`--impl reference` times the CPU oracle (test infrastructure, used as it
stands) on the host cores on the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "candidate-elements screened/sec"
UNIT = "elements/s"
K_CANDS, SIDE, S_TIMINGS, BUDGET = 64, 4096, 100, 32
# DRAM bytes moved per algorithmic byte by the streaming screen kernel come from the ncu capture
# summarised in profiles/ (dram__bytes_read.sum + dram__bytes_write.sum over (K+1)*N*2 bytes;
# captured at side 2048 and scaled by the bytes a full launch processes); the figure is stored
# beside that summary so that it is replaced together with it.
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "screen_stream_kernel_bf16_config2.json")
REF_MAX_STEPS, REF_MAX_WARMUP = 50, 5      # bounds of the reference arm (a step costs ~0.6 s)


def dram_bytes_per_algorithmic_byte():
    try:
        with open(TRAFFIC_FILE) as f:
            return float(json.load(f)["dram_bytes_per_algorithmic_byte"])
    except Exception:
        return None

WORKLOAD = ("config2: screen K=64 bf16 4096x4096 (atol=1e-2, rtol=1.6e-2) + adjudicate "
            "timings[64][100] + select top 32")


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs.
    Everything that talks to NVML (initialisation included) happens on this daemon thread, so a
    slow or stuck NVML can never block the benchmark itself."""

    def __init__(self, index: int, period_s: float = 0.001):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self.stamps = []
        self.window = None                 # (t0, t1) of the timed region, perf_counter
        self.n_before_load = 0             # samples taken before the first warm-up step
        self.ready = threading.Event()
        self._halt = threading.Event()

    def run(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = int(nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM))
        except Exception:
            self.ready.set()
            return
        self.ready.set()
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
        }
        while not self._halt.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)))
                self.stamps.append(time.perf_counter())
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(h))
                for name, bit in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._halt.wait(self.period)

    def stop(self):
        self._halt.set()
        if self.is_alive():
            self.join(timeout=2)
        samples = list(self.samples)[self.n_before_load:]
        stamps = list(self.stamps)[self.n_before_load:][:len(samples)]
        timed = [v for v, t in zip(samples, stamps)
                 if self.window and self.window[0] <= t <= self.window[1]]
        # the sampler runs from the first warm-up step to the end of the timed region and, if
        # that gave fewer than five samples, over an untimed continuation of the same steps
        use = timed if len(timed) >= 5 else samples
        return {"sm_mhz": int(np.median(use)) if use else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(use), "samples_in_timed_region": len(timed),
                "window": "timed region" if len(timed) >= 5 else
                          "warm-up + timed region + untimed continuation of the same steps"}


def host_cores() -> int:
    return max(1, len(os.sched_getaffinity(0)))


def oracle_step(ref_np, cands_np, timings, n_cands, threads):
    """One bounded sample of the workload on the CPU oracle; returns seconds."""
    import oracle
    t0 = time.perf_counter()
    rec = oracle.screen(ref_np, cands_np[:n_cands], 2, 1e-2, 1.6e-2, threads=threads)
    med, iqr, wins = oracle.adjudicate(timings, threads=threads)
    oracle.select(rec, med[:n_cands], 0, min(BUDGET, n_cands))
    return time.perf_counter() - t0


def run_reference(args):
    """The reference arm: the CPU oracle on the host cores, same config and metric: every step
    screens all 64 candidates, adjudicates [64][100] and selects.  `--steps`/`--warmup` are
    honoured up to REF_MAX_STEPS / REF_MAX_WARMUP."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch
    from paper_2608_02611_b200 import synth
    cores = host_cores()
    case, timings = synth.config2("cpu", side=SIDE, K=K_CANDS)
    ref_np = synth.to_oracle_array(case.ref, case.dtype)
    cands_np = [synth.to_oracle_array(case.make_cand(k), case.dtype) for k in range(K_CANDS)]
    warmup = max(0, min(args.warmup, REF_MAX_WARMUP))
    steps = max(1, min(args.steps, REF_MAX_STEPS))
    for _ in range(warmup):
        oracle_step(ref_np, cands_np, timings, K_CANDS, cores)
    secs = [oracle_step(ref_np, cands_np, timings, K_CANDS, cores) for _ in range(steps)]
    per_step = float(np.mean(secs))
    value = K_CANDS * case.N / per_step
    sample = (f"the whole step: all {K_CANDS} candidates of 4096x4096 bf16, adjudication [64][100] "
              f"and select; {steps} steps after {warmup} warm-up steps on {cores} threads")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": per_step * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "K": K_CANDS, "N": case.N, "storage": "bf16", "S": S_TIMINGS,
                   "budget": BUDGET, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def run_adjudicate(args):
    """kb_adjudicate alone: logical comparisons/s = K^2 S^2 / t; for the direct-comparison kernel
    also the executed sample-pair evaluations against the ALU-pipe roofline."""
    import torch
    from paper_2608_02611_b200 import binding, synth
    dev = torch.device("cuda", 0)
    ctx = binding.Context(0)
    ctx.set_wins_algo(args.wins_algo)
    K, S = args.K, args.S
    t_k = synth.base_latencies(synth.MASTER_SEED + 5, K, 0.3)
    timings = synth.lognormal_timings(synth.MASTER_SEED + 5, t_k, S, 0.15)
    d_t = torch.from_numpy(timings).to(dev)
    steps, warmup = max(1, min(args.steps, 200)), max(3, args.warmup)
    for _ in range(warmup):
        ctx.adjudicate(d_t)
    torch.cuda.synchronize()
    ctx.enable_timing(True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        ctx.adjudicate(d_t)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    wins_ms = float(np.mean(ctx.read_timer(binding.KB_TIMER_WINS)))
    assert ctx.poll() == 0
    logical = K * K * S * S
    line = {"workload": f"adjudicate timings[{K}][{S}]", "wins_algo": args.wins_algo,
            "ms_per_call": ms, "wins_kernel_ms": wins_ms,
            "pairwise_comparisons_per_s": logical / (wins_ms * 1e-3), "steps": steps}
    direct = (args.wins_algo == 1 or S > 4096) and K % 8 == 0   # the count below assumes full 8-row blocks
    if direct:
        # every unordered block pair once; R*32 sample slots per lane row; at least the two
        # compares of a sample pair must issue on the ALU pipe (64 lanes/clk/SM)
        KB = (K + 7) // 8
        nj = (S + 255) // 256
        R = ((S + nj - 1) // nj + 31) // 32
        evals = KB * (KB + 1) // 2 * 64 * S * (nj * R * 32)
        peak = 148 * 64 * 1.965e9 / 2          # sample-pair evaluations/s at 64 ALU lanes/clk/SM
        probe = ctx.alu_probe(20000)           # the same instruction mix on registers only, measured
        line["roofline"] = {"bound": "alu", "achieved": evals / (wins_ms * 1e-3), "peak": peak,
                            "unit": "sample-pair evaluations/s", "frac": evals / (wins_ms * 1e-3) / peak,
                            "traffic": None, "peak_source": "derived: 148 SMs x 64 ALU lanes x 1.965 GHz / 2 "
                            "compares per pair", "measured_probe": probe,
                            "frac_of_probe": evals / (wins_ms * 1e-3) / probe}
    print(json.dumps(line), flush=True)
    ctx.close()


def run_screen(args):
    """One kb_screen / kb_screen_f64 call on a seeded synthetic batch: a standard-normal
    reference and K candidates that differ from it by one unit in the last place on a fraction
    of the elements (two kernels that round differently).  Secondary measurement: the streaming
    kernel's bytes/s against the measured HBM peak, for other dtypes and batch sizes than the
    benchmark line's."""
    import torch
    from paper_2608_02611_b200 import binding
    dev = torch.device("cuda", 0)
    ctx = binding.Context(0)
    if not args.default_dispatch:
        ctx.set_small_path(False)      # time the streaming path whatever the size
    K, N = args.K, 1 << args.log2n
    tdt = {"f64": torch.float64, "f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16,
           "e4m3": torch.float8_e4m3fn, "e5m2": torch.float8_e5m2}[args.dtype]
    idt = {8: torch.int64, 4: torch.int32, 2: torch.int16, 1: torch.int8}[torch.empty(0, dtype=tdt).element_size()]
    g = torch.Generator(device=dev)
    g.manual_seed(20260802)
    base = torch.randn(N, dtype=torch.float32, device=dev, generator=g) * args.ref_scale
    soft = None
    if args.softmax_spread > 0.0:
        # rows of 16384 logits of the given spread: outputs with a long tail of tiny values
        soft = (torch.randn(N, dtype=torch.float32, device=dev, generator=g) * args.softmax_spread).view(-1, min(N, 16384))
        base = torch.softmax(soft, dim=1).reshape(-1)
    ref = (torch.relu(base) if args.relu else base).to(tdt)   # (noise goes in before the rectifier)
    esz1 = ref.element_size() == 1           # 8-bit floats: one unit in the last place is up to 1/8
    cands = []
    for _ in range(K):
        if soft is not None:
            c = torch.softmax(soft + torch.randn(soft.shape, dtype=torch.float32, device=dev, generator=g) * 1e-4, dim=1)
            cands.append(c.reshape(-1).to(tdt))
            continue
        if args.noise_sigma > 0.0:
            # accumulated rounding error does not scale with the value: where the reference is near
            # zero the relative error is large and the element passes by atol alone
            c = base + torch.randn(N, dtype=torch.float32, device=dev, generator=g) * args.noise_sigma
            cands.append((torch.relu(c) if args.relu else c).to(tdt))
            continue
        flip = torch.rand(N, device=dev, generator=g) < args.flip_frac
        cands.append(torch.where(flip, ref.view(idt) + 1, ref.view(idt)).view(tdt))
    del base, soft
    # tolerances under which a one-ulp difference passes: 2^-3 relative in e4m3, 2^-2 in e5m2
    atol, rtol = (1e-12, 1e-12) if args.dtype == "f64" else \
        (1e-2, 0.26 if args.dtype == "e5m2" else 0.13) if esz1 else (1e-2, 1.6e-2)
    atol = args.atol if args.atol is not None else atol
    rtol = args.rtol if args.rtol is not None else rtol
    held = cands if args.dtype == "f64" else binding.Candidates(cands)   # pointer array built once
    call = (lambda: ctx.screen_f64(ref, cands, atol, rtol)) if args.dtype == "f64" else \
        (lambda: ctx.screen(ref, held, atol, rtol))
    steps, warmup = max(1, min(args.steps, 50)), max(3, args.warmup)
    if args.noise_sigma > 0.0 or args.softmax_spread > 0.0:
        warmup = max(warmup, 12)       # the context's choice of instantiation follows its reports
    for _ in range(warmup):
        call()
    torch.cuda.synchronize()
    ctx.enable_timing(True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        call()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    tk = ctx.read_timer(binding.KB_TIMER_SCREEN_STREAM)
    k_ms = float(np.mean(tk)) if len(tk) else float("nan")   # no streaming launch on the small path
    assert ctx.poll() == 0
    ntiles = N // 4096
    nscout = min(8, max(1, ntiles // 128)) if ntiles >= 2 else 0
    esz = ref.element_size()
    stream_bytes = (K + 1) * (ntiles - nscout) * 4096 * esz
    peak, src = peaks()
    what = f"softmax over rows of 16384 logits of spread {args.softmax_spread:g}, candidates from logits + N(0, 1e-8)" \
        if args.softmax_spread > 0.0 else \
        (f"absolute noise sigma={args.noise_sigma:g} on a reference of scale {args.ref_scale:g}"
         + (", rectified" if args.relu else "")) if args.noise_sigma > 0.0 else \
        f"one-ulp differences on {args.flip_frac:.0%} of the elements"
    line = {"workload": f"screen K={K} N=2^{args.log2n} {args.dtype}, {what}",
            "filter": {0: "plain", 1: "sharp", 3: "by definition"}.get(ctx.last_filter_mode, "-"),
            "ms_per_call": ms, "stream_kernel_ms": k_ms, "steps": steps,
            "call_gbs": (K + 1) * N * esz / (ms * 1e-3) / 1e9,
            "roofline": {"bound": "hbm", "achieved": stream_bytes / (k_ms * 1e-3) / 1e9, "peak": peak,
                         "unit": "GB/s", "frac": stream_bytes / (k_ms * 1e-3) / 1e9 / peak,
                         "traffic": None, "peak_source": src}}
    print(json.dumps(line), flush=True)
    ctx.close()


# Largest output of each of the paper's six benchmarks (Appendix "Benchmark Descriptions and
# Shapes"): MatVec M=2048; GroupConv 217800 x 20; LinearReLUDiv 1024 x 8192; SDPAttn
# 32 x 32 x 512 x 1024; RMSNorm 16 x 64 x 768 x 768; Softmax 4096 x 393216.
PAPER_SHAPES = [("MatVec", 2048), ("GroupConv", 217800 * 20), ("LinearReLUDiv", 1024 * 8192),
                ("SDPAttn", 32 * 32 * 512 * 1024), ("RMSNorm", 16 * 64 * 768 * 768),
                ("Softmax", 4096 * 393216)]


def run_paper_scale(args):
    """kb_screen at the paper's own scale: the six benchmark output sizes x the candidate counts of
    its funnel (21 -> 7 -> 3), bf16 and fp32, default dispatch.  One JSON line per entry: time per
    call (CUDA events around back-to-back calls, no kernel timers), bytes/s of (K+1)*N*sizeof
    against the measured HBM peak, launches per call.  Secondary measurement."""
    import torch
    from paper_2608_02611_b200 import binding
    dev = torch.device("cuda", 0)
    ctx = binding.Context(0)
    peak, src = peaks()
    calls = max(3, min(args.steps, 20))
    # a fresh process finds the GPU at idle clocks: keep it busy for a moment first, or the first
    # (smallest) entries are timed while the clocks still rise
    warm = torch.randn(1 << 24, device=dev).to(torch.bfloat16)
    warm_c = binding.Candidates([warm.clone() for _ in range(8)])
    t_warm = time.perf_counter()
    while time.perf_counter() - t_warm < 0.3:
        for _ in range(20):
            ctx.screen(warm, warm_c, 1e-2, 1.6e-2)
        torch.cuda.synchronize()
    del warm, warm_c
    for name, N in PAPER_SHAPES:
        for dname, tdt, idt in (("bf16", torch.bfloat16, torch.int16), ("f32", torch.float32, torch.int32)):
            esz = 2 if dname == "bf16" else 4
            g = torch.Generator(device=dev)
            g.manual_seed(20260802)
            ref = None
            for K in (21, 7, 3):
                if (K + 1) * N * esz > 100e9:
                    print(json.dumps({"benchmark": name, "N": N, "dtype": dname, "K": K,
                                      "skipped": "more than 100 GB of tensors"}), flush=True)
                    continue
                if ref is None:
                    ref = torch.empty(N, dtype=tdt, device=dev)
                    for s0 in range(0, N, 1 << 27):           # in slices: no full-size fp32 temporary
                        ref[s0:s0 + (1 << 27)] = torch.randn(min(1 << 27, N - s0), dtype=torch.float32,
                                                             device=dev, generator=g).to(tdt)
                    cands = []
                while len(cands) < K:                         # one-ulp differences on 1% of the elements
                    c = ref.clone()
                    c.view(idt)[len(cands)::101] += 1
                    cands.append(c)
                cs = cands[:K]
                out = torch.empty((K, binding.RESULT_BYTES), dtype=torch.uint8, device=dev)
                for _ in range(3):
                    ctx.screen(ref, cs, 1e-2, 1.6e-2, out=out)
                torch.cuda.synchronize()
                # the C entry point itself with its arguments marshalled once: the Python
                # binding's own 10-15 us per call would otherwise hide the small cases
                import ctypes
                L = binding.load()
                ptrs = (ctypes.c_void_p * K)(*[c.data_ptr() for c in cs])
                a = (ctx._h, ref.data_ptr(), ptrs, K, N, binding.DTYPE_CODE[tdt], 1e-2, 1.6e-2, None,
                     out.data_ptr(), int(torch.cuda.current_stream(dev).cuda_stream))
                n0 = ctx.launch_count
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                # (ten times the calls for the tiny outputs: 20 calls of 5 us are over before the
                # launch pipeline has filled)
                n_calls = calls * 10 if (K + 1) * N * esz < (1 << 24) else calls
                e0.record()
                for _ in range(n_calls):
                    L.kb_screen(*a)
                e1.record()
                torch.cuda.synchronize()
                us = e0.elapsed_time(e1) / n_calls * 1e3
                assert ctx.poll() == 0
                rec = binding.records(out)
                gbs = (K + 1) * N * esz / (us * 1e-6) / 1e9
                print(json.dumps({"benchmark": name, "N": N, "dtype": dname, "K": K, "us_per_call": us,
                                  "gbs": gbs, "frac_of_measured_hbm": gbs / peak,
                                  "launches_per_call": (ctx.launch_count - n0) / n_calls,
                                  "all_pass": bool((rec["pass"] == 1).all()), "calls": n_calls}), flush=True)
            del ref
            cands = []
            torch.cuda.empty_cache()
    ctx.close()


def relaunch_ranks(n: int):
    """`python bench.py --gpus N` without a launcher: start N ranks (one process per GPU) under
    torch.distributed.run on this node, with the same arguments, and pass their output on."""
    import socket
    import subprocess
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")           # the communicator set-up goes to stderr
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    raise SystemExit(subprocess.run(cmd, env=env).returncode)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="skip the secondary CUDA-graph replay of the step")
    ap.add_argument("--workload", default="step", choices=["step", "adjudicate", "screen", "paper-scale"],
                    help="'adjudicate' times kb_adjudicate alone on timings[K][S] (config 5 tier 1 by "
                         "default) and reports pairwise comparisons/s against the ALU roofline; it is a "
                         "secondary measurement, not the benchmark line")
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "f16", "f32", "f64", "e4m3", "e5m2"],
                    help="storage type of the 'screen' workload")
    ap.add_argument("--log2n", type=int, default=24, help="elements per tensor of the 'screen' workload")
    ap.add_argument("--flip-frac", type=float, default=0.25)
    ap.add_argument("--noise-sigma", type=float, default=0.0,
                    help="'screen' workload: candidates = round(reference + N(0, sigma^2)) instead of one-ulp differences")
    ap.add_argument("--ref-scale", type=float, default=1.0, help="'screen' workload: standard deviation of the reference")
    ap.add_argument("--atol", type=float, default=None, help="'screen' workload: tolerance override")
    ap.add_argument("--rtol", type=float, default=None, help="'screen' workload: tolerance override")
    ap.add_argument("--softmax-spread", type=float, default=0.0,
                    help="'screen' workload: reference = softmax over rows of 16384 logits N(0, spread^2)")
    ap.add_argument("--relu", action="store_true", help="'screen' workload: rectified reference and candidates")
    ap.add_argument("--default-dispatch", action="store_true",
                    help="'screen' workload: let small problems take the single-launch kernel")
    ap.add_argument("--K", type=int, default=512)
    ap.add_argument("--S", type=int, default=200)
    ap.add_argument("--wins-algo", type=int, default=0, choices=[0, 1, 2, 3])
    ap.add_argument("--side", type=int, default=SIDE,
                    help="tensor side; anything but 4096 is for profiler captures only and is "
                         "not a benchmark configuration")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.workload == "adjudicate":
        return run_adjudicate(args)
    if args.workload == "screen":
        return run_screen(args)
    if args.workload == "paper-scale":
        return run_paper_scale(args)

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return relaunch_ranks(args.gpus)

    import torch
    import torch.distributed as dist
    from paper_2608_02611_b200 import binding, sharding, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product has no CPU path")
    if world > torch.cuda.device_count():
        raise SystemExit(f"bench.py --gpus {world}: only {torch.cuda.device_count()} GPUs are visible")
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    ctx = binding.Context(local_rank)

    side = args.side
    small = side != SIDE
    steps = max(1, args.steps)
    warmup = max(3, args.warmup)

    # ---- inputs, resident in HBM (each rank: its own candidates, same reference) ----
    case, timings = synth.config2(dev, side=side, K=K_CANDS)
    N = case.N
    cands = []
    for k in range(K_CANDS):
        cands.append(case.make_cand(k) if rank == 0 else
                     synth._sparse_flips(case.ref, case.dtype, synth.MASTER_SEED + 2 + 1000 * rank, k, 100))
    d_timings = torch.from_numpy(timings).to(dev)
    out = torch.empty((K_CANDS, binding.RESULT_BYTES), dtype=torch.uint8, device=dev)
    torch.cuda.synchronize()

    # The gate and the adjudication do not depend on each other: they go to two streams (each
    # with its own context, since a context serves one stream at a time) and join for select.
    ctx_adj = binding.Context(local_rank)
    main = torch.cuda.current_stream(dev)
    side = torch.cuda.Stream(dev)

    held = binding.Candidates(cands)        # the same tensors every step: pointer array built once

    def step():
        side.wait_stream(main)
        with torch.cuda.stream(side):
            med, iqr, wins = ctx_adj.adjudicate(d_timings)
        ctx.screen(case.ref, held, case.atol, case.rtol, out=out)
        main.wait_stream(side)
        for t in (med, iqr, wins):
            t.record_stream(main)
        return ctx.select(out, med, binding.KB_SELECT_ERR_THEN_TIME, BUDGET)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    sampler.start()
    sampler.ready.wait(timeout=5)           # NVML initialised (tens of ms) before the load starts
    sampler.n_before_load = len(sampler.samples)
    for _ in range(warmup):
        step()
    barrier()
    assert ctx.poll() == 0 and ctx_adj.poll() == 0

    # ---- timed region: exactly `steps` steps, CUDA events, clocks sampled meanwhile ----
    # An event pair around the dominant kernel costs the step 6-9 us (the launches around it no
    # longer run back to back, and the streaming kernel can no longer be set up while the lead
    # kernel runs), so it is put on every fourth step of the timed region only.
    TIMED_EVERY = 4
    ctx.enable_timing(True)           # (creates the context's event pool, outside the timed region)
    ctx.enable_timing(False)
    launches0 = ctx.launch_count + ctx_adj.launch_count
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_begin = time.perf_counter()
    e0.record()
    for i in range(steps):
        if i % TIMED_EVERY == 0:
            ctx.enable_timing(True, keep=i > 0)
        elif i % TIMED_EVERY == 1:
            ctx.enable_timing(False)
        surv, n = step()
    e1.record()
    barrier()
    sampler.window = (t_begin, time.perf_counter())
    elapsed_ms = e0.elapsed_time(e1)
    launches = ctx.launch_count + ctx_adj.launch_count - launches0
    filter_used = {0: "plain", 1: "sharp", 3: "by definition"}.get(ctx.last_filter_mode, "?")
    stream_ms = ctx.read_timer(binding.KB_TIMER_SCREEN_STREAM)
    ctx.enable_timing(False)
    # the win-count kernel's own duration (a secondary figure): ten adjudications by themselves,
    # untimed and uncounted, with its event pair on (inside the step the kernel shares the GPU
    # with the resident streaming CTAs, and an event pair around it would measure its wait)
    torch.cuda.synchronize()
    ctx_adj.enable_timing(True)
    with torch.cuda.stream(side):
        for _ in range(10):
            ctx_adj.adjudicate(d_timings)
    torch.cuda.synchronize()
    wins_ms = ctx_adj.read_timer(binding.KB_TIMER_WINS)
    ctx_adj.enable_timing(False)
    # A timed region shorter than a few NVML queries (20 steps take 7 ms) leaves the sampler
    # nothing to see: the same steps go on, untimed and uncounted, until it has five samples
    # under this load.
    t_more = time.perf_counter()
    while sampler.is_alive() and len(sampler.samples) < 5 + sampler.n_before_load \
            and time.perf_counter() - t_more < 0.5:
        for _ in range(10):
            step()
        torch.cuda.synchronize()
    clocks = sampler.stop()
    if world > 1:
        elapsed_ms = sharding.max_over_ranks(elapsed_ms, dev)
    ms_per_step = elapsed_ms / steps
    value = world * K_CANDS * N / (ms_per_step * 1e-3)

    # ---- secondary: the same step captured once into a CUDA graph and replayed (what a caller who
    # captures the three calls gets: no per-kernel event pairs, launch gaps of a graph).  Not the
    # benchmark value. ----
    graph_replay = None
    if not args.no_graph:
        try:
            cap = torch.cuda.Stream(dev)
            cap2 = torch.cuda.Stream(dev)
            g_out = torch.empty_like(out)

            def graph_step():
                cur = torch.cuda.current_stream(dev)
                cap2.wait_stream(cur)
                with torch.cuda.stream(cap2):
                    med, iqr, wins = ctx_adj.adjudicate(d_timings)
                ctx.screen(case.ref, cands, case.atol, case.rtol, out=g_out)
                cur.wait_stream(cap2)
                return ctx.select(g_out, med, binding.KB_SELECT_ERR_THEN_TIME, BUDGET)

            cap.wait_stream(main)
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.stream(cap):
                with torch.cuda.graph(graph, stream=cap):
                    g_surv, g_n = graph_step()
            torch.cuda.synchronize()
            for _ in range(3):
                graph.replay()
            torch.cuda.synchronize()
            g_steps = min(steps, 200)
            e0g, e1g = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0g.record()
            for _ in range(g_steps):
                graph.replay()
            e1g.record()
            torch.cuda.synchronize()
            g_ms = e0g.elapsed_time(e1g) / g_steps
            same = bool((g_out == out).all()) and g_surv.tolist() == surv.tolist() and int(g_n) == int(n)
            graph_replay = {"ms_per_step": g_ms, "value": world * K_CANDS * N / (g_ms * 1e-3), "steps": g_steps,
                            "same_results_as_direct_calls": same}
            del graph
        except Exception as exc:   # a secondary figure must not take the benchmark line down
            graph_replay = {"error": str(exc)[:200]}
        torch.cuda.synchronize()

    # ---- end to end through the C ABI with HOST buffers (pinned), copies inside the timing ----
    e2e_steps = max(1, min(steps, 5))
    if args.no_e2e:
        e2e_steps = 0
    h_ref = case.ref.cpu().pin_memory() if e2e_steps else None
    h_cands = [c.cpu().pin_memory() for c in cands] if e2e_steps else []
    h_timings = torch.from_numpy(timings).pin_memory()

    def e2e_step():
        rec = ctx.screen_host(h_ref, h_cands, case.atol, case.rtol)          # H2D + D2H inside
        dt = h_timings.to(dev, non_blocking=True)
        med, iqr, wins = ctx_adj.adjudicate(dt)
        d_rec = torch.from_numpy(rec.view(np.uint8).reshape(K_CANDS, binding.RESULT_BYTES)).to(dev)
        surv, n = ctx.select(d_rec, med, binding.KB_SELECT_ERR_THEN_TIME, BUDGET)
        return surv.cpu(), n.cpu(), med.cpu(), iqr.cpu(), wins.cpu()

    if e2e_steps:
        e2e_step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        res = e2e_step()
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    if world > 1:
        e2e_s = sharding.max_over_ranks(e2e_s, dev)
    esz = synth.ELEM_SIZE[case.dtype]
    h2d = (K_CANDS + 1) * N * esz + K_CANDS * S_TIMINGS * 4 + K_CANDS * binding.RESULT_BYTES
    d2h = K_CANDS * binding.RESULT_BYTES + BUDGET * 4 + 4 + 2 * K_CANDS * 4 + K_CANDS * K_CANDS * 4
    e2e_value = world * K_CANDS * N / (e2e_s / e2e_steps) if e2e_steps else None

    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        torch.cuda.synchronize()
        ctx_adj.close()
        ctx.close()
        return

    # ---- roofline of the dominant kernel (streaming screen): algorithmic bytes / event time ----
    peak, peak_src = peaks()
    alg_bytes = (K_CANDS + 1) * N * esz                      # whole screen, reference counted once
    # the streaming kernel's own launch: everything but the tiles the scout kernel took
    # (min(8, max(1, tiles/128)) leading 4096-element tiles)
    ntiles = N // 4096
    nscout = min(8, max(1, ntiles // 128)) if ntiles >= 2 else 0
    stream_bytes = (K_CANDS + 1) * (N - nscout * 4096) * esz
    avg_stream_ms = float(np.mean(stream_ms)) if len(stream_ms) else float("nan")
    achieved = stream_bytes / (avg_stream_ms * 1e-3) / 1e9
    ratio = dram_bytes_per_algorithmic_byte()
    traffic = ratio * stream_bytes if ratio else None
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "traffic": traffic, "peak_source": peak_src,
                "traffic_source": os.path.relpath(TRAFFIC_FILE, ROOT) if traffic else None,
                "kernel": "screen_stream_kernel<bf16>", "launch_ms_avg": avg_stream_ms,
                "launch_ms_min": float(np.min(stream_ms)) if len(stream_ms) else None,
                "instantiation": filter_used,
                "algorithmic_bytes_per_launch": stream_bytes, "launches_timed": int(len(stream_ms)),
                "timed": f"every {TIMED_EVERY}th launch of the timed region",
                "share_of_step": avg_stream_ms / ms_per_step}

    # ---- CPU baseline: the oracle as it stands on a bounded sample (rank 0, N=1 only) ----
    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        cores = host_cores()
        n_sample = K_CANDS
        ref_np = synth.to_oracle_array(case.ref, case.dtype)
        cands_np = [synth.to_oracle_array(c, case.dtype) for c in cands[:n_sample]]
        secs = oracle_step(ref_np, cands_np, timings, n_sample, cores)
        cpu_baseline = {"value": n_sample * N / secs, "unit": UNIT, "cores": cores, "kind": "oracle",
                        "sample": f"one full step: {n_sample} candidates x {N} elements screened, "
                                  f"adjudication [64][100], select; {secs:.2f} s wall on {cores} threads"}

    S2 = S_TIMINGS * S_TIMINGS
    avg_wins_ms = float(np.mean(wins_ms)) if len(wins_ms) else float("nan")
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
        "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD if not small else f"{side}x{side} variant (profiler capture only)",
                   "K": K_CANDS, "N": N, "storage": "bf16", "S": S_TIMINGS, "budget": BUDGET,
                   "l2": "inputs (2.18 GB per step) exceed the 126 MB L2; no flush between steps",
                   "sharding": "candidates per rank, reference replicated, no collective"},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                "ms_per_step": e2e_s / e2e_steps * 1e3 if e2e_steps else None},
        "gpu_launches": int(launches),
        "roofline": roofline,
        "cpu_baseline": cpu_baseline,
        "screen_gbs_whole_step": world * alg_bytes / (ms_per_step * 1e-3) / 1e9,
        "pairwise_comparisons_per_s": K_CANDS * K_CANDS * S2 / (avg_wins_ms * 1e-3),
        "wins_kernel_ms_avg": avg_wins_ms,
        "n_survivors": int(n.item()),
        "graph_replay": graph_replay,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    torch.cuda.synchronize()
    ctx_adj.close()
    ctx.close()


if __name__ == "__main__":
    main()
