"""Seeded synthetic inputs for the screen / adjudicate / select path.

The paper's workloads are the output tensors of six benchmark kernels
(Appendix, Benchmark Descriptions and Shapes) and their repeated timings
(Appendix, Relative Variability Metrics); neither the candidates nor the
measurements are available, so these generators build stand-ins with the same
shapes, value ranges and failure structure.  The module holds NO arithmetic of
the method itself: it only produces tensors and timing matrices, plus the
ground truth that follows in closed form from how a candidate was built
(e.g. "3 NaN and 1 Inf were written").  Both the CUDA path and the CPU oracle
consume the bytes produced here.

Dense per-element noise is integer-only (a counter-based 64-bit hash of
(seed, candidate, index) driving +-1-ulp steps on the sign-magnitude bit
pattern), so it gives identical bytes on any torch device.  Floating-point
draws (the reference values, the timings) are made on the host in double
precision with a Philox generator and rounded once.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Callable, Dict, List, Optional, Tuple

import numpy as np
import torch

MASTER_SEED = 260802611

# dtype codes at the C boundary
F32, F16, BF16, F8E4M3, F8E5M2 = 0, 1, 2, 3, 4
TORCH_DTYPE = {F32: torch.float32, F16: torch.float16, BF16: torch.bfloat16,
               F8E4M3: torch.float8_e4m3fn, F8E5M2: torch.float8_e5m2}
ELEM_SIZE = {F32: 4, F16: 2, BF16: 2, F8E4M3: 1, F8E5M2: 1}
_INT_VIEW = {F32: torch.int32, F16: torch.int16, BF16: torch.int16, F8E4M3: torch.int8, F8E5M2: torch.int8}
_MAG_MASK = {F32: 0x7FFFFFFF, F16: 0x7FFF, BF16: 0x7FFF, F8E4M3: 0x7F, F8E5M2: 0x7F}
# first magnitude pattern that is not a finite number (e4m3fn has no Inf: 0x7F is its NaN)
_INF_MAG = {F32: 0x7F800000, F16: 0x7C00, BF16: 0x7F80, F8E4M3: 0x7F, F8E5M2: 0x7C}
_SIGN_BIT = {F32: 0x80000000, F16: 0x8000, BF16: 0x8000, F8E4M3: 0x80, F8E5M2: 0x80}
_BITS = {F32: 32, F16: 16, BF16: 16, F8E4M3: 8, F8E5M2: 8}


# --------------------------------------------------------------------------
# counter-based hash (integer only; identical on CPU and CUDA)
# --------------------------------------------------------------------------

def _s64(v: int) -> int:
    """Python int -> the same 64 bits as a signed value."""
    v &= (1 << 64) - 1
    return v - (1 << 64) if v >= (1 << 63) else v


_C1 = _s64(0xBF58476D1CE4E5B9)
_C2 = _s64(0x94D049BB133111EB)
_GOLD = _s64(0x9E3779B97F4A7C15)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of int64."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def mix64(x: torch.Tensor) -> torch.Tensor:
    """splitmix64 finaliser on an int64 tensor (wrapping arithmetic)."""
    x = (x ^ _lsr(x, 30)) * _C1
    x = (x ^ _lsr(x, 27)) * _C2
    return x ^ _lsr(x, 31)


def mix64_int(v: int) -> int:
    """The same finaliser on one Python int (for host-side structure draws)."""
    m = (1 << 64) - 1
    v &= m
    v = ((v ^ (v >> 30)) * 0xBF58476D1CE4E5B9) & m
    v = ((v ^ (v >> 27)) * 0x94D049BB133111EB) & m
    return v ^ (v >> 31)


def hash_elems(seed: int, k: int, idx: torch.Tensor) -> torch.Tensor:
    """Non-negative 62-bit hash of (seed, k, idx) for an int64 index tensor."""
    base = _s64(mix64_int(seed * 0x9E3779B97F4A7C15 + (k + 1) * 0xD1B54A32D192ED03))
    h = mix64(idx * _GOLD + base)
    return _lsr(h, 2)


def host_rng(seed: int, stream: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed & ((1 << 64) - 1), stream]))


# --------------------------------------------------------------------------
# bit-pattern helpers
# --------------------------------------------------------------------------

def _bits(t: torch.Tensor, dtype: int) -> torch.Tensor:
    """int64 tensor holding the unsigned bit pattern of each element."""
    b = t.view(_INT_VIEW[dtype]).to(torch.int64)
    return b & ((1 << _BITS[dtype]) - 1)


def _from_bits(b: torch.Tensor, dtype: int) -> torch.Tensor:
    n = _BITS[dtype]
    b = torch.where(b >= (1 << (n - 1)), b - (1 << n), b).to(_INT_VIEW[dtype])
    return b.view(TORCH_DTYPE[dtype])


def ulp_step(t: torch.Tensor, dtype: int, step: torch.Tensor) -> torch.Tensor:
    """Move each element by `step` (int64, any small integer) units in the last
    place of its sign-magnitude pattern.  A magnitude never goes below 0 (a
    zero only moves up) and never reaches the Inf pattern (it moves down
    instead)."""
    b = _bits(t, dtype)
    sign = b & _SIGN_BIT[dtype]
    mag = b & _MAG_MASK[dtype]
    new = mag + step
    new = torch.where(new < 0, mag - step, new)
    new = torch.where(new >= _INF_MAG[dtype], mag - step.abs(), new)
    return _from_bits(sign | new, dtype)


def _round_to(x64: np.ndarray, dtype: int, device) -> torch.Tensor:
    return torch.from_numpy(x64).to(TORCH_DTYPE[dtype]).to(device)


# --------------------------------------------------------------------------
# case containers
# --------------------------------------------------------------------------

@dataclass
class ScreenCase:
    name: str
    dtype: int
    N: int
    K: int
    atol: float
    rtol: float
    ref: torch.Tensor
    make_cand: Callable[[int], torch.Tensor]
    truth: Dict[int, dict] = field(default_factory=dict)   # per-candidate closed-form facts
    mask: Optional[tuple] = None                           # ("strided", log2_tile, stride, phase)
    notes: str = ""

    def cands(self) -> List[torch.Tensor]:
        return [self.make_cand(k) for k in range(self.K)]


def to_oracle_array(t: torch.Tensor, dtype: int) -> np.ndarray:
    """Raw bytes of a tensor as the numpy array the oracle expects."""
    t = t.detach().contiguous().cpu().reshape(-1)
    if dtype == F32:
        return t.numpy()
    if _BITS[dtype] == 8:
        return t.view(torch.int8).numpy().view(np.uint8)
    return t.view(torch.int16).numpy().view(np.uint16)


# --------------------------------------------------------------------------
# timings (host, double precision, rounded once)
# --------------------------------------------------------------------------

def lognormal_timings(seed: int, t_k: np.ndarray, S: int, sigma: float,
                      outlier_prob: float = 0.0, outlier_factor: float = 1.0,
                      quantum_ms: float = 0.0) -> np.ndarray:
    """timings[K][S] = t_k * exp(sigma*z), optional xfactor outliers, optional
    quantisation to a grid (ties).  float32 milliseconds."""
    rng = host_rng(seed, 7)
    K = len(t_k)
    z = rng.standard_normal((K, S))
    t = np.asarray(t_k, dtype=np.float64)[:, None] * np.exp(sigma * z)
    if outlier_prob > 0.0:
        u = rng.random((K, S))
        t = np.where(u < outlier_prob, t * outlier_factor, t)
    if quantum_ms > 0.0:
        per_ms = np.float32(round(1.0 / quantum_ms))
        t32 = np.round(t / quantum_ms).astype(np.float32) / per_ms
        return np.ascontiguousarray(t32, dtype=np.float32)
    return np.ascontiguousarray(t.astype(np.float32))


def base_latencies(seed: int, K: int, spread_sigma: float) -> np.ndarray:
    """Per-candidate true latency t_k = exp(spread_sigma * z_k) ms."""
    rng = host_rng(seed, 11)
    return np.exp(spread_sigma * rng.standard_normal(K))


# --------------------------------------------------------------------------
# config 1: fp32, N = 65536, K = 4
# --------------------------------------------------------------------------

def config1(device="cpu", N: int = 65536) -> Tuple[ScreenCase, np.ndarray]:
    seed = MASTER_SEED + 1
    rng = host_rng(seed, 0)
    ref64 = rng.standard_normal(N)
    ref = _round_to(ref64, F32, device)
    noise = rng.standard_normal(N) * 1e-6
    cand1 = (torch.from_numpy(ref64.astype(np.float32)) +
             torch.from_numpy(noise.astype(np.float32))).to(device)
    bad_idx = rng.choice(N, size=4, replace=False)
    burst_len = min(100, N)
    burst_start = int(rng.integers(0, N - burst_len + 1))

    def make(k: int) -> torch.Tensor:
        if k == 0:
            return ref.clone()
        if k == 1:
            return cand1.clone()
        if k == 2:
            c = ref.clone()
            c[torch.as_tensor(bad_idx[:3], device=device)] = float("nan")
            c[int(bad_idx[3])] = float("inf")
            return c
        c = ref.clone()
        c[burst_start:burst_start + burst_len] += 0.01  # fp32 add of (float)0.01
        return c

    truth = {
        0: dict(kind="copy", passes=True, mismatch=0, nan=0, inf=0),
        1: dict(kind="tiny_noise", passes=True, mismatch=0, nan=0, inf=0),
        2: dict(kind="nan_inf", passes=False, mismatch=4, nan=3, inf=1, max_abs=0.0,
                idx=sorted(int(i) for i in bad_idx)),
        3: dict(kind="burst", passes=False, mismatch=burst_len, nan=0, inf=0,
                burst=(burst_start, burst_len)),
    }
    case = ScreenCase("config1", F32, N, 4, 1e-5, 1e-3, ref, make, truth)
    timings = lognormal_timings(seed, np.array([1.0, 0.9, 0.9, 1.2]), 20, 0.05)
    return case, timings


# --------------------------------------------------------------------------
# config 2: bf16 GEMM-output-like, side x side, K = 64
# --------------------------------------------------------------------------

def _normal_ref(seed: int, N: int, sigma: float, dtype: int, device) -> torch.Tensor:
    rng = host_rng(seed, 0)
    out = torch.empty(N, dtype=TORCH_DTYPE[dtype], device=device)
    chunk = 1 << 24
    for s in range(0, N, chunk):
        n = min(chunk, N - s)
        out[s:s + n] = _round_to(rng.standard_normal(n) * sigma, dtype, device)
    return out


def _sparse_flips(ref: torch.Tensor, dtype: int, seed: int, k: int, one_in: int,
                  ulps: int = 1) -> torch.Tensor:
    """Copy of ref with +-ulps steps where hash % one_in == 0 (direction: next bit)."""
    N = ref.numel()
    out = torch.empty_like(ref)
    chunk = 1 << 24
    for s in range(0, N, chunk):
        n = min(chunk, N - s)
        idx = torch.arange(s, s + n, dtype=torch.int64, device=ref.device)
        h = hash_elems(seed, k, idx)
        hit = (h % one_in) == 0
        direction = 1 - 2 * ((h // one_in) & 1)
        step = torch.where(hit, direction * ulps, torch.zeros_like(direction))
        out[s:s + n] = ulp_step(ref[s:s + n], dtype, step)
    return out


def config2(device="cpu", side: int = 4096, K: int = 64, n_bad: int = 10,
            block: int = 128) -> Tuple[ScreenCase, np.ndarray]:
    seed = MASTER_SEED + 2
    N = side * side
    ref = _normal_ref(seed, N, 4.0, BF16, device)
    rng = host_rng(seed, 1)
    bad = sorted(int(x) for x in rng.choice(K, size=min(n_bad, K), replace=False))
    nblk = side // block
    blocks = {k: (int(rng.integers(0, nblk)), int(rng.integers(0, nblk))) for k in bad}

    def make(k: int) -> torch.Tensor:
        if k not in blocks:
            return _sparse_flips(ref, BF16, seed, k, 100)
        c = ref.clone().view(side, side)
        br, bc = blocks[k]
        rows = torch.arange(br * block, (br + 1) * block, dtype=torch.int64, device=device)
        cols = torch.arange(bc * block, (bc + 1) * block, dtype=torch.int64, device=device)
        flat = (rows[:, None] * side + cols[None, :]).reshape(-1)
        src = hash_elems(seed, k, flat) % N            # values drawn from the same distribution
        c.view(-1)[flat] = ref[src]
        return c.view(-1)

    truth = {}
    for k in range(K):
        if k in blocks:
            truth[k] = dict(kind="wrong_block", passes=False, block=blocks[k],
                            mismatch_max=block * block, nan=0, inf=0)
        else:
            truth[k] = dict(kind="ulp_flips", passes=True, mismatch=0, nan=0, inf=0,
                            rel_bound=2.0 ** -7)
    case = ScreenCase("config2", BF16, N, K, 1e-2, 1.6e-2, ref, make, truth)
    t_k = base_latencies(seed, K, 0.1)
    timings = lognormal_timings(seed, t_k, 100, 0.08)
    return case, timings


# --------------------------------------------------------------------------
# config 3: fp16 attention-output-like (B, H, S, D), K = 256
# --------------------------------------------------------------------------

def config3(device="cpu", B: int = 8, H: int = 32, S: int = 2048, D: int = 128, K: int = 256,
            n_nan: int = 13, n_transposed: int = 13, S_t: int = 200) -> Tuple[ScreenCase, np.ndarray]:
    seed = MASTER_SEED + 3
    rng = host_rng(seed, 0)
    T = 64                                              # table entries per head
    V = torch.from_numpy(rng.uniform(-3.0, 3.0, size=(H, T, D)).astype(np.float32)).to(device)
    N = B * H * S * D
    ref = torch.empty(N, dtype=torch.float16, device=device)
    ref4 = ref.view(B, H, S, D)
    for b in range(B):
        idx = torch.from_numpy(rng.integers(0, T, size=(H, S, 4))).to(device)
        logits = torch.from_numpy(rng.standard_normal((H, S, 4)).astype(np.float32)).to(device)
        w = torch.softmax(logits, dim=-1)
        acc = torch.zeros(H, S, D, dtype=torch.float32, device=device)
        harange = torch.arange(H, device=device)[:, None]
        for j in range(4):
            acc += w[:, :, j, None] * V[harange, idx[:, :, j]]
        ref4[b] = acc.to(torch.float16)
    special = rng.choice(K, size=min(K, n_nan + n_transposed), replace=False)
    nan_c = {int(k): int(rng.integers(0, B * H * S)) for k in special[:n_nan]}
    tr_c = {int(k): int(rng.integers(0, B * H)) for k in special[n_nan:]}
    L = S * D

    def make(k: int) -> torch.Tensor:
        c = torch.empty_like(ref)
        chunk = 1 << 24
        for s in range(0, N, chunk):
            n = min(chunk, N - s)
            i = torch.arange(s, s + n, dtype=torch.int64, device=device)
            step = (hash_elems(seed, k, i) % 3) - 1
            c[s:s + n] = ulp_step(ref[s:s + n], F16, step)
        if k in nan_c:
            row = nan_c[k]
            c[row * D:(row + 1) * D] = float("nan")
        if k in tr_c:
            blk = tr_c[k]
            src = c[blk * L:(blk + 1) * L].clone()
            c[blk * L:(blk + 1) * L] = src.view(D, S).t().contiguous().view(-1)
        return c

    truth = {}
    for k in range(K):
        if k in nan_c:
            truth[k] = dict(kind="nan_row", passes=False, nan=D, inf=0, mismatch_min=D,
                            row=nan_c[k])
        elif k in tr_c:
            truth[k] = dict(kind="transposed_head", passes=False, nan=0, inf=0, head=tr_c[k])
        else:
            truth[k] = dict(kind="ulp_noise", passes=True, mismatch=0, nan=0, inf=0)
    case = ScreenCase("config3", F16, N, K, 1e-3, 1e-2, ref, make, truth)
    t_k = base_latencies(seed, K, 0.1)
    timings = lognormal_timings(seed, t_k, S_t, 0.1, outlier_prob=0.02, outlier_factor=3.0)
    return case, timings


# --------------------------------------------------------------------------
# config 4: fp32 heavy-tailed, N = 2^20, K = 1024
# --------------------------------------------------------------------------

def config4(device="cpu", N: int = 1 << 20, K: int = 1024, S_t: int = 64) -> Tuple[ScreenCase, np.ndarray]:
    seed = MASTER_SEED + 4
    rng = host_rng(seed, 0)
    z = rng.standard_normal(N)
    sign = np.where(rng.random(N) < 0.5, -1.0, 1.0)
    ref64 = sign * np.exp(4.0 * z)
    zero_idx = rng.choice(N, size=max(1, N // 100), replace=False)
    ref64[zero_idx] = 0.0
    ref = _round_to(ref64, F32, device)
    n_inf = max(1, (K * 5) // 100)
    n_rel = max(1, (K * 5) // 100) if K >= 3 else 0
    special = rng.choice(K, size=min(K, n_inf + n_rel), replace=False)
    inf_c = {}
    for k in special[:n_inf]:
        cnt = int(rng.integers(1, 9))
        pos = rng.choice(N, size=cnt, replace=False)
        sg = rng.random(cnt) < 0.5
        inf_c[int(k)] = [(int(p), bool(s)) for p, s in zip(pos, sg)]
    rel_c = set(int(k) for k in special[n_inf:])
    up = torch.tensor(1.0 + 2e-3, dtype=torch.float32, device=device)
    dn = torch.tensor(1.0 - 2e-3, dtype=torch.float32, device=device)

    def make(k: int) -> torch.Tensor:
        if k in inf_c:
            c = ref.clone()
            for p, neg in inf_c[k]:
                c[p] = float("-inf") if neg else float("inf")
            return c
        if k in rel_c:
            i = torch.arange(N, dtype=torch.int64, device=device)
            s = (hash_elems(seed, k, i) & 1) == 1
            return ref * torch.where(s, up, dn)
        return _sparse_flips(ref, F32, seed, k, 100)

    truth = {}
    for k in range(K):
        if k in inf_c:
            truth[k] = dict(kind="inf", passes=False, nan=0, inf=len(inf_c[k]),
                            mismatch=len(inf_c[k]), max_abs=0.0)
        elif k in rel_c:
            truth[k] = dict(kind="rel_2e-3", passes=False, nan=0, inf=0)
        else:
            truth[k] = dict(kind="ulp_flips", passes=True, mismatch=0, nan=0, inf=0,
                            rel_bound=2.0 ** -23)
    case = ScreenCase("config4", F32, N, K, 1e-6, 1e-3, ref, make, truth)
    t_k = base_latencies(seed, K, 0.2)
    timings = lognormal_timings(seed, t_k, S_t, 0.05, quantum_ms=1e-3)
    return case, timings


# --------------------------------------------------------------------------
# config 5: two-tier bf16, N = 2^28, K = 512, tier-1 mask 1/16 of 4096-tiles
# --------------------------------------------------------------------------

def config5(device="cpu", N: int = 1 << 28, K: int = 512, budget: int = 32, S1: int = 200,
            S2: int = 2000, log2_tile: int = 12, stride: int = 16,
            burst_len: int = 16384) -> dict:
    """Returns a dict: case (tier-1 ScreenCase with its mask), timings1,
    make_timings2(survivors) and the population labels."""
    seed = MASTER_SEED + 5
    phase = seed % stride
    ref = _normal_ref(seed, N, 4.0, BF16, device)
    rng = host_rng(seed, 1)
    # population in proportion 128 : 128 : 64 : 128 : 64 of 512
    counts = [K * 128 // 512, K * 128 // 512, K * 64 // 512, K * 128 // 512]
    counts.append(K - sum(counts))
    labels = (["clean"] * counts[0] + ["hidden_burst"] * counts[1] + ["visible_burst"] * counts[2]
              + ["ulp4"] * counts[3] + ["nan_inf"] * counts[4])
    perm = rng.permutation(K)
    label_of = {int(perm[i]): labels[i] for i in range(K)}
    tile = 1 << log2_tile
    ntiles = (N + tile - 1) // tile
    burst_tiles = max(1, burst_len // tile)
    blen = min(burst_len, burst_tiles * tile)
    params: Dict[int, dict] = {}
    for k in range(K):
        lab = label_of[k]
        if lab == "hidden_burst":
            # a run of tiles none of which is selected: fits between two selected tiles
            assert burst_tiles < stride
            g = int(rng.integers(0, max(1, ntiles // stride - 1)))
            start_tile = g * stride + phase + 1
            params[k] = dict(start=start_tile * tile, length=blen)
        elif lab == "visible_burst":
            g = int(rng.integers(0, max(1, ntiles // stride - 1)))
            start_tile = g * stride + phase         # begins inside a selected tile
            params[k] = dict(start=start_tile * tile, length=blen)
        elif lab == "nan_inf":
            cnt = int(rng.integers(1, 9))
            tiles_sel = rng.integers(0, max(1, ntiles // stride), size=cnt) * stride + phase
            offs = rng.integers(0, tile, size=cnt)
            pos = sorted(set(int(min(N - 1, t * tile + o)) for t, o in zip(tiles_sel, offs)))
            kinds = [bool(x) for x in (rng.random(len(pos)) < 0.5)]
            params[k] = dict(pos=pos, is_nan=kinds)

    def make(k: int) -> torch.Tensor:
        lab = label_of[k]
        if lab == "ulp4":
            return _sparse_flips(ref, BF16, seed, k, 1000, ulps=4)
        c = _sparse_flips(ref, BF16, seed, k, 100)
        if lab in ("hidden_burst", "visible_burst"):
            p = params[k]
            i = torch.arange(p["start"], p["start"] + p["length"], dtype=torch.int64, device=device)
            src = hash_elems(seed, k, i) % N
            c[p["start"]:p["start"] + p["length"]] = ref[src]
        elif lab == "nan_inf":
            p = params[k]
            for pos, is_nan in zip(p["pos"], p["is_nan"]):
                c[pos] = float("nan") if is_nan else float("inf")
        return c

    truth = {}
    for k in range(K):
        lab = label_of[k]
        if lab == "clean":
            truth[k] = dict(kind=lab, tier1_pass=True, tier2_pass=True)
        elif lab == "hidden_burst":
            truth[k] = dict(kind=lab, tier1_pass=True, tier2_pass=False, **params[k])
        elif lab == "visible_burst":
            truth[k] = dict(kind=lab, tier1_pass=False, tier2_pass=False, **params[k])
        elif lab == "ulp4":
            truth[k] = dict(kind=lab, tier1_pass=False, tier2_pass=False)
        else:
            p = params[k]
            truth[k] = dict(kind=lab, tier1_pass=False, tier2_pass=False,
                            nan=sum(p["is_nan"]), inf=len(p["pos"]) - sum(p["is_nan"]))
    case = ScreenCase("config5", BF16, N, K, 1e-2, 1.6e-2, ref, make, truth,
                      mask=("strided", log2_tile, stride, phase))
    t_k = base_latencies(seed, K, 0.3)
    timings1 = lognormal_timings(seed, t_k, S1, 0.15)

    def make_timings2(survivors) -> np.ndarray:
        return lognormal_timings(seed + 1000, t_k[np.asarray(survivors, dtype=np.int64)], S2, 0.15)

    return dict(case=case, timings1=timings1, make_timings2=make_timings2, labels=label_of,
                budget=budget, t_k=t_k)


# --------------------------------------------------------------------------
# sharding helper for the multi-GPU bench / tests (candidates are independent)
# --------------------------------------------------------------------------

def shard_range(K: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous block of candidate indices owned by `rank` (balanced to +-1)."""
    base, extra = divmod(K, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)
