"""Candidate sharding across ranks (one process per GPU).

The gate has no exchange step: candidates are independent, so a job with one
global K gives each rank a contiguous block of candidates (`synth.shard_range`)
and a replica of the reference, and gathers K 48-byte records at the end.  The
only other cross-rank value is the step time, taken as the maximum over ranks.
These helpers work with any torch.distributed backend (NCCL on GPUs; the CPU
tests use gloo).
"""
from __future__ import annotations

import numpy as np
import torch
import torch.distributed as dist

from .synth import shard_range

RECORD_BYTES = 48


def gather_records(local: np.ndarray, K: int, device="cpu") -> np.ndarray:
    """All-gather per-rank record blocks (uint8 view, [k_local, 48]) into [K, 48] in
    candidate order.  `local` must hold exactly the records of shard_range(K, rank, world)."""
    world, rank = dist.get_world_size(), dist.get_rank()
    lo, hi = shard_range(K, rank, world)
    local = np.ascontiguousarray(local).view(np.uint8).reshape(-1, RECORD_BYTES)
    if local.shape[0] != hi - lo:
        raise ValueError(f"rank {rank} holds {local.shape[0]} records, its shard has {hi - lo}")
    width = max(shard_range(K, r, world)[1] - shard_range(K, r, world)[0] for r in range(world))
    pad = torch.zeros((width, RECORD_BYTES), dtype=torch.uint8, device=device)
    pad[: hi - lo] = torch.from_numpy(local).to(device)
    parts = [torch.empty_like(pad) for _ in range(world)]
    dist.all_gather(parts, pad)
    out = np.zeros((K, RECORD_BYTES), dtype=np.uint8)
    for r in range(world):
        a, b = shard_range(K, r, world)
        out[a:b] = parts[r][: b - a].cpu().numpy()
    return out


def max_over_ranks(value: float, device="cpu") -> float:
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def screen_sharded(ctx, ref: torch.Tensor, make_cand, K: int, atol: float, rtol: float,
                   mask=None) -> np.ndarray:
    """The gate over ONE global set of K candidates, sharded by candidate across the ranks of
    the default process group (one process per GPU).

    Every rank holds a replica of the reference on its own GPU; `make_cand(k)` returns
    candidate k as a tensor on this rank's device and is called only for the rank's own block
    `shard_range(K, rank, world)`.  Each rank runs kb_screen on its block through `ctx` (a
    binding.Context on its device); the K 48-byte records are then all-gathered (NCCL on GPUs),
    so every rank returns all K records in candidate order.  The collective moves the library's
    outputs only: no kernel is ever handed another GPU's memory.

    The adjudication is not sharded: its input is K x S floats and the whole call takes well
    under 0.1 ms on one GPU, less than an all-gather of the win matrix's rows would.
    """
    from . import binding
    world, rank = dist.get_world_size(), dist.get_rank()
    lo, hi = shard_range(K, rank, world)
    if hi > lo:
        cands = [make_cand(k) for k in range(lo, hi)]
        local = binding.records(ctx.screen(ref, cands, atol, rtol, mask))
        local = local.view(np.uint8).reshape(-1, RECORD_BYTES)
    else:
        local = np.zeros((0, RECORD_BYTES), dtype=np.uint8)
    out = gather_records(local, K, device=ref.device)
    return out.reshape(-1).view(binding.RESULT_DTYPE)



# ---------------------------------------------------------------------------------------------
# Element-range sharding: few, large tensors (the last rungs of a funnel: 3 candidates of 1.6e9
# elements).  Every rank holds one contiguous part of the reference and of every candidate,
# screens it, and the K records of the parts are merged into the records of the whole range
# (kb_merge_ranges).  The only exchange is an all-gather of R x K 48-byte records.
# ---------------------------------------------------------------------------------------------

RANGE_ALIGN = 4096          # elements: parts start on kernel-tile boundaries (and so 16-byte aligned)


def element_range(N: int, rank: int, world: int, align: int = RANGE_ALIGN):
    """[lo, hi) of rank's part of N elements: consecutive, covering, every part but the last a
    whole number of `align`-element tiles; trailing ranks get an empty part when there are
    fewer tiles than ranks."""
    tiles = (N + align - 1) // align
    per, extra = divmod(tiles, world)
    t_lo = rank * per + min(rank, extra)
    t_hi = t_lo + per + (1 if rank < extra else 0)
    return min(t_lo * align, N), min(t_hi * align, N)


def gather_parts(local: torch.Tensor, lo: int, hi: int):
    """All-gather every rank's [K, 48] records and range start.  Returns (parts, firsts): the
    records of the non-empty parts as one uint8 tensor [R, K, 48] on `local`'s device, in
    ascending range order, and their first global indices."""
    world = dist.get_world_size()
    local = local.contiguous().view(torch.uint8).reshape(-1, RECORD_BYTES)
    got = [torch.empty_like(local) for _ in range(world)]
    dist.all_gather(got, local)
    bounds = torch.tensor([lo, hi], dtype=torch.int64, device=local.device)
    all_bounds = [torch.empty_like(bounds) for _ in range(world)]
    dist.all_gather(all_bounds, bounds)
    keep = [(int(b[0]), r) for r, b in enumerate(all_bounds) if int(b[1]) > int(b[0])]
    keep.sort()
    parts = torch.stack([got[r] for _, r in keep])
    return parts, [f for f, _ in keep]


def screen_range_sharded(ctx, ref_part: torch.Tensor, cand_parts, lo: int, hi: int,
                         atol: float, rtol: float) -> np.ndarray:
    """The gate over tensors whose ELEMENTS are spread over the ranks of the default process
    group: this rank holds elements [lo, hi) of the reference (`ref_part`) and of each of the
    K candidates (`cand_parts`), with `lo` a multiple of RANGE_ALIGN (see `element_range`).
    Each rank screens its part through `ctx`; the records are all-gathered and merged on the
    device by kb_merge_ranges, so every rank returns the K records of the whole range.  A rank
    with an empty part (hi == lo) passes any tensors of K candidates' shape [0]."""
    from . import binding
    K = len(cand_parts)
    if hi > lo:
        local = ctx.screen(ref_part, cand_parts, atol, rtol)
    else:
        local = torch.zeros((K, RECORD_BYTES), dtype=torch.uint8, device=ref_part.device)
    parts, firsts = gather_parts(local, lo, hi)
    merged = ctx.merge_ranges(parts, firsts)
    return binding.records(merged)
