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

