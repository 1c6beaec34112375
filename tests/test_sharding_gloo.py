"""The multi-rank host logic on CPU: two gloo ranks shard the candidates, each produces the
records of its block (here with the oracle standing in for the GPU), and the gathered result
equals the single-process result in candidate order; the step time is the maximum over ranks."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2608_02611_b200 import sharding, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, K, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        case, _ = synth.config2("cpu", side=128, K=K, n_bad=2, block=32)
        lo, hi = synth.shard_range(K, rank, world)
        ref = synth.to_oracle_array(case.ref, case.dtype)
        local = oracle.screen(ref, [synth.to_oracle_array(case.make_cand(k), case.dtype)
                                    for k in range(lo, hi)], case.dtype, case.atol, case.rtol)
        gathered = sharding.gather_records(local.view(np.uint8).reshape(-1, 48), K)
        slowest = sharding.max_over_ranks(1.0 + rank)
        if rank == 0:
            q.put((gathered.tobytes(), slowest))
    finally:
        dist.destroy_process_group()


import pytest


@pytest.mark.parametrize("K", [7, 1])     # an odd K: the shards differ in size; K = 1: one is empty
def test_two_ranks_shard_and_gather(K):
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, K, q)) for r in range(world)]
    for p in procs:
        p.start()
    blob, slowest = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    case, _ = synth.config2("cpu", side=128, K=K, n_bad=2, block=32)
    ref = synth.to_oracle_array(case.ref, case.dtype)
    want = oracle.screen(ref, [synth.to_oracle_array(case.make_cand(k), case.dtype) for k in range(K)],
                         case.dtype, case.atol, case.rtol)
    assert blob == want.tobytes()
    assert slowest == 2.0


# ---- element-range sharding: partition arithmetic and the all-gather of part records --------

def test_element_ranges_are_consecutive_aligned_and_cover():
    for N in (1, 4095, 4096, 4097, 3 * 4096 + 77, 1 << 20, (1 << 20) + 5):
        for world in (1, 2, 3, 8):
            prev = 0
            for r in range(world):
                lo, hi = sharding.element_range(N, r, world)
                assert lo == prev and lo <= hi <= N
                assert lo % sharding.RANGE_ALIGN == 0 or lo == N
                prev = hi
            assert prev == N


def _range_worker(rank, world, port, N, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        rng = np.random.default_rng(5)                       # the same tensors on every rank
        ref = rng.standard_normal(N).astype(np.float32)
        cands = [ref.copy() for _ in range(3)]
        cands[1][rng.integers(0, N, 20)] += 0.5
        cands[2][N - 1] = np.nan
        lo, hi = sharding.element_range(N, rank, world)
        if hi > lo:                                          # the oracle stands in for the GPU
            local = oracle.screen(ref[lo:hi], [c[lo:hi] for c in cands], oracle.F32, 1e-3, 1e-3)
        else:
            local = np.zeros(3, dtype=oracle.RESULT_DTYPE)
        parts, firsts = sharding.gather_parts(torch.from_numpy(local.view(np.uint8).reshape(-1, 48).copy()), lo, hi)
        merged = oracle.merge_ranges([p.numpy().reshape(-1).view(oracle.RESULT_DTYPE) for p in parts], firsts)
        if rank == world - 1:
            want = oracle.screen(ref, cands, oracle.F32, 1e-3, 1e-3)
            q.put((merged.tobytes() == want.tobytes(), len(firsts)))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("N,n_parts", [(5 * 4096 + 9, 2), (100, 1)])   # 100 elements: one rank's part is empty
def test_two_ranks_shard_the_elements(N, n_parts):
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_range_worker, args=(r, world, port, N, q)) for r in range(world)]
    for p in procs:
        p.start()
    same, parts = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert same and parts == n_parts
