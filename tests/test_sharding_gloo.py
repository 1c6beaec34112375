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
