"""Candidate-sharded screening on two GPUs: one process per GPU over NCCL, one global K, each
rank screens its block against its replica of the reference, the records are all-gathered and
compared with the oracle; and element-range sharding of a few large tensors (each rank screens
its part, the parts' records are all-gathered and merged on the device).  Skipped where fewer
than two GPUs are visible.  The collectives carry the library's outputs only (no peer memory
reaches any kernel)."""
import os
import socket

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, K, side, q):
    import torch.distributed as dist
    import oracle
    from paper_2608_02611_b200 import binding, sharding, synth
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    torch.cuda.set_device(rank)
    dev = torch.device("cuda", rank)
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    ctx = binding.Context(rank)
    try:
        case, _ = synth.config2(dev, side=side, K=K, n_bad=3)
        got = sharding.screen_sharded(ctx, case.ref, case.make_cand, K, case.atol, case.rtol)
        assert ctx.poll() == 0
        slowest = sharding.max_over_ranks(1.0 + rank, dev)
        if rank == 0:
            ref = synth.to_oracle_array(case.ref, case.dtype)
            want = oracle.screen(ref, [synth.to_oracle_array(case.make_cand(k), case.dtype) for k in range(K)],
                                 case.dtype, case.atol, case.rtol, threads=8)
            q.put((got.tobytes() == want.tobytes(), slowest))
        dist.barrier()
    finally:
        ctx.close()
        dist.destroy_process_group()


@pytest.mark.parametrize("K,side", [(7, 256), (21, 1024)])
def test_two_gpus_shard_one_global_candidate_set(K, side):
    if torch.cuda.device_count() < 2:
        pytest.skip("needs two GPUs")
    import torch.multiprocessing as mp
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, K, side, q)) for r in range(world)]
    for p in procs:
        p.start()
    same, slowest = q.get(timeout=300)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert same and slowest == 2.0


def _range_worker(rank, world, port, K, N, q):
    import torch.distributed as dist
    import oracle
    from paper_2608_02611_b200 import binding, sharding, synth
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    torch.cuda.set_device(rank)
    dev = torch.device("cuda", rank)
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    ctx = binding.Context(rank)
    try:
        g = torch.Generator().manual_seed(77)                       # the same host tensors on every rank
        ref = torch.randn(N, generator=g).to(torch.bfloat16)
        cands = []
        for k in range(K):
            c = ref.clone()
            idx = torch.randint(0, N, (50,), generator=g)
            c[idx] = (c[idx].float() * 1.05).to(torch.bfloat16)
            cands.append(c)
        lo, hi = sharding.element_range(N, rank, world)
        got = sharding.screen_range_sharded(ctx, ref[lo:hi].to(dev), [c[lo:hi].to(dev) for c in cands],
                                            lo, hi, 1e-2, 1.6e-2)
        assert ctx.poll() == 0
        if rank == 0:
            want = oracle.screen(synth.to_oracle_array(ref, synth.BF16),
                                 [synth.to_oracle_array(c, synth.BF16) for c in cands], synth.BF16, 1e-2, 1.6e-2)
            q.put(got.tobytes() == want.tobytes())
        dist.barrier()
    finally:
        ctx.close()
        dist.destroy_process_group()


@pytest.mark.parametrize("K,N", [(3, 1 << 20), (2, 3 * 4096 + 77)])
def test_two_gpus_shard_the_elements_of_a_few_large_tensors(K, N):
    if torch.cuda.device_count() < 2:
        pytest.skip("needs two GPUs")
    import torch.multiprocessing as mp
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_range_worker, args=(r, world, port, K, N, q)) for r in range(world)]
    for p in procs:
        p.start()
    same = q.get(timeout=300)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert same
