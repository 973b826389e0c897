"""The N>1 host path on CPU: two gloo ranks shard the workload, time a dummy region, reduce with MAX."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    from paper_2402_06082_b200 import sharding, synth
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = sharding.rank_workload(synth.CFG3.scaled(B=1, H=2, Hkv=2, ncomp=4), rank)
    K, _, _ = synth.sequence_stream(w, 0, 16)
    dist.barrier()
    ms = sharding.max_over_ranks(10.0 * (rank + 1), dist)
    q.put((rank, w.data_seed, float(K.float().sum()), ms, sharding.job_steps_per_s(world, 5, ms)))
    dist.destroy_process_group()


def test_two_ranks_shard_and_reduce():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, seed0, sum0, ms0, v0), (r1, seed1, sum1, ms1, v1) = res
    assert seed0 != seed1 and sum0 != sum1            # each rank serves its own sequences
    assert ms0 == ms1 == 20.0                         # the slowest rank defines the time
    assert v0 == v1 == 2 * 5 / 0.020


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    from paper_2402_06082_b200 import sharding
    assert sharding.max_over_ranks(3.5) == 3.5
    assert sharding.job_steps_per_s(1, 10, 100.0) == 100.0
