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


# ---- a job cut over two ranks gives the unsharded job's outputs --------------------------------------------
def _job():
    sys.path.insert(0, ROOT)
    from paper_2402_06082_b200 import synth
    w = synth.CFG3.scaled(B=3, H=8, Hkv=4, d=64, dtype="fp32", n_prompt=0, ncomp=6, s=24, t=3, window=5, m_max=64)
    return w, 70


def _oracle_outputs(w, n, units, unit_ids):
    """Outputs [len(units), G, n, d] of the CPU oracle for the given (seq, kvhead) units keyed with unit_ids."""
    import numpy as np
    from oracle import subgen_oracle as orc
    from paper_2402_06082_b200 import synth
    G = w.H // w.Hkv
    out = np.zeros((len(units), G, n, w.d))
    for i, ((b, h), uid) in enumerate(zip(units, unit_ids)):
        K, V, Q = (synth.to_f32_numpy(x) for x in synth.sequence_stream(w, b, n, "cpu"))
        o = orc.OracleUnit(w.d, w.delta, w.t, w.s, w.window, seed=w.philox_seed, unit_id=uid, m_max=w.m_max)
        for j in range(n):
            o.push(K[h, j], V[h, j])
            for g in range(G):
                out[i, g, j] = o.query(Q[h * G + g, j])
    return out


def _shard_worker(rank, world, port, mode, q):
    sys.path.insert(0, ROOT)
    import numpy as np
    from paper_2402_06082_b200 import sharding
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w, n = _job()
    shards = sharding.partition(w.B, w.H, w.Hkv, world, mode)
    me = shards[rank]
    units = [(me.b0 + lb, me.h0 + lh) for lb in range(me.B_local) for lh in range(me.Hkv_local)]
    ids = [me.unit_id(lb, lh) for lb in range(me.B_local) for lh in range(me.Hkv_local)]
    o = _oracle_outputs(w, n, units, ids)                       # [units, G, n, d]
    G = me.G
    last = torch.from_numpy(o[:, :, n - 1]).reshape(me.B_local, me.Hkv_local * G, w.d)      # the last step's [B_l, H_l, d]
    full = sharding.gather_outputs(last, shards, rank, dist)
    q.put((rank, [s.unit_offset for s in shards], full.numpy()))
    dist.destroy_process_group()


def _run_sharded(mode):
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + os.getpid() % 2000 + (7 if mode == "head" else 0)
    procs = [ctx.Process(target=_shard_worker, args=(r, 2, port, mode, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted((q.get(timeout=300) for _ in procs), key=lambda x: x[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    return res


def test_sharded_job_equals_unsharded_job():
    """Two gloo ranks each run the oracle on their shard (units numbered as in the whole job) and gather the step's
    output; the result equals the unsharded job's, number for number, whether the job is cut by sequence (3 sequences:
    shards of 2 and 1) or by KV head."""
    import numpy as np
    w, n = _job()
    units = [(b, h) for b in range(w.B) for h in range(w.Hkv)]
    ref = _oracle_outputs(w, n, units, [b * w.Hkv + h for b, h in units])[:, :, n - 1]     # [B*Hkv, G, d]
    ref = ref.reshape(w.B, w.H, w.d)
    for mode, offsets in (("sequence", [0, 2 * w.Hkv]), ("head", [0, 2])):
        res = _run_sharded(mode)
        for rank, offs, full in res:
            assert offs == offsets
            np.testing.assert_array_equal(full, ref, err_msg="%s sharding, as seen by rank %d" % (mode, rank))


def test_partition_shapes():
    sys.path.insert(0, ROOT)
    from paper_2402_06082_b200 import sharding
    sh = sharding.partition(8, 32, 8, 3, "sequence")
    assert [(s.b0, s.b1) for s in sh] == [(0, 3), (3, 6), (6, 8)] and all(s.Hkv_local == 8 for s in sh)
    assert [s.unit_offset for s in sh] == [0, 24, 48] and all(s.unit_stride == 8 for s in sh)
    sh = sharding.partition(1, 32, 8, 4, "auto")                 # one sequence: cut by KV head
    assert [(s.h0, s.h1) for s in sh] == [(0, 2), (2, 4), (4, 6), (6, 8)] and all(s.H_local == 8 for s in sh)
    assert sh[2].unit_id(0, 1) == 5 and sh[2].handle_kwargs() == dict(B=1, H=8, Hkv=2, unit_stride=8, unit_offset=4)
    sh = sharding.partition(2, 4, 4, 3, "sequence")              # more ranks than sequences: the last rank idles
    assert sh[2].empty and not sh[1].empty
    q = torch.arange(2 * 4 * 3).reshape(2, 4, 3)
    assert torch.equal(sh[1].q_rows(q), q[1:2])
    import pytest
    with pytest.raises(ValueError):
        sharding.partition(1, 6, 3, 2, "head")
