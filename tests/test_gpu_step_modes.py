"""The two ways a bf16 handle can run a stream step (one fused kernel, or insertion + cluster scan + value scan)
against the CPU oracle and against each other.

Both must leave the same integer state, bit for bit, and give outputs within the bf16 tolerance of the oracle
(main loop of Algorithm 1 with the window of Section 3.2). The fused kernel scans the state as it was before the
step's insertion and corrects for the insertion afterwards, so the cases below aim at that correction: a token that
joins a singleton cluster, one that opens a cluster, value slots replaced during the scan, windows of 0 and 1 row,
a window that is not yet full, grouped queries, many blocks per unit and a single one.
"""
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))

import numpy as np
import pytest
import torch

import helpers as hp
from helpers import f32
from paper_2402_06082_b200 import synth

pytestmark = pytest.mark.gpu

MODES = ["fused", "split"]


def _sg(w, **kw):
    from paper_2402_06082_b200.binding import SubGen
    args = dict(Hkv=w.Hkv, dtype=w.torch_dtype, m_max=w.m_max)
    args.update(kw)
    return SubGen(w.B, w.H, w.d, w.delta, w.t, w.s, w.window, w.philox_seed, **args)


def _stream(w, n_prefill, n_steps, mode, **kw):
    """Prefill, then n_steps stream steps with every output checked per coordinate; final state bit for bit."""
    n = n_prefill + n_steps
    K, V, Q = synth.batch_stream(w, n, "cuda")
    sg = _sg(w, step_mode=mode, **kw)
    assert sg.step_kernels == (1 if mode == "fused" else 3)
    units = [(b, h) for b in range(w.B) for h in range(w.Hkv)]
    orcs = {bh: hp.oracle_unit(w, *bh) for bh in units}
    Kn, Vn, Qn = f32(K), f32(V), f32(Q)
    if n_prefill:
        sg.prefill(K[:, :, :n_prefill].contiguous(), V[:, :, :n_prefill].contiguous())
        for (b, h), o in orcs.items():
            o.push_many(Kn[b, h, :n_prefill], Vn[b, h, :n_prefill])
    outs = [f32(sg.step(Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous())) for i in range(n_prefill, n)]
    G = w.H // w.Hkv
    opened = joined_singleton = replaced = 0
    for j, i in enumerate(range(n_prefill, n)):
        for (b, h), o in orcs.items():
            m0, cnt0, mt0 = o.m, o.counts.copy(), o.m_tok.copy()
            o.push(Kn[b, h, i], Vn[b, h, i])
            if o.inserted:
                e = o.inserted - 1
                c = int(o.assign[e])
                opened += int(o.m > m0)
                joined_singleton += int(o.m == m0 and c < len(cnt0) and cnt0[c] == 1)
                replaced += int(np.sum(o.m_tok != mt0))
            for g in range(G):
                hp.assert_output(outs[j][b, h * G + g], o.query(Qn[b, h * G + g, i]), w.torch_dtype,
                                 "%s step %d unit %s head %d" % (mode, i, (b, h), g))
    for (b, h), o in orcs.items():
        st = sg.export_state(b, h)
        hp.assert_state_equal(st, o, "%s after steps unit %s" % (mode, (b, h)))
        hp.assert_rows_match_tokens(sg, b, h, st, K[b, h], V[b, h])
    assert sg.status() == 0
    return dict(opened=opened, joined_singleton=joined_singleton, replaced=replaced), sg


@pytest.mark.parametrize("mode", MODES)
def test_outliers_gqa(mode):
    """Outliers open clusters and leave singletons that later members join; G = 4 heads share a unit."""
    w = synth.CFG3.scaled(B=2, H=8, Hkv=2, n_prompt=700, ncomp=24, s=256, window=32, m_max=512)
    ev, _ = _stream(w, 700, 80, mode)
    assert ev["opened"] > 0 and ev["replaced"] > 0


@pytest.mark.parametrize("mode", MODES)
def test_from_empty_through_window_fill(mode):
    """A stream from nothing: steps before the window is full, the first insertion (M takes the token in every
    slot), then ordinary steps; a small s / n ratio makes value slots change in most steps."""
    w = synth.CFG2.scaled(B=1, H=2, Hkv=2, ncomp=6, s=48, t=4, window=9, m_max=128)
    ev, _ = _stream(w, 0, 120, mode)
    assert ev["replaced"] > 48 and ev["joined_singleton"] > 0


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("window", [0, 1])
def test_tiny_windows(mode, window):
    w = synth.CFG2.scaled(B=1, H=4, Hkv=2, ncomp=5, s=40, t=3, window=window, m_max=128, outlier_frac=0.1)
    _stream(w, 50, 70, mode)
    _stream(w, 0, 5, mode)


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("splits", [1, 2, 7, 23])
def test_block_splits(mode, splits):
    """One block per unit (no arrival ticket), a few, and more blocks than the unit has work items."""
    w = synth.CFG3.scaled(B=1, H=2, Hkv=2, n_prompt=400, ncomp=12, s=96, window=24, m_max=256)
    _stream(w, 400, 30, mode, splits=splits)


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("d,G,t", [(64, 1, 5), (64, 8, 8), (128, 2, 16), (128, 8, 33)])
def test_geometries(mode, d, G, t):
    """Both head dimensions, group sizes up to 8, t beyond 16 (no slot merging) and beyond 32 (two coin words)."""
    w = synth.CFG2.scaled(B=1, H=2 * G, Hkv=2, d=d, n_prompt=300, ncomp=8, s=64, t=t, window=16, m_max=128)
    _stream(w, 300, 40, mode)


def test_modes_agree_and_many_units_fused():
    """More units than the automatic choice would fuse (one block per unit, several waves): fused and split handles
    fed the same stream end in the same state and give the same outputs up to rounding."""
    w = synth.CFG3.scaled(B=5, H=32, Hkv=32, n_prompt=300, ncomp=8, s=64, window=16, m_max=128)
    n0, nd = 300, 12
    K, V, Q = synth.batch_stream(w, n0 + nd, "cuda")
    a, b = _sg(w, step_mode="fused"), _sg(w, step_mode="split")
    for sg in (a, b):
        sg.prefill(K[:, :, :n0].contiguous(), V[:, :, :n0].contiguous())
    for i in range(n0, n0 + nd):
        q, k, v = Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous()
        oa, ob = f32(a.step(q, k, v)), f32(b.step(q, k, v))
        for bb in range(w.B):
            for h in range(w.H):
                hp.assert_output(oa[bb, h], ob[bb, h], w.torch_dtype, "step %d seq %d head %d" % (i, bb, h))
    for bb in range(w.B):
        for h in range(0, w.Hkv, 5):
            sa, sb = a.export_state(bb, h), b.export_state(bb, h)
            for key in ("n", "m", "mu", "last_cluster", "last_opened"):
                assert sa[key] == sb[key], key
            for key in ("counts", "centre_tok", "slot_tok", "m_tok", "m_w"):
                np.testing.assert_array_equal(sa[key], sb[key], err_msg=key)
    o = hp.oracle_unit(w, 4, 31)
    Kn, Vn = f32(K[4, 31]), f32(V[4, 31])
    o.push_many(Kn, Vn)
    hp.assert_state_equal(a.export_state(4, 31), o, "fused, last unit")
    assert a.status() == 0 and b.status() == 0


def test_fused_capacity_overflow_sets_status():
    """A key that needs a cluster when none is free: status bit, NaN outputs, no fault (fused path)."""
    w = synth.CFG1.scaled(dtype="bf16", d=64, delta=0.0, window=2, s=16, m_max=8)
    K, V, Q = synth.batch_stream(w, 40, "cuda")
    sg = _sg(w, step_mode="fused")
    out = None
    for i in range(40):
        out = sg.step(Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous())
    assert sg.status() & 1
    assert torch.isnan(out.float()).all()


@pytest.mark.parametrize("mode", ["sequence", "head"])
def test_sharded_handles_reproduce_the_whole_job(mode):
    """A job cut in two shards (by sequence: 2 + 1 sequences; by KV head: 2 + 2 heads), each shard on a handle of its
    own with the whole job's unit numbering: every shard ends in exactly the state the unsharded handle has for those
    units (same Philox draws), and the outputs put back in place agree with the unsharded outputs up to rounding."""
    from paper_2402_06082_b200 import sharding
    from paper_2402_06082_b200.binding import SubGen
    w = synth.CFG3.scaled(B=3, H=8, Hkv=4, n_prompt=500, ncomp=12, s=64, window=16, m_max=256)
    n0, nd = w.n_prompt, 10
    K, V, Q = synth.batch_stream(w, n0 + nd, "cuda")
    whole = _sg(w)
    whole.prefill(K[:, :, :n0].contiguous(), V[:, :, :n0].contiguous())
    shards = sharding.partition(w.B, w.H, w.Hkv, 2, mode)
    handles = []
    for sh in shards:
        kw = sh.handle_kwargs()
        sg = SubGen(kw.pop("B"), kw.pop("H"), w.d, w.delta, w.t, w.s, w.window, w.philox_seed, dtype=w.torch_dtype,
                    m_max=w.m_max, **kw)
        sg.prefill(sh.kv_rows(K[:, :, :n0]), sh.kv_rows(V[:, :, :n0]))
        handles.append(sg)
    for i in range(n0, n0 + nd):
        q, k, v = Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous()
        ref = f32(whole.step(q, k, v))
        full = torch.zeros(w.B, w.H, w.d, dtype=w.torch_dtype, device="cuda")
        for sh, sg in zip(shards, handles):
            sharding.scatter_outputs(full, sh, sg.step(sh.q_rows(q), sh.kv_rows(k), sh.kv_rows(v)))
        got = f32(full)
        for b in range(w.B):
            for h in range(w.H):
                hp.assert_output(got[b, h], ref[b, h], w.torch_dtype, "step %d seq %d head %d" % (i, b, h))
    for sh, sg in zip(shards, handles):
        for lb in range(sh.B_local):
            for lh in range(sh.Hkv_local):
                a, c = sg.export_state(lb, lh), whole.export_state(sh.b0 + lb, sh.h0 + lh)
                for key in ("n", "m", "mu", "last_cluster", "last_opened", "last_d2"):
                    assert a[key] == c[key], key
                for key in ("counts", "centre_tok", "slot_tok", "m_tok", "m_w"):
                    np.testing.assert_array_equal(a[key], c[key], err_msg=key)
    o = hp.oracle_unit(w, 2, 3)
    o.push_many(f32(K[2, 3]), f32(V[2, 3]))
    last = handles[1]
    hp.assert_state_equal(last.export_state(last.B - 1, last.Hkv - 1), o, "last unit of the job, on its shard")


def test_ragged_prompts_many_units():
    """Prompts of very different lengths on a handle with more units than SMs: the three-kernel step serves the units
    largest first (an order built after the prefill); every unit must still be served exactly once per step."""
    w = synth.CFG5.scaled(B=6, H=32, Hkv=32, ncomp=16, s=64, window=16, m_max=512)
    lens = [40, 700, 120, 350, 17, 500]
    n_dec = 6
    streams = [synth.sequence_stream(w, b, lens[b] + n_dec, "cuda") for b in range(w.B)]
    cu = np.concatenate([[0], np.cumsum(lens)])
    Kp = torch.cat([streams[b][0][:, :lens[b]] for b in range(w.B)], dim=1).contiguous()
    Vp = torch.cat([streams[b][1][:, :lens[b]] for b in range(w.B)], dim=1).contiguous()
    sg = _sg(w)
    assert sg.step_kernels == 3
    sg.prefill_varlen(Kp, Vp, cu)
    orcs = {}
    for b in range(w.B):
        for h in range(w.Hkv):
            o = hp.oracle_unit(w, b, h)
            o.push_many(f32(streams[b][0][h, :lens[b]]), f32(streams[b][1][h, :lens[b]]))
            orcs[(b, h)] = o
    ms = [o.m for o in orcs.values()]
    assert max(ms) > 2 * max(min(ms), 1)
    for i in range(n_dec):
        q = torch.stack([streams[b][2][:, lens[b] + i] for b in range(w.B)]).contiguous()
        k = torch.stack([streams[b][0][:, lens[b] + i] for b in range(w.B)]).contiguous()
        v = torch.stack([streams[b][1][:, lens[b] + i] for b in range(w.B)]).contiguous()
        if i % 2:                                         # host buffers: the next step applies a search made ahead
            hout = torch.empty(w.B, w.H, w.d, dtype=torch.bfloat16).pin_memory()
            sg.step_host(q.cpu().pin_memory(), k.cpu().pin_memory(), v.cpu().pin_memory(), hout)
            out = f32(hout)
        else:
            out = f32(sg.step(q, k, v))
        kn, vn, qn = f32(k), f32(v), f32(q)
        for (b, h), o in orcs.items():
            o.push(kn[b, h], vn[b, h])
            hp.assert_output(out[b, h], o.query(qn[b, h]), torch.bfloat16, "step %d unit %s" % (i, (b, h)))
    for (b, h), o in orcs.items():
        hp.assert_state_equal(sg.export_state(b, h), o, "ragged, ordered units %s" % ((b, h),))
    assert sg.status() == 0


@pytest.mark.parametrize("window", [1, 2, 64])
def test_long_split_stream_many_blocks_per_unit(window):
    """Three-kernel steps back to back with few units and 64 blocks per unit: every kernel of a step starts work before
    its dependency wait (the insertion searches under the previous value scan, the value scan runs beside the cluster
    scan), which rests on the order in which the kernels let each other be scheduled. 1200 steps with frequent
    openings must end in the oracle's state."""
    w = synth.CFG3.scaled(B=2, H=8, Hkv=4, n_prompt=64, ncomp=10, s=48, t=4, window=window, m_max=2048, outlier_frac=0.3)
    n0, nd = 64, 1200
    K, V, Q = synth.batch_stream(w, n0 + nd, "cuda")
    sg = _sg(w, step_mode="split", splits=64)
    sg.prefill(K[:, :, :n0].contiguous(), V[:, :, :n0].contiguous())
    last = None
    for i in range(n0, n0 + nd):
        last = sg.step(Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous())
    last = f32(last)
    Kn, Vn, Qn = f32(K), f32(V), f32(Q)
    G = w.H // w.Hkv
    for b in range(w.B):
        for h in range(w.Hkv):
            o = hp.oracle_unit(w, b, h)
            o.push_many(Kn[b, h], Vn[b, h])
            hp.assert_state_equal(sg.export_state(b, h), o, "window %d, unit %s" % (window, (b, h)))
            for g in range(G):
                hp.assert_output(last[b, h * G + g], o.query(Qn[b, h * G + g, n0 + nd - 1]), w.torch_dtype, "last step")
    assert sg.status() == 0


@pytest.mark.parametrize("window", [2, 3, 64])
def test_long_fused_stream_with_frequent_openings(window):
    """The one-kernel step works on the leaving token before it waits for the previous step (windows of two rows or
    more), from a cluster count that is two steps old, and looks at the cluster the previous step may have opened
    afterwards. A long back-to-back stream in which many steps open a cluster (so that the nearest representative is
    often the one opened by the step before) must end in the oracle's state; every 50th step's outputs are checked."""
    w = synth.CFG3.scaled(B=2, H=8, Hkv=4, n_prompt=64, ncomp=10, s=48, t=4, window=window, m_max=2048, outlier_frac=0.3)
    n0, nd = 64, 1500
    K, V, Q = synth.batch_stream(w, n0 + nd, "cuda")
    sg = _sg(w, step_mode="fused")
    sg.prefill(K[:, :, :n0].contiguous(), V[:, :, :n0].contiguous())
    outs = {}
    for i in range(n0, n0 + nd):
        o = sg.step(Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous())
        if i % 50 == 0:
            outs[i] = f32(o)
    Kn, Vn, Qn = f32(K), f32(V), f32(Q)
    G = w.H // w.Hkv
    opened = 0
    for b in range(w.B):
        for h in range(w.Hkv):
            o = hp.oracle_unit(w, b, h)
            o.push_many(Kn[b, h, :n0], Vn[b, h, :n0])
            m0 = o.m
            for i in range(n0, n0 + nd):
                o.push(Kn[b, h, i], Vn[b, h, i])
                if i in outs:
                    for g in range(G):
                        hp.assert_output(outs[i][b, h * G + g], o.query(Qn[b, h * G + g, i]), w.torch_dtype,
                                         "step %d unit %s head %d" % (i, (b, h), g))
            opened += o.m - m0
            hp.assert_state_equal(sg.export_state(b, h), o, "window %d, unit %s" % (window, (b, h)))
    assert opened > 200
    assert sg.status() == 0


@pytest.mark.parametrize("window", [1, 2, 24])
def test_host_buffer_steps_search_ahead(window):
    """Host-buffer steps of a three-kernel handle leave the search for the next step's leaving token running behind
    them; the next step (host or device buffers) only applies it; a prefill in between throws it away. Mixed sequence
    of calls against the oracle: state bit for bit, every output within tolerance."""
    w = synth.CFG3.scaled(B=2, H=4, Hkv=2, n_prompt=200, ncomp=12, s=48, t=4, window=window, m_max=1024, outlier_frac=0.2)
    n0, n = 200, 200 + 90
    K, V, Q = synth.batch_stream(w, n, "cuda")
    Kn, Vn, Qn = f32(K), f32(V), f32(Q)
    units = [(b, h) for b in range(w.B) for h in range(w.Hkv)]
    orcs = {bh: hp.oracle_unit(w, *bh) for bh in units}
    G = w.H // w.Hkv
    sg = _sg(w, step_mode="split")
    sg.prefill(K[:, :, :n0].contiguous(), V[:, :, :n0].contiguous())
    for (b, h), o in orcs.items():
        o.push_many(Kn[b, h, :n0], Vn[b, h, :n0])
    pin = lambda x: x.contiguous().cpu().pin_memory()
    hout = torch.empty(w.B, w.H, w.d, dtype=w.torch_dtype).pin_memory()
    i = n0
    launches = []
    while i < n:
        phase = (i - n0) % 30
        if phase == 20:                                   # a prefill of 5 tokens between steps
            sg.prefill(K[:, :, i:i + 5].contiguous(), V[:, :, i:i + 5].contiguous())
            for (b, h), o in orcs.items():
                o.push_many(Kn[b, h, i:i + 5], Vn[b, h, i:i + 5])
            i += 5
            continue
        l0 = sg.launch_count
        if phase % 3 == 2:                                # device buffers
            out = f32(sg.step(Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous()))
        else:
            sg.step_host(pin(Q[:, :, i]), pin(K[:, :, i]), pin(V[:, :, i]), hout)
            out = f32(hout)
        launches.append(sg.launch_count - l0)
        for (b, h), o in orcs.items():
            o.push(Kn[b, h, i], Vn[b, h, i])
            for g in range(G):
                hp.assert_output(out[b, h * G + g], o.query(Qn[b, h * G + g, i]), w.torch_dtype,
                                 "step %d unit %s head %d" % (i, (b, h), g))
        i += 1
    for (b, h), o in orcs.items():
        st = sg.export_state(b, h)
        hp.assert_state_equal(st, o, "window %d unit %s" % (window, (b, h)))
        hp.assert_rows_match_tokens(sg, b, h, st, K[b, h], V[b, h])
    assert sg.status() == 0
    assert 4 in launches, "host-buffer steps launch the search for the next step behind their three kernels"
