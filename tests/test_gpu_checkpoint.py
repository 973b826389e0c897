"""Checkpoint and resume: a loaded handle continues the stream exactly as the saved one (and the oracle) would."""
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


def _sg(w, **kw):
    from paper_2402_06082_b200.binding import SubGen
    args = dict(Hkv=w.Hkv, dtype=w.torch_dtype, m_max=w.m_max)
    args.update(kw)
    return SubGen(w.B, w.H, w.d, w.delta, w.t, w.s, w.window, w.philox_seed, **args)


@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("fp32", 64)])
def test_resume_continues_the_stream(dtype, d):
    w = synth.CFG3.scaled(B=2, H=4, Hkv=2, d=d, dtype=dtype, n_prompt=700, ncomp=24, s=64, window=48, m_max=256)
    n0, n1, n2, n3 = 700, 6, 150, 8          # prefill, steps, [checkpoint], prefill again, steps
    n = n0 + n1 + n2 + n3
    K, V, Q = synth.batch_stream(w, n, "cuda")
    Kn, Vn, Qn = f32(K), f32(V), f32(Q)
    units = [(b, h) for b in range(w.B) for h in range(w.Hkv)]
    orcs = {bh: hp.oracle_unit(w, *bh) for bh in units}
    G = w.H // w.Hkv

    def step(sg, i):
        return f32(sg.step(Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous()))

    a = _sg(w)
    a.prefill(K[:, :, :n0].contiguous(), V[:, :, :n0].contiguous())
    for i in range(n0, n0 + n1):
        step(a, i)
    blob = a.checkpoint_save()
    # the second handle has a larger capacity and another split of the units over thread blocks
    b = _sg(w, m_max=2 * w.m_max, splits=3)
    b.prefill(K[:, :, :5].contiguous(), V[:, :, :5].contiguous())       # whatever it held is discarded
    b.checkpoint_load(blob.clone())
    for (bb, h), o in orcs.items():
        o.push_many(Kn[bb, h, : n0 + n1], Vn[bb, h, : n0 + n1])
        hp.assert_state_equal(b.export_state(bb, h), o, "after load, unit %s" % ((bb, h),))
    for sg in (a, b):
        sg.prefill(K[:, :, n0 + n1:n0 + n1 + n2].contiguous(), V[:, :, n0 + n1:n0 + n1 + n2].contiguous())
    for o_key, o in orcs.items():
        o.push_many(Kn[o_key[0], o_key[1], n0 + n1:n0 + n1 + n2], Vn[o_key[0], o_key[1], n0 + n1:n0 + n1 + n2])
    for i in range(n0 + n1 + n2, n):
        oa, ob = step(a, i), step(b, i)
        for (bb, h), o in orcs.items():
            o.push(Kn[bb, h, i], Vn[bb, h, i])
            for g in range(G):
                want = o.query(Qn[bb, h * G + g, i])
                hp.assert_output(ob[bb, h * G + g], want, w.torch_dtype)
                hp.assert_output(oa[bb, h * G + g], want, w.torch_dtype)
    want = sum(len(set(r.tolist())) for o in orcs.values() for r in o.slot_tok[o.counts > 1])
    assert a.cache_stats()["distinct_sample_rows"] == b.cache_stats()["distinct_sample_rows"] == want
    for (bb, h), o in orcs.items():
        sa, sb = a.export_state(bb, h), b.export_state(bb, h)
        hp.assert_state_equal(sb, o, "resumed handle, unit %s" % ((bb, h),))
        for key in ("n", "m", "mu", "last_cluster", "last_opened"):
            assert sa[key] == sb[key]
        for key in ("counts", "centre_tok", "slot_tok", "m_tok", "m_w"):
            np.testing.assert_array_equal(sa[key], sb[key])
        hp.assert_rows_match_tokens(b, bb, h, sb, K[bb, h], V[bb, h])


def test_checkpoint_of_an_empty_handle_and_rejections():
    w = synth.CFG2.scaled(B=1, H=2, Hkv=2, n_prompt=60, ncomp=4, s=16, window=8, m_max=32)
    K, V, Q = synth.batch_stream(w, 61, "cuda")
    a = _sg(w)
    empty = a.checkpoint_save()
    a.prefill(K[:, :, :60].contiguous(), V[:, :, :60].contiguous())
    full = a.checkpoint_save()
    assert full.numel() > empty.numel()
    a.checkpoint_load(empty)                                      # back to a fresh stream
    assert a.export_state(0, 0)["n"] == 0 and a.export_state(0, 1)["m"] == 0
    a.checkpoint_load(full)
    assert a.export_state(0, 0)["n"] == 60
    m_now = max(a.export_state(0, h)["m"] for h in range(2))
    with pytest.raises(RuntimeError, match="configuration"):
        _sg(w.scaled(t=w.t + 1)).checkpoint_load(full)
    with pytest.raises(RuntimeError, match="configuration"):
        _sg(w.scaled(philox_seed=5)).checkpoint_load(full)
    with pytest.raises(RuntimeError, match="truncated"):
        _sg(w).checkpoint_load(full[:-8].clone())
    with pytest.raises(RuntimeError, match="not a checkpoint"):
        _sg(w).checkpoint_load(torch.zeros(4096, dtype=torch.uint8))
    if m_now > 1:
        with pytest.raises(RuntimeError, match="m_max"):
            _sg(w, m_max=m_now - 1).checkpoint_load(full)
    # the handle is still usable after a rejected load
    out = a.step(Q[:, :, 60].contiguous(), K[:, :, 60].contiguous(), V[:, :, 60].contiguous())
    assert torch.isfinite(out.float()).all()


@pytest.mark.parametrize("dtype,d,mode", [("bf16", 128, "fused"), ("bf16", 128, "split"), ("bf16", 64, "auto"), ("fp32", 64, "auto")])
def test_grow_keeps_the_stream(dtype, d, mode):
    """A handle created with room for few clusters is grown twice while outliers keep opening clusters (delta small
    enough that the first capacity would overflow): prefill, steps, grow, prefill again, steps, grow, steps. State and
    outputs must be those of the oracle, which never had a bound; the rows stored before a growth must still be the
    tokens' rows after it."""
    big = 1024
    w = synth.CFG3.scaled(B=2, H=4, Hkv=2, d=d, dtype=dtype, n_prompt=300, ncomp=24, s=64, window=16, m_max=big,
                          outlier_frac=0.15)
    n0, n1, n2, n3, n4 = 300, 20, 200, 20, 30
    n = n0 + n1 + n2 + n3 + n4
    K, V, Q = synth.batch_stream(w, n, "cuda")
    Kn, Vn, Qn = f32(K), f32(V), f32(Q)
    units = [(b, h) for b in range(w.B) for h in range(w.Hkv)]
    orcs = {bh: hp.oracle_unit(w, *bh) for bh in units}
    G = w.H // w.Hkv
    for (b, h), o in orcs.items():
        o.push_many(Kn[b, h, :n0 + n1], Vn[b, h, :n0 + n1])
    m1 = max(o.m for o in orcs.values())
    for (b, h), o in orcs.items():
        o.push_many(Kn[b, h, n0 + n1:n0 + n1 + n2 + n3], Vn[b, h, n0 + n1:n0 + n1 + n2 + n3])
    m2 = max(o.m for o in orcs.values())
    cap0, cap1 = m1 + 2, m2 + 2
    assert m1 < m2 and cap0 < m2, "the first capacity must be too small for the second phase"
    orcs = {bh: hp.oracle_unit(w, *bh) for bh in units}

    def steps(sg, lo, hi):
        for i in range(lo, hi):
            out = f32(sg.step(Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous()))
            for (b, h), o in orcs.items():
                o.push(Kn[b, h, i], Vn[b, h, i])
                for g in range(G):
                    hp.assert_output(out[b, h * G + g], o.query(Qn[b, h * G + g, i]), w.torch_dtype,
                                     "step %d unit %s head %d" % (i, (b, h), g))

    kw = dict(step_mode=mode) if mode != "auto" else {}
    sg = _sg(w, m_max=cap0, **kw)
    sg.prefill(K[:, :, :n0].contiguous(), V[:, :, :n0].contiguous())
    for (b, h), o in orcs.items():
        o.push_many(Kn[b, h, :n0], Vn[b, h, :n0])
    steps(sg, n0, n0 + n1)
    with pytest.raises(Exception):
        sg.grow(cap0)                                   # not larger
    sg.grow(cap1)
    assert sg.m_max == cap1
    for (b, h), o in orcs.items():
        st = sg.export_state(b, h)
        hp.assert_state_equal(st, o, "right after the first growth, unit %s" % ((b, h),))
        hp.assert_rows_match_tokens(sg, b, h, st, K[b, h], V[b, h])
    lo = n0 + n1
    sg.prefill(K[:, :, lo:lo + n2].contiguous(), V[:, :, lo:lo + n2].contiguous())
    for (b, h), o in orcs.items():
        o.push_many(Kn[b, h, lo:lo + n2], Vn[b, h, lo:lo + n2])
    steps(sg, lo + n2, lo + n2 + n3)
    sg.grow(big)
    steps(sg, lo + n2 + n3, n)
    for (b, h), o in orcs.items():
        st = sg.export_state(b, h)
        hp.assert_state_equal(st, o, "end, unit %s" % ((b, h),))
        hp.assert_rows_match_tokens(sg, b, h, st, K[b, h], V[b, h])
    assert sg.status() == 0


def test_grow_is_refused_where_it_does_not_apply():
    from paper_2402_06082_b200.binding import SubGen
    w = synth.CFG2.scaled(B=1, H=2, Hkv=2, s=32, window=8, m_max=64)
    bounded = SubGen(w.B, w.H, w.d, w.delta, w.t, w.s, w.window, w.philox_seed, Hkv=w.Hkv, dtype=w.torch_dtype,
                     m_max=64, bounded=True)
    with pytest.raises(Exception):
        bounded.grow(128)


def test_grow_with_a_library_owned_workspace():
    """The C call with workspace = NULL (the library allocates and frees) on a handle created without a workspace."""
    import ctypes as C
    from paper_2402_06082_b200 import binding
    L = binding.load()
    w = synth.CFG3.scaled(B=1, H=2, Hkv=2, n_prompt=200, ncomp=12, s=32, window=8, m_max=512, outlier_frac=0.15)
    K, V, Q = synth.batch_stream(w, 260, "cuda")
    m_prompt = 0
    for hh in range(w.Hkv):
        o = hp.oracle_unit(w, 0, hh)
        o.push_many(f32(K)[0, hh, :200], f32(V)[0, hh, :200])
        m_prompt = max(m_prompt, o.m)
    cap0 = m_prompt + 1
    cfg = binding.SubgenConfig(w.B, w.H, w.Hkv, w.d, float(w.delta), w.t, w.s, w.window, int(w.philox_seed), 1, cap0, 0, None, 0,
                               torch.cuda.current_stream().cuda_stream, 1, 0, 0, 0, 0)
    h = L.subgen_create_ex(C.byref(cfg))
    assert h
    try:
        k0, v0 = K[:, :, :200].contiguous(), V[:, :, :200].contiguous()
        assert L.subgen_prefill(h, k0.data_ptr(), v0.data_ptr(), 200) == 0
        assert L.subgen_grow(h, 512, None, 0) == 0
        out = torch.empty(w.B, w.H, w.d, dtype=torch.bfloat16, device="cuda")
        for i in range(200, 260):
            q, k, v = Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous()
            assert L.subgen_step(h, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr()) == 0
        assert L.subgen_status(h) == 0
        ref = _sg(w)
        ref.prefill(k0, v0)
        for i in range(200, 260):
            o2 = ref.step(Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous())
        torch.cuda.synchronize()
        assert hp.rel_err(f32(out).reshape(-1, w.d), f32(o2).reshape(-1, w.d)) <= 1e-2
        o = hp.oracle_unit(w, 0, 1)
        o.push_many(f32(K)[0, 1], f32(V)[0, 1])
        assert o.m > cap0, "the first capacity must have been too small"
        assert ref.export_state(0, 1)["m"] == o.m
    finally:
        L.subgen_destroy(h)
