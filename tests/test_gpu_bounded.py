"""Parity of the bounded-m variant (cluster budget, threshold doubling, merging) with the CPU oracle."""
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))

import numpy as np
import pytest
import torch

import helpers as hp
from helpers import f32
from oracle import subgen_oracle as orc
from paper_2402_06082_b200 import synth

pytestmark = pytest.mark.gpu


def _sg(w, **kw):
    from paper_2402_06082_b200.binding import SubGen
    args = dict(Hkv=w.Hkv, dtype=w.torch_dtype, m_max=w.m_max, bounded=True)
    args.update(kw)
    return SubGen(w.B, w.H, w.d, w.delta, w.t, w.s, w.window, w.philox_seed, **args)


def _oracle(w, seq, h, bounded=True):
    return orc.OracleUnit(w.d, w.delta, w.t, w.s, w.window, seed=w.philox_seed, unit_id=seq * w.Hkv + h,
                          m_max=w.m_max, bounded=bounded)


def _same(sg, o, b, h, where):
    st = sg.export_state(b, h)
    hp.assert_state_equal(st, o, where)
    assert st["threshold2"] == o.thr2_fx and st["doublings"] == o.level, where
    return st


@pytest.mark.parametrize("dtype,d,G,m_max", [("bf16", 128, 2, 24), ("fp32", 64, 1, 17), ("bf16", 64, 4, 40), ("bf16", 128, 1, 1)])
def test_budgeted_stream_matches_oracle(dtype, d, G, m_max):
    w = synth.CFG3.scaled(B=2, H=2 * G, Hkv=2, d=d, dtype=dtype, n_prompt=500, ncomp=60, s=64, window=32,
                          m_max=m_max, delta=0.5)
    n0, n1, n2, n3 = 300, 25, 175, 40            # prefill, steps, prefill again, steps
    n = n0 + n1 + n2 + n3
    K, V, Q = synth.batch_stream(w, n, "cuda")
    Kn, Vn, Qn = f32(K), f32(V), f32(Q)
    units = [(b, h) for b in range(w.B) for h in range(w.Hkv)]
    orcs = {bh: _oracle(w, *bh) for bh in units}
    sg = _sg(w)

    def prefill(a, b_):
        sg.prefill(K[:, :, a:b_].contiguous(), V[:, :, a:b_].contiguous())
        for (b, h), o in orcs.items():
            o.push_many(Kn[b, h, a:b_], Vn[b, h, a:b_])
            _same(sg, o, b, h, "after prefill to %d, unit %s" % (b_, (b, h)))

    def steps(a, b_):
        for i in range(a, b_):
            out = f32(sg.step(Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous()))
            for (b, h), o in orcs.items():
                o.push(Kn[b, h, i], Vn[b, h, i])
                for g in range(G):
                    err = hp.rel_err(out[b, h * G + g], o.query(Qn[b, h * G + g, i]))
                    hp.assert_output(out[b, h * G + g], o.query(Qn[b, h * G + g, i]), w.torch_dtype, "step %d unit %s head %d: rel err %.3g" % (i, (b, h), g, err))
            if i % 8 == 0 or i == b_ - 1:
                for (b, h), o in orcs.items():
                    _same(sg, o, b, h, "after step %d, unit %s" % (i, (b, h)))

    prefill(0, n0)
    lv0 = [o.level for o in orcs.values()]
    steps(n0, n0 + n1)
    prefill(n0 + n1, n0 + n1 + n2)
    steps(n0 + n1 + n2, n)
    assert sg.status() == 0
    assert min(lv0) >= 1                                           # the budget was hit during the prompt already
    if dtype == "bf16":                                            # the slot aliases survived the merges and moves
        want = sum(len(set(r.tolist())) for o in orcs.values() for r in o.slot_tok[o.counts > 1])
        assert sg.cache_stats()["distinct_sample_rows"] == want
    for (b, h), o in orcs.items():
        assert o.m <= m_max
        st = _same(sg, o, b, h, "end, unit %s" % ((b, h),))
        hp.assert_rows_match_tokens(sg, b, h, st, K[b, h], V[b, h])


def test_doubling_inside_decode_steps():
    """The budget is first exhausted by a stream step (not by the prompt), several units at different tokens."""
    w = synth.CFG3.scaled(B=3, H=2, Hkv=2, n_prompt=0, ncomp=50, s=32, window=0, m_max=12, delta=0.5)
    n = 120
    K, V, Q = synth.batch_stream(w, n, "cuda")
    Kn, Vn, Qn = f32(K), f32(V), f32(Q)
    orcs = {(b, h): _oracle(w, b, h) for b in range(w.B) for h in range(w.Hkv)}
    sg = _sg(w)
    seen = set()
    for i in range(n):
        out = f32(sg.step(Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous()))
        for (b, h), o in orcs.items():
            lv = o.level
            o.push(Kn[b, h, i], Vn[b, h, i])
            if o.level > lv:
                seen.add(i)
                _same(sg, o, b, h, "right after a doubling at token %d, unit %s" % (i, (b, h)))
            hp.assert_output(out[b, h], o.query(Qn[b, h, i]), w.torch_dtype)
    assert len(seen) >= 3
    for (b, h), o in orcs.items():
        _same(sg, o, b, h, "end")


def test_unreached_budget_equals_plain_handle():
    w = synth.CFG2.scaled(B=1, H=2, Hkv=2, n_prompt=400, ncomp=10, s=32, window=16, m_max=128)
    K, V, Q = synth.batch_stream(w, 410, "cuda")
    a, b = _sg(w), _sg(w, bounded=False)
    for sg in (a, b):
        sg.prefill(K[:, :, :400].contiguous(), V[:, :, :400].contiguous())
        for i in range(400, 410):
            sg.step(Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous())
    for h in range(2):
        o = _oracle(w, 0, h, bounded=False)
        o.push_many(f32(K)[0, h], f32(V)[0, h])
        sa, sb = a.export_state(0, h), b.export_state(0, h)
        hp.assert_state_equal(sa, o, "bounded handle below its budget")
        hp.assert_state_equal(sb, o, "plain handle")
        assert sa["doublings"] == 0 and sa["threshold2"] == sb["threshold2"] == o.delta2_fx


def test_bounded_checkpoint_resume():
    w = synth.CFG3.scaled(B=1, H=2, Hkv=2, n_prompt=300, ncomp=40, s=32, window=8, m_max=10, delta=0.5)
    K, V, Q = synth.batch_stream(w, 400, "cuda")
    a = _sg(w)
    a.prefill(K[:, :, :300].contiguous(), V[:, :, :300].contiguous())
    blob = a.checkpoint_save()
    b = _sg(w, m_max=10)
    b.checkpoint_load(blob)
    from paper_2402_06082_b200.binding import SubgenError
    with pytest.raises(SubgenError, match="configuration"):
        _sg(w, bounded=False).checkpoint_load(blob)
    for i in range(300, 400):
        b.step(Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous())
    for h in range(2):
        o = _oracle(w, 0, h)
        o.push_many(f32(K)[0, h], f32(V)[0, h])
        _same(b, o, 0, h, "resumed bounded handle")
        assert o.level >= 2


def test_chunked_prefill_of_a_bounded_handle(monkeypatch):
    """bf16 handles with d = 128 prefill chunk by chunk also when they are bounded: a chunk ends at the key that finds
    the budget used up, that key is inserted on its own (doubling, merge sweep) and the walk resumes behind it. A long
    prompt with several doublings, cut at awkward places, against the oracle and against the token-by-token kernel."""
    w = synth.CFG3.scaled(B=2, H=4, Hkv=2, n_prompt=2600, ncomp=300, s=64, window=24, m_max=48, delta=0.5)
    K, V, Q = synth.batch_stream(w, w.n_prompt + 6, "cuda")
    Kn, Vn, Qn = f32(K), f32(V), f32(Q)
    a = _sg(w)
    cuts = [0, 1, 129, 130, 1000, 2600]
    orcs = {(b, h): _oracle(w, b, h) for b in range(w.B) for h in range(w.Hkv)}
    launches = a.launch_count
    for lo, hi in zip(cuts[:-1], cuts[1:]):
        a.prefill(K[:, :, lo:hi].contiguous(), V[:, :, lo:hi].contiguous())
        for (b, h), o in orcs.items():
            o.push_many(Kn[b, h, lo:hi], Vn[b, h, lo:hi])
            _same(a, o, b, h, "chunked, after prefill to %d, unit %s" % (hi, (b, h)))
    assert a.launch_count - launches < 80                 # a handful of kernels per call, not one pass per token
    assert min(o.level for o in orcs.values()) >= 2        # the budget was exhausted more than once
    monkeypatch.setenv("SUBGEN_PREFILL", "seq")
    s = _sg(w)
    s.prefill(K[:, :, :w.n_prompt].contiguous(), V[:, :, :w.n_prompt].contiguous())
    for (b, h), o in orcs.items():
        _same(s, o, b, h, "token by token, unit %s" % ((b, h),))
    G = w.H // w.Hkv
    for i in range(w.n_prompt, w.n_prompt + 6):
        out = f32(a.step(Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous()))
        for (b, h), o in orcs.items():
            o.push(Kn[b, h, i], Vn[b, h, i])
            for g in range(G):
                hp.assert_output(out[b, h * G + g], o.query(Qn[b, h * G + g, i]), w.torch_dtype, "step %d" % i)
    for (b, h), o in orcs.items():
        st = _same(a, o, b, h, "end, unit %s" % ((b, h),))
        hp.assert_rows_match_tokens(a, b, h, st, K[b, h], V[b, h])
    assert a.status() == 0
