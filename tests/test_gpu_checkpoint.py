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
