"""Read-only multi-query calls (procedure QueryStreamAttn for several queries per head) against the CPU oracle."""
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


@pytest.mark.parametrize("dtype,d,G,nq,window,n0", [("bf16", 128, 1, 4, 48, 700), ("bf16", 128, 2, 4, 48, 700), ("bf16", 64, 1, 8, 0, 300),
                                                    ("fp32", 64, 1, 2, 16, 300), ("fp32", 128, 4, 2, 16, 200), ("bf16", 128, 1, 2, 64, 20)])
def test_multi_query_matches_oracle_and_changes_nothing(dtype, d, G, nq, window, n0):
    w = synth.CFG3.scaled(B=2, H=2 * G, Hkv=2, d=d, dtype=dtype, n_prompt=n0, ncomp=20, s=64, window=window, m_max=256)
    nd = 6
    K, V, Q = synth.batch_stream(w, n0 + nd, "cuda")
    Kn, Vn, Qn = f32(K), f32(V), f32(Q)
    units = [(b, h) for b in range(w.B) for h in range(w.Hkv)]
    orcs = {bh: hp.oracle_unit(w, *bh) for bh in units}
    sg = _sg(w, nq_max=nq)
    sg.prefill(K[:, :, :n0].contiguous(), V[:, :, :n0].contiguous())
    for (b, h), o in orcs.items():
        o.push_many(Kn[b, h, :n0], Vn[b, h, :n0])
    gen = torch.Generator(device="cuda").manual_seed(5)
    for i in range(n0, n0 + nd):
        # nq probes per head against the state before this step's token
        probes = torch.randn(w.B, w.H, nq, d, device="cuda", generator=gen).to(w.torch_dtype)
        before = {bh: sg.export_state(*bh) for bh in units}
        got = f32(sg.query(probes))
        pn = f32(probes)
        for (b, h), o in orcs.items():
            for g in range(G):
                for j in range(nq):
                    err = hp.rel_err(got[b, h * G + g, j], o.query(pn[b, h * G + g, j]))
                    hp.assert_output(got[b, h * G + g, j], o.query(pn[b, h * G + g, j]), w.torch_dtype, "probe %d of head %d, unit %s, n=%d: rel err %.3g" % (j, g, (b, h), i, err))
            after = sg.export_state(b, h)
            for key in ("n", "m", "mu", "status"):
                assert after[key] == before[(b, h)][key]
            np.testing.assert_array_equal(after["slot_tok"], before[(b, h)]["slot_tok"])
        # the stream goes on as if the probes had never been asked
        out = f32(sg.step(Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous()))
        for (b, h), o in orcs.items():
            o.push(Kn[b, h, i], Vn[b, h, i])
            for g in range(G):
                hp.assert_output(out[b, h * G + g], o.query(Qn[b, h * G + g, i]), w.torch_dtype)
    for (b, h), o in orcs.items():
        hp.assert_state_equal(sg.export_state(b, h), o, "end, unit %s" % ((b, h),))


def test_multi_query_rejections():
    from paper_2402_06082_b200.binding import SubgenError
    w = synth.CFG2.scaled(B=1, H=4, Hkv=2, n_prompt=10, ncomp=4, s=16, window=4, m_max=32)
    K, V, _ = synth.batch_stream(w, 10, "cuda")
    with pytest.raises(SubgenError, match="nq_max"):
        _sg(w, nq_max=8)                                   # 2 heads per KV head * 8 > 8 columns
    sg = _sg(w, nq_max=2)
    q = torch.zeros(1, 4, 2, w.d, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(SubgenError, match="no tokens"):
        sg.query(q)
    sg.prefill(K, V)
    sg.query(q)
    with pytest.raises(SubgenError, match="nq"):
        sg.query(torch.zeros(1, 4, 4, w.d, dtype=torch.bfloat16, device="cuda"))
