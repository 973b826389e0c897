"""More units than one wave of value-scan blocks: the value scan then cuts its work evenly over the grid, so a block
serves parts of several consecutive units and a unit's partials come from several blocks."""
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


@pytest.mark.parametrize("d,G,s,window,n0", [(64, 1, 48, 40, 200), (128, 2, 100, 16, 120), (128, 1, 33, 0, 90), (64, 1, 48, 64, 30)])
def test_evenly_cut_value_scan_matches_oracle(d, G, s, window, n0):
    from paper_2402_06082_b200.binding import SubGen
    w = synth.CFG3.scaled(B=40, H=16 * G, Hkv=16, d=d, n_prompt=n0, ncomp=12, s=s, window=window, m_max=64, t=4)
    nd = 5
    sample = [(0, 0), (0, 15), (17, 3), (39, 15), (25, 8)]
    K = torch.empty(w.B, w.Hkv, n0 + nd, d, dtype=torch.bfloat16, device="cuda")
    V = torch.empty_like(K)
    Q = torch.empty(w.B, w.H, n0 + nd, d, dtype=torch.bfloat16, device="cuda")
    for b in range(w.B):
        K[b], V[b], Q[b] = synth.sequence_stream(w, b, n0 + nd, "cuda")
    sg = SubGen(w.B, w.H, d, w.delta, w.t, s, window, w.philox_seed, Hkv=w.Hkv, dtype=torch.bfloat16, m_max=w.m_max, nq_max=2)
    sg.prefill(K[:, :, :n0].contiguous(), V[:, :, :n0].contiguous())
    orcs = {bh: hp.oracle_unit(w, *bh) for bh in sample}
    for (b, h), o in orcs.items():
        o.push_many(f32(K[b, h, :n0]), f32(V[b, h, :n0]))
    for i in range(n0, n0 + nd):
        out = f32(sg.step(Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous()))
        for (b, h), o in orcs.items():
            o.push(f32(K[b, h, i]), f32(V[b, h, i]))
            for g in range(G):
                err = hp.rel_err(out[b, h * G + g], o.query(f32(Q[b, h * G + g, i])))
                hp.assert_output(out[b, h * G + g], o.query(f32(Q[b, h * G + g, i])), torch.bfloat16, "step %d unit %s head %d: rel err %.3g" % (i, (b, h), g, err))
    # the read-only multi-query call takes the same path
    probes = Q[:, :, n0:n0 + 2].contiguous()
    got = f32(sg.query(probes))
    for (b, h), o in orcs.items():
        hp.assert_state_equal(sg.export_state(b, h), o, "unit %s" % ((b, h),))
        for g in range(G):
            for j in range(2):
                hp.assert_output(got[b, h * G + g, j], o.query(f32(probes[b, h * G + g, j])), torch.bfloat16)
    assert sg.status() == 0
