"""Parity of the offline greedy k-center compression (Section 3.2 variant) with the CPU oracle."""
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


def _exact(w, n_max):
    from paper_2402_06082_b200.binding import ExactAttention
    return ExactAttention(w.B, w.H, w.d, n_max, Hkv=w.Hkv, dtype=w.torch_dtype)


@pytest.mark.parametrize("dtype,d,G", [("bf16", 128, 1), ("fp32", 64, 2), ("bf16", 64, 4)])
def test_kcenter_selection_and_attention_match_oracle(dtype, d, G):
    w = synth.CFG3.scaled(B=2, H=2 * G, Hkv=2, d=d, dtype=dtype, n_prompt=1500, ncomp=40)
    n0, nd, k, r = 1500, 5, 96, 64
    K, V, Q = synth.batch_stream(w, n0 + nd, "cuda")
    ex = _exact(w, n0 + nd)
    ex.append(K[:, :, :n0].contiguous(), V[:, :, :n0].contiguous())
    ex.kcenter_compress(k, r)
    Kn, Vn, Qn = f32(K), f32(V), f32(Q)
    keeps = {}
    for b in range(w.B):
        for h in range(w.Hkv):
            cent, _ = orc.kcenter(Kn[b, h, : n0 - r], k)
            keep = np.concatenate([cent.astype(np.int64), np.arange(n0 - r, n0)])
            np.testing.assert_array_equal(ex.export_tokens(b, h), keep)          # bit-exact selection, same order
            keeps[(b, h)] = keep
    assert ex.bytes_per_step() == 2 * w.B * w.Hkv * (k + r) * d * (4 if dtype == "fp32" else 2)
    for i in range(n0, n0 + nd):                                                  # later tokens are appended and attended exactly
        out = f32(ex.step(Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous()))
        for (b, h), keep in keeps.items():
            rows = np.concatenate([keep, np.arange(n0, i + 1)])
            for g in range(G):
                want = orc.exact_attention(Kn[b, h, rows], Vn[b, h, rows], Qn[b, h * G + g, i])
                assert hp.rel_err(out[b, h * G + g], want) <= hp.TOL[w.torch_dtype]
    assert len(ex.export_tokens(0, 0)) == k + r + nd


def test_kcenter_edge_cases():
    w = synth.CFG2.scaled(B=1, H=2, Hkv=2, n_prompt=50, ncomp=4)
    K, V, Q = synth.batch_stream(w, 51, "cuda")
    # fewer old tokens than k: everything is kept, in order
    ex = _exact(w, 64)
    ex.append(K[:, :, :50].contiguous(), V[:, :, :50].contiguous())
    ex.kcenter_compress(100, 10)
    np.testing.assert_array_equal(np.sort(ex.export_tokens(0, 0)), np.arange(50))
    # window longer than the stream: nothing changes
    ex.kcenter_compress(3, 500)
    assert len(ex.export_tokens(0, 1)) == 50
    # r = 0 and k = 1: only the first token survives
    ex.kcenter_compress(1, 0)
    assert ex.export_tokens(0, 0).tolist() == [0]
    out = f32(ex.step(Q[:, :, 50].contiguous(), K[:, :, 50].contiguous(), V[:, :, 50].contiguous()))
    want = orc.exact_attention(f32(K)[0, 0, [0, 50]], f32(V)[0, 0, [0, 50]], f32(Q)[0, 0, 50])
    assert hp.rel_err(out[0, 0], want) <= hp.TOL[torch.bfloat16]
    # empty cache
    ex2 = _exact(w, 8)
    ex2.kcenter_compress(4, 2)
    assert len(ex2.export_tokens(0, 0)) == 0


def test_kcenter_varlen():
    w = synth.CFG5.scaled(B=3, H=2, Hkv=2, ncomp=16)
    lens = [30, 700, 333]
    streams = [synth.sequence_stream(w, b, lens[b], "cuda") for b in range(w.B)]
    cu = np.concatenate([[0], np.cumsum(lens)])
    Kp = torch.cat([s[0] for s in streams], dim=1).contiguous()
    Vp = torch.cat([s[1] for s in streams], dim=1).contiguous()
    ex = _exact(w, 800)
    ex.append_varlen(Kp, Vp, cu)
    ex.kcenter_compress(40, 25)
    for b in range(w.B):
        for h in range(w.Hkv):
            n = lens[b]
            cent, _ = orc.kcenter(f32(streams[b][0])[h, : n - 25], 40)
            keep = np.concatenate([cent.astype(np.int64), np.arange(n - 25, n)])
            np.testing.assert_array_equal(ex.export_tokens(b, h), keep)
