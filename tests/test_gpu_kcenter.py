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
                hp.assert_output(out[b, h * G + g], want, w.torch_dtype)
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
    hp.assert_output(out[0, 0], want, torch.bfloat16)
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


def _check_selection(ex, Kn, units, n_old, k, r):
    for b, h in units:
        cent, _ = orc.kcenter(Kn[b, h, :n_old], k)
        keep = np.concatenate([cent.astype(np.int64), np.arange(n_old, n_old + r)])
        np.testing.assert_array_equal(ex.export_tokens(b, h), keep)


def test_kcenter_ties_and_uninformative_heads():
    """Inputs on which the early lower bound is tight, useless or decides between equal distances.

    Unit 0: a coarse lattice with many duplicates (equal distances everywhere, ties go to the lowest index).
    Unit 1: keys equal in the first 16 coordinates (the head bound is 0, every comparison needs the full row).
    Unit 2: keys that differ in the first 16 coordinates only (the head bound is the whole distance).
    Unit 3: clustered keys plus exact copies of earlier rows.
    """
    rng = np.random.default_rng(7)
    n, d, k, r = 3000, 128, 200, 17
    K = np.zeros((1, 4, n, d), np.float32)
    K[0, 0] = rng.integers(-1, 2, (n, d)) * 0.5
    K[0, 0, :, 4:] = 0.0
    K[0, 1, :, :16] = 0.25
    K[0, 1, :, 16:] = rng.normal(size=(n, d - 16))
    K[0, 2, :, :16] = rng.normal(size=(n, 16))
    K[0, 2, :, 16:] = -1.5
    cl = rng.normal(size=(12, d))
    K[0, 3] = cl[rng.integers(0, 12, n)] + 0.01 * rng.normal(size=(n, d))
    K[0, 3, 1500:] = K[0, 3, :1500]
    Kt = torch.tensor(K, dtype=torch.bfloat16, device="cuda")
    Vt = torch.randn(1, 4, n, d, device="cuda").to(torch.bfloat16)
    from paper_2402_06082_b200.binding import ExactAttention
    ex = ExactAttention(1, 4, d, n, Hkv=4, dtype=torch.bfloat16)
    ex.append(Kt, Vt)
    ex.kcenter_compress(k, r)
    _check_selection(ex, f32(Kt), [(0, h) for h in range(4)], n - r, k, r)
    looked, full = ex.kcenter_counters()
    assert 0 < full <= looked


def test_kcenter_long_slices_many_units():
    """More units than one wave of blocks and more than 16384 older tokens: every unit is cut into two slices."""
    w = synth.CFG3.scaled(B=150, H=8, Hkv=8, d=64, n_prompt=16500, ncomp=64)
    n, k, r = 16500, 24, 50
    K = torch.empty(w.B, w.Hkv, n, w.d, dtype=torch.bfloat16, device="cuda")
    for b in range(w.B):
        K[b] = synth.sequence_stream(w.scaled(data_seed=1003 + b % 3), b, n, "cuda")[0]
    ex = _exact(w, n)
    ex.append(K, K)
    ex.kcenter_compress(k, r)
    Kn = {b: f32(K[b:b + 1]) for b in (0, 77, 149)}
    for b, Kb in Kn.items():
        for h in (0, 7):
            cent, _ = orc.kcenter(Kb[0, h, : n - r], k)
            np.testing.assert_array_equal(ex.export_tokens(b, h)[:k], cent.astype(np.int64))
