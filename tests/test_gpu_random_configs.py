"""Randomly drawn configurations (seeded): shapes, sample counts, windows, budgets, prefill cuts, a checkpoint round
trip, multi-query calls and a second prefill in the middle of a stream, every unit compared with the CPU oracle."""
import os
import random
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


def _draw(seed):
    rnd = random.Random(seed)
    cfg = dict(
        dtype=rnd.choice(["bf16", "bf16", "bf16", "fp32"]), d=rnd.choice([64, 128]), G=rnd.choice([1, 1, 2, 4, 8]),
        Hkv=rnd.choice([1, 2, 5]), B=rnd.choice([1, 2, 3]), t=rnd.choice([1, 2, 3, 8, 8, 16, 17, 33, 64]),
        s=rnd.choice([1, 7, 16, 33, 100]), window=rnd.choice([0, 1, 5, 16, 40]), bounded=rnd.random() < 0.35)
    cfg["m_max"] = rnd.choice([6, 20]) if cfg["bounded"] else 512
    cfg.update(ncomp=rnd.choice([3, 10, 40]), delta=rnd.choice([0.3, 0.5, 0.8]), n0=rnd.choice([0, 1, 50, 200, 390]),
               nd=rnd.choice([3, 9]), philox=rnd.randrange(1 << 40))
    nq = 1
    while cfg["G"] * nq * 2 <= 8 and rnd.random() < 0.5:
        nq *= 2
    cfg["nq"] = nq
    cfg["cuts"] = sorted(set([0, cfg["n0"]] + [rnd.randrange(0, cfg["n0"] + 1) for _ in range(rnd.choice([0, 1, 2]))]))
    cfg["checkpoint"] = rnd.random() < 0.5
    cfg["extra"] = rnd.choice([0, 30])
    return cfg


@pytest.mark.parametrize("seed", list(range(40)))
def test_random_configuration(seed, monkeypatch):
    from paper_2402_06082_b200.binding import SubGen
    c = _draw(seed)
    # unbounded bf16 handles with d = 128 have two prefill paths (a score and a resolve kernel per chunk, or one
    # persistent kernel per call); the default picks by unit count, so odd seeds force the persistent one
    if seed % 2:
        monkeypatch.setenv("SUBGEN_PREFILL", "persist")
    B, Hkv, G, d, t, s, window = c["B"], c["Hkv"], c["G"], c["d"], c["t"], c["s"], c["window"]
    w = synth.CFG3.scaled(B=B, H=Hkv * G, Hkv=Hkv, d=d, dtype=c["dtype"], n_prompt=c["n0"], ncomp=c["ncomp"], s=s, window=window,
                          m_max=c["m_max"], t=t, delta=c["delta"], philox_seed=c["philox"], data_seed=seed)
    n0, nd, nq = c["n0"], c["nd"], c["nq"]
    K, V, Q = synth.batch_stream(w, n0 + nd + 40, "cuda")
    Kn, Vn, Qn = f32(K), f32(V), f32(Q)
    tol = hp.TOL[w.torch_dtype]

    def make():
        return SubGen(B, w.H, d, w.delta, t, s, window, w.philox_seed, Hkv=Hkv, dtype=w.torch_dtype, m_max=w.m_max,
                      bounded=c["bounded"], nq_max=nq)

    sg = make()
    orcs = {(b, h): orc.OracleUnit(d, w.delta, t, s, window, seed=w.philox_seed, unit_id=b * Hkv + h, m_max=w.m_max,
                                   bounded=c["bounded"]) for b in range(B) for h in range(Hkv)}

    def steps(pos, count):
        for i in range(pos, pos + count):
            out = f32(sg.step(Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous()))
            for (b, h), o in orcs.items():
                o.push(Kn[b, h, i], Vn[b, h, i])
                for g in range(G):
                    hp.assert_output(out[b, h * G + g], o.query(Qn[b, h * G + g, i]), w.torch_dtype, (c, i))
        return pos + count

    for a, b_ in zip(c["cuts"][:-1], c["cuts"][1:]):
        sg.prefill(K[:, :, a:b_].contiguous(), V[:, :, a:b_].contiguous())
    for (b, h), o in orcs.items():
        o.push_many(Kn[b, h, :n0], Vn[b, h, :n0])
        hp.assert_state_equal(sg.export_state(b, h), o, "after prefill %s" % (c,))
    pos = steps(n0, nd)
    if c["checkpoint"]:
        blob = sg.checkpoint_save()
        sg.close()
        sg = make()
        sg.checkpoint_load(blob)
    if c["extra"]:
        sg.prefill(K[:, :, pos:pos + c["extra"]].contiguous(), V[:, :, pos:pos + c["extra"]].contiguous())
        for (b, h), o in orcs.items():
            o.push_many(Kn[b, h, pos:pos + c["extra"]], Vn[b, h, pos:pos + c["extra"]])
        pos += c["extra"]
    probes = Q[:, :, pos:pos + nq].contiguous()
    got = f32(sg.query(probes))
    for (b, h), o in orcs.items():
        for g in range(G):
            for j in range(nq):
                hp.assert_output(got[b, h * G + g, j], o.query(f32(probes[b, h * G + g, j])), w.torch_dtype, c)
    pos = steps(pos, 3)
    distinct = 0
    for (b, h), o in orcs.items():
        st = sg.export_state(b, h)
        hp.assert_state_equal(st, o, "end %s" % (c,))
        assert st["threshold2"] == o.thr2_fx and st["doublings"] == o.level
        hp.assert_rows_match_tokens(sg, b, h, st, K[b, h], V[b, h])
        distinct += sum(len(set(r.tolist())) if t <= 16 else t for r in o.slot_tok[o.counts > 1])
    assert sg.cache_stats()["distinct_sample_rows"] == distinct
    assert sg.status() == 0
    sg.close()
