"""Shared pieces of the GPU parity tests: run the CPU oracle on the same inputs and compare."""
import numpy as np
import torch

from oracle import subgen_oracle as orc
from paper_2402_06082_b200 import synth

TOL = {torch.float32: 1e-4, torch.bfloat16: 2e-2}     # relative L2 error of an output vector


def f32(x: torch.Tensor) -> np.ndarray:
    return synth.to_f32_numpy(x)


def oracle_unit(w, seq, kvhead, m_max=None):
    return orc.OracleUnit(w.d, w.delta, w.t, w.s, w.window, seed=w.philox_seed, unit_id=seq * w.Hkv + kvhead,
                          m_max=m_max or w.m_max)


def assert_state_equal(gpu: dict, o, where=""):
    """Bit-exact comparison of everything that is an integer decision."""
    assert gpu["status"] == 0, "%s: device status %d" % (where, gpu["status"])
    assert gpu["n"] == o.n, where
    assert gpu["inserted"] == o.inserted, where
    assert gpu["m"] == o.m, "%s: m gpu %d oracle %d" % (where, gpu["m"], o.m)
    assert gpu["mu"] == o.mu, where
    np.testing.assert_array_equal(gpu["counts"], o.counts, err_msg=where + " counts")
    np.testing.assert_array_equal(gpu["centre_tok"], o.centre_tok, err_msg=where + " centre tokens")
    np.testing.assert_array_equal(gpu["slot_tok"], o.slot_tok, err_msg=where + " cluster slot tokens")
    np.testing.assert_array_equal(gpu["m_tok"], o.m_tok, err_msg=where + " value slot tokens")
    w = o.w
    mt = o.m_tok
    exp_w = np.where(mt >= 0, w[np.maximum(mt, 0)] if o.n else 0, 0).astype(np.uint64)
    np.testing.assert_array_equal(gpu["m_w"], exp_w, err_msg=where + " value slot weights")
    if o.inserted:
        e = o.inserted - 1
        opened = int(o.centre_tok[o.assign[e]] == e)
        assert gpu["last_cluster"] == int(o.assign[e]), where
        assert gpu["last_opened"] == opened, where
        if not opened:          # the fixed-point distance to the joined representative, bit for bit
            d2 = int(o.ins_d2[e])
            assert gpu["last_d2"] == d2, "%s: last D2 gpu %d oracle %d" % (where, gpu["last_d2"], d2)


def rel_err(got: np.ndarray, want: np.ndarray) -> float:
    got = np.asarray(got, np.float64); want = np.asarray(want, np.float64)
    return float(np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-30))


def out_ulp(want: np.ndarray, dtype) -> np.ndarray:
    """One unit in the last place of the OUTPUT format at each wanted value (bf16: 8 significant bits; fp32: 24)."""
    a = np.abs(np.asarray(want, np.float64))
    bits = 8 if dtype == torch.bfloat16 else 24
    e = np.floor(np.log2(np.maximum(a, 2.0 ** -126)))
    return 2.0 ** (e - (bits - 1))


def elem_err(got: np.ndarray, want: np.ndarray, dtype) -> float:
    """Largest per-coordinate error in units of the tolerance: (|got_j - want_j| - ulp_j) / (tol * max_j |want_j|).
    A norm can hide a wrong small coordinate under a few large ones; this cannot."""
    got = np.asarray(got, np.float64); want = np.asarray(want, np.float64)
    scale = TOL[dtype] * max(float(np.max(np.abs(want))), 1e-30)
    return float(np.max((np.abs(got - want) - out_ulp(want, dtype)) / scale))


def assert_output(got: np.ndarray, want: np.ndarray, dtype, where="") -> None:
    """An output vector against the oracle's: relative L2 error within the tolerance of the dtype AND every
    coordinate within tol * max|want| plus one unit in the last place of the output format."""
    assert np.all(np.isfinite(np.asarray(got, np.float64))), "%s: non-finite output" % (where,)
    r = rel_err(got, want)
    assert r <= TOL[dtype], "%s: relative L2 error %.3g > %.3g" % (where, r, TOL[dtype])
    e = elem_err(got, want, dtype)
    assert e <= 1.0, "%s: a coordinate is off by %.3g x the per-element tolerance" % (where, e)


def assert_rows_match_tokens(sg, seq, kvhead, gpu_state, K_unit: torch.Tensor, V_unit: torch.Tensor):
    """Stored vectors are bit copies of the input rows named by the token indices."""
    st = gpu_state
    m, t = st["m"], sg.t
    X = sg.export_rows(seq, kvhead, 0)[:m]
    assert torch.equal(X, K_unit[st["centre_tok"]].cpu())
    S = sg.export_rows(seq, kvhead, 1).reshape(sg.m_max, t, sg.d)[:m]
    mat = st["counts"] > 1                                   # sample rows exist once a second member arrived
    if mat.any():
        idx = torch.from_numpy(st["slot_tok"][mat].astype(np.int64))
        assert torch.equal(S[torch.from_numpy(mat)], K_unit.cpu()[idx])
    filled = st["m_tok"] >= 0
    if filled.any():
        idx = torch.from_numpy(st["m_tok"][filled].astype(np.int64))
        f = torch.from_numpy(filled)
        assert torch.equal(sg.export_rows(seq, kvhead, 2)[f], K_unit.cpu()[idx])
        assert torch.equal(sg.export_rows(seq, kvhead, 3)[f], V_unit.cpu()[idx])
    if sg.window:
        n = st["n"]
        toks = np.arange(max(0, n - sg.window), n)
        rk = sg.export_rows(seq, kvhead, 4); rv = sg.export_rows(seq, kvhead, 5)
        assert torch.equal(rk[toks % sg.window], K_unit.cpu()[toks])
        assert torch.equal(rv[toks % sg.window], V_unit.cpu()[toks])
