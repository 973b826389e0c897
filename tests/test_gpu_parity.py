"""Parity of the CUDA library (through its C ABI) with the CPU oracle on the same seeded inputs.

Integer decisions (cluster of every key, counts, sampled token indices, mu, the fixed-point distance
of the latest insertion) must match bit for bit; outputs within 1e-4 (fp32) / 2e-2 (bf16) relative L2.
"""
import sys, os
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
    args = dict(Hkv=w.Hkv, dtype=w.torch_dtype, m_max=w.m_max)
    args.update(kw)
    return SubGen(w.B, w.H, w.d, w.delta, w.t, w.s, w.window, w.philox_seed, **args)


def _run_stream(w, n_prefill, n_steps, check_every=0, prefill_chunks=(), **kw):
    """prefill n_prefill tokens (optionally in chunks), then n_steps stream steps; compares every unit."""
    n = n_prefill + n_steps
    K, V, Q = synth.batch_stream(w, n, "cuda")            # [B,Hkv,n,d], [B,H,n,d]
    sg = _sg(w, **kw)
    units = [(b, h) for b in range(w.B) for h in range(w.Hkv)]
    orcs = {bh: hp.oracle_unit(w, *bh) for bh in units}
    Kn, Vn, Qn = f32(K), f32(V), f32(Q)
    cuts = [0] + list(prefill_chunks) + [n_prefill]
    for a, b_ in zip(cuts[:-1], cuts[1:]):
        if b_ > a:
            sg.prefill(K[:, :, a:b_].contiguous(), V[:, :, a:b_].contiguous())
    for (b, h), o in orcs.items():
        o.push_many(Kn[b, h, :n_prefill], Vn[b, h, :n_prefill])
        hp.assert_state_equal(sg.export_state(b, h), o, "after prefill unit %s" % ((b, h),))
    G = w.H // w.Hkv
    worst = 0.0
    outs = []
    for i in range(n_prefill, n):
        outs.append(sg.step(Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous()))
    outs = [f32(o) for o in outs]
    for j, i in enumerate(range(n_prefill, n)):
        for (b, h), o in orcs.items():
            o.push(Kn[b, h, i], Vn[b, h, i])
            for g in range(G):
                want = o.query(Qn[b, h * G + g, i])
                err = hp.rel_err(outs[j][b, h * G + g], want)
                worst = max(worst, err)
                assert err <= hp.TOL[w.torch_dtype], "step %d unit %s head %d: rel err %.3g" % (i, (b, h), g, err)
        # the device state is only observable at the end; intermediate checkpoints replay a fresh handle
    for (b, h), o in orcs.items():
        st = sg.export_state(b, h)
        hp.assert_state_equal(st, o, "after steps unit %s" % ((b, h),))
        hp.assert_rows_match_tokens(sg, b, h, st, K[b, h], V[b, h])
    assert sg.status() == 0
    return sg, orcs, worst


def test_cfg1_full_stream_fp32():
    """The 4096-token fp32 stream (16-component mixture, delta 0.5, t 4, s 256, window 64), every step compared."""
    w = synth.CFG1
    sg, orcs, worst = _run_stream(w, 0, w.n_decode)
    o = orcs[(0, 0)]
    assert o.m == 16 and o.inserted == w.n_decode - w.window
    print("cfg1 worst rel err %.3g" % worst)


@pytest.mark.parametrize("splits", [1, 3, 8])
def test_stream_state_checkpoints_fp32(splits):
    """State compared at several stream lengths (a fresh handle per length), for several block splits."""
    w = synth.CFG1.scaled(outlier_frac=0.1, m_max=512, s=37, t=3)
    for n in (1, 63, 64, 65, 200, 701):
        _run_stream(w, 0, n, splits=splits)


def test_prefill_equals_steps_and_chunking_is_invariant():
    w = synth.CFG2.scaled(B=2, H=4, Hkv=4, n_prompt=1500, ncomp=32, s=128, window=64, m_max=256)
    sg1, orcs, _ = _run_stream(w, 1500, 8)
    sg2, _, _ = _run_stream(w, 1500, 8, prefill_chunks=(1, 63, 64, 65, 700, 1499))
    sg3, _, _ = _run_stream(w, 0, 1508)
    for b in range(w.B):
        for h in range(w.Hkv):
            a, c, e = sg1.export_state(b, h), sg2.export_state(b, h), sg3.export_state(b, h)
            for key in ("m", "mu", "n"):
                assert a[key] == c[key] == e[key]
            for key in ("counts", "centre_tok", "slot_tok", "m_tok", "m_w"):
                np.testing.assert_array_equal(a[key], c[key]); np.testing.assert_array_equal(a[key], e[key])


def test_bf16_gqa_outliers():
    w = synth.CFG3.scaled(B=2, H=8, Hkv=2, n_prompt=900, ncomp=24, s=256, window=32, m_max=512)
    _, orcs, worst = _run_stream(w, 900, 24)
    assert any((o.counts == 1).sum() > 10 for o in orcs.values())      # singleton clusters are exercised
    print("bf16 gqa worst rel err %.3g" % worst)


@pytest.mark.parametrize("dtype,d", [("fp32", 128), ("bf16", 64), ("fp32", 64), ("bf16", 128)])
def test_all_row_geometries(dtype, d):
    w = synth.CFG2.scaled(B=1, H=2, Hkv=2, d=d, dtype=dtype, n_prompt=300, ncomp=8, s=64, t=5, window=16, m_max=128)
    _run_stream(w, 300, 12)


@pytest.mark.parametrize("G", [2, 8])
def test_gqa_group_sizes(G):
    w = synth.CFG2.scaled(B=1, H=2 * G, Hkv=2, n_prompt=200, ncomp=8, s=64, window=16, m_max=128)
    _run_stream(w, 200, 6)


def test_drifting_centres():
    w = synth.CFG4.scaled(H=4, Hkv=1, n_prompt=3000, ncomp=64, s=256, window=128, m_max=3000, drift_step=0.05)
    _, orcs, _ = _run_stream(w, 3000, 10)
    assert orcs[(0, 0)].m > 200


@pytest.mark.parametrize("window", [0, 1, 5])
def test_small_windows(window):
    w = synth.CFG1.scaled(window=window, s=20, t=2, m_max=64)
    _run_stream(w, 40, 60)
    _run_stream(w, 0, 3)


def test_degenerate_parameters():
    _run_stream(synth.CFG1.scaled(t=1, s=1, window=3, m_max=64), 50, 20)
    _run_stream(synth.CFG1.scaled(t=64, s=5, window=3, m_max=64), 50, 20)
    # delta = 0: every distinct key opens its own cluster
    w = synth.CFG1.scaled(delta=0.0, window=2, s=16, m_max=128)
    _, orcs, _ = _run_stream(w, 30, 40)
    assert orcs[(0, 0)].m == 68
    # window longer than the stream: exact attention, nothing inserted
    w = synth.CFG1.scaled(window=512, s=16, m_max=8)
    sg, orcs, _ = _run_stream(w, 100, 50)
    assert orcs[(0, 0)].m == 0 and sg.export_state(0, 0)["mu"] == 0


def test_empty_prefill_and_zero_values():
    from paper_2402_06082_b200.binding import SubGen
    w = synth.CFG1.scaled(window=0, s=8, m_max=16)
    sg = _sg(w)
    sg.prefill(torch.empty(1, 1, 0, w.d, device="cuda"), torch.empty(1, 1, 0, w.d, device="cuda"))
    assert sg.export_state(0, 0)["n"] == 0
    o = hp.oracle_unit(w, 0, 0)
    q = torch.ones(1, 1, w.d, device="cuda"); k = torch.ones(1, 1, w.d, device="cuda")
    z = torch.zeros(1, 1, w.d, device="cuda")
    out = sg.step(q, k, z)                                   # zero value: never sampled, output 0
    o.push(f32(k)[0, 0], f32(z)[0, 0])
    np.testing.assert_array_equal(f32(out)[0, 0], o.query(f32(q)[0, 0]))
    hp.assert_state_equal(sg.export_state(0, 0), o, "zero value")
    out = sg.step(q, k, 2 * q)
    o.push(f32(k)[0, 0], 2 * f32(q)[0, 0])
    assert hp.rel_err(f32(out)[0, 0], o.query(f32(q)[0, 0])) < 1e-5
    hp.assert_state_equal(sg.export_state(0, 0), o, "after zero value")


@pytest.mark.parametrize("mode", ["chunk", "persist"])
def test_varlen_prefill_bf16(mode, monkeypatch):
    monkeypatch.setenv("SUBGEN_PREFILL", mode)
    w = synth.CFG5.scaled(B=3, H=4, Hkv=2, ncomp=16, s=64, window=32, m_max=256)
    lens = [5, 333, 90]
    n_dec = 6
    streams = [synth.sequence_stream(w, b, lens[b] + n_dec, "cuda") for b in range(w.B)]
    cu = np.concatenate([[0], np.cumsum(lens)])
    Kp = torch.cat([streams[b][0][:, :lens[b]] for b in range(w.B)], dim=1).contiguous()     # [Hkv,total,d]
    Vp = torch.cat([streams[b][1][:, :lens[b]] for b in range(w.B)], dim=1).contiguous()
    sg = _sg(w)
    sg.prefill_varlen(Kp, Vp, cu)
    orcs = {}
    for b in range(w.B):
        for h in range(w.Hkv):
            o = hp.oracle_unit(w, b, h)
            o.push_many(f32(streams[b][0][h, :lens[b]]), f32(streams[b][1][h, :lens[b]]))
            hp.assert_state_equal(sg.export_state(b, h), o, "varlen prefill %s" % ((b, h),))
            orcs[(b, h)] = o
    G = w.H // w.Hkv
    for i in range(n_dec):
        q = torch.stack([streams[b][2][:, lens[b] + i] for b in range(w.B)]).contiguous()
        k = torch.stack([streams[b][0][:, lens[b] + i] for b in range(w.B)]).contiguous()
        v = torch.stack([streams[b][1][:, lens[b] + i] for b in range(w.B)]).contiguous()
        out = f32(sg.step(q, k, v))
        for (b, h), o in orcs.items():
            o.push(f32(k)[b, h], f32(v)[b, h])
            for g in range(G):
                hp.assert_output(out[b, h * G + g], o.query(f32(q)[b, h * G + g]), torch.bfloat16)
    for (b, h), o in orcs.items():
        hp.assert_state_equal(sg.export_state(b, h), o, "varlen steps %s" % ((b, h),))


def test_capacity_overflow_sets_status_and_poisons_output():
    from paper_2402_06082_b200 import binding
    w = synth.CFG1.scaled(delta=0.0, window=0, s=8, m_max=4)
    K, V, Q = synth.batch_stream(w, 6, "cuda")
    sg = _sg(w)
    outs = [sg.step(Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous()) for i in range(6)]
    assert sg.status() == binding.ST_CAPACITY
    assert torch.isfinite(outs[3]).all() and torch.isnan(outs[4]).all() and torch.isnan(outs[5]).all()
    assert sg.export_state(0, 0)["m"] == 4
    o = hp.oracle_unit(w, 0, 0)
    with pytest.raises(OverflowError):
        o.push_many(f32(K)[0, 0], f32(V)[0, 0])
    assert o.overflow_at == 4


def test_non_finite_input_sets_status():
    from paper_2402_06082_b200 import binding
    w = synth.CFG1.scaled(window=0, s=8, m_max=16)
    sg = _sg(w)
    q = torch.ones(1, 1, w.d, device="cuda")
    bad = q.clone(); bad[0, 0, 3] = float("inf")
    sg.step(q, q, q)
    assert sg.status() == 0
    sg.step(q, q, bad)
    assert sg.status() == binding.ST_RANGE


def test_host_argument_errors():
    from paper_2402_06082_b200 import binding
    w = synth.CFG1.scaled(window=4, s=8, m_max=16)
    sg = _sg(w)
    L = binding.load()
    assert L.subgen_step(sg._h, None, None, None, None) == -1
    assert L.subgen_prefill(sg._h, None, None, -1) == -1
    assert L.subgen_prefill(sg._h, None, None, 5) == -1
    assert L.subgen_export_state(sg._h, 3, 0, None) == -1
    with pytest.raises(ValueError):
        sg.step(torch.ones(1, 1, 8, device="cuda"), torch.ones(1, 1, w.d, device="cuda"), torch.ones(1, 1, w.d, device="cuda"))
    assert sg.export_state(0, 0)["n"] == 0
    L.subgen_destroy(None)


@pytest.mark.parametrize("how", ["pinned_staged", "pinned_direct", "pageable"])
def test_step_host_matches_step(how):
    """Pinned buffers: the result is written by the kernels directly; the inputs are read by them directly (few blocks
    per unit) or brought over by one staging kernel first (many blocks per unit). Pageable buffers go through staging
    copies."""
    w = synth.CFG2.scaled(B=2, H=4, Hkv=2, n_prompt=100, ncomp=8, s=32, window=16, m_max=64)
    K, V, Q = synth.batch_stream(w, 110, "cuda")
    kw = dict(splits=2) if how == "pinned_direct" else {}
    a, b = _sg(w, **kw), _sg(w, **kw)
    a.prefill(K[:, :, :100].contiguous(), V[:, :, :100].contiguous())
    b.prefill(K[:, :, :100].contiguous(), V[:, :, :100].contiguous())
    host = (lambda x: x.cpu()) if how == "pageable" else (lambda x: x.cpu().pin_memory())
    for i in range(100, 110):
        q, k, v = Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous()
        o1 = a.step(q, k, v)
        out = host(torch.empty(o1.shape, dtype=o1.dtype))
        b.step_host(host(q), host(k), host(v), out)
        # same arithmetic, but the order in which partial sums meet depends on scheduling: compare to rounding
        err = hp.rel_err(f32(o1).reshape(-1, w.d), f32(out).reshape(-1, w.d))
        assert err <= 1e-2
    for bb in range(w.B):
        for h in range(w.Hkv):
            s1, s2 = a.export_state(bb, h), b.export_state(bb, h)
            for key in ("m", "mu", "n"):
                assert s1[key] == s2[key]
            for key in ("counts", "centre_tok", "slot_tok", "m_tok"):
                np.testing.assert_array_equal(s1[key], s2[key])


@pytest.mark.parametrize("mode", ["split", "fused"])
def test_cache_stats_and_profile(mode):
    w = synth.CFG3.scaled(B=1, H=2, Hkv=2, n_prompt=600, ncomp=16, s=64, window=32, m_max=256)
    sg, orcs, _ = _run_stream(w, 600, 4, step_mode=mode)
    st = sg.cache_stats()
    assert st["units"] == 2 and st["tokens"] == 2 * 604 and st["window_rows"] == 64
    assert st["clusters"] == sum(o.m for o in orcs.values())
    assert st["singleton_clusters"] == sum(int((o.counts == 1).sum()) for o in orcs.values())
    assert st["m_filled"] == sum(int((o.m_tok >= 0).sum()) for o in orcs.values())
    row = w.d * 2
    assert st["insert_bytes"] == st["clusters"] * (32 * 2 + 4)      # bf16: packed heads and their norms
    distinct = sum(len(set(r.tolist())) for o in orcs.values() for r in o.slot_tok[o.counts > 1])
    assert st["distinct_sample_rows"] == distinct
    assert distinct < (st["clusters"] - st["singleton_clusters"]) * w.t          # reservoirs do repeat tokens
    crow = st["singleton_clusters"] + distinct
    assert st["cluster_bytes"] == crow * row + st["clusters"] * (4 + w.t)
    assert st["value_bytes"] == (2 * st["m_filled"] + 2 * 64) * row + 2 * w.s * 4
    assert st["query_bytes"] == st["cluster_bytes"] + st["value_bytes"]
    sg.profile_enable(True)
    K, V, Q = synth.batch_stream(w, 3, "cuda")
    before = sg.launch_count
    for i in range(3):
        sg.step(Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous())
    ins, tau, zz, steps = sg.profile_read()
    nk = sg.step_kernels
    assert nk == (3 if mode == "split" else 1) and steps == 3 and sg.launch_count == before + 3 * nk
    assert tau > 0 and ((ins > 0 and zz > 0) if nk == 3 else (ins < tau and zz < tau))     # one kernel: its time is in tau


def test_chunked_prefill_equals_token_by_token_prefill(monkeypatch):
    """bf16 handles prefill chunk by chunk on the tensor cores; SUBGEN_PREFILL=seq selects the token-by-token
    kernel. Both must leave the same state, also when a call continues a stream whose tail is in the window."""
    w = synth.CFG3.scaled(B=2, H=4, Hkv=2, n_prompt=1000, ncomp=24, s=96, t=6, window=48, m_max=512)
    K, V, _ = synth.batch_stream(w, 1000, "cuda")
    a = _sg(w)                                   # d = 128: chunk scoring with tcgen05
    monkeypatch.setenv("SUBGEN_PREFILL", "seq")
    b = _sg(w)
    monkeypatch.setenv("SUBGEN_PREFILL", "mma")  # chunk scoring with warp-level MMAs
    c = _sg(w)
    monkeypatch.setenv("SUBGEN_PREFILL", "persist")  # all chunks of a call in one persistent kernel (tcgen05)
    p = _sg(w)
    monkeypatch.delenv("SUBGEN_PREFILL")
    for lo, hi in ((0, 7), (7, 300), (300, 301), (301, 1000)):
        for sg in (a, b, c, p):
            sg.prefill(K[:, :, lo:hi].contiguous(), V[:, :, lo:hi].contiguous())
        for bb in range(w.B):
            for h in range(w.Hkv):
                s2 = b.export_state(bb, h)
                hp.assert_rows_match_tokens(b, bb, h, s2, K[bb, h], V[bb, h])
                for sg in (a, c, p):
                    s1 = sg.export_state(bb, h)
                    for key in ("m", "mu", "n", "last_cluster", "last_opened", "status"):
                        assert s1[key] == s2[key], (key, lo, hi)
                    for key in ("counts", "centre_tok", "slot_tok", "m_tok", "m_w"):
                        np.testing.assert_array_equal(s1[key], s2[key], err_msg="%s after [%d,%d)" % (key, lo, hi))
                    hp.assert_rows_match_tokens(sg, bb, h, s1, K[bb, h], V[bb, h])
    assert a.launch_count > p.launch_count > b.launch_count


@pytest.mark.parametrize("mode", ["chunk", "persist"])
def test_tcgen05_scoring_many_tiles_and_dense_candidates(mode, monkeypatch):
    """Several 128-representative tiles per chunk, and a radius so large that every pair is inside the guard band
    (the exhaustive path of the score kernel): state must equal the oracle's. Both tcgen05 prefill paths."""
    monkeypatch.setenv("SUBGEN_PREFILL", mode)
    w = synth.CFG3.scaled(B=1, H=2, Hkv=2, n_prompt=2500, ncomp=400, s=64, t=4, window=16, m_max=1024)
    _run_stream(w, 2500, 4)
    w = synth.CFG2.scaled(B=1, H=1, Hkv=1, n_prompt=600, ncomp=4, sigma=0.5, delta=30.0, s=32, t=4, window=8, m_max=64)
    _, orcs, _ = _run_stream(w, 600, 4)
    assert orcs[(0, 0)].m == 1


@pytest.mark.parametrize("mode", ["chunk", "persist"])
def test_prefill_capacity_overflow_is_reported(mode, monkeypatch):
    from paper_2402_06082_b200 import binding
    monkeypatch.setenv("SUBGEN_PREFILL", mode)
    w = synth.CFG3.scaled(B=1, H=2, Hkv=2, n_prompt=400, ncomp=64, s=32, window=8, m_max=16)
    K, V, _ = synth.batch_stream(w, 400, "cuda")
    sg = _sg(w)
    sg.prefill(K, V)
    assert sg.status() == binding.ST_CAPACITY
    assert sg.export_state(0, 0)["m"] == 16


# ------------------------------------------------------------------------------------------- exact path
@pytest.mark.parametrize("dtype,G", [("fp32", 1), ("bf16", 4)])
def test_exact_attention_matches_eq1(dtype, G):
    from paper_2402_06082_b200.binding import ExactAttention
    w = synth.CFG2.scaled(B=2, H=2 * G, Hkv=2, dtype=dtype, n_prompt=777, ncomp=8)
    n0, nd = 777, 5
    K, V, Q = synth.batch_stream(w, n0 + nd, "cuda")
    ex = ExactAttention(w.B, w.H, w.d, n0 + nd, Hkv=w.Hkv, dtype=w.torch_dtype)
    ex.append(K[:, :, :500].contiguous(), V[:, :, :500].contiguous())
    ex.append(K[:, :, 500:n0].contiguous(), V[:, :, 500:n0].contiguous())
    Kn, Vn, Qn = f32(K), f32(V), f32(Q)
    for i in range(n0, n0 + nd):
        out = f32(ex.step(Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous()))
        for b in range(w.B):
            for hq in range(w.H):
                want = orc.exact_attention(Kn[b, hq // G, : i + 1], Vn[b, hq // G, : i + 1], Qn[b, hq, i])
                hp.assert_output(out[b, hq], want, w.torch_dtype)
    assert ex.bytes_per_step() == 2 * w.B * w.Hkv * (n0 + nd) * w.d * (4 if dtype == "fp32" else 2)
    with pytest.raises(Exception):
        ex.step(Q[:, :, 0].contiguous(), K[:, :, 0].contiguous(), V[:, :, 0].contiguous())   # cache full


def test_exact_varlen_and_short_window_agreement():
    """While nothing has left the window SubGen IS exact attention: both kernels must agree."""
    from paper_2402_06082_b200.binding import ExactAttention
    w = synth.CFG5.scaled(B=2, H=4, Hkv=2, ncomp=8, s=16, window=256, m_max=8)
    lens = [17, 120]
    streams = [synth.sequence_stream(w, b, lens[b] + 3, "cuda") for b in range(w.B)]
    cu = [0, 17, 137]
    Kp = torch.cat([streams[b][0][:, :lens[b]] for b in range(w.B)], dim=1).contiguous()
    Vp = torch.cat([streams[b][1][:, :lens[b]] for b in range(w.B)], dim=1).contiguous()
    ex = ExactAttention(w.B, w.H, w.d, 200, Hkv=w.Hkv, dtype=w.torch_dtype)
    ex.append_varlen(Kp, Vp, cu)
    sg = _sg(w)
    sg.prefill_varlen(Kp, Vp, cu)
    for i in range(3):
        q = torch.stack([streams[b][2][:, lens[b] + i] for b in range(w.B)]).contiguous()
        k = torch.stack([streams[b][0][:, lens[b] + i] for b in range(w.B)]).contiguous()
        v = torch.stack([streams[b][1][:, lens[b] + i] for b in range(w.B)]).contiguous()
        a, e = f32(sg.step(q, k, v)), f32(ex.step(q, k, v))
        for b in range(w.B):
            for hq in range(w.H):
                want = orc.exact_attention(f32(streams[b][0])[hq // 2, : lens[b] + i + 1],
                                           f32(streams[b][1])[hq // 2, : lens[b] + i + 1], f32(q)[b, hq])
                hp.assert_output(a[b, hq], want, torch.bfloat16)
                hp.assert_output(e[b, hq], want, torch.bfloat16)


# ------------------------------------------------------------------------------------------- full size
def test_benchmark_workload_full_size_sampled_units():
    """The benchmark's workload (cfg3: 8 x 32 heads, 32768-token prompts, bf16) in the benchmark's launch
    configuration; the oracle replays a seeded sample of (sequence, head) units in full."""
    from concurrent.futures import ThreadPoolExecutor
    w = synth.CFG3
    n0, nd = w.n_prompt, 6
    sg = _sg(w)
    rng = np.random.default_rng(5)
    sample = [(int(b), int(h)) for b, h in zip(rng.integers(0, w.B, 3), rng.integers(0, w.Hkv, 3))]
    Kp = torch.empty(w.B, w.Hkv, n0, w.d, dtype=w.torch_dtype, device="cuda")
    Vp = torch.empty_like(Kp)
    dec, host = [], {}
    for b in range(w.B):
        K, V, Q = synth.sequence_stream(w, b, n0 + nd, "cuda")
        Kp[b], Vp[b] = K[:, :n0], V[:, :n0]
        dec.append((K[:, n0:].clone(), V[:, n0:].clone(), Q[:, n0:].clone()))
        for (bb, h) in sample:
            if bb == b:
                host[(b, h)] = (f32(K[h]), f32(V[h]), f32(Q[h]))
        del K, V, Q
    sg.prefill(Kp, Vp)
    del Kp, Vp
    orcs = {bh: hp.oracle_unit(w, *bh) for bh in sample}

    def replay(bh):
        orcs[bh].push_many(host[bh][0][:n0], host[bh][1][:n0])
    with ThreadPoolExecutor(len(sample)) as ex:
        list(ex.map(replay, sample))
    for bh in sample:
        hp.assert_state_equal(sg.export_state(*bh), orcs[bh], "full-size prefill unit %s" % (bh,))
        assert orcs[bh].m > 1500
    for i in range(nd):
        q = torch.stack([d[2][:, i] for d in dec]).contiguous()
        k = torch.stack([d[0][:, i] for d in dec]).contiguous()
        v = torch.stack([d[1][:, i] for d in dec]).contiguous()
        out = f32(sg.step(q, k, v))
        for (b, h) in sample:
            Kh, Vh, Qh = host[(b, h)]
            orcs[(b, h)].push(Kh[n0 + i], Vh[n0 + i])
            err = hp.rel_err(out[b, h], orcs[(b, h)].query(Qh[n0 + i]))
            hp.assert_output(out[b, h], orcs[(b, h)].query(Qh[n0 + i]), torch.bfloat16, "step %d unit %s: %.3g" % (i, (b, h), err))
    for bh in sample:
        hp.assert_state_equal(sg.export_state(*bh), orcs[bh], "full-size steps unit %s" % (bh,))
    assert sg.status() == 0


@pytest.mark.parametrize("t,m_max,bounded", [(3, 512, False), (3, 6, True), (17, 512, False), (33, 7, True), (64, 512, False), (1, 512, False)])
def test_odd_sample_counts_and_unaligned_units(t, m_max, bounded):
    """t that is not a multiple of 4 (the per-unit alias rows then start at odd byte offsets) and t > 16 (alias
    lists keep every slot; the cluster scan goes through its rows in several passes)."""
    from paper_2402_06082_b200.binding import SubGen
    from oracle import subgen_oracle as orc
    w = synth.CFG3.scaled(B=1, H=5, Hkv=5, d=128, n_prompt=150, ncomp=10, s=7, window=1, m_max=m_max, t=t, delta=0.5)
    n0, nd = 150, 9
    K, V, Q = synth.batch_stream(w, n0 + nd, "cuda")
    sg = SubGen(1, 5, 128, w.delta, t, w.s, w.window, w.philox_seed, Hkv=5, dtype=torch.bfloat16, m_max=m_max, bounded=bounded)
    orcs = {h: orc.OracleUnit(128, w.delta, t, w.s, w.window, seed=w.philox_seed, unit_id=h, m_max=m_max, bounded=bounded) for h in range(5)}
    sg.prefill(K[:, :, :n0].contiguous(), V[:, :, :n0].contiguous())
    for h, o in orcs.items():
        o.push_many(f32(K[0, h, :n0]), f32(V[0, h, :n0]))
    for i in range(n0, n0 + nd):
        out = f32(sg.step(Q[:, :, i].contiguous(), K[:, :, i].contiguous(), V[:, :, i].contiguous()))
        for h, o in orcs.items():
            o.push(f32(K[0, h, i]), f32(V[0, h, i]))
            hp.assert_output(out[0, h], o.query(f32(Q[0, h, i])), torch.bfloat16)
    want = 0
    for h, o in orcs.items():
        hp.assert_state_equal(sg.export_state(0, h), o, "unit %d" % h)
        want += sum(len(set(r.tolist())) if t <= 16 else t for r in o.slot_tok[o.counts > 1])
    assert sg.cache_stats()["distinct_sample_rows"] == want
