"""Pins of the CPU oracle against what the paper and the mathematics fix.

Nothing here touches the CUDA path. Each test names the passage it pins.
"""
import os
from fractions import Fraction

import numpy as np
import pytest
import scipy.special
import scipy.stats

from oracle import subgen_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# --------------------------------------------------------------------------- Philox
def test_philox_published_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) >= 2
    for r in rows:
        w = [int(x, 16) for x in r]
        assert orc.philox4x32_10(w[0:4], w[4:6]) == w[6:10]


def _philox_py(ctr, key):
    """Philox4x32-10 with Python integers (second, independent statement)."""
    c = list(ctr); k = list(key)
    for r in range(10):
        if r:
            k = [(k[0] + 0x9E3779B9) & 0xFFFFFFFF, (k[1] + 0xBB67AE85) & 0xFFFFFFFF]
        p0 = 0xD2511F53 * c[0]; p1 = 0xCD9E8D57 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k[0], p1 & 0xFFFFFFFF, (p0 >> 32) ^ c[3] ^ k[1], p0 & 0xFFFFFFFF]
    return c


def test_philox_python_bigint_agrees():
    rng = np.random.default_rng(1)
    for _ in range(200):
        ctr = [int(x) for x in rng.integers(0, 2 ** 32, 4)]
        key = [int(x) for x in rng.integers(0, 2 ** 32, 2)]
        assert orc.philox4x32_10(ctr, key) == _philox_py(ctr, key)


def test_philox_words_uniform():
    words = np.array([orc.philox4x32_10([i, 7, 0, 1], [0, 0]) for i in range(20000)], dtype=np.uint64).ravel()
    hist = np.bincount((words >> 28).astype(np.int64), minlength=16)
    assert scipy.stats.chisquare(hist).pvalue > 1e-4
    bits = ((words[:, None] >> np.arange(32, dtype=np.uint64)) & 1).mean(axis=0)
    assert np.all(np.abs(bits - 0.5) < 5 * 0.5 / np.sqrt(words.size))


# --------------------------------------------------------------------------- fixed-point norms / distances
def test_fixed_point_distance_and_norm_track_the_real_values():
    rng = np.random.default_rng(2)
    for d in (8, 64, 128):
        x = rng.standard_normal(d).astype(np.float32); k = (x + 0.05 * rng.standard_normal(d)).astype(np.float32)
        real = float(np.sum((x.astype(np.float64) - k.astype(np.float64)) ** 2))
        assert abs(orc.dist2_fx(x, k) / 2 ** 32 - real) <= 1e-6 * real + d * 2.0 ** -32
        nv = float(np.sum(x.astype(np.float64) ** 2))
        assert abs(orc.norm2_fx(x) / 2 ** 24 - nv) <= 1e-6 * nv + d * 2.0 ** -24
        p = rng.permutation(d)      # order independence: any coordinate order gives the same bits
        assert orc.dist2_fx(x[p], k[p]) == orc.dist2_fx(x, k)
        assert orc.norm2_fx(x[p]) == orc.norm2_fx(x)
    assert orc.dist2_fx(np.ones(4), np.ones(4)) == 0
    assert orc.norm2_fx(np.array([1.0, 2.0, 0.5])) == (1 + 4) * 2 ** 24 + 2 ** 22


# --------------------------------------------------------------------------- exact special cases
def _softmax_attention(K, V, q):
    K = K.astype(np.float64); V = V.astype(np.float64); q = q.astype(np.float64)
    return scipy.special.softmax(K @ q) @ V


def test_exact_attention_is_eq1():
    rng = np.random.default_rng(3)
    K = rng.standard_normal((37, 16)).astype(np.float32); V = rng.standard_normal((37, 16)).astype(np.float32)
    q = rng.standard_normal(16).astype(np.float32)
    np.testing.assert_allclose(orc.exact_attention(K, V, q), _softmax_attention(K, V, q), rtol=1e-12, atol=1e-14)
    # V is indexed by row, not transposed: one-hot softmax picks a row of V
    Kb = np.zeros((5, 4), np.float32); Kb[3] = 50.0
    Vb = np.arange(20, dtype=np.float32).reshape(5, 4)
    np.testing.assert_allclose(orc.exact_attention(Kb, Vb, np.ones(4, np.float32)), Vb[3], atol=1e-12)


@pytest.mark.parametrize("window,n", [(64, 64), (64, 10), (7, 7), (1, 1)])
def test_stream_not_longer_than_window_is_exact_attention(window, n):
    """Window reading: while nothing has left the window the output is Eq. 1."""
    rng = np.random.default_rng(4)
    d = 8
    u = orc.OracleUnit(d, 0.5, 4, 16, window)
    K = rng.standard_normal((n, d)).astype(np.float32); V = rng.standard_normal((n, d)).astype(np.float32)
    for i in range(n):
        q = rng.standard_normal(d).astype(np.float32)
        out = u.step(q, K[i], V[i])
        np.testing.assert_allclose(out, _softmax_attention(K[: i + 1], V[: i + 1], q), rtol=1e-11, atol=1e-13)
    assert u.m == 0 and u.inserted == 0 and u.mu == 0 and np.all(u.m_tok == -1)


def test_first_token_fills_everything_and_output_is_v1():
    """After token 1, M is s copies of (k_1, v_1) (Section 2.2) and D one cluster of t copies: z/tau = v_1."""
    rng = np.random.default_rng(5)
    d = 8
    u = orc.OracleUnit(d, 0.5, 4, 32, 0, seed=9)
    k = rng.standard_normal(d).astype(np.float32); v = rng.standard_normal(d).astype(np.float32)
    out = u.step(rng.standard_normal(d), k, v)
    assert np.all(u.m_tok == 0) and u.m == 1 and np.all(u.slot_tok == 0) and u.counts[0] == 1
    np.testing.assert_allclose(out, v.astype(np.float64), rtol=1e-12)


def test_delta_zero_partition_function_is_exact():
    """delta = 0: distinct keys are singleton clusters of t copies, so tau = sum_i exp<q,k_i>; a repeated
    key joins its twin and tau stays exact."""
    rng = np.random.default_rng(6)
    d, n = 6, 50
    K = (0.3 * rng.standard_normal((n, d))).astype(np.float32)
    K[17] = K[3]; K[40] = K[3]
    V = rng.standard_normal((n, d)).astype(np.float32)
    u = orc.OracleUnit(d, 0.0, 3, 8, 0)
    u.push_many(K, V)
    assert u.m == n - 2 and u.counts[3] == 3
    q = rng.standard_normal(d).astype(np.float32)
    _, _, tau, shift = u.query_parts(q)
    np.testing.assert_allclose(tau * np.exp(shift), np.exp(K.astype(np.float64) @ q.astype(np.float64)).sum(), rtol=1e-12)


def test_zero_values_never_enter_M_and_null_slots_add_nothing():
    d = 4
    u = orc.OracleUnit(d, 10.0, 2, 8, 0)
    u.push(np.ones(d), np.zeros(d))
    assert np.all(u.m_tok == -1) and u.mu == 0
    np.testing.assert_array_equal(u.query(np.ones(d)), np.zeros(d))
    u.push(np.ones(d), np.full(d, 2.0))
    assert np.all(u.m_tok == 1)              # mu was 0, W > 0: probability one
    np.testing.assert_allclose(u.query(np.ones(d)), np.full(d, 2.0) / 2, rtol=1e-12)  # tau counts both keys


# --------------------------------------------------------------------------- Lemma 2 invariants
def _mixture(rng, n, d, ncomp, sigma, outlier=0.0):
    cent = rng.standard_normal((ncomp, d))
    comp = rng.integers(0, ncomp, n)
    K = cent[comp] + sigma / np.sqrt(d) * rng.standard_normal((n, d))
    if outlier:
        o = rng.random(n) < outlier
        g = rng.standard_normal((n, d)); K[o] = 3 * g[o] / np.linalg.norm(g[o], axis=1, keepdims=True)
    return K.astype(np.float32)


@pytest.mark.parametrize("window", [0, 16])
def test_lemma2_invariants_and_nearest_centre_rule(window):
    rng = np.random.default_rng(7)
    d, n, delta, t = 16, 600, 0.5, 4
    K = _mixture(rng, n, d, 12, 0.25, outlier=0.05)
    V = rng.standard_normal((n, d)).astype(np.float32)
    u = orc.OracleUnit(d, delta, t, 32, window)
    u.push_many(K, V)
    ins = n - window
    assert u.inserted == ins and u.n == n
    a = u.assign
    assert np.all(a[:ins] >= 0) and np.all(a[ins:] == -1)          # oldest tokens leave the window first
    m = u.m
    K64 = K.astype(np.float64)
    cent = u.centre_tok
    assert 12 <= m < ins                                           # some compression, some outliers
    np.testing.assert_array_equal(u.counts, np.bincount(a[:ins], minlength=m))     # (2) n_i = |C_i|
    assert u.counts.sum() == ins
    slots = u.slot_tok
    for c in range(m):
        members = np.flatnonzero(a[:ins] == c)
        assert cent[c] == members[0]                               # (1) representative = first member
        dist = np.linalg.norm(K64[members] - K64[cent[c]], axis=1)
        assert np.all(dist <= delta * (1 + 1e-6))                  # (3)
        assert np.all(np.isin(slots[c], members))                  # (5) samples are members
    G = np.linalg.norm(K64[cent][:, None] - K64[cent][None], axis=2)
    assert np.all(G[~np.eye(m, dtype=bool)] > delta * (1 - 1e-6))  # (4)
    # UpdateSoftmaxNormalizer: every token went to the nearest representative existing at its time,
    # and opened a cluster exactly when that one was farther than delta.
    order_open = {int(tok): c for c, tok in enumerate(cent)}
    existing = []
    for e in range(ins):
        if existing:
            dist = np.linalg.norm(K64[cent[existing]] - K64[e], axis=1)
            j = int(np.argmin(dist))
            if dist[j] <= delta * (1 - 1e-6):
                assert a[e] == existing[j] or abs(dist[a[e]] - dist[j]) <= 1e-6 * delta
                assert e not in order_open
            elif dist[j] > delta * (1 + 1e-6):
                assert order_open.get(e) == len(existing)
        if e in order_open:
            assert a[e] == order_open[e] == len(existing)
            existing.append(order_open[e])
    # mu invariant of Lemma 1 over the inserted tokens
    assert u.mu == int(u.w[:ins].astype(object).sum())
    np.testing.assert_allclose(u.mu / 2 ** 24, (V[:ins].astype(np.float64) ** 2).sum(), rtol=1e-6)


def test_threshold_is_inclusive():
    """'<= delta' joins (Algorithm 1 and Lemma 2)."""
    d = 4
    x = np.zeros(d, np.float32)
    k_on = np.array([0.5, 0, 0, 0], np.float32)           # exactly at distance delta
    k_out = np.array([0.5000001, 0, 0, 0], np.float32)
    u = orc.OracleUnit(d, 0.5, 2, 4, 0)
    u.push(x, np.ones(d)); u.push(k_on, np.ones(d))
    assert u.m == 1 and u.counts[0] == 2
    u.push(k_out, np.ones(d))
    assert u.m == 2


def test_argmin_ties_go_to_the_lowest_index():
    d = 2
    u = orc.OracleUnit(d, 1.0, 2, 4, 0)
    u.push(np.array([-1.0, 0.0]), np.ones(d)); u.push(np.array([1.0, 0.0]), np.ones(d))
    assert u.m == 2
    u.push(np.array([0.0, 0.0]), np.ones(d))               # equidistant, both within delta
    assert u.m == 2 and list(u.counts) == [2, 1]


# --------------------------------------------------------------------------- sampling laws
def test_lemma1_value_slots_follow_squared_norms():
    """Pr[M(j) = (k_i, v_i)] = ||v_i||^2 / sum_l ||v_l||^2, slots independent (Lemma 1)."""
    rng = np.random.default_rng(8)
    d, n, s = 4, 6, 512
    scale = np.array([0.5, 2.0, 1.0, 0.2, 1.5, 1.0])
    V = (scale[:, None] * rng.standard_normal((n, d))).astype(np.float32)
    K = rng.standard_normal((n, d)).astype(np.float32)
    hist = np.zeros(n)
    for seed in range(40):
        u = orc.OracleUnit(d, 100.0, 2, s, 0, seed=seed)
        u.push_many(K, V)
        hist += np.bincount(u.m_tok, minlength=n)
        w = u.w
    p = w.astype(np.float64) / w.astype(np.float64).sum()
    assert scipy.stats.chisquare(hist, p * hist.sum()).pvalue > 1e-4
    # a coin that used the new mu (mu + 2W in the denominator) would give the last token W/(mu_old+2W)
    wrong_last = w[-1] / (w.sum() + w[-1])
    assert abs(hist[-1] / hist.sum() - p[-1]) < 0.25 * abs(wrong_last - p[-1])
    # independence across slots: neighbouring slots agree no more often than sum p^2
    u = orc.OracleUnit(d, 100.0, 2, 8192, 0, seed=123); u.push_many(K, V)
    mt = u.m_tok
    agree = np.mean(mt[0::2] == mt[1::2])
    assert abs(agree - np.sum(p ** 2)) < 5 * np.sqrt(0.25 / (mt.size / 2))


def test_lemma2_cluster_slots_are_uniform_over_members():
    rng = np.random.default_rng(9)
    d, n, t = 4, 7, 64
    K = (0.01 * rng.standard_normal((n, d))).astype(np.float32)
    V = rng.standard_normal((n, d)).astype(np.float32)
    hist = np.zeros(n)
    for seed in range(60):
        u = orc.OracleUnit(d, 1.0, t, 4, 0, seed=seed)
        u.push_many(K, V)
        assert u.m == 1 and u.counts[0] == n
        hist += np.bincount(u.slot_tok.ravel(), minlength=n)
    assert scipy.stats.chisquare(hist).pvalue > 1e-4


def test_coins_differ_between_units_tokens_and_domains():
    d, n = 4, 40
    rng = np.random.default_rng(10)
    K = (0.01 * rng.standard_normal((n, d))).astype(np.float32); V = rng.standard_normal((n, d)).astype(np.float32)
    res = []
    for unit in (0, 1):
        u = orc.OracleUnit(d, 1.0, 16, 64, 0, seed=5, unit_id=unit); u.push_many(K, V)
        res.append((u.slot_tok.copy(), u.m_tok.copy()))
    assert not np.array_equal(res[0][0], res[1][0]) and not np.array_equal(res[0][1], res[1][1])
    u = orc.OracleUnit(d, 1.0, 16, 64, 0, seed=5, unit_id=0); u.push_many(K, V)
    np.testing.assert_array_equal(u.slot_tok, res[0][0]); np.testing.assert_array_equal(u.m_tok, res[0][1])


# --------------------------------------------------------------------------- estimator: mean and variance
def _estimator_samples(K, V, q, delta, t, s, window, seeds):
    d = K.shape[1]
    zs, taus = [], []
    for seed in seeds:
        u = orc.OracleUnit(d, delta, t, s, window, seed=seed)
        u.push_many(K, V)
        _, z, tau, shift = u.query_parts(q)
        zs.append(z * np.exp(shift)); taus.append(tau * np.exp(shift))
        part = u.assign[: u.inserted].copy()
    return np.array(zs), np.array(taus), part


@pytest.mark.parametrize("window", [0, 8])
def test_estimator_unbiased_with_closed_form_variance(window):
    """E z = exp(Kq)^T V and E tau = sum exp<q,k>; E||z - A||^2 = (mu ||e||^2 - ||A||^2)/s over the sampled
    part (row-norm sampling, Section 2.1) and Var tau = sum_c n_c^2/t Var_{k~U(C_c)} exp<q,k>."""
    rng = np.random.default_rng(11)
    d, n, t, s, R = 4, 48, 3, 16, 4000
    K = _mixture(rng, n, d, 4, 0.6)
    V = (rng.lognormal(0, 0.5, n)[:, None] * rng.standard_normal((n, d))).astype(np.float32)
    q = (0.7 * rng.standard_normal(d)).astype(np.float32)
    zs, taus, part = _estimator_samples(K, V, q, 0.8, t, s, window, range(R))
    K64, V64, q64 = K.astype(np.float64), V.astype(np.float64), q.astype(np.float64)
    e = np.exp(K64 @ q64)
    ins = n - window
    A_all = e @ V64
    A_ins = e[:ins] @ V64[:ins]
    # mean
    se_z = zs.std(axis=0) / np.sqrt(R)
    assert np.all(np.abs(zs.mean(axis=0) - A_all) < 4.5 * se_z)
    assert abs(taus.mean() - e.sum()) < 4.5 * taus.std() / np.sqrt(R)
    # variance of the numerator
    mu = (V64[:ins] ** 2).sum()
    var_z = (mu * (e[:ins] ** 2).sum() - A_ins @ A_ins) / s
    mse = ((zs - A_all) ** 2).sum(axis=1)
    assert abs(mse.mean() - var_z) < 5 * mse.std() / np.sqrt(R) + 1e-3 * var_z
    # variance of the partition function given the (deterministic) partition
    var_tau = sum((np.sum(part == c) ** 2) / t * e[:ins][part == c].var() for c in np.unique(part))
    emp = taus.var()
    assert abs(emp - var_tau) < 0.12 * var_tau
    # the constant-free part of the error bound (Eq. 3 with ||V||_F^2 <= d ||V||_op^2)
    rms = np.sqrt(mse.mean())
    assert rms <= np.sqrt(d / s) * np.linalg.norm(e[:ins]) * np.linalg.norm(V64[:ins], 2) * 1.05


def test_update_precedes_query_and_new_mu_is_used():
    """Main loop of Algorithm 1: the token of a step is visible to that step's query (window = 0)."""
    rng = np.random.default_rng(12)
    d = 4
    u = orc.OracleUnit(d, 100.0, 64, 256, 0, seed=3)
    K = rng.standard_normal((2, d)).astype(np.float32) * 0.1
    V = np.stack([np.full(d, 1.0), np.full(d, -3.0)]).astype(np.float32)
    u.step(np.zeros(d), K[0], V[0])
    out = u.step(np.zeros(d), K[1], V[1])        # q = 0: exact answer is the mean of the values
    # z = mu/(s) sum_j v/||v||^2 over the slots; with mu = new mu the expectation is v_1 + v_2, tau = 2
    mt = u.m_tok
    w = u.w.astype(np.float64)
    z = sum(u.mu / (u.s * w[e]) * V[e].astype(np.float64) for e in mt)
    np.testing.assert_allclose(out, z / 2.0, rtol=1e-12)
    assert 0 < np.sum(mt == 1) < u.s


# --------------------------------------------------------------------------- brute force with Python integers
def _brute(K, V, delta, t, s, window, seed, unit):
    """The same stream semantics written again with Python integers and Fractions (tiny inputs)."""
    f32 = np.float32
    def d2(x, k):
        return sum(int(f32(f32(a - b) * f32(a - b)) * f32(2 ** 32)) for a, b in zip(x, k))
    def w2(v):
        return sum(int(f32(a * a) * f32(2 ** 24)) for a in v)
    key = [seed & 0xFFFFFFFF, seed >> 32]
    thr = int(Fraction(float(f32(delta))) ** 2 * 2 ** 32)
    cent, cnt, slots, M, mu = [], [], [], [-1] * s, 0
    n = K.shape[0]
    for e in range(max(0, n - window)):
        ds = [d2(K[c], K[e]) for c in cent]
        if ds and min(ds) <= thr:
            i = ds.index(min(ds)); cnt[i] += 1
            for j in range(t):
                if _philox_py([e, unit, j // 4, 0], key)[j % 4] * cnt[i] < 2 ** 32:
                    slots[i][j] = e
        else:
            cent.append(e); cnt.append(1); slots.append([e] * t)
        W = w2(V[e])
        for j in range(s):
            if W and Fraction(_philox_py([e, unit, j // 4, 1], key)[j % 4], 2 ** 32) < Fraction(W, mu + W):
                M[j] = e
        mu += W
    return cent, cnt, slots, M, mu


@pytest.mark.parametrize("window,seed,unit", [(0, 0, 0), (5, 2 ** 40 + 17, 3)])
def test_state_matches_python_integer_enumeration(window, seed, unit):
    rng = np.random.default_rng(13)
    d, n, t, s = 5, 60, 5, 9
    K = _mixture(rng, n, d, 3, 0.5); V = rng.standard_normal((n, d)).astype(np.float32)
    u = orc.OracleUnit(d, 0.45, t, s, window, seed=seed, unit_id=unit)
    u.push_many(K, V)
    cent, cnt, slots, M, mu = _brute(K, V, 0.45, t, s, window, seed, unit)
    assert list(u.centre_tok) == cent and list(u.counts) == cnt
    assert u.slot_tok.tolist() == slots and list(u.m_tok) == M and u.mu == mu
    assert 3 <= u.m < n - window
