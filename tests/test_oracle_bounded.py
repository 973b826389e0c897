"""Pins of the oracle's bounded-m variant (cluster budget with threshold doubling and merging).

The paper fixes no rule for an exhausted budget, so these pins check what any such rule must keep (the properties
of Lemma 2 that the estimator relies on, with the threshold in force), that the variant is Algorithm 1 unchanged
while the budget is not reached, and the reading itself against a second statement in Python integers.
"""
import os
import sys
from fractions import Fraction

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))

import numpy as np
import pytest
from scipy import stats

from oracle import subgen_oracle as orc


def _mixture(rng, n, d, ncomp, sigma, spread=1.0):
    cent = spread * rng.standard_normal((ncomp, d))
    return (cent[rng.integers(0, ncomp, n)] + sigma / np.sqrt(d) * rng.standard_normal((n, d))).astype(np.float32)


def _state(u):
    return (u.m, u.mu, u.counts.tolist(), u.centre_tok.tolist(), u.slot_tok.tolist(), u.m_tok.tolist(), u.assign.tolist())


def test_unreached_budget_is_algorithm_1_unchanged():
    rng = np.random.default_rng(3)
    K = _mixture(rng, 400, 16, 9, 0.2); V = rng.standard_normal((400, 16)).astype(np.float32)
    a = orc.OracleUnit(16, 0.5, 4, 16, 7, seed=5, unit_id=2, m_max=64)
    b = orc.OracleUnit(16, 0.5, 4, 16, 7, seed=5, unit_id=2, m_max=64, bounded=True)
    a.push_many(K, V); b.push_many(K, V)
    assert a.m < 64 and _state(a) == _state(b)
    assert b.level == 0 and b.thr2_fx == b.delta2_fx


@pytest.mark.parametrize("window,m_max", [(0, 5), (6, 12), (0, 1)])
def test_budget_holds_and_lemma2_properties_survive_merging(window, m_max):
    rng = np.random.default_rng(11)
    n, d, t = 600, 12, 6
    K = _mixture(rng, n, d, 40, 0.3); V = rng.standard_normal((n, d)).astype(np.float32)
    u = orc.OracleUnit(d, 0.4, t, 8, window, seed=9, unit_id=1, m_max=m_max, bounded=True)
    levels = []
    for i in range(n):
        u.push(K[i], V[i])                      # never raises: the budget is not an error any more
        assert u.m <= m_max
        levels.append(u.level)
    assert u.overflow_at == -1 and u.level >= 1 and levels == sorted(levels)
    # the threshold in force is delta^2 * 4^level in fixed point
    assert u.thr2_fx == u.delta2_fx * 4 ** u.level
    ins = u.inserted
    assign, cent, cnt, slots = u.assign[:ins], u.centre_tok, u.counts, u.slot_tok
    assert ins == n - window and cnt.sum() == ins
    # (1) counts are the cluster sizes, (2) the representative is a member, its first one
    for c in range(u.m):
        members = np.flatnonzero(assign == c)
        assert len(members) == cnt[c] and cent[c] == members[0]
        # (5) every sample is a member
        assert set(slots[c].tolist()) <= set(members.tolist())
    # (4) representatives are pairwise farther apart than the threshold in force
    for a in range(u.m):
        for b in range(a):
            assert orc.dist2_fx(K[cent[a]], K[cent[b]]) > u.thr2_fx
    # (3) members lie within twice the threshold radius of their representative: a member joined within the
    # threshold of its time and every later merge moved its representative by at most the threshold of that
    # time; thresholds double, so the distances sum to less than twice the last one
    r_now = np.sqrt(u.thr2_fx / 2.0 ** 32)
    dist = np.linalg.norm(K[:ins].astype(np.float64) - K[cent[assign]].astype(np.float64), axis=1)
    assert dist.max() <= 2.0 * r_now * (1 + 1e-6)
    # mu and M are untouched by merging: same as the unbounded structure on the same stream
    ref = orc.OracleUnit(d, 0.4, t, 8, window, seed=9, unit_id=1, m_max=n)
    ref.push_many(K, V)
    assert ref.mu == u.mu and ref.m_tok.tolist() == u.m_tok.tolist()


def _philox_py(ctr, key):
    c = list(ctr); k = list(key)
    for r in range(10):
        if r:
            k = [(k[0] + 0x9E3779B9) & 0xFFFFFFFF, (k[1] + 0xBB67AE85) & 0xFFFFFFFF]
        p0 = 0xD2511F53 * c[0]; p1 = 0xCD9E8D57 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k[0], p1 & 0xFFFFFFFF, (p0 >> 32) ^ c[3] ^ k[1], p0 & 0xFFFFFFFF]
    return c


def _brute_bounded(K, delta, t, window, seed, unit, m_max):
    """The clustering half of the bounded variant written again with Python integers and Fractions."""
    f32 = np.float32
    def d2(x, k):
        return sum(int(f32(f32(a - b) * f32(a - b)) * f32(2 ** 32)) for a, b in zip(x, k))
    key = [seed & 0xFFFFFFFF, seed >> 32]
    thr = int(Fraction(float(f32(delta))) ** 2 * 2 ** 32)
    cent, cnt, slots, level = [], [], [], 0
    for e in range(max(0, K.shape[0] - window)):
        while True:
            ds = [d2(K[c], K[e]) for c in cent]
            if ds and min(ds) <= thr:
                i = ds.index(min(ds)); cnt[i] += 1
                for j in range(t):
                    if _philox_py([e, unit, j // 4, 0], key)[j % 4] * cnt[i] < 2 ** 32:
                        slots[i][j] = e
                break
            if len(cent) < m_max:
                cent.append(e); cnt.append(1); slots.append([e] * t)
                break
            level += 1
            thr = max(4 * thr, 1)
            kc, kn, ks = [], [], []
            for i in range(len(cent)):
                ds = [d2(K[c], K[cent[i]]) for c in kc]
                if ds and min(ds) <= thr:
                    j = ds.index(min(ds))
                    total = kn[j] + cnt[i]
                    for q in range(t):
                        word = _philox_py([e, unit, q // 4 + 256 * i, 2 + 4 * level], key)[q % 4]
                        if Fraction(word, 2 ** 32) < Fraction(cnt[i], total):
                            ks[j][q] = slots[i][q]
                    kn[j] = total
                else:
                    kc.append(cent[i]); kn.append(cnt[i]); ks.append(list(slots[i]))
            cent, cnt, slots = kc, kn, ks
    return cent, cnt, slots, level, thr


@pytest.mark.parametrize("window,seed,unit,m_max", [(0, 0, 0, 4), (3, 2 ** 41 + 5, 6, 7)])
def test_bounded_state_matches_python_integer_enumeration(window, seed, unit, m_max):
    rng = np.random.default_rng(21)
    d, n, t = 4, 90, 5
    K = _mixture(rng, n, d, 12, 0.4); V = rng.standard_normal((n, d)).astype(np.float32)
    u = orc.OracleUnit(d, 0.35, t, 4, window, seed=seed, unit_id=unit, m_max=m_max, bounded=True)
    u.push_many(K, V)
    cent, cnt, slots, level, thr = _brute_bounded(K, 0.35, t, window, seed, unit, m_max)
    assert level >= 2
    assert (u.centre_tok.tolist(), u.counts.tolist(), u.slot_tok.tolist(), u.level, u.thr2_fx) == (cent, cnt, slots, level, thr)


def test_samples_stay_uniform_over_merged_clusters():
    """Property (5) of Lemma 2 after merges: a slot of a cluster is uniform over ALL its members, whichever of the
    merged clusters they first belonged to. Cluster membership does not depend on the coins, so the law can be
    tested over seeds."""
    rng = np.random.default_rng(4)
    n, d, t, m_max = 60, 3, 2, 3
    K = _mixture(rng, n, d, 8, 0.3); V = np.ones((n, d), np.float32)
    seeds = 3000
    first = None
    hits = None
    for sd in range(seeds):
        u = orc.OracleUnit(d, 0.3, t, 1, 0, seed=sd, unit_id=0, m_max=m_max, bounded=True)
        u.push_many(K, V)
        if first is None:
            first = (u.assign.copy(), u.counts.copy(), u.level)
            hits = np.zeros((u.m, t, n))
        assert np.array_equal(u.assign, first[0])
        for c in range(u.m):
            for q in range(t):
                hits[c, q, u.slot_tok[c, q]] += 1
    assign, counts, level = first
    assert level >= 1 and counts.max() >= 10
    for c in range(len(counts)):
        members = np.flatnonzero(assign == c)
        if len(members) < 2:
            continue
        for q in range(t):
            assert hits[c, q].sum() == hits[c, q, members].sum() == seeds
            p = stats.chisquare(hits[c, q, members]).pvalue
            assert p > 1e-4, "cluster %d slot %d: p = %.2g" % (c, q, p)


def test_partition_function_estimate_stays_unbiased_under_merging():
    """tau-hat = sum_i n_i / t sum_{k in S_i} exp<q,k> is unbiased for any partition with uniform samples."""
    rng = np.random.default_rng(8)
    n, d, t, m_max = 80, 4, 3, 4
    K = _mixture(rng, n, d, 10, 0.5, spread=0.7); V = np.ones((n, d), np.float32)
    q = (0.5 * rng.standard_normal(d)).astype(np.float32)
    exact = np.exp(K.astype(np.float64) @ q.astype(np.float64)).sum()
    taus = []
    for sd in range(1500):
        u = orc.OracleUnit(d, 0.3, t, 1, 0, seed=sd, unit_id=3, m_max=m_max, bounded=True)
        u.push_many(K, V)
        _, _, tau, shift = u.query_parts(q)
        taus.append(tau * np.exp(shift))
    taus = np.array(taus)
    assert u.level >= 1
    se = taus.std(ddof=1) / np.sqrt(len(taus))
    assert abs(taus.mean() - exact) <= 4.5 * se, (taus.mean(), exact, se)
    assert se > 0          # there is sampling noise to average over: the clusters are not singletons
