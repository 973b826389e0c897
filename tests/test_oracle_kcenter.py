"""Pins of the oracle's greedy k-center compression (Section 3.2 variant) against textbook facts."""
import itertools

import numpy as np
import scipy.special

from oracle import subgen_oracle as orc


def _radius(K, centres):
    d = np.linalg.norm(K[:, None, :].astype(np.float64) - K[centres][None].astype(np.float64), axis=2)
    return d.min(axis=1).max()


def test_each_centre_is_the_farthest_point_from_the_earlier_ones():
    rng = np.random.default_rng(1)
    K = rng.standard_normal((300, 12)).astype(np.float32)
    cent, rad2 = orc.kcenter(K, 20)
    assert cent[0] == 0 and len(set(cent.tolist())) == 20
    K64 = K.astype(np.float64)
    for t in range(1, 20):
        dist = np.linalg.norm(K64[:, None] - K64[cent[:t]][None], axis=2).min(axis=1)
        assert dist[cent[t]] >= dist.max() * (1 - 1e-6)          # farthest-point rule
    np.testing.assert_allclose(np.sqrt(rad2 / 2 ** 32), _radius(K, cent), rtol=1e-5)


def test_two_approximation_of_the_optimal_radius():
    """Gonzalez: the greedy covering radius is at most twice the optimum (brute force over all k-subsets)."""
    rng = np.random.default_rng(2)
    for n, k in ((9, 2), (10, 3), (8, 4)):
        K = rng.standard_normal((n, 3)).astype(np.float32)
        cent, _ = orc.kcenter(K, k)
        opt = min(_radius(K, list(c)) for c in itertools.combinations(range(n), k))
        assert _radius(K, cent) <= 2 * opt * (1 + 1e-6)


def test_separated_clusters_get_one_centre_each_and_ties_take_the_lowest_index():
    rng = np.random.default_rng(3)
    means = 50 * np.eye(6, 8)
    lab = rng.integers(0, 6, 200); lab[:6] = np.arange(6)
    K = (means[lab] + 0.01 * rng.standard_normal((200, 8))).astype(np.float32)
    cent, rad2 = orc.kcenter(K, 6)
    assert sorted(lab[cent].tolist()) == list(range(6)) and np.sqrt(rad2 / 2 ** 32) < 0.2
    Kt = np.array([[0, 0], [1, 0], [-1, 0], [0, 1]], np.float32)      # rows 1, 2, 3 are equally far from row 0
    cent, _ = orc.kcenter(Kt, 2)
    assert cent.tolist() == [0, 1]


def test_keeping_everything_is_exact_attention_and_kept_tokens_are_centres_then_window():
    rng = np.random.default_rng(4)
    n, d = 40, 6
    K = rng.standard_normal((n, d)).astype(np.float32); V = rng.standard_normal((n, d)).astype(np.float32)
    q = rng.standard_normal(d).astype(np.float32)
    full = scipy.special.softmax(K.astype(np.float64) @ q.astype(np.float64)) @ V.astype(np.float64)
    out, keep = orc.kcenter_window_attention(K, V, q, 100, 10)           # k >= n - r: every token kept
    assert sorted(keep.tolist()) == list(range(n))
    np.testing.assert_allclose(out, full, rtol=1e-11)
    out, keep = orc.kcenter_window_attention(K, V, q, 5, 8)
    assert len(keep) == 13 and keep[-8:].tolist() == list(range(32, 40)) and keep[0] == 0 and keep[:5].max() < 32
    sub = scipy.special.softmax(K[keep].astype(np.float64) @ q.astype(np.float64)) @ V[keep].astype(np.float64)
    np.testing.assert_allclose(out, sub, rtol=1e-11)
    out, keep = orc.kcenter_window_attention(K, V, q, 5, 64)             # window covers the stream
    assert keep.tolist() == list(range(n))
