"""Pins of the oracle for Section 4.3's augmented variant (tokens with strongly anti-correlated keys are
preserved exactly, the standard procedure runs on the rest).  The paper fixes neither the measure nor
the threshold; the reading -- cosine of a key with the block's mean key at most tau -- is pinned by
hand cases, and the composition by the invariants of Theorem 3.3's estimator."""
import numpy as np

import oracle
from oracle import PreservingOracle, anticorrelated


def test_hand_cases_of_the_anticorrelation_rule():
    # mean of the block = (1, 0): cosines 1, 1, 1, -1 -> only the last key points against the mean
    K = np.array([[2.0, 0.0], [2.0, 0.0], [1.0, 0.0], [-1.0, 0.0]])
    assert anticorrelated(K, -0.5).tolist() == [False, False, False, True]
    assert anticorrelated(K, -1.0).tolist() == [False, False, False, True]     # exact opposite: cosine -1 <= -1
    assert anticorrelated(K, 1.0).tolist() == [True] * 4                       # everything has cosine <= 1
    # orthogonal key: cosine 0 with mean (1, 1)/2 ... keys (1,0), (0,1), (1,1): all positive cosines
    K2 = np.array([[1.0, 0.0], [0.0, 1.0], [1.0, 1.0]])
    assert anticorrelated(K2, 0.0).tolist() == [False, False, False]
    assert anticorrelated(K2, 0.8).tolist() == [True, True, False]             # cos((1,0),(2,2)/3) = 0.7071
    # the rule is the cosine, not the inner product: scaling a key does not change its class
    K3 = np.array([[1.0, 0.2], [1.0, -0.1], [-0.3, 0.05], [-30.0, 5.0], [3.0, 0.0]])
    m = anticorrelated(K3, -0.9)
    mean = K3.mean(0)
    cos = K3 @ mean / (np.linalg.norm(K3, axis=1) * np.linalg.norm(mean))
    assert m.tolist() == (cos <= -0.9).tolist() and m[2] == m[3]
    # a zero key counts as cosine 0
    assert anticorrelated(np.array([[0.0, 0.0], [1.0, 0.0]]), -0.1).tolist() == [False, False]
    assert anticorrelated(np.array([[0.0, 0.0], [1.0, 0.0]]), 0.0).tolist() == [True, False]


def _data(n, d, seed, n_anti):
    rng = np.random.default_rng(seed)
    mu = rng.standard_normal(d)
    K = 0.4 * rng.standard_normal((n, d)) + mu
    where = rng.choice(n, n_anti, replace=False)
    K[where] = -1.5 * mu + 0.1 * rng.standard_normal((n_anti, d))
    return K, rng.standard_normal((n, d)), np.sort(where)


def test_preserved_tokens_keep_weight_one_and_never_enter_a_call():
    d, t, T, n = 16, 32, 2, 32 * 9 + 7
    K, V, where = _data(n, d, 1, 7)
    o = PreservingOracle(d=d, t=t, T=T, tau=-0.5, max_tokens=n, seed=3, c_override=0.5)
    m = o.append(K, V)
    assert np.flatnonzero(m).tolist() == where.tolist()
    o.compress()
    keep, rest = o.views()
    assert np.array_equal(keep[3], where) and np.all(keep[2] == 1.0)
    assert np.array_equal(keep[0], K[where]) and np.array_equal(keep[1], V[where])
    assert not set(rest[3].tolist()) & set(where.tolist())                   # disjoint: a preserved token is in no call
    assert keep[2].sum() + rest[2].sum() == n                                 # Theorem 3.3's weights: tokens seen
    # the rest is exactly the plain BalanceKV stream of the remaining tokens (same coins: layer coordinate 1)
    plain = oracle.OracleStream(oracle.OracleParams(d=d, t=t, T=T, layer=1, head=0, max_tokens=n, seed=3, c_override=0.5))
    plain.append(K[~m], V[~m])
    plain.compress()
    for a, b in zip(plain.view()[:3], rest[:3]):
        assert np.array_equal(a, b)
    assert np.array_equal(np.flatnonzero(~m)[plain.view()[3]], rest[3])


def test_estimate_is_exact_without_compression_and_chunking_respects_the_block_mean():
    d, n = 8, 96
    K, V, _ = _data(n, d, 2, 5)
    q = np.random.default_rng(5).standard_normal((3, d))
    o = PreservingOracle(d=d, t=32, T=0, tau=-0.5, max_tokens=n)
    o.append(K, V)
    assert np.allclose(o.estimate(q), oracle.weighted_attention(K, V, None, q), rtol=1e-12, atol=1e-12)
    # the mean is the appended block's: two appends classify with two means
    o2 = PreservingOracle(d=d, t=32, T=0, tau=-0.5, max_tokens=n)
    m2 = np.concatenate([o2.append(K[:40], V[:40]), o2.append(K[40:], V[40:])])
    assert m2.tolist() == np.concatenate([anticorrelated(K[:40], -0.5), anticorrelated(K[40:], -0.5)]).tolist()
    assert np.allclose(o2.estimate(q), oracle.weighted_attention(K, V, None, q), rtol=1e-12, atol=1e-12)
