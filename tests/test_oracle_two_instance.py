"""Pins of the oracle's form of Algorithm 1 with a separate denominator instance: the numerator
comes from MergeAndReduce on (k_j, v_j), the denominator from a second MergeAndReduce on
(k_j, 1) (here the unit value (1, 0, ..., 0), whose pairwise kernel is exp(<k_i,k_j>/sqrt d))."""
import math

import numpy as np
import pytest

import oracle
from oracle import OracleParams, OracleStream


def _unit(n, d):
    E = np.zeros((n, d))
    E[:, 0] = 1.0
    return E


def test_unnormalised_sums_against_a_direct_evaluation_and_the_pinned_ratio():
    rng = np.random.default_rng(0)
    n, d = 37, 8
    K, V, w = rng.standard_normal((n, d)), rng.standard_normal((n, d)), 2.0 ** rng.integers(0, 4, n)
    q = rng.standard_normal((3, d))
    num, den, mx = oracle.weighted_sums(K, V, w, q)
    e = w[None, :] * np.exp(q @ K.T / math.sqrt(d))                    # written out, no max shift
    assert np.allclose(num * np.exp(mx)[:, None], e @ V, rtol=1e-12)
    assert np.allclose(den * np.exp(mx), e.sum(1), rtol=1e-12)
    assert np.allclose(num / den[:, None], oracle.weighted_attention(K, V, w, q), rtol=1e-12, atol=1e-15)
    assert np.allclose(mx, np.max(q @ K.T / math.sqrt(d) + np.log(w)[None, :], axis=1))
    # large logits: the shifted form stays finite where the plain one overflows
    num2, den2, mx2 = oracle.weighted_sums(60.0 * K, V, None, q)
    assert np.all(np.isfinite(num2)) and np.all(den2 >= 1.0) and np.all(den2 <= n)


def test_denominator_instance_walks_on_the_key_kernel_alone():
    """(k, 1): S_j = sum_{i<j} eta_i exp((<k_i,k_j> - r_key^2)/sqrt d), written out in numpy."""
    rng = np.random.default_rng(1)
    m, d = 24, 8
    K = 0.9 * rng.standard_normal((m, d))
    P = OracleParams(d=d, t=m, T=1, max_tokens=1024, seed=3, c_override=0.7)
    r = oracle.softmax_balance(P, K, _unit(m, d))
    assert r["rv2"] == 1.0
    rk2 = np.max(np.sum(K * K, axis=1))
    G = np.exp((K @ K.T - rk2) / math.sqrt(d))
    S = np.array([np.clip(np.dot(G[j, :j], r["eta"][:j]), -0.7, 0.7) for j in range(m)])
    assert np.allclose(r["S"], S, atol=1e-13) and np.allclose(r["p"], 0.5 - S / 1.4, atol=1e-13)
    assert np.array_equal(r["eta"], np.where(r["u"] < r["p"], 1, -1))


def test_T0_two_instances_give_exact_attention_and_equal_subsets_give_the_shared_ratio():
    rng = np.random.default_rng(2)
    n, d, t = 64, 8, 16
    K, V = rng.standard_normal((n, d)), rng.standard_normal((n, d))
    q = rng.standard_normal((4, d))
    exact = oracle.weighted_attention(K, V, None, q)
    a, b = OracleStream(OracleParams(d=d, t=t, T=0, layer=0)), OracleStream(OracleParams(d=d, t=t, T=0, layer=1))
    a.append(K, V); b.append(K, _unit(n, d)); a.compress(); b.compress()
    assert np.allclose(oracle.two_instance_estimate(a.view(), b.view(), q), exact, rtol=1e-12, atol=1e-14)
    # forcing the same signs in both instances selects the same subset: Algorithm 1's ratio then
    # equals the ratio over one shared set
    eta = [np.where(rng.random(t) < 0.5, 1, -1) for _ in range(n // t)]
    a, b = OracleStream(OracleParams(d=d, t=t, T=1, layer=0)), OracleStream(OracleParams(d=d, t=t, T=1, layer=1))
    for o, e in enumerate(eta):
        a.force_eta(0, o, e); b.force_eta(0, o, e)
    a.append(K, V); b.append(K, _unit(n, d)); a.compress(); b.compress()
    assert np.array_equal(a.view()[3], b.view()[3])
    Ka, Va, wa, _ = a.view()
    assert np.allclose(oracle.two_instance_estimate(a.view(), b.view(), q), oracle.weighted_attention(Ka, Va, wa, q),
                       rtol=1e-12, atol=1e-14)


def test_instances_draw_independent_coins_and_keep_their_own_subsets():
    rng = np.random.default_rng(3)
    n, d, t = 128, 8, 32
    K, V = rng.standard_normal((n, d)), rng.standard_normal((n, d))
    a, b = OracleStream(OracleParams(d=d, t=t, T=2, layer=0, seed=5)), OracleStream(OracleParams(d=d, t=t, T=2, layer=1, seed=5))
    a.append(K, V); b.append(K, _unit(n, d)); a.compress(); b.compress()
    ia, ib = a.view()[3], b.view()[3]
    assert len(ia) == len(ib) == n // 4 and not np.array_equal(ia, ib)
    assert a.view()[2].sum() == n and b.view()[2].sum() == n           # both estimators count every token
    ua = np.concatenate([c["u"] for c in a.calls()])
    ub = np.concatenate([c["u"] for c in b.calls()])
    assert not np.any(ua == ub)                                         # the slot index enters the coin's counter


def test_denominator_discrepancy_inside_the_theorem_3_2_style_bound():
    """|sum_j eta_j e^{<k_j,q>/sqrt d}| <= sqrt(s) c e^{|q|^2/(2 sqrt d)} e^{r_key^2/(2 sqrt d)} r_value for |q| <= r_key,
    with the explicit constant c, r_value = 1 and s = d (the unit values are stored as vectors of
    R^d), the same reading of Theorem 3.2 as the numerator's pin."""
    rng = np.random.default_rng(4)
    m, d = 64, 8
    K = 0.8 * rng.standard_normal((m, d))
    P = OracleParams(d=d, t=m, T=1, max_tokens=1024, seed=1, c_override=0.5)
    r = oracle.softmax_balance(P, K, _unit(m, d))
    assert r["fails"] == 0
    for _ in range(50):
        q = rng.standard_normal(d)
        q *= rng.random() * math.sqrt(r["rk2"]) / np.linalg.norm(q)
        lhs = abs(np.dot(r["eta"], np.exp(K @ q / math.sqrt(d))))
        assert lhs <= math.sqrt(d) * 0.5 * math.exp((q @ q) / (2 * math.sqrt(d)) + r["rk2"] / (2 * math.sqrt(d)))


def test_merged_estimate_over_a_partition_equals_the_estimate_over_the_whole_set():
    """Splitting a weighted set into slots and merging their un-normalised parts changes nothing
    (up to rounding), whatever the split and however different the slots' largest logits."""
    rng = np.random.default_rng(5)
    n, d = 90, 8
    K, V, w = 3.0 * rng.standard_normal((n, d)), rng.standard_normal((n, d)), 2.0 ** rng.integers(0, 3, n)
    q = rng.standard_normal((5, d))
    whole = oracle.weighted_attention(K, V, w, q)
    cuts = [0, 7, 40, 40, 90]                                  # one slot is empty
    views = [(K[a:b], V[a:b], w[a:b]) for a, b in zip(cuts[:-1], cuts[1:])]
    assert np.allclose(oracle.merged_estimate(views, views, q), whole, rtol=1e-12, atol=1e-14)
    # one numerator and one denominator view: the two-instance form
    assert np.allclose(oracle.merged_estimate([views[1]], [views[3]], q),
                       oracle.two_instance_estimate(views[1], views[3], q), rtol=1e-12, atol=1e-14)


def test_first_tokens_kept_exactly_beside_a_compressed_middle():
    """The single-layer setting of Appendix B: the first tokens and a recent window at weight 1, the
    walk on the tokens in between; every token is counted once, and with T = 0 the result is exact."""
    rng = np.random.default_rng(6)
    n, d, t, sink, W = 200, 8, 16, 24, 10
    K, V = rng.standard_normal((n, d)), rng.standard_normal((n, d))
    q = rng.standard_normal((3, d))
    for T in (0, 2):
        head = OracleStream(OracleParams(d=d, t=t, T=T, layer=0))        # never compressed
        rest = OracleStream(OracleParams(d=d, t=t, T=T, W=W, layer=1, c_override=0.5))
        head.append(K[:sink], V[:sink])
        rest.append(K[sink:], V[sink:])
        rest.compress()
        views = [head.view(), rest.view()]
        assert views[0][2].sum() + views[1][2].sum() == n
        assert np.all(views[1][2][-W:] == 1.0)
        z = oracle.merged_estimate(views, views, q)
        if T == 0:
            assert np.allclose(z, oracle.weighted_attention(K, V, None, q), rtol=1e-12, atol=1e-14)
        else:
            assert len(views[1][3]) < n - sink and np.all(np.isfinite(z))
