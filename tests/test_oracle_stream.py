"""Pins of the oracle's MergeAndReduce driver (Algorithm 3) and of the estimator.

The streaming driver is compared with the offline recursive description the proof of
Theorem 3.3 gives (implemented separately below), and with the invariants the paper states.
"""
import math

import numpy as np
import pytest

import oracle
from oracle import OracleParams, OracleStream
from paper_2502_07861_b200 import synth


def _params(d, t, T, W=0, seed=0, c_override=0.0, n=None, **kw):
    return OracleParams(d=d, t=t, T=T, W=W, seed=seed, c_override=c_override,
                        max_tokens=n if n else 1 << 20, **kw)


def _offline_tree(P: OracleParams, K, V, n_eligible):
    """Offline form: split the eligible prefix into batches of t, halve every batch, merge
    neighbouring halves into batches of the next level, repeat up to level T; an odd batch
    at a level stays in that level's set.  Returns {level: [original indices]}."""
    t, T = P.t, P.T
    p = n_eligible // t
    batches = [list(range(b * t, (b + 1) * t)) for b in range(p)]
    sets = {i: [] for i in range(1, T + 1)}
    level = 0
    while batches and level < T:
        halves = []
        for ordinal, idx in enumerate(batches):
            r = oracle.softmax_balance(P, K[idx], V[idx], ordinal=ordinal, level=level)
            halves.append([idx[j] for j in r["kept"]])
        level += 1
        if level == T:
            for h in halves:
                sets[level] += h
            break
        merged = [halves[2 * l] + halves[2 * l + 1] for l in range(len(halves) // 2)]
        if len(halves) % 2 == 1:
            sets[level] += halves[-1]
        batches = merged
    return sets


@pytest.mark.parametrize("n,t,T,W", [(64, 8, 1, 0), (8 * 13, 8, 3, 0), (16 * 11 + 5, 16, 2, 0),
                                      (16 * 8, 16, 4, 0), (200, 16, 3, 24), (40, 8, 2, 40)])
def test_streaming_tree_equals_offline_recursion(n, t, T, W):
    rng = np.random.default_rng(n + t + T)
    d = 8
    K, V = rng.standard_normal((n, d)), rng.standard_normal((n, d))
    P = _params(d, t, T, W, seed=5, c_override=0.4)
    s = OracleStream(P)
    s.append(K, V)
    s.compress()
    eligible = max(0, n - W)
    sets = _offline_tree(P, K, V, eligible)
    Kc, Vc, w, idx = s.view()
    sizes = s.level_sizes()
    pos = 0
    for lvl in range(T, 0, -1):
        got = list(idx[pos:pos + sizes[lvl]])
        assert got == sets[lvl], (lvl, got, sets[lvl])
        assert np.all(w[pos:pos + sizes[lvl]] == 2.0**lvl)
        pos += sizes[lvl]
    rest = list(range((eligible // t) * t, n))
    assert list(idx[pos:]) == rest and np.all(w[pos:] == 1.0)
    assert np.array_equal(Kc, K[idx]) and np.array_equal(Vc, V[idx])
    assert np.all(np.diff(idx) > 0)


def test_call_schedule_ordinals_and_levels():
    d, t, T = 4, 4, 3
    n = t * 8
    rng = np.random.default_rng(0)
    s = OracleStream(_params(d, t, T))
    s.append(rng.standard_normal((n, d)), rng.standard_normal((n, d)))
    assert s.compress() == 8 + 4 + 2
    got = [(c["level"], c["ordinal"]) for c in s.calls()]
    want = [(0, 0), (0, 1), (1, 0), (0, 2), (0, 3), (1, 1), (2, 0),
            (0, 4), (0, 5), (1, 2), (0, 6), (0, 7), (1, 3), (2, 1)]
    assert got == want
    for c in s.calls():
        assert c["m"] == t and len(c["kept"]) == t // 2
        assert np.all(np.diff(c["idx"]) > 0)
        if c["level"] == 0:
            assert list(c["idx"]) == list(range(c["ordinal"] * t, (c["ordinal"] + 1) * t))


@pytest.mark.parametrize("W", [0, 7])
def test_weights_sum_to_tokens_seen_at_every_step_and_lazy_equals_eager(W):
    rng = np.random.default_rng(1)
    d, t, T, n = 4, 8, 3, 150
    K, V = rng.standard_normal((n, d)), rng.standard_normal((n, d))
    P = _params(d, t, T, W, seed=9, c_override=0.5)
    eager, lazy = OracleStream(P), OracleStream(P)
    for j in range(n):
        eager.append(K[j:j + 1], V[j:j + 1])
        eager.compress()
        _, _, w, idx = eager.view()
        assert w.sum() == j + 1                       # sum_l 2^l |C^l| = tokens seen
        sizes = eager.level_sizes()
        assert all(sizes[l] <= t for l in range(1, T)) and sizes[0] < t + W + 1
        assert set(np.unique(w)) <= {2.0**l for l in range(T + 1)}
        if W:
            assert list(idx[-min(W, j + 1):]) == list(range(j + 1 - min(W, j + 1), j + 1))
            assert np.all(w[-min(W, j + 1):] == 1.0)
    lazy.append(K[:60], V[:60])
    lazy.compress()
    lazy.append(K[60:], V[60:])
    lazy.compress()
    for a, b in zip(eager.view(), lazy.view()):
        assert np.array_equal(a, b)
    assert [(c["level"], c["ordinal"]) for c in eager.calls()] == [(c["level"], c["ordinal"]) for c in lazy.calls()]


def test_tokens_after_the_last_compress_stay_at_weight_one():
    rng = np.random.default_rng(2)
    d, t, T = 4, 8, 2
    s = OracleStream(_params(d, t, T, c_override=0.5))
    s.append(rng.standard_normal((32, d)), rng.standard_normal((32, d)))
    s.compress()
    s.append(rng.standard_normal((20, d)), rng.standard_normal((20, d)))   # e.g. decode-phase tokens
    _, _, w, idx = s.view()
    assert list(idx[-20:]) == list(range(32, 52)) and np.all(w[-20:] == 1) and w.sum() == 52


def test_forced_signs_drive_the_tree():
    rng = np.random.default_rng(3)
    d, t, T = 4, 8, 2
    K, V = rng.standard_normal((16, d)), rng.standard_normal((16, d))
    s = OracleStream(_params(d, t, T))
    s.force_eta(0, 0, [1, -1, -1, -1, -1, -1, -1, 1])     # keeps 0, 7 + latest two of the rest: 5, 6
    s.force_eta(0, 1, [-1] * 4 + [1] * 4)                 # tie -> +1 class: 12..15
    s.force_eta(1, 0, [1, 1, 1, 1, -1, -1, -1, -1])       # tie -> first four
    s.append(K, V)
    s.compress()
    calls = s.calls()
    assert list(calls[0]["kept"]) == [0, 5, 6, 7]
    assert list(calls[2]["idx"]) == [0, 5, 6, 7, 12, 13, 14, 15]
    _, _, w, idx = s.view()
    assert list(idx) == [0, 5, 6, 7] and np.all(w == 4.0)


def test_estimator_error_is_small_and_inside_theorem_3_3_style_bound():
    """z_j = sum_l 2^l sum_{C^l} e^{<k,q>/sqrt d} v against the full sum: the error of each
    level-l call is at most 2^l times the Theorem 3.2 bound (explicit constant c, plus the
    strict-half completion term), summed over the calls (triangle inequality of the proof)."""
    rng = np.random.default_rng(4)
    d, t, T, n = 8, 32, 2, 32 * 8
    K, V = 0.8 * rng.standard_normal((n, d)), rng.standard_normal((n, d))
    P = _params(d, t, T, seed=2, c_override=0.5)
    s = OracleStream(P)
    s.append(K, V)
    s.compress()
    Kc, Vc, w, _ = s.view()
    for _ in range(20):
        q = rng.standard_normal(d)
        q *= 0.9 * math.sqrt(min(c["rk2"] for c in s.calls())) / np.linalg.norm(q)
        full = np.exp(K @ q / math.sqrt(d)) @ V
        est = (w * np.exp(Kc @ q / math.sqrt(d))) @ Vc
        bound = 0.0
        for c in s.calls():
            kk, vv = K[c["idx"]], V[c["idx"]]
            plus, minus = (c["eta"] > 0).sum(), (c["eta"] < 0).sum()
            deficit = t // 2 - min(plus, minus)
            walk = math.sqrt(d) * c["c"] * math.exp((q @ q) / (2 * math.sqrt(d)) + c["rk2"] / (2 * math.sqrt(d))) * math.sqrt(c["rv2"])
            fix = 2 * deficit * np.max(np.exp(kk @ q / math.sqrt(d)) * np.linalg.norm(vv, axis=1))
            bound += 2.0 ** c["level"] * (walk + fix)
        assert np.linalg.norm(full - est) <= bound


def test_balancekv_beats_uniform_sampling_on_clustered_keys():
    """Qualitative expectation of the single-layer experiment (Fig. 1): at equal rate, the
    walk (with a constant small enough to matter) has lower attention error than keeping a
    uniformly random half, averaged over seeds, on keys with near-duplicates."""
    rng = np.random.default_rng(5)
    d, t, T, n = 16, 64, 1, 256
    unit = lambda a: a / np.linalg.norm(a, axis=1, keepdims=True)
    centers = 6.0 * unit(rng.standard_normal((8, d)))        # equal norms: G-hat ~ 1 inside a cluster
    lab = rng.integers(0, 8, n)
    K = centers[lab] + 0.02 * rng.standard_normal((n, d))
    V = unit(rng.standard_normal((8, d)))[lab] + 0.02 * rng.standard_normal((n, d))
    qs = 0.5 * (centers[:4] + centers[4:])                   # queries that mix two clusters
    exact = oracle.weighted_attention(K, V, None, qs)
    err_walk, err_unif = [], []
    for seed in range(30):
        s = OracleStream(_params(d, t, T, seed=seed, c_override=0.25))
        s.append(K, V)
        s.compress()
        z = s.decode(qs)
        err_walk.append(np.linalg.norm(z - exact) / np.linalg.norm(exact))
        keep = np.sort(np.random.default_rng(100 + seed).choice(n, n // 2, replace=False))
        zu = oracle.weighted_attention(K[keep], V[keep], None, qs)
        err_unif.append(np.linalg.norm(zu - exact) / np.linalg.norm(exact))
    assert np.mean(err_walk) < 0.8 * np.mean(err_unif)


def test_tiny_config_shape_512_kept_all_weight_two():
    """The tiny single-head case: 1024 tokens in blocks of 256, T=1 -> 4 calls, 512 kept."""
    K, V = synth.stream_kv("outlier2", 1001, 0, 0, 0, 1024, 64, "fp32")
    s = OracleStream(OracleParams(d=64, t=256, T=1, max_tokens=1024, seed=0))
    s.append(K, V)
    assert s.compress() == 4
    _, _, w, idx = s.view()
    assert len(idx) == 512 and np.all(w == 2.0) and w.sum() == 1024
    assert sum(c["fails"] for c in s.calls()) == 0
    for c in s.calls():
        assert np.all(np.abs(c["S"]) <= c["c"]) and np.all((c["p"] >= 0) & (c["p"] <= 1))
