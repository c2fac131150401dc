"""Pins of the oracle's value-norm buckets (Algorithm 1: bucketing step, erasure of small-norm
buckets, union of the instances' sets in the numerator of the output ratio)."""
import math

import numpy as np
import pytest

import oracle
from oracle import BucketedOracle, OracleParams, OracleStream, value_bucket


def _unit(n, d):
    E = np.zeros((n, d))
    E[:, 0] = 1.0
    return E


def _with_norm(rng, d, norm):
    v = rng.standard_normal(d)
    return v * (norm / np.linalg.norm(v))


def test_bucket_index_hand_cases():
    """2^(i-1) < ||v|| <= 2^i, norms written out by hand."""
    e = np.zeros(4)
    for norm, i in ((1.0, 0), (1.0001, 1), (2.0, 1), (2.0001, 2), (3.0, 2), (4.0, 2), (0.75, 0), (0.5, -1),
                    (0.5001, 0), (0.3, -1), (0.25, -2), (1000.0, 10), (1024.0, 10), (1025.0, 11)):
        e[2] = norm
        assert value_bucket(e) == i, norm
    assert value_bucket(np.array([3.0, 4.0])) == 3            # norm 5
    assert value_bucket(np.array([1.0, 1.0, 1.0, 1.0])) == 1  # norm 2: the boundary belongs to the lower index
    assert value_bucket(np.zeros(8)) == oracle.NO_BUCKET


def test_bucket_index_brackets_the_norm_and_shifts_with_scaling():
    rng = np.random.default_rng(0)
    for _ in range(300):
        v = rng.standard_normal(16) * 10.0 ** rng.uniform(-3, 3)
        i = value_bucket(v)
        nrm = math.sqrt(math.fsum(x * x for x in v))
        assert 2.0 ** (i - 1) < nrm <= 2.0 ** i
        assert value_bucket(2.0 * v) == i + 1 and value_bucket(0.25 * v) == i - 2


def _mixed_stream(rng, n, d, lo=-6, hi=2):
    K = 0.5 * rng.standard_normal((n, d))
    V = np.stack([_with_norm(rng, d, 2.0 ** rng.uniform(lo, hi)) for _ in range(n)])
    return K, V


def test_every_token_lands_in_exactly_one_bucket_or_is_dropped():
    rng = np.random.default_rng(1)
    n, d = 200, 8
    K, V = _mixed_stream(rng, n, d)
    V[17] = 0.0
    o = BucketedOracle(d=d, t=16, T=1, i_top=2, n_buckets=5, erase_ratio=2.0 ** -5.5, max_tokens=n)
    o.append(K, V)
    seen = sorted(o.erased + [j for r in o.route.values() for j in r])
    assert seen == list(range(n))
    assert 17 in o.erased
    for b, r in o.route.items():
        assert r == sorted(r)
        for j in r:
            assert value_bucket(V[j]) == 2 - b


def test_final_state_equals_the_closed_form_of_the_erase_rule():
    """The threshold only grows, so after the stream the surviving buckets are exactly those with
    2^i > rho * max_j ||v_j|| (and inside the instantiated range), each holding all of its tokens."""
    rng = np.random.default_rng(2)
    n, d, i_top, nb = 300, 8, 3, 6
    for rho in (0.0, 2.0 ** -7.3, 2.0 ** -4.5, 2.0 ** -2.5):
        K, V = _mixed_stream(rng, n, d, lo=-7, hi=3)
        o = BucketedOracle(d=d, t=32, T=0, i_top=i_top, n_buckets=nb, erase_ratio=rho, max_tokens=n)
        o.append(K, V)
        vmax = max(np.linalg.norm(v) for v in V)
        want = {}
        for j, v in enumerate(V):
            i = math.ceil(math.log2(np.linalg.norm(v)))
            if 2.0 ** i > rho * vmax and i_top - i < nb:
                want.setdefault(i_top - i, []).append(j)
        assert o.route == want


def test_chunking_of_the_stream_does_not_change_routes_or_erasure():
    rng = np.random.default_rng(3)
    n, d = 257, 8
    K, V = _mixed_stream(rng, n, d)
    # norms grow along the stream so that buckets are erased in the middle of it
    V *= (2.0 ** np.linspace(-4, 0, n))[:, None]
    ref = None
    for cuts in ([n], [1] * n, [100, 57, 100], [3, 250, 4]):
        o = BucketedOracle(d=d, t=16, T=2, i_top=2, n_buckets=8, erase_ratio=2.0 ** -4.2, max_tokens=n, c_override=0.5)
        p = 0
        for c in cuts:
            o.append(K[p:p + c], V[p:p + c])
            p += c
        o.compress()
        state = (o.route, sorted(o.erased), [tuple(v[3]) for v in o.views()])
        if ref is None:
            ref = state
            assert len(o.erased) > 0 and len(o.route) >= 3
        assert state == ref


def test_T0_without_erasure_is_exact_attention():
    rng = np.random.default_rng(4)
    n, d = 96, 8
    K, V = _mixed_stream(rng, n, d, lo=-3, hi=2)
    q = rng.standard_normal((5, d))
    o = BucketedOracle(d=d, t=16, T=0, i_top=2, n_buckets=8, max_tokens=n)
    o.append(K, V)
    den = OracleStream(OracleParams(d=d, t=16, T=0, layer=9, max_tokens=n))
    den.append(K, _unit(n, d))
    assert len(o.erased) == 0 and len(o.views()) >= 4
    assert np.allclose(o.estimate(q, [den.view()]), oracle.weighted_attention(K, V, None, q), rtol=1e-12, atol=1e-14)


def test_erased_part_is_the_dropped_term_and_obeys_the_bound_in_the_proof_of_theorem_1_1():
    """With T = 0 the only error is the erased buckets' term of the numerator; its norm is at most
    rho * v_max (weighted average of norms <= 2^i <= rho * v_max)."""
    rng = np.random.default_rng(5)
    n, d = 400, 8
    K, V = _mixed_stream(rng, n, d, lo=-9, hi=1)
    q = rng.standard_normal((6, d))
    eps = 0.5
    rho = eps / math.sqrt(n)
    o = BucketedOracle(d=d, t=16, T=0, i_top=1, n_buckets=12, erase_ratio=rho, max_tokens=n)
    o.append(K, V)
    den = OracleStream(OracleParams(d=d, t=16, T=0, layer=20, max_tokens=n))
    den.append(K, _unit(n, d))
    assert 0 < len(o.erased) < n
    e = np.exp(q @ K.T / math.sqrt(d))
    dropped = (e[:, o.erased] @ V[o.erased]) / e.sum(1)[:, None]
    exact = (e @ V) / e.sum(1)[:, None]
    est = o.estimate(q, [den.view()])
    assert np.allclose(exact - est, dropped, rtol=1e-10, atol=1e-14)
    vmax = max(np.linalg.norm(v) for v in V)
    assert np.all(np.linalg.norm(dropped, axis=1) <= rho * vmax)
    # ... which is within the error budget of Eq. (2): eps * ||softmax||_2 * ||V||_F
    sm = e / e.sum(1)[:, None]
    assert np.all(np.linalg.norm(dropped, axis=1) <= eps * np.linalg.norm(sm, axis=1) * np.linalg.norm(V))


def test_bucket_instances_are_independent_merge_and_reduce_runs_with_their_own_coins():
    rng = np.random.default_rng(6)
    n, d, t = 256, 8, 16
    K, V = _mixed_stream(rng, n, d, lo=-1.9, hi=1.9)
    o = BucketedOracle(d=d, t=t, T=2, i_top=2, n_buckets=4, layer0=3, head=1, seed=7, max_tokens=n, c_override=0.4)
    o.append(K, V)
    o.compress()
    tot = 0.0
    for b, view in zip(sorted(o.inst), o.views()):
        r = np.asarray(o.route[b])
        # Theorem 3.3's weights: the bucket's sets still stand for every token it received
        assert view[2].sum() == len(r)
        tot += view[2].sum()
        assert np.all(np.isin(view[3], r)) and np.all(np.diff(view[3][view[2] == view[2].max()]) > 0)
        # coins of slot b are keyed by layer0 + b: the first level-0 call replays from Philox alone
        calls = [c for c in o.inst[b].calls() if c["level"] == 0 and c["ordinal"] == 0]
        if calls:
            u = [oracle.walk_uniform(7, 3 + b, 1, 0, 0, j) for j in range(t)]
            assert np.allclose(calls[0]["u"], u, atol=0)
    assert tot + len(o.erased) == n


def test_a_norm_above_the_top_bucket_is_refused():
    o = BucketedOracle(d=4, t=16, T=1, i_top=0, n_buckets=2)
    with pytest.raises(ValueError):
        o.append(np.zeros((1, 4)), np.array([[1.5, 0, 0, 0]]))
