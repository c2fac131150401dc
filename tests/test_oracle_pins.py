"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests re-types the oracle's own loop: each compares it with a closed form,
an invariant, a library routine, a known-answer vector or a brute-force enumeration
written independently here in numpy.
"""
import ctypes
import glob
import itertools
import math
import os

import numpy as np
import pytest

import oracle
from oracle import OracleParams, OracleStream

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# --------------------------------------------------------------------------- RNG
def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) if l[0] != "#"]
    assert len(rows) >= 2
    for r in rows:
        v = [int(x, 16) for x in r]
        out = oracle.philox4x32_10(v[4:6], v[0:4])
        assert [int(x) for x in out] == v[6:10]


def _curand():
    pats = ["/usr/local/cuda/lib64/libcurand.so*"]
    try:
        import nvidia.curand  # type: ignore

        pats.append(os.path.join(os.path.dirname(nvidia.curand.__path__[0]), "curand/lib/libcurand.so*"))
    except Exception:
        pass
    for p in pats:
        for f in sorted(glob.glob(p)):
            if "stubs" in f:
                continue
            try:
                return ctypes.CDLL(f)
            except OSError:
                continue
    return None


def test_philox_against_curand_host_generator():
    """Library cross-check: the first blocks of cuRAND's host Philox4_32_10 generator (a CPU
    routine, used as a black box) are philox(key=seed, ctr=(0,0,i,0)), i = 0,1,2,...: its
    consecutive 4-word blocks walk the subsequence word of the counter."""
    lib = _curand()
    if lib is None:
        pytest.skip("libcurand not found")
    gen = ctypes.c_void_p()
    if lib.curandCreateGeneratorHost(ctypes.byref(gen), 161) != 0:
        pytest.skip("cuRAND host generator unavailable")
    for seed in (0, 1, 0x299F31D0A4093822, 2**64 - 1):
        assert lib.curandSetPseudoRandomGeneratorSeed(gen, ctypes.c_ulonglong(seed)) == 0
        assert lib.curandSetGeneratorOffset(gen, ctypes.c_ulonglong(0)) == 0
        out = np.zeros(4 * 64, np.uint32)
        assert lib.curandGenerate(gen, out.ctypes.data_as(ctypes.c_void_p), ctypes.c_size_t(out.size)) == 0
        key = [seed & 0xFFFFFFFF, seed >> 32]
        for i in (0, 1, 2, 17, 63):
            mine = oracle.philox4x32_10(key, [0, 0, i, 0])
            assert list(mine) == list(out[4 * i:4 * i + 4])
    lib.curandDestroyGenerator(gen)


def test_walk_uniform_is_top_24_bits_of_word0():
    for (seed, layer, head, ordinal, level, j) in [(0, 0, 0, 0, 0, 0), (5, 3, 7, 11, 2, 1023),
                                                    (2**40 + 17, 31, 6, 63, 1, 2047)]:
        w = oracle.philox4x32_10([seed & 0xFFFFFFFF, seed >> 32], [j, ordinal, level, (layer << 16) | head])
        assert oracle.walk_uniform(seed, layer, head, ordinal, level, j) == (int(w[0]) >> 8) / 2.0**24
    us = np.array([oracle.walk_uniform(9, 0, 0, 0, 0, j) for j in range(20000)])
    assert 0 <= us.min() and us.max() < 1
    assert abs(us.mean() - 0.5) < 0.01 and abs(us.var() - 1 / 12) < 0.005
    hist = np.histogram(us, bins=16, range=(0, 1))[0]
    chi2 = ((hist - 1250.0) ** 2 / 1250.0).sum()
    assert chi2 < 45.0  # 15 dof, p ~ 1e-4


# --------------------------------------------------------------------------- attention
def _softmax_attn(q, K, V, w=None):
    d = K.shape[1]
    logit = K @ q / math.sqrt(d)
    if w is not None:
        logit = logit + np.log(w)
    e = np.exp(logit - logit.max())
    return (e[:, None] * V).sum(0) / e.sum()


def test_T0_is_exact_attention():
    rng = np.random.default_rng(0)
    n, d = 300, 32
    K, V = rng.standard_normal((n, d)), rng.standard_normal((n, d))
    q = rng.standard_normal((5, d))
    s = OracleStream(OracleParams(d=d, t=64, T=0, max_tokens=n))
    s.append(K, V)
    assert s.compress() == 0 and len(s) == n
    z = s.decode(q)
    for a in range(5):
        ref = _softmax_attn(q[a], K, V)
        assert np.linalg.norm(z[a] - ref) <= 1e-12 * np.linalg.norm(ref)
    assert np.allclose(z, s.exact(q), rtol=0, atol=1e-14)


def test_weighted_attention_closed_forms():
    rng = np.random.default_rng(1)
    n, d = 50, 16
    K, V, q = rng.standard_normal((n, d)), rng.standard_normal((n, d)), rng.standard_normal((3, d))
    base = oracle.weighted_attention(K, V, None, q)
    # equal weights cancel in the ratio
    assert np.allclose(oracle.weighted_attention(K, V, np.full(n, 8.0), q), base, atol=1e-13)
    # a token counted twice == the token with weight 2
    w = np.ones(n)
    w[:10] = 2.0
    Kd, Vd = np.concatenate([K, K[:10]]), np.concatenate([V, V[:10]])
    assert np.allclose(oracle.weighted_attention(K, V, w, q), oracle.weighted_attention(Kd, Vd, None, q), atol=1e-13)
    # general weights against the numpy definition
    w = rng.choice([1.0, 2.0, 4.0, 8.0], size=n)
    for a in range(3):
        assert np.allclose(oracle.weighted_attention(K, V, w, q)[a], _softmax_attn(q[a], K, V, w), atol=1e-13)
    # one dominating key: output -> that token's value
    Kb = K.copy()
    Kb[7] = 200.0 * q[0] / np.linalg.norm(q[0])
    assert np.allclose(oracle.weighted_attention(Kb, V, None, q[:1])[0], V[7], atol=1e-9)


# --------------------------------------------------------------------------- kernel / probabilities
def _printed_walk_quantities(K, V, eta, c):
    """y^T eta, R^2 and p_j exactly as Algorithm 2 prints them (un-normalised kernel)."""
    m, d = K.shape
    G = np.exp(K @ K.T / math.sqrt(d)) * (V @ V.T)
    R2 = math.exp(max((K * K).sum(1)) / math.sqrt(d)) * max((V * V).sum(1))
    y_eta = np.array([sum(eta[i] * G[i, j] for i in range(j)) for j in range(m)])
    return y_eta, R2, 0.5 - y_eta / (2 * c * R2)


def test_probabilities_match_printed_formula():
    rng = np.random.default_rng(2)
    m, d = 24, 8
    K, V = 0.7 * rng.standard_normal((m, d)), rng.standard_normal((m, d))
    P = OracleParams(d=d, t=m, c_override=0.75, seed=3)
    r = oracle.softmax_balance(P, K, V)
    y_eta, R2, p = _printed_walk_quantities(K, V, r["eta"].astype(float), r["c"])
    assert np.allclose(r["S"], y_eta / R2, rtol=1e-12, atol=1e-15)
    ok = np.abs(y_eta / R2) <= r["c"]
    assert np.allclose(r["p"][ok], p[ok], rtol=0, atol=1e-13)
    assert np.all((r["p"] >= 0) & (r["p"] <= 1))
    assert np.array_equal(r["eta"] > 0, r["u"] < r["p"])
    assert abs(r["rk2"] - max((K * K).sum(1))) < 1e-12 and abs(r["rv2"] - max((V * V).sum(1))) < 1e-12


def test_default_constant_is_30_ln_m_over_delta():
    P = OracleParams(d=8, t=256, max_tokens=4096)
    c = oracle.walk_constant(P, 256)
    assert c == float(np.float32(30.0 * math.log(256 * 4096.0**2)))
    P2 = OracleParams(d=8, t=256, max_tokens=4096, delta=1e-3)
    assert oracle.walk_constant(P2, 64) == float(np.float32(30.0 * math.log(64 / 1e-3)))


def test_zero_keys_reduce_to_plain_walk_on_values():
    rng = np.random.default_rng(3)
    m, d = 40, 12
    V = rng.standard_normal((m, d))
    P = OracleParams(d=d, t=m, c_override=2.0, seed=11)
    r = oracle.softmax_balance(P, np.zeros((m, d)), V)
    eta = r["eta"].astype(float)
    rv2 = max((V * V).sum(1))
    S = np.array([sum(eta[i] * (V[i] @ V[j]) for i in range(j)) for j in range(m)]) / rv2
    assert np.allclose(r["S"], S, atol=1e-13)
    assert r["rk2"] == 0.0


def test_two_identical_max_norm_tokens():
    d = 8
    k = np.array([[1.0, 2, 0, 0, 0, 0, 0, 1]])
    v = np.array([[0.5, 0, 1, 0, 0, 0, 2, 0]])
    K, V = np.repeat(k, 2, 0), np.repeat(v, 2, 0)
    for seed in range(8):
        r = oracle.softmax_balance(OracleParams(d=d, t=2, c_override=3.0, seed=seed), K, V)
        assert r["p"][0] == 0.5
        assert abs(r["p"][1] - (0.5 - r["eta"][0] / (2 * 3.0))) < 1e-15   # G-hat = 1 exactly


def test_orthogonal_values_make_signs_a_pure_function_of_the_rng():
    rng = np.random.default_rng(4)
    m = d = 16
    K = rng.standard_normal((m, d))
    V = np.eye(m)
    P = OracleParams(d=d, t=m, seed=21, layer=2, head=3, c_override=0.01)
    r = oracle.softmax_balance(P, K, V, ordinal=5, level=1)
    assert np.all(r["p"] == 0.5) and np.all(r["S"] == 0)
    u = np.array([oracle.walk_uniform(21, 2, 3, 5, 1, j) for j in range(m)])
    assert np.array_equal(r["eta"], np.where(u < 0.5, 1, -1))


def test_kernel_bounds_cauchy_schwarz():
    rng = np.random.default_rng(5)
    m, d = 30, 16
    K, V = rng.standard_normal((m, d)) * 2, rng.standard_normal((m, d))
    # |G-hat_ij| <= 1: with eta forced to the sign of G-hat_ij's column, |S_j| <= j
    P = OracleParams(d=d, t=m, c_override=1e9)
    for j_star in (5, 17, 29):
        rk2, rv2 = max((K * K).sum(1)), max((V * V).sum(1))
        g = np.exp((K @ K[j_star] - rk2) / math.sqrt(d)) * (V @ V[j_star]) / rv2
        forced = np.where(g >= 0, 1, -1).astype(np.int8)
        r = oracle.softmax_balance(P, K, V, forced=forced)
        assert abs(r["S"][j_star] - np.abs(g[:j_star]).sum()) < 1e-12
        assert np.all(np.abs(g) <= 1 + 1e-12)


def test_fail_is_counted_and_clamped():
    d = 4
    K = np.zeros((6, d))
    V = np.tile(np.array([[1.0, 0, 0, 0]]), (6, 1))          # G-hat = 1 for every pair
    r = oracle.softmax_balance(OracleParams(d=d, t=6, c_override=1.5), K, V,
                               forced=np.ones(6, np.int8))
    assert list(r["S"]) == [0, 1, 2, 3, 4, 5]
    assert r["fails"] == 4                                        # |S| > 1.5 at j = 2..5
    assert list(r["p"][2:]) == [0.0] * 4 and r["p"][1] == 0.5 - 1 / 3.0


def test_key_centering_is_shift_invariant():
    rng = np.random.default_rng(6)
    m, d = 32, 8
    K, V = rng.standard_normal((m, d)), rng.standard_normal((m, d))
    P = OracleParams(d=d, t=m, c_override=0.5, center_keys=1, seed=4)
    a = oracle.softmax_balance(P, K, V)
    b = oracle.softmax_balance(P, K + 3.0 * rng.standard_normal(d), V)
    assert np.allclose(a["S"], b["S"], atol=1e-10) and np.array_equal(a["eta"], b["eta"])
    Kc = K - K.mean(0)
    c = oracle.softmax_balance(OracleParams(d=d, t=m, c_override=0.5, seed=4), Kc, V)
    assert np.allclose(a["S"], c["S"], atol=1e-12)


# --------------------------------------------------------------------------- walk law, brute force
def _walk_law(G_hat, c):
    """P(eta) for every sign vector under Algorithm 2's rule, enumerated in numpy."""
    m = G_hat.shape[0]
    law = {}
    for bits in itertools.product((1, -1), repeat=m):
        eta = np.array(bits, float)
        pr = 1.0
        for j in range(m):
            S = float(eta[:j] @ G_hat[:j, j])
            S = max(-c, min(c, S))
            p = 0.5 - S / (2 * c)
            pr *= p if bits[j] == 1 else (1 - p)
        law[bits] = pr
    return law


def _ghat(K, V):
    d = K.shape[1]
    return np.exp((K @ K.T - max((K * K).sum(1))) / math.sqrt(d)) * (V @ V.T) / max((V * V).sum(1))


@pytest.mark.parametrize("m", [3, 6, 10])
def test_probabilities_for_every_prefix_brute_force(m):
    rng = np.random.default_rng(7 + m)
    d, c = 4, 0.8
    K, V = 0.8 * rng.standard_normal((m, d)), rng.standard_normal((m, d))
    G = _ghat(K, V)
    P = OracleParams(d=d, t=m, c_override=c)
    for bits in itertools.product((1, -1), repeat=m):
        r = oracle.softmax_balance(P, K, V, forced=np.array(bits, np.int8))
        eta = np.array(bits, float)
        S = np.array([eta[:j] @ G[:j, j] for j in range(m)])
        assert np.allclose(r["S"], S, atol=1e-13)
        assert np.allclose(r["p"], 0.5 - np.clip(S, -c, c) / (2 * c), atol=1e-13)


def test_walk_law_sums_to_one_and_matches_empirical_distribution():
    rng = np.random.default_rng(8)
    m, d, c = 4, 4, 0.45
    K, V = 0.2 * rng.standard_normal((m, d)), rng.standard_normal((m, d))
    law = _walk_law(_ghat(K, V), c)
    assert abs(sum(law.values()) - 1.0) < 1e-12
    n_seeds = 40000
    counts = dict.fromkeys(law, 0)
    for seed in range(n_seeds):
        r = oracle.softmax_balance(OracleParams(d=d, t=m, c_override=c, seed=seed), K, V)
        counts[tuple(int(x) for x in r["eta"])] += 1
    chi2 = sum((counts[k] - n_seeds * law[k]) ** 2 / (n_seeds * law[k]) for k in law if law[k] > 0)
    assert all(counts[k] == 0 for k in law if law[k] == 0)
    assert chi2 < 44.0  # 15 dof, p ~ 1e-4
    # the law is far from uniform here, so the chi-square test has power
    assert max(law.values()) / min(v for v in law.values() if v > 0) > 3


def test_walk_lowers_discrepancy_below_fair_coin():
    """E[eta^T G-hat eta] (feature-space squared discrepancy) under the walk law is below
    the fair-coin value trace(G-hat); both by enumeration (m=12) and by Monte Carlo."""
    rng = np.random.default_rng(9)
    m, d, c = 12, 4, 0.7
    K, V = 0.5 * rng.standard_normal((m, d)), rng.standard_normal((m, d))
    G = _ghat(K, V)
    law = _walk_law(G, c)
    assert abs(sum(law.values()) - 1) < 1e-10
    exp_disc = sum(pr * (np.array(b, float) @ G @ np.array(b, float)) for b, pr in law.items())
    assert exp_disc < 0.8 * np.trace(G)
    mc = []
    for seed in range(6000):
        e = oracle.softmax_balance(OracleParams(d=d, t=m, c_override=c, seed=seed), K, V)["eta"].astype(float)
        mc.append(e @ G @ e)
    assert abs(np.mean(mc) - exp_disc) < 5 * np.std(mc) / math.sqrt(len(mc))


# --------------------------------------------------------------------------- selection
def test_strict_half_selection_hand_cases():
    d = 2
    P = lambda m: OracleParams(d=d, t=m, c_override=1e6)
    K = lambda m: np.zeros((m, d))
    V = lambda m: np.ones((m, d))
    sel = lambda eta: list(oracle.softmax_balance(P(len(eta)), K(len(eta)), V(len(eta)),
                                                  forced=np.array(eta, np.int8))["kept"])
    assert sel([1, -1]) == [0]                 # tie -> the +1 class
    assert sel([-1, 1]) == [1]
    assert sel([1, 1]) == [1]                  # minority empty -> latest of the other class
    assert sel([-1, -1]) == [1]
    assert sel([1, -1, -1, -1]) == [0, 3]      # minority {0} + latest of the majority
    assert sel([-1, 1, 1, 1]) == [0, 3]
    assert sel([1, 1, -1, -1]) == [0, 1]       # tie
    assert sel([1, -1, 1, -1, -1, -1, 1, -1]) == [0, 2, 6, 7]
    assert sel([1, 1, 1, 1, 1, 1, -1, 1]) == [4, 5, 6, 7]
    assert sel([1] * 8) == [4, 5, 6, 7]
    assert sel([-1, 1, -1, 1, 1, -1, -1, 1]) == [1, 3, 4, 7]   # balanced: exactly the +1 class


def test_selection_equals_smaller_class_when_balanced():
    rng = np.random.default_rng(10)
    m, d = 64, 8
    K, V = rng.standard_normal((m, d)), rng.standard_normal((m, d))
    for seed in range(20):
        r = oracle.softmax_balance(OracleParams(d=d, t=m, c_override=0.3, seed=seed), K, V)
        plus = np.flatnonzero(r["eta"] > 0)
        minus = np.flatnonzero(r["eta"] < 0)
        small = plus if len(plus) <= len(minus) else minus
        assert len(r["kept"]) == m // 2 and np.all(np.diff(r["kept"]) > 0)
        assert set(small) <= set(r["kept"])
        extra = sorted(set(r["kept"]) - set(small))
        other = minus if small is plus else plus
        assert extra == sorted(other[len(other) - len(extra):]) if extra else True


# --------------------------------------------------------------------------- discrepancy bound (Theorem 3.2)
def test_discrepancy_within_theorem_bound_with_explicit_constant():
    rng = np.random.default_rng(11)
    m, d = 128, 16
    K, V = rng.standard_normal((m, d)) * 1.5, rng.standard_normal((m, d))
    for P in (OracleParams(d=d, t=m, max_tokens=m, seed=1), OracleParams(d=d, t=m, c_override=1.0, seed=1)):
        r = oracle.softmax_balance(P, K, V)
        eta = r["eta"].astype(float)
        rk = math.sqrt(r["rk2"])
        for _ in range(50):
            q = rng.standard_normal(d)
            q *= rng.uniform(0, 1) * rk / np.linalg.norm(q)
            disc = np.linalg.norm((eta * np.exp(K @ q / math.sqrt(d))) @ V)
            log_bound = (math.log(math.sqrt(d) * r["c"]) + (q @ q) / (2 * math.sqrt(d))
                         + r["rk2"] / (2 * math.sqrt(d)) + 0.5 * math.log(r["rv2"]))
            assert math.log(disc) <= log_bound
        assert r["fails"] == 0
