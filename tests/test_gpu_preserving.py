"""GPU parity of Section 4.3's augmented variant: rows whose key has cosine <= tau with the block's mean
key are preserved exactly in their own layer slot, the rest is an ordinary BalanceKV stream.  The routing
is compared bit for bit with the oracle (inputs kept away from the threshold, where fp32 and double
agree), the rest by the teacher-forced procedure, the union by the oracle's estimator."""
import numpy as np
import pytest
import torch

from oracle import PreservingOracle, anticorrelated
from paper_2502_07861_b200 import synth
from parity_util import Harness, rel_l2, to_device

pytestmark = pytest.mark.gpu


def _stream(seed, b, h, n, d, dtype, frac):
    rng = np.random.default_rng([seed, b, h])
    mu = rng.standard_normal(d).astype(np.float32)
    K = (0.06 * (4.0 * mu + rng.standard_normal((n, d)))).astype(np.float32)
    anti = rng.random(n) < frac
    K[anti] = (0.06 * (-5.0 * mu + 0.3 * rng.standard_normal((int(anti.sum()), d)))).astype(np.float32)
    return synth.round_to(K, dtype), synth.round_to(rng.standard_normal((n, d)).astype(np.float32), dtype)


def _margin_ok(K, tau):
    K = K.astype(np.float64)
    mean = K.mean(0)
    cos = K @ mean / (np.linalg.norm(K, axis=1) * np.linalg.norm(mean))
    return np.min(np.abs(cos - tau)) > 1e-4


@pytest.mark.parametrize("dtype,d,t,T,tau", [("bf16", 128, 128, 2, -0.5), ("fp32", 64, 64, 1, -0.3)])
def test_preserving_append_compress_decode(cuda_lib, dtype, d, t, T, tau):
    B, H, g = 2, 2, 4
    chunks = [900, 333, 1100]
    n = sum(chunks)
    K = np.empty((B, H, n, d), np.float32)
    V = np.empty_like(K)
    for b in range(B):
        for h in range(H):
            K[b, h], V[b, h] = _stream(5, b, h, n, d, dtype, 0.02)
    hz = Harness(cuda_lib, B=B, L=2, H=H, g=g, d=d, dtype=dtype, t=t, T=T, N=n, seed=21, c_override=0.7)
    po = {(b, h): PreservingOracle(d=d, t=t, T=T, tau=tau, layer0=0, head=h, max_tokens=n, seed=21 + b, c_override=0.7)
          for b in range(B) for h in range(H)}
    kept = {k: [] for k in po}
    p = 0
    for m in chunks:
        Kc, Vc = np.ascontiguousarray(K[:, :, p:p + m]), np.ascontiguousarray(V[:, :, p:p + m])
        counts, slots = hz.ctx.stream_append_layer_preserving(0, to_device(Kc, dtype), to_device(Vc, dtype), tau, want_slots=True)
        slots = slots.cpu().numpy()
        for b in range(B):
            for h in range(H):
                assert _margin_ok(Kc[b, h], tau)
                mask = po[(b, h)].append(Kc[b, h], Vc[b, h])
                assert np.array_equal(slots[b, h] == 0, mask), (b, h, np.flatnonzero((slots[b, h] == 0) != mask)[:8])
                assert [int(x) for x in counts[b * H + h]] == [int(mask.sum()), int((~mask).sum()), 0]
                assert 0 < mask.sum() < m // 4
                kept[(b, h)].append((Kc[b, h][mask], Vc[b, h][mask]))
                hz.events.append(("append_stream", b, 1, h, Kc[b, h][~mask], Vc[b, h][~mask]))
        hz.ctx.compress_layer(1)                     # the slot of the preserved tokens is never compressed
        hz.events.append(("compress",))
        p += m
    tot, _ = hz.check_all(2e-4 if dtype == "bf16" else 2e-5, streams={(b, 1, h) for b in range(B) for h in range(H)})
    assert tot > 0
    for (b, h), o in po.items():
        for (lvl, od), (eta, _, _) in hz.recs[(b, 1, h)].items():
            o.force_eta(lvl, od, eta)
        o.compress()
        keep, rest = o.views()
        Kg, Vg, wg, ig = hz.ctx.cache_view(b, 0, h)
        assert np.array_equal(Kg.float().cpu().numpy().astype(np.float64), keep[0])
        assert np.array_equal(Vg.float().cpu().numpy().astype(np.float64), keep[1])
        assert np.all(wg.cpu().numpy() == 1.0) and np.array_equal(ig.cpu().numpy(), np.arange(len(keep[3])))
        ref = hz.oracles[(b, 1, h)].view()
        assert np.array_equal(rest[0], ref[0]) and np.array_equal(rest[2], ref[2])
        assert keep[2].sum() + rest[2].sum() == n                           # Theorem 3.3's weights: tokens seen
    if dtype != "bf16":
        return
    q = synth.queries(5, 0, 0, B, H * g, d, dtype)
    out = hz.ctx.decode_attn_merged([0, 1], [0, 1], to_device(q, dtype)).float().cpu().numpy()
    for (b, h), o in po.items():
        assert rel_l2(out[b, h * g:(h + 1) * g], o.estimate(q[b, h * g:(h + 1) * g])) <= 2e-3
    assert hz.ctx.stats()["device_status"] == 0
