"""GPU parity of Algorithm 1's value-norm buckets: the library routes every row of a block to the
MergeAndReduce instance of its bucket 2^(i-1) < ||v|| <= 2^i (one layer slot per bucket), erases the
instances with 2^i <= rho * v_max, compresses every instance with its own coins, and decodes the
union of the instances over a separate denominator instance.  Routing, erasure and counts are
compared with the oracle's token-by-token form of Algorithm 1, every surviving instance by the
teacher-forced procedure, and the decode output with the oracle's ratio."""
import math

import numpy as np
import pytest
import torch

import oracle
from oracle import BucketedOracle
from paper_2502_07861_b200 import synth
from parity_util import Harness, rel_l2, to_device

pytestmark = pytest.mark.gpu


def _unit(shape):
    E = np.zeros(shape, np.float32)
    E[..., 0] = 1.0
    return E


def _stream(seed, b, h, n, d, dtype, key_scale):
    """Keys as the llama recipe (scaled), values N(0,1) rows with norms spread over ~7 octaves that
    grow along the stream (so that buckets are erased after they have received rows)."""
    k, v = synth.stream_kv("llama", seed, b, 0, h, n, d, dtype)
    rng = np.random.default_rng([seed, b, h])
    scale = 2.0 ** (rng.uniform(-4.5, 0.0, n) + np.linspace(-2.0, 0.0, n))
    v = synth.round_to((v * scale[:, None] * math.sqrt(128.0 / d)).astype(np.float32), dtype)
    v[5] = 0.0                                                    # a zero value has no bucket
    return synth.round_to(k * key_scale, dtype), v


def _not_borderline(V, rho):
    """The library decides on fp32 squared norms, the oracle in double: keep the inputs away from
    the bucket boundaries and the erase threshold (relative 1e-5), where both readings agree."""
    ns = np.sum(V.astype(np.float64) ** 2, axis=-1).ravel()
    ns = ns[ns > 0]
    frac = 0.5 * np.log2(ns)
    assert np.min(np.abs(frac - np.round(frac))) > 1e-5
    if rho > 0:
        run = 0.5 * np.log2(np.maximum.accumulate(ns) * rho * rho)
        assert np.min(np.abs(run - np.round(run))) > 1e-5


@pytest.mark.parametrize("dtype,d,t,T,rho,c,W", [("bf16", 128, 128, 2, 2.0 ** -3.3, 0.75, 0), ("fp32", 64, 64, 1, 2.0 ** -3.3, 0.5, 0),
                                                 ("bf16", 128, 256, 1, 0.0, 0.0, 0), ("bf16", 128, 64, 3, 2.0 ** -3.3, 0.75, 48)])
def test_bucketed_append_compress_decode(cuda_lib, dtype, d, t, T, rho, c, W):
    B, H, g, nb, i_top = 2, 2, 4, 5, 4
    chunks = [700, 300, 1048]
    n = sum(chunks)
    K = np.empty((B, H, n, d), np.float32)
    V = np.empty_like(K)
    for b in range(B):
        for h in range(H):
            K[b, h], V[b, h] = _stream(77, b, h, n, d, dtype, 0.06 if c > 0 else 1.0)
    _not_borderline(V, rho)
    assert math.sqrt(np.max(np.sum(V.astype(np.float64) ** 2, -1))) <= 2.0 ** i_top
    # W > 0: every instance keeps the newest W tokens of its own sub-stream out of the batches
    hz = Harness(cuda_lib, B=B, L=nb + 1, H=H, g=g, d=d, dtype=dtype, t=t, T=T, N=n, W=W, seed=11, c_override=c)
    bo = {(b, h): BucketedOracle(d=d, t=t, T=T, i_top=i_top, n_buckets=nb, erase_ratio=rho, layer0=0, head=h,
                                 max_tokens=n, seed=11 + b, c_override=c, W=W) for b in range(B) for h in range(H)}
    per_slot_events = {}
    p = 0
    for m in chunks:
        Kc, Vc = np.ascontiguousarray(K[:, :, p:p + m]), np.ascontiguousarray(V[:, :, p:p + m])
        counts, slots = hz.ctx.stream_append_layer_bucketed(0, nb, i_top, to_device(Kc, dtype), to_device(Vc, dtype),
                                                            erase_ratio=rho, want_slots=True)
        if dtype == "bf16":
            hz.ctx.stream_append_layer_keys(nb, to_device(Kc, dtype))        # MR-Denominator on (k_j, 1)
            hz.events.append(("append", nb, Kc, _unit(Kc.shape)))
        slots = slots.cpu().numpy()
        for b in range(B):
            for h in range(H):
                o = bo[(b, h)]
                before = {s: len(r) for s, r in o.route.items()}
                o.append(Kc[b, h], Vc[b, h])
                want = np.full(m, -1, np.int8)
                for s, r in o.route.items():
                    new = np.asarray(r[before.get(s, 0):], np.int64) - p
                    want[new] = s
                    hz.events.append(("append_stream", b, s, h, Kc[b, h][new], Vc[b, h][new], p))
                # rows the oracle sent to an instance that this very block erased count as dropped
                assert np.array_equal(slots[b, h], want), (b, h, np.flatnonzero(slots[b, h] != want)[:8])
                row = counts[b * H + h]
                assert [int(x) for x in row[:nb]] == [int(np.sum(want == s)) for s in range(nb)]
                assert int(row[nb]) == int(np.sum(want == -1))
        hz.compress()
        p += m
    # instances erased along the way are empty on the GPU; drop their earlier rows from the replay
    alive = {(b, s, h) for (b, h), o in bo.items() for s in o.inst}
    hz.events = [e for e in hz.events if e[0] != "append_stream" or (e[1], e[2], e[3]) in alive]
    hz.events = [e[:6] if e[0] == "append_stream" else e for e in hz.events]
    erased_slots = 0
    for b in range(B):
        for h in range(H):
            assert (rho > 0) == (len(bo[(b, h)].inst) < nb)
            for s in range(nb):
                if (b, s, h) not in alive:
                    erased_slots += 1
                    assert sum(hz.ctx.level_sizes(b, s, h)) == 0
    streams = alive | ({(b, nb, h) for b in range(B) for h in range(H)} if dtype == "bf16" else set())
    tot, _ = hz.check_all(2e-4 if dtype == "bf16" else 2e-5, streams=streams)
    assert tot > 0
    # the oracle's own Algorithm 1 object, following the same signs, holds the same sets
    for (b, h), o in bo.items():
        for s in o.inst:
            for (lvl, od), (eta, _, _) in hz.recs[(b, s, h)].items():
                o.force_eta(s, lvl, od, eta)
        o.compress()
        for s, view in zip(sorted(o.inst), o.views()):
            ref = hz.oracles[(b, s, h)].view()
            assert np.array_equal(view[0], ref[0]) and np.array_equal(view[1], ref[1]) and np.array_equal(view[2], ref[2])
            assert np.array_equal(view[3], np.asarray(o.route[s])[ref[3]])
            assert view[2].sum() == len(o.route[s])                          # Theorem 3.3's weights
    if dtype != "bf16":
        return
    for step in range(2):
        q = synth.queries(77, 0, step, B, H * g, d, dtype)
        out = hz.ctx.decode_attn_merged(list(range(nb)), [nb], to_device(q, dtype)).float().cpu().numpy()
        for (b, h), o in bo.items():
            qs = q[b, h * g:(h + 1) * g]
            ref = o.estimate(qs, [hz.oracles[(b, nb, h)].view()])
            assert rel_l2(out[b, h * g:(h + 1) * g], ref) <= 2e-3
            if T == 0 or rho == 0.0:
                continue
    assert hz.ctx.stats()["device_status"] == 0


@pytest.mark.parametrize("capacity", [500, 300])
def test_bucketed_per_stream_entry_and_refusals(cuda_lib, capacity):
    """capacity 500: every instance could take the whole block; capacity 300: only the actual per-bucket
    counts fit, and repeating the block overflows an instance (refused as a whole)."""
    d, t, n = 128, 64, 500
    ctx = cuda_lib.Context(n_seqs=1, n_layers=4, n_kv_heads=2, n_q_heads=8, head_dim=d, dtype="bf16", block=t, levels=1,
                           max_tokens=capacity)
    k, v = _stream(78, 0, 1, n, d, "bf16", 1.0)
    _not_borderline(v, 0.0)
    Kd, Vd = to_device(k, "bf16"), to_device(v, "bf16")
    # a norm above 2^i_top refuses the whole block and leaves every instance untouched
    with pytest.raises(Exception):
        ctx.stream_append_bucketed(0, 0, 4, 1, 1, Kd, Vd)
    assert all(sum(ctx.level_sizes(0, s, 1)) == 0 for s in range(4))
    counts, slots = ctx.stream_append_bucketed(0, 0, 4, 4, 1, Kd, Vd, want_slots=True)
    want = np.array([4 - oracle.value_bucket(x) if np.any(x) else 99 for x in v.astype(np.float64)])
    want = np.where(want < 4, want, -1)
    assert np.array_equal(slots.cpu().numpy(), want)
    assert [int(x) for x in counts] == [int(np.sum(want == s)) for s in range(4)] + [int(np.sum(want == -1))]
    for s in range(4):
        rows = np.flatnonzero(want == s)
        Kg, Vg, wg, ig = ctx.cache_view(0, s, 1)
        assert np.array_equal(Vg.float().cpu().numpy(), v[rows]) and np.array_equal(Kg.float().cpu().numpy(), k[rows])
        assert np.array_equal(ig.cpu().numpy(), np.arange(len(rows))) and np.all(wg.cpu().numpy() == 1)
        assert sum(ctx.level_sizes(0, s, 0)) == 0                 # the other head's instances are untouched
    with pytest.raises(Exception):
        ctx.stream_append_bucketed(0, 2, 4, 4, 1, Kd, Vd)         # slots beyond the context's layers
    if capacity == 300:
        with pytest.raises(Exception):                            # an instance would overflow: refused, nothing appended
            for _ in range(3):
                ctx.stream_append_bucketed(0, 0, 4, 4, 1, Kd, Vd)
        assert all(sum(ctx.level_sizes(0, s, 1)) <= capacity for s in range(4))


def test_bucketed_llama_layer_full_size_sampled_instances(cuda_lib):
    """The one-layer Llama-3.1-8B-shaped workload (8 KV heads x 32768 tokens, d = 128, bf16, block
    1024, T = 2) through the bucketed path: routing of every row of every stream against a direct
    evaluation of the bucket rule, size-independent properties of every instance, teacher-forced
    replay of two sampled instances, and the merged decode of a sampled head."""
    B, H, g, d, n, t, T, nb, i_top = 1, 8, 4, 128, 32768, 1024, 2, 4, 4
    K = np.empty((B, H, n, d), np.float32)
    V = np.empty_like(K)
    for h in range(H):
        k, v = synth.stream_kv("llama", 1002, 0, 0, h, n, d, "bf16")
        scale = 2.0 ** np.random.default_rng([1002, h]).uniform(-3.9, 0.0, n)
        K[0, h], V[0, h] = k, synth.round_to((v * scale[:, None]).astype(np.float32), "bf16")
    # rows whose norm sits within rounding of a bucket boundary are moved off it (see _not_borderline)
    frac = 0.5 * np.log2(np.sum(V.astype(np.float64) ** 2, -1))
    near = np.abs(frac - np.round(frac)) <= 1e-4
    V[near] = synth.round_to(V[near] * np.float32(1.0625), "bf16")
    _not_borderline(V, 0.0)
    ns = np.sum(V.astype(np.float64) ** 2, -1)
    want = i_top - np.ceil(0.5 * np.log2(ns)).astype(np.int64)           # the bucket rule, written out
    assert want.min() >= 0
    want = np.where(want < nb, want, -1)
    ctx = cuda_lib.Context(n_seqs=B, n_layers=nb + 1, n_kv_heads=H, n_q_heads=H * g, head_dim=d, dtype="bf16", block=t,
                           levels=T, max_tokens=n, seed=7)
    ctx.debug_enable(True)
    Kd, Vd = to_device(K, "bf16"), to_device(V, "bf16")
    counts, slots = ctx.stream_append_layer_bucketed(0, nb, i_top, Kd, Vd, want_slots=True)
    ctx.stream_append_layer_keys(nb, Kd)
    ctx.compress()
    assert np.array_equal(slots.cpu().numpy(), want)
    for h in range(H):
        assert [int(x) for x in counts[h]] == [int(np.sum(want[0, h] == s)) for s in range(nb)] + [int(np.sum(want[0, h] < 0))]
        for s in range(nb):
            m = int(counts[h, s])
            _, _, w, idx = ctx.cache_view(0, s, h)
            sizes = ctx.level_sizes(0, s, h)
            assert float(w.sum()) == m                                   # Theorem 3.3's weights stand for every row
            assert sizes[0] == m % t
            assert sizes[T] == (m // (2 * t)) * (t // 2) and torch.all(idx[: sizes[T]][1:] > idx[: sizes[T]][:-1])
    st = ctx.stats()
    assert st["device_status"] == 0
    from oracle import OracleStream
    from parity_util import check_stream, gpu_call_records, oracle_params
    tot = marg = 0
    for (h, s) in ((2, 1), (5, 3)):
        rows = np.flatnonzero(want[0, h] == s)
        rec = gpu_call_records(ctx, 0, s, h, len(rows) // t)
        o = OracleStream(oracle_params(ctx, 0, s, h))
        for (lvl, od), (eta, _, _) in rec.items():
            o.force_eta(lvl, od, eta)
        o.append(K[0, h][rows], V[0, h][rows])
        o.compress()
        a, b = check_stream(ctx, 0, s, h, o, rec, 2e-4)
        tot, marg = tot + a, marg + b
    assert tot > 0 and marg <= 1e-3 * tot
    # merged decode of every head against the oracle's ratio evaluated on the library's own sets
    q = synth.queries(1002, 0, 0, B, H * g, d, "bf16")
    out = ctx.decode_attn_merged(list(range(nb)), [nb], to_device(q, "bf16")).float().cpu().numpy()
    for h in (0, 5):
        views = []
        for s in range(nb + 1):
            Kg, Vg, wg, _ = ctx.cache_view(0, s, h)
            views.append((Kg.float().cpu().numpy().astype(np.float64), Vg.float().cpu().numpy().astype(np.float64),
                          wg.cpu().numpy().astype(np.float64)))
        ref = oracle.merged_estimate(views[:nb], [views[nb]], q[0, h * g:(h + 1) * g])
        assert rel_l2(out[0, h * g:(h + 1) * g], ref) <= 2e-3


def test_error_sweep_point_buckets_beat_uniform_on_mixed_value_norms(cuda_lib):
    """One point of the error-against-rate sweep with value norms spread over three octaves: a walk
    that is not a fair coin needs Algorithm 1's buckets (without them it is no better than uniform
    sampling, with them clearly better)."""
    from paper_2502_07861_b200 import error_sweep

    acc = {}
    for seed in range(4):
        for k, v in error_sweep.run_point("clustered_norms", seed, 2, 8192, 128, 128, 1, 0.25, 0, buckets=4).items():
            acc[k] = acc.get(k, 0.0) + v / 4
    assert acc["algorithm1_small_c"] < 0.8 * acc["uniform"]
    assert acc["algorithm1_small_c"] < 0.8 * acc["balancekv_small_c"]
    assert 0.5 * acc["uniform"] < acc["algorithm1_paper_c"] < 2.0 * acc["uniform"]
