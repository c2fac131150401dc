"""GPU parity at the full size of the one-layer Llama-3.1-8B-shaped workload (32 query / 8 KV
heads, d = 128, 32768 context tokens, bf16, block 1024, T = 2), driven the way the benchmark
drives it: one whole-layer append, one compress, then stream_step per decode token.  Two of the
eight streams are replayed by the oracle (the others are covered by size-independent
properties), plus the small cases of stream_step and of the sampled profiler."""
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

from oracle import OracleStream
from paper_2502_07861_b200 import synth
from parity_util import check_stream, gpu_call_records, oracle_params, rel_l2, to_device

pytestmark = pytest.mark.gpu

B, H, G, D, N, T_BLOCK, LEVELS, STEPS = 1, 8, 4, 128, 32768, 1024, 2, 12
SAMPLED = (1, 6)


def _inputs():
    K = np.empty((B, H, N + STEPS, D), np.float32)
    V = np.empty_like(K)
    for h in range(H):
        K[0, h], V[0, h] = synth.stream_kv("llama", 1002, 0, 0, h, N + STEPS, D, "bf16")
    return K, V


def test_llama_layer_full_size_sampled_streams(cuda_lib):
    K, V = _inputs()
    Kd, Vd = to_device(K, "bf16"), to_device(V, "bf16")
    make = lambda: cuda_lib.Context(n_seqs=B, n_layers=1, n_kv_heads=H, n_q_heads=H * G, head_dim=D, dtype="bf16",
                                    block=T_BLOCK, levels=LEVELS, max_tokens=N + STEPS, seed=7)
    ctx = make()
    ctx.debug_enable(True)
    ctx.stream_append_layer(0, Kd[:, :, :N].contiguous(), Vd[:, :, :N].contiguous())
    ctx.compress()
    # the benchmark's configuration has the debug record off: same kept sets, bit for bit
    plain = make()
    plain.stream_append_layer(0, Kd[:, :, :N].contiguous(), Vd[:, :, :N].contiguous())
    plain.compress()
    for h in range(H):
        a, b = ctx.cache_view(0, 0, h), plain.cache_view(0, 0, h)
        assert all(torch.equal(x, y) for x, y in zip(a, b))
        # size-independent properties of every stream (Algorithm 3): 4x compression, weights 2^T,
        # increasing original positions
        _, _, w, idx = a
        assert len(idx) == N >> LEVELS and torch.all(w == 2.0 ** LEVELS) and torch.all(idx[1:] > idx[:-1])
    st = ctx.stats()
    assert st["device_status"] == 0 and st["walk_fails"] == 0 and st["calls_run"] == H * (32 + 16)

    # teacher-forced replay of the sampled streams (threads: the oracle call releases the GIL)
    recs = {h: gpu_call_records(ctx, 0, 0, h, N // T_BLOCK) for h in SAMPLED}

    def replay(h):
        o = OracleStream(oracle_params(ctx, 0, 0, h))
        for (lvl, ordinal), (eta, _, _) in recs[h].items():
            o.force_eta(lvl, ordinal, eta)
        o.append(K[0, h, :N], V[0, h, :N])
        o.compress()
        return o

    with ThreadPoolExecutor(len(SAMPLED)) as ex:
        oracles = dict(zip(SAMPLED, ex.map(replay, SAMPLED)))
    decisions = margin = 0
    for h in SAMPLED:
        n, m = check_stream(ctx, 0, 0, h, oracles[h], recs[h], 2e-4)
        decisions += n
        margin += m
    assert decisions == len(SAMPLED) * 48 * T_BLOCK and margin <= 1e-3 * decisions

    # decode steps through stream_step on the plain context (append one token per stream, attend)
    out = torch.empty(B, H * G, D, dtype=torch.bfloat16, device="cuda")
    for s in range(STEPS):
        q = synth.queries(1002, 0, s, B, H * G, D, "bf16")
        plain.stream_step(0, to_device(q, "bf16"), Kd[:, :, N + s:N + s + 1].contiguous(),
                          Vd[:, :, N + s:N + s + 1].contiguous(), out)
        got = out.float().cpu().numpy()
        for h in SAMPLED:
            oracles[h].append(K[0, h, N + s:N + s + 1], V[0, h, N + s:N + s + 1])
            ref = oracles[h].decode(q[0, h * G:(h + 1) * G])
            assert rel_l2(got[0, h * G:(h + 1) * G], ref) <= 2e-3
    sizes = plain.level_sizes(0, 0, 3)
    assert list(sizes) == [STEPS, 0, N >> LEVELS]
    assert plain.stats()["device_status"] == 0


def test_stream_step_equals_append_then_decode(cuda_lib):
    Bs, Hs, g, d, n = 2, 2, 4, 128, 300
    mk = lambda: cuda_lib.Context(n_seqs=Bs, n_layers=1, n_kv_heads=Hs, n_q_heads=Hs * g, head_dim=d, dtype="bf16",
                                  block=64, levels=1, max_tokens=n + 4, seed=1)
    rng = np.random.default_rng(0)
    K = to_device(rng.standard_normal((Bs, Hs, n + 4, d)).astype(np.float32), "bf16")
    V = to_device(rng.standard_normal((Bs, Hs, n + 4, d)).astype(np.float32), "bf16")
    a, b = mk(), mk()
    for c in (a, b):
        c.stream_append_layer(0, K[:, :, :n].contiguous(), V[:, :, :n].contiguous())
        c.compress()
    for s in range(4):
        q = to_device(rng.standard_normal((Bs, Hs * g, d)).astype(np.float32), "bf16")
        k1, v1 = K[:, :, n + s:n + s + 1].contiguous(), V[:, :, n + s:n + s + 1].contiguous()
        out_a = torch.empty_like(q)
        a.stream_step(0, q, k1, v1, out_a)
        b.stream_append_layer(0, k1, v1)
        out_b = b.decode_attn(0, q)
        # the fused step scores the new token in fp32 outside the tiles: same value up to rounding
        assert rel_l2(out_a.float().cpu().numpy(), out_b.float().cpu().numpy()) <= 2e-3
    for h in range(Hs):
        assert all(torch.equal(x, y) for x, y in zip(a.cache_view(1, 0, h), b.cache_view(1, 0, h)))


def test_profiler_class_mask_and_sampling(cuda_lib):
    Bs, Hs, g, d, n = 1, 2, 2, 128, 256
    ctx = cuda_lib.Context(n_seqs=Bs, n_layers=1, n_kv_heads=Hs, n_q_heads=Hs * g, head_dim=d, dtype="bf16", block=64,
                           levels=1, max_tokens=n, seed=1)
    K = torch.randn(Bs, Hs, n, d, device="cuda").to(torch.bfloat16)
    q = torch.randn(Bs, Hs * g, d, device="cuda").to(torch.bfloat16)
    ctx.profile_enable(True, classes=("decode", "compact"))
    ctx.profile_sample("decode", 4)
    ctx.profile_read()
    ctx.stream_append_layer(0, K, K)
    ctx.compress()
    for _ in range(10):
        ctx.decode_attn(0, q)
    prof = ctx.profile_read()
    assert prof["append"][0] == 0 and prof["gram_walk"][0] == 0        # masked out
    assert prof["compact"][0] == 1 and prof["compact"][1] > 0
    assert prof["decode"][0] == 3 and prof["decode"][1] > 0            # launches 0, 4, 8 of 10
    ctx.profile_enable(False)
    ctx.decode_attn(0, q)
    assert ctx.profile_read()["decode"][0] == 0


def test_host_buffer_entry_points_match_the_device_ones(cuda_lib):
    """append / decode / step through host buffers (pinned, one step pageable; more steps than staging slots) give
    bit-identical caches and outputs to the device-pointer calls."""
    Bs, Hs, g, d, n, steps = 2, 2, 4, 128, 200, 70
    mk = lambda: cuda_lib.Context(n_seqs=Bs, n_layers=1, n_kv_heads=Hs, n_q_heads=Hs * g, head_dim=d, dtype="bf16",
                                  block=64, levels=1, max_tokens=n + steps, seed=1)
    rng = np.random.default_rng(1)
    bf = lambda shape: torch.from_numpy(rng.standard_normal(shape).astype(np.float32)).to(torch.bfloat16)
    K_h, V_h = bf((Bs, Hs, n, d)).pin_memory(), bf((Bs, Hs, n, d)).pin_memory()
    a, b = mk(), mk()
    a.stream_append_layer(0, K_h.cuda(), V_h.cuda())
    b.stream_append_layer_host(0, K_h, V_h)
    a.compress()
    b.compress()
    q_h = bf((Bs, Hs * g, d)).pin_memory()
    out_h = torch.empty_like(q_h).pin_memory()
    b.decode_attn_host(0, q_h, out_h)
    torch.cuda.synchronize()
    assert torch.equal(a.decode_attn(0, q_h.cuda()).cpu(), out_h)
    qs, ks, vs = bf((steps, Bs, Hs * g, d)).pin_memory(), bf((steps, Bs, Hs, 1, d)).pin_memory(), bf((steps, Bs, Hs, 1, d)).pin_memory()
    outs_h = torch.empty_like(qs).pin_memory()
    out_d = torch.empty(Bs, Hs * g, d, dtype=torch.bfloat16, device="cuda")
    pageable = torch.empty_like(qs[0])                      # not pinned: goes through the device buffer and a copy
    for s in range(steps):
        b.stream_step_host(0, qs[s], ks[s], vs[s], pageable if s == 1 else outs_h[s])
        if s == 1:
            torch.cuda.synchronize()
            outs_h[1].copy_(pageable)
    for s in range(steps):
        a.stream_step(0, qs[s].cuda(), ks[s].cuda(), vs[s].cuda(), out_d)
        if s in (0, steps // 2, steps - 1):
            torch.cuda.synchronize()
            assert torch.equal(out_d.cpu(), outs_h[s])
    for h in range(Hs):
        assert all(torch.equal(x, y) for x, y in zip(a.cache_view(1, 0, h), b.cache_view(1, 0, h)))


def test_tokens_appended_by_decode_steps_compress_like_appended_ones(cuda_lib):
    """More decode steps than a block, then compress: the rows (and the row norms from which the radii
    of Algorithm 2 are taken) written by the fused decode step must be those an append writes --
    same running correlations S_j, bit for bit, and same caches."""
    Bs, Hs, g, d, t, n0, steps = 1, 2, 4, 128, 64, 100, 160
    mk = lambda: cuda_lib.Context(n_seqs=Bs, n_layers=1, n_kv_heads=Hs, n_q_heads=Hs * g, head_dim=d, dtype="bf16",
                                  block=t, levels=2, max_tokens=n0 + steps, seed=2, c_override=0.6)
    rng = np.random.default_rng(3)
    K = to_device(0.08 * rng.standard_normal((Bs, Hs, n0 + steps, d)).astype(np.float32), "bf16")
    V = to_device(rng.standard_normal((Bs, Hs, n0 + steps, d)).astype(np.float32), "bf16")
    q = to_device(rng.standard_normal((Bs, Hs * g, d)).astype(np.float32), "bf16")
    a, b = mk(), mk()
    for c in (a, b):
        c.debug_enable(True)
        c.stream_append_layer(0, K[:, :, :n0].contiguous(), V[:, :, :n0].contiguous())
        c.compress()
    out = torch.empty_like(q)
    for s in range(steps):
        a.stream_step(0, q, K[:, :, n0 + s:n0 + s + 1].contiguous(), V[:, :, n0 + s:n0 + s + 1].contiguous(), out)
    b.stream_append_layer(0, K[:, :, n0:].contiguous(), V[:, :, n0:].contiguous())
    a.compress()
    b.compress()
    blocks = (n0 + steps) // t
    for h in range(Hs):
        assert all(torch.equal(x, y) for x, y in zip(a.cache_view(0, 0, h), b.cache_view(0, 0, h)))
        for lvl in range(2):
            for o in range(blocks >> lvl):
                ea, Sa, _ = a.debug_call(0, 0, h, lvl, o)
                eb, Sb, _ = b.debug_call(0, 0, h, lvl, o)
                assert torch.equal(ea, eb) and torch.equal(Sa, Sb)
    assert torch.equal(a.decode_attn(0, q), b.decode_attn(0, q))
    assert a.stats()["device_status"] == 0 and a.stats()["calls_run"] == Hs * (blocks + blocks // 2)
