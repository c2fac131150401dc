"""GPU parity: the CUDA library against the CPU oracle on the same seeded inputs, through the
C ABI.  Tolerances: kept indices / weights / stored rows bit-exact given the signs; sign
decisions equal unless the walk margin is below 1e-5 (counted, < 0.1 %); S_j within the
stated tolerance; decode within 2e-3 (bf16) / 1e-5 (fp32) relative L2."""
import numpy as np
import pytest
import torch

from oracle import OracleParams, OracleStream
import oracle
from paper_2502_07861_b200 import synth
from parity_util import Harness, rel_l2, to_device

pytestmark = pytest.mark.gpu

S_TOL = {"fp32": 2e-5, "bf16": 2e-4}
DEC_TOL = {"fp32": 1e-5, "bf16": 2e-3}


def _layer_inputs(recipe, data_seed, B, L, H, n, d, dtype, key_scale=1.0):
    K = np.empty((B, L, H, n, d), np.float32)
    V = np.empty_like(K)
    for b in range(B):
        for l in range(L):
            for h in range(H):
                k, v = synth.stream_kv(recipe, data_seed, b, l, h, n, d, dtype)
                K[b, l, h] = synth.round_to(k * key_scale, dtype)
                V[b, l, h] = v
    return K, V


def test_tiny_single_head_fp32(cuda_lib):
    """1 layer, 1 KV head, d=64, 1024 tokens in blocks of 256, T=1, fp32, seed 0, 16 queries."""
    K, V = _layer_inputs("outlier2", 1001, 1, 1, 1, 1024, 64, "fp32")
    hz = Harness(cuda_lib, B=1, L=1, H=1, g=1, d=64, dtype="fp32", t=256, T=1, N=1024, seed=0)
    for b in range(4):
        hz.append_layer(0, K[:, 0, :, b * 256:(b + 1) * 256], V[:, 0, :, b * 256:(b + 1) * 256])
        hz.compress()
    tot, marg = hz.check_all(S_TOL["fp32"])
    assert tot == 1024
    Kc, Vc, w, idx = hz.ctx.cache_view(0, 0, 0)
    assert len(idx) == 512 and torch.all(w == 2.0) and float(w.sum()) == 1024
    for step in range(16):
        q = synth.queries(1001, 0, step, 1, 1, 64, "fp32")
        hz.check_decode(0, q, DEC_TOL["fp32"])
    st = hz.ctx.stats()
    assert st["device_status"] == 0 and st["calls_run"] == 4 and st["walk_fails"] == 0


@pytest.mark.parametrize("dtype,d,t,T,gram", [("fp32", 128, 256, 2, 1), ("bf16", 128, 256, 2, 1), ("bf16", 64, 128, 3, 1),
                                              ("fp32", 64, 64, 1, 1), ("bf16", 128, 128, 1, 2), ("bf16", 128, 256, 2, 2),
                                              ("bf16", 128, 1024, 2, 2)])
def test_aggressive_walk_exercises_the_gram_arithmetic(cuda_lib, dtype, d, t, T, gram):
    """Small c and small keys make p_j stray far from 1/2, so S_j parity tests every Gram entry."""
    B, L, H, g = 1, 2, 2, 4
    n = t * (8 if t < 1024 else 4) + 37
    K, V = _layer_inputs("llama", 77, B, L, H, n, d, dtype, key_scale=0.06)
    hz = Harness(cuda_lib, B=B, L=L, H=H, g=g, d=d, dtype=dtype, t=t, T=T, N=n, seed=3, c_override=0.75, gram_path=gram)
    for l in range(L):
        hz.append_layer(l, K[:, l], V[:, l])
    hz.compress()
    tot, marg = hz.check_all(S_TOL[dtype])
    assert tot > 0
    # the walk really is non-degenerate here
    ps = np.concatenate([c["p"] for o in hz.oracles.values() for c in o.calls()])
    assert np.mean(np.abs(ps - 0.5) > 0.05) > 0.2
    for l in range(L):
        q = synth.queries(77, l, 0, B, H * g, d, dtype)
        hz.check_decode(l, q, DEC_TOL[dtype])
    assert hz.ctx.stats()["device_status"] == 0


def test_student_t_keys_window_and_three_levels_streamed_in_chunks(cuda_lib):
    """14B-shaped case, reduced: g=5, T=3, recent window 128, heavy-tailed keys, chunked prefill,
    then decode steps that append one token per stream (kept uncompressed)."""
    B, L, H, g, d, t, T, W = 2, 1, 2, 5, 128, 128, 3, 128
    n, chunk = 128 * 19 + 60, 512
    K, V = _layer_inputs("student_t", 1004, B, L, H, n + 8, d, "bf16")
    hz = Harness(cuda_lib, B=B, L=L, H=H, g=g, d=d, dtype="bf16", t=t, T=T, N=n + 8, W=W, seed=1, max_pending=chunk)
    for c0 in range(0, n, chunk):
        c1 = min(n, c0 + chunk)
        hz.append_layer(0, K[:, 0, :, c0:c1], V[:, 0, :, c0:c1])
        hz.compress()
    hz.check_all(S_TOL["bf16"])
    sizes = hz.ctx.level_sizes(0, 0, 0)
    eligible = n - W
    assert sum(int(sizes[l]) << l for l in range(T + 1)) == n
    assert sizes[0] == eligible % t + W
    for step in range(8):
        q = synth.queries(1004, 0, step, B, H * g, d, "bf16")
        hz.check_decode(0, q, DEC_TOL["bf16"])
        hz.append_layer(0, K[:, 0, :, n + step:n + step + 1], V[:, 0, :, n + step:n + step + 1])   # decode-phase token
        # no new calls fire (compress is not called in the decode phase): replay with the same signs
        hz.oracles = {k: hz.oracle_replay(*k, rec=hz.recs[k]) for k in hz.oracles}
        for (s_, l_, h_), o in hz.oracles.items():
            Kg, Vg, wg, ig = hz.ctx.cache_view(s_, l_, h_)
            assert np.array_equal(ig.cpu().numpy(), o.view()[3])
            assert np.all(wg.cpu().numpy()[-(step + 1):] == 1.0)


def test_T0_is_exact_attention_and_empty_streams_give_zeros(cuda_lib):
    B, L, H, g, d = 2, 1, 2, 4, 128
    ctx = cuda_lib.Context(n_seqs=B, n_layers=L, n_kv_heads=H, n_q_heads=H * g, head_dim=d, dtype="bf16", block=64,
                           levels=0, max_tokens=700)
    q = synth.queries(5, 0, 0, B, H * g, d, "bf16")
    out = ctx.decode_attn(0, to_device(q, "bf16")).float().cpu().numpy()
    assert np.all(out == 0)
    n = 333                                  # ragged: not a multiple of any tile
    K, V = _layer_inputs("llama", 5, B, L, H, n, d, "bf16")
    ctx.stream_append_layer(0, to_device(K[:, 0], "bf16"), to_device(V[:, 0], "bf16"))
    ctx.compress()
    out = ctx.decode_attn(0, to_device(q, "bf16")).float().cpu().numpy()
    for b in range(B):
        for h in range(H):
            ref = oracle.weighted_attention(K[b, 0, h], V[b, 0, h], None, q[b, h * g:(h + 1) * g])
            assert rel_l2(out[b, h * g:(h + 1) * g], ref) <= DEC_TOL["bf16"]
    assert ctx.stats()["tokens_stored"] == B * H * n


def test_per_stream_append_ragged_lengths_and_errors(cuda_lib):
    bk = cuda_lib
    B, L, H, g, d, t = 2, 2, 2, 2, 64, 64
    ctx = bk.Context(n_seqs=B, n_layers=L, n_kv_heads=H, n_q_heads=H * g, head_dim=d, dtype="fp32", block=t, levels=2,
                     max_tokens=1000, seed=9, c_override=0.5)
    ctx.debug_enable(True)
    lens = {(0, 0, 0): 64 * 5 + 3, (0, 0, 1): 10, (1, 1, 0): 64 * 4, (1, 1, 1): 0, (1, 0, 1): 64 * 2 + 63}
    data = {}
    for (s, l, h), n in lens.items():
        k, v = synth.stream_kv("llama", 31, s, l, h, max(n, 1), d, "fp32")
        k = synth.round_to(0.1 * k, "fp32")
        data[(s, l, h)] = (k[:n], v[:n])
        if n:
            ctx.stream_append(s, l, h, to_device(k[:n], "fp32"), to_device(v[:n], "fp32"))
    ctx.compress()
    for (s, l, h), n in lens.items():
        o = OracleStream(OracleParams(d=d, t=t, T=2, layer=l, head=h, max_tokens=1000, seed=9 + s, c_override=0.5))
        if n:
            o.append(*data[(s, l, h)])
        o.compress()
        # follow the GPU's signs
        blocks = n // t
        o2 = OracleStream(OracleParams(d=d, t=t, T=2, layer=l, head=h, max_tokens=1000, seed=9 + s, c_override=0.5))
        for lvl in range(2):
            for od in range(blocks >> lvl):
                e, _, _ = ctx.debug_call(s, l, h, lvl, od)
                o2.force_eta(lvl, od, e.cpu().numpy())
        if n:
            o2.append(*data[(s, l, h)])
        o2.compress()
        Kg, Vg, wg, ig = ctx.cache_view(s, l, h)
        assert np.array_equal(ig.cpu().numpy(), o2.view()[3]) and np.array_equal(wg.cpu().numpy(), o2.view()[2])
        for c in o2.calls():
            want = np.where(c["u"] < c["p"], 1, -1)
            bad = want != c["eta"]
            assert np.all(np.abs(c["u"] - c["p"])[bad] < 1e-5)
    # decode over streams of different lengths (one empty) in one launch
    for l in range(L):
        q = synth.queries(31, l, 0, B, H * g, d, "fp32")
        out = ctx.decode_attn(l, to_device(q, "fp32")).float().cpu().numpy()
        for s in range(B):
            for h in range(H):
                Kg, Vg, wg, _ = ctx.cache_view(s, l, h)
                if len(wg) == 0:
                    assert np.all(out[s, h * g:(h + 1) * g] == 0)
                    continue
                ref = oracle.weighted_attention(Kg.cpu().numpy(), Vg.cpu().numpy(), wg.cpu().numpy(), q[s, h * g:(h + 1) * g])
                assert rel_l2(out[s, h * g:(h + 1) * g], ref) <= DEC_TOL["fp32"]
    # errors
    k = torch.zeros(2000, d, device="cuda")
    with pytest.raises(bk.BalanceKVError) as ei:
        ctx.stream_append(0, 0, 0, k, k)
    assert ei.value.code == bk.binding.E_NOMEM
    with pytest.raises(bk.BalanceKVError) as ei:
        ctx.compress(T=1)
    assert ei.value.code == bk.binding.E_INVAL
    with pytest.raises(bk.BalanceKVError):
        ctx.stream_append(5, 0, 0, k[:1], k[:1])
    with pytest.raises(bk.BalanceKVError):
        bk.Context(head_dim=96)


@pytest.mark.parametrize("gram", [1, 2])
def test_key_centering_flag(cuda_lib, gram):
    B, L, H, g, d, t = 1, 1, 2, 1, 128, 128
    n = t * 4
    K, V = _layer_inputs("llama", 41, B, L, H, n, d, "bf16", key_scale=0.06)
    K = synth.round_to(K + 1.5, "bf16")       # a large common offset that centering removes
    hz = Harness(cuda_lib, B=B, L=L, H=H, g=g, d=d, dtype="bf16", t=t, T=1, N=n, seed=2, c_override=0.75, center_keys=1,
                 gram_path=gram)
    hz.append_layer(0, K[:, 0], V[:, 0])
    hz.compress()
    hz.check_all(5e-4)


def test_two_runs_are_bit_identical(cuda_lib):
    B, L, H, g, d, t = 1, 1, 4, 4, 128, 256
    n = t * 4
    K, V = _layer_inputs("llama", 51, B, L, H, n, d, "bf16", key_scale=0.06)
    q = to_device(synth.queries(51, 0, 0, B, H * g, d, "bf16"), "bf16")
    outs = []
    for _ in range(2):
        ctx = cuda_lib.Context(n_seqs=B, n_layers=L, n_kv_heads=H, n_q_heads=H * g, head_dim=d, dtype="bf16", block=t,
                               levels=2, max_tokens=n, seed=4, c_override=0.75)
        ctx.debug_enable(True)
        ctx.stream_append_layer(0, to_device(K[:, 0], "bf16"), to_device(V[:, 0], "bf16"))
        ctx.compress()
        S = torch.cat([ctx.debug_call(0, 0, h, 0, o)[1] for h in range(H) for o in range(4)])
        view = [ctx.cache_view(0, 0, h)[3] for h in range(H)]
        outs.append((S.clone(), view, ctx.decode_attn(0, q).clone()))
        ctx.close()
    assert torch.equal(outs[0][0], outs[1][0])
    assert all(torch.equal(a, b) for a, b in zip(outs[0][1], outs[1][1]))
    assert torch.equal(outs[0][2], outs[1][2])


def test_loaded_cache_decode_sweep_shape(cuda_lib):
    """Decode-sweep case, reduced: cache built directly at level T with weights 2^T and
    uniform-random kept positions, g=5."""
    B, L, H, g, d = 3, 1, 2, 5, 128
    for T, Lc in ((1, 1000), (3, 2048 + 17)):
        ctx = cuda_lib.Context(n_seqs=B, n_layers=L, n_kv_heads=H, n_q_heads=H * g, head_dim=d, dtype="bf16", block=64,
                               levels=T, max_tokens=Lc << T)
        K, V = _layer_inputs("llama", 1005, B, L, H, Lc, d, "bf16")
        idx = np.stack([np.stack([synth.kept_positions(1005, b, 0, h, Lc, T) for h in range(H)]) for b in range(B)])
        ctx.cache_load_level(0, T, to_device(K[:, 0], "bf16"), to_device(V[:, 0], "bf16"),
                             torch.from_numpy(idx).cuda().contiguous())
        q = synth.queries(1005, 0, 0, B, H * g, d, "bf16")
        out = ctx.decode_attn(0, to_device(q, "bf16")).float().cpu().numpy()
        for b in range(B):
            for h in range(H):
                Kg, Vg, wg, ig = ctx.cache_view(b, 0, h)
                assert torch.all(wg == 2.0 ** T) and np.array_equal(ig.cpu().numpy(), idx[b, h])
                ref = oracle.weighted_attention(K[b, 0, h], V[b, 0, h], np.full(Lc, 2.0 ** T), q[b, h * g:(h + 1) * g])
                assert rel_l2(out[b, h * g:(h + 1) * g], ref) <= DEC_TOL["bf16"]
        ctx.close()


@pytest.mark.parametrize("gram", [1, 2])
def test_degenerate_inputs_zero_values_and_duplicate_tokens(cuda_lib, gram):
    """All-zero values (r_value = 0: the kernel vanishes and the signs are the coins alone) and
    identical tokens (Ghat = 1 everywhere: with a small constant every other step hits the FAIL clamp,
    and both sides must count the same FAILs)."""
    B, L, H, g, d, t = 1, 2, 1, 2, 128, 128
    n = t * 4
    K, V = _layer_inputs("llama", 61, B, L, H, n, d, "bf16", key_scale=0.06)
    V[:, 0] = 0.0                                              # layer 0: zero values
    K[:, 1] = K[:, 1, :, :1]                                   # layer 1: every token equals the first one
    V[:, 1] = V[:, 1, :, :1]
    hz = Harness(cuda_lib, B=B, L=L, H=H, g=g, d=d, dtype="bf16", t=t, T=2, N=n, seed=8, c_override=0.3, gram_path=gram)
    for l in range(L):
        hz.append_layer(l, K[:, l], V[:, l])
    hz.compress()
    hz.check_all(S_TOL["bf16"])
    zero = hz.oracles[(0, 0, 0)].calls()
    assert all(np.all(c["S"] == 0) and np.all(c["p"] == 0.5) for c in zero)
    dup_fails = sum(c["fails"] for c in hz.oracles[(0, 1, 0)].calls())
    assert dup_fails >= 0.4 * sum(len(c["eta"]) for c in hz.oracles[(0, 1, 0)].calls())   # every other step: S swings past c and back
    assert hz.ctx.stats()["walk_fails"] == dup_fails + sum(c["fails"] for c in zero)
    for l in range(L):
        q = synth.queries(61, l, 0, B, H * g, d, "bf16")
        if l == 0:
            assert np.all(hz.ctx.decode_attn(0, to_device(q, "bf16")).float().cpu().numpy() == 0)
        else:
            hz.check_decode(l, q, DEC_TOL["bf16"])


def test_a_timed_out_wait_surfaces_as_an_error_code_and_reset_clears_it(cuda_lib):
    """A bounded device-side wait that gives up sets the context's status word; here the word is set
    from the host (no kernel is made to hang).  stats() then reports it, every call that would
    enqueue work is refused with BALANCEKV_E_TIMEOUT, and reset() makes the context usable again."""
    bk = cuda_lib
    ctx = bk.Context(n_seqs=1, n_layers=1, n_kv_heads=2, n_q_heads=8, head_dim=128, dtype="bf16", block=128, levels=1,
                     max_tokens=1024)
    K = torch.randn(1, 2, 256, 128, device="cuda").to(torch.bfloat16)
    q = torch.randn(1, 8, 128, device="cuda").to(torch.bfloat16)
    ctx.stream_append_layer(0, K, K)
    ctx.compress()
    st = ctx.stats()
    assert st["device_status"] == 0 and st["walk_kernel"] == 2 and st["decode_kernel"] == 2
    ctx.debug_set_status(1)
    assert ctx.stats()["device_status"] == 1
    for call in (lambda: ctx.decode_attn(0, q), lambda: ctx.stream_append_layer(0, K, K), lambda: ctx.compress()):
        with pytest.raises(bk.BalanceKVError) as ei:
            call()
        assert ei.value.code == bk.binding.E_TIMEOUT
    ctx.reset()
    ctx.stream_append_layer(0, K, K)
    ctx.compress()
    ctx.decode_attn(0, q)
    assert ctx.stats()["device_status"] == 0
    ctx.close()


@pytest.mark.parametrize("g", [1, 2, 3, 5, 6, 7, 8])
@pytest.mark.parametrize("splits", [1, 5, 24, 64])
def test_decode_kernel_every_group_size_and_split_factor(cuda_lib, g, splits):
    """The tensor-core decode kernel against the oracle's weighted attention for every group size (g <= 4 packs the
    high and low parts of the probabilities into one MMA) and for split factors that take each of its combine
    paths: a single split (the result stays in the CTA), a few splits, more splits than tiles (empty partial rows),
    and a grid of several waves (64 splits + g - 1 combining CTAs per stream).  Two levels with ragged lengths, one
    of them shorter than a tile.  Behind every launch the split-K scratch is empty again."""
    B, H, d, T, n_heavy, n_tail = 1, 2, 128, 2, 2500, 37
    ctx = cuda_lib.Context(n_seqs=B, n_layers=1, n_kv_heads=H, n_q_heads=H * g, head_dim=d, dtype="bf16", block=64, levels=T,
                           max_tokens=(n_heavy << T) + 64, decode_splits=splits)
    K, V = synth.layer_kv("llama", 31, 0, B, H, n_heavy + n_tail, d, "bf16")
    ctx.cache_load_level(0, T, to_device(K[:, :, :n_heavy], "bf16"), to_device(V[:, :, :n_heavy], "bf16"))
    ctx.stream_append_layer(0, to_device(K[:, :, n_heavy:], "bf16"), to_device(V[:, :, n_heavy:], "bf16"))
    w = np.concatenate([np.full(n_heavy, 4.0), np.ones(n_tail)])
    for step in range(2):                                   # twice: the scratch is reused
        q = synth.queries(31, 0, step, B, H * g, d, "bf16")
        out = ctx.decode_attn(0, to_device(q, "bf16")).float().cpu().numpy()
        assert ctx.debug_scratch_used() == 0
        for h in range(H):
            ref = oracle.weighted_attention(K[0, h], V[0, h], w, q[0, h * g:(h + 1) * g])
            assert rel_l2(out[0, h * g:(h + 1) * g], ref) <= 2e-3, (g, splits, h)
    st = ctx.stats()
    assert st["device_status"] == 0 and st["decode_kernel"] == 2
    ctx.close()


def test_decode_scratch_is_empty_behind_every_launch_while_the_split_factor_moves(cuda_lib):
    """The partial rows of the tensor-core decode kernel are their own arrival flags: a launch must find and leave
    every word of the split-K scratch empty, whatever split factor the launch before it used.  Decode steps (attend +
    append) with compress points in between walk the automatic split factor through several values; every output is
    checked against the oracle's weighted attention over the library's own cache view."""
    B, H, g, d, t, T = 1, 2, 4, 128, 64, 2
    ctx = cuda_lib.Context(n_seqs=B, n_layers=1, n_kv_heads=H, n_q_heads=H * g, head_dim=d, dtype="bf16", block=t, levels=T,
                           max_tokens=8192)
    K, V = synth.layer_kv("llama", 77, 0, B, H, 6000, d, "bf16")
    pos = 0
    for n_new in (130, 700, 64, 2100, 1500):
        ctx.stream_append_layer(0, to_device(K[:, :, pos:pos + n_new], "bf16"), to_device(V[:, :, pos:pos + n_new], "bf16"))
        pos += n_new
        ctx.compress()
        for step in range(3):
            q = synth.queries(77, 0, pos + step, B, H * g, d, "bf16")
            kn, vn = K[:, :, pos], V[:, :, pos]                                  # [B, H, d]
            views = [ctx.cache_view(0, 0, h) for h in range(H)]                  # the weighted set before the step
            q_t = to_device(q, "bf16")
            out_t = q_t.clone()
            ctx.stream_step(0, q_t, to_device(kn, "bf16"), to_device(vn, "bf16"), out_t)
            out = out_t.float().cpu().numpy()
            pos += 1
            assert ctx.debug_scratch_used() == 0
            for h in range(H):
                vK, vV, vw, _ = views[h]
                Kh = np.concatenate([vK.float().cpu().numpy().astype(np.float64), kn[0, h][None].astype(np.float64)])
                Vh = np.concatenate([vV.float().cpu().numpy().astype(np.float64), vn[0, h][None].astype(np.float64)])
                wh = np.concatenate([vw.float().cpu().numpy().astype(np.float64), np.ones(1)])
                ref = oracle.weighted_attention(Kh, Vh, wh, q[0, h * g:(h + 1) * g])
                assert rel_l2(out[0, h * g:(h + 1) * g], ref) <= 2e-3, (pos, h, len(wh))
    st = ctx.stats()
    assert st["device_status"] == 0 and st["decode_kernel"] == 2
    ctx.close()
