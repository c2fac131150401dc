"""GPU parity of Algorithm 1 with its separate denominator instance (no value-norm buckets):
slot 0 of the context holds (k_j, v_j), slot 1 holds (k_j, 1); both are compressed by the same
MergeAndReduce machinery with independent coins, and decode divides the numerator of slot 0 by
the denominator of slot 1."""
import numpy as np
import pytest
import torch

import oracle
from paper_2502_07861_b200 import synth
from parity_util import Harness, rel_l2, to_device

pytestmark = pytest.mark.gpu


def _unit(shape):
    E = np.zeros(shape, np.float32)
    E[..., 0] = 1.0
    return E


@pytest.mark.parametrize("t,T,key_scale,c", [(128, 2, 0.06, 0.75), (256, 1, 1.0, 0.0)])
def test_two_instance_estimator(cuda_lib, t, T, key_scale, c):
    B, H, g, d = 2, 2, 4, 128
    n = t * 6 + 29
    K = np.empty((B, H, n, d), np.float32)
    V = np.empty_like(K)
    for b in range(B):
        for h in range(H):
            k, v = synth.stream_kv("llama", 91, b, 0, h, n, d, "bf16")
            K[b, h], V[b, h] = synth.round_to(k * key_scale, "bf16"), v
    hz = Harness(cuda_lib, B=B, L=2, H=H, g=g, d=d, dtype="bf16", t=t, T=T, N=n, seed=4, c_override=c)
    hz.append_layer(0, K, V)                                   # numerator instance
    hz.ctx.stream_append_layer_keys(1, to_device(K, "bf16"))   # denominator instance: the library supplies the 1
    hz.events.append(("append", 1, K, _unit(K.shape)))
    hz.compress()
    tot, _ = hz.check_all(2e-4)        # signs, kept sets, weights and stored rows (unit values included) of both slots
    assert tot == 2 * B * H * sum((n // t) >> l for l in range(T)) * t
    kept = [hz.oracles[(0, l, 1)].view()[3] for l in (0, 1)]
    if c > 0:
        assert not np.array_equal(kept[0], kept[1])            # the two instances keep their own subsets
    for step in range(3):
        q = synth.queries(91, 0, step, B, H * g, d, "bf16")
        out = hz.ctx.decode_attn_two(0, 1, to_device(q, "bf16")).float().cpu().numpy()
        for b in range(B):
            for h in range(H):
                ref = oracle.two_instance_estimate(hz.oracles[(b, 0, h)].view(), hz.oracles[(b, 1, h)].view(),
                                                   q[b, h * g:(h + 1) * g])
                assert rel_l2(out[b, h * g:(h + 1) * g], ref) <= 2e-3
    assert hz.ctx.stats()["device_status"] == 0


def test_two_instance_T0_is_exact_attention_and_empty_slots_give_zeros(cuda_lib):
    B, H, g, d, n = 1, 2, 4, 128, 333
    ctx = cuda_lib.Context(n_seqs=B, n_layers=2, n_kv_heads=H, n_q_heads=H * g, head_dim=d, dtype="bf16", block=64,
                           levels=0, max_tokens=n)
    q = synth.queries(92, 0, 0, B, H * g, d, "bf16")
    assert np.all(ctx.decode_attn_two(0, 1, to_device(q, "bf16")).float().cpu().numpy() == 0)
    K = np.stack([np.stack([synth.stream_kv("llama", 92, 0, 0, h, n, d, "bf16")[0] for h in range(H)])])
    V = np.stack([np.stack([synth.stream_kv("llama", 92, 0, 0, h, n, d, "bf16")[1] for h in range(H)])])
    ctx.stream_append_layer(0, to_device(K, "bf16"), to_device(V, "bf16"))
    ctx.stream_append_layer_keys(1, to_device(K, "bf16"))
    ctx.compress()
    out = ctx.decode_attn_two(0, 1, to_device(q, "bf16")).float().cpu().numpy()
    for h in range(H):
        ref = oracle.weighted_attention(K[0, h], V[0, h], None, q[0, h * g:(h + 1) * g])
        assert rel_l2(out[0, h * g:(h + 1) * g], ref) <= 2e-3
    with pytest.raises(cuda_lib.BalanceKVError):
        cuda_lib.Context(n_seqs=1, n_layers=2, n_kv_heads=1, n_q_heads=1, head_dim=64, dtype="fp32", block=64, levels=0,
                         max_tokens=64).decode_attn_two(0, 1, torch.zeros(1, 1, 64, device="cuda"))


def test_error_sweep_point_small_c_beats_uniform_on_clustered_keys(cuda_lib):
    """One point of the error-against-rate sweep: on near-duplicate keys a small walk constant gives a
    clearly lower attention error than uniform sampling at the same rate, the paper's constant about
    the same (its walk is almost a fair coin at these norms)."""
    from paper_2502_07861_b200 import error_sweep

    acc = {}
    for seed in range(4):
        for k, v in error_sweep.run_point("clustered", seed, 2, 4096, 128, 128, 2, 0.25, 0).items():
            acc[k] = acc.get(k, 0.0) + v / 4
    assert acc["balancekv_small_c"] < 0.7 * acc["uniform"]
    assert 0.5 * acc["uniform"] < acc["balancekv_paper_c"] < 2.0 * acc["uniform"]
    assert acc["balancekv_paper_c_fails"] == 0


def test_merged_decode_first_tokens_exact_recent_window_and_compressed_middle(cuda_lib):
    """The paper's single-layer setting: slot 0 keeps the first 256 tokens and is never compressed,
    slot 1 runs BalanceKV on the rest with a recent window; decode merges the two slots."""
    B, H, g, d, t, T, W, sink = 1, 2, 4, 128, 128, 2, 64, 256
    n = sink + t * 8 + 50
    K = np.empty((B, H, n, d), np.float32)
    V = np.empty_like(K)
    for h in range(H):
        k, v = synth.stream_kv("llama", 93, 0, 0, h, n, d, "bf16")
        K[0, h], V[0, h] = synth.round_to(0.06 * k, "bf16"), v
    hz = Harness(cuda_lib, B=B, L=2, H=H, g=g, d=d, dtype="bf16", t=t, T=T, N=n, W=W, seed=6, c_override=0.75)
    hz.append_layer(0, K[:, :, :sink], V[:, :, :sink])
    hz.append_layer(1, K[:, :, sink:], V[:, :, sink:])
    hz.ctx.compress_layer(1)                                    # slot 0 stays as it is
    # the oracle side: only slot 1's stream compresses
    hz.events.append(("compress",))
    hz.oracle_replay_orig = hz.oracle_replay

    def replay(seq, layer, head, rec=None):
        saved = hz.events
        hz.events = [e for e in saved if not (e[0] == "compress" and layer == 0)]
        try:
            return hz.oracle_replay_orig(seq, layer, head, rec)
        finally:
            hz.events = saved

    hz.oracle_replay = replay
    hz.check_all(2e-4)
    assert list(hz.ctx.level_sizes(0, 0, 0)) == [sink, 0, 0]
    for step in range(2):
        q = synth.queries(93, 0, step, B, H * g, d, "bf16")
        out = hz.ctx.decode_attn_merged([0, 1], [0, 1], to_device(q, "bf16")).float().cpu().numpy()
        for h in range(H):
            views = [hz.oracles[(0, 0, h)].view(), hz.oracles[(0, 1, h)].view()]
            assert views[0][2].sum() + views[1][2].sum() == n
            ref = oracle.merged_estimate(views, views, q[0, h * g:(h + 1) * g])
            assert rel_l2(out[0, h * g:(h + 1) * g], ref) <= 2e-3
    with pytest.raises(cuda_lib.BalanceKVError):
        hz.ctx.decode_attn_merged([0, 0], [1], to_device(q, "bf16"))
    assert hz.ctx.stats()["device_status"] == 0
