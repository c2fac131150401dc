"""GPU parity at the full per-stream sizes of the larger workloads: the 8B-shaped stack (block
2048, 131072 tokens, chunked prefill; two of its 32 identical layers), the 14B-shaped case (T = 3,
recent window 128, heavy-tailed keys; one layer) and the decode sweep at batch 32.  The inputs are
drawn on the device (seeded) and the oracle consumes the same bytes copied back; what the oracle
replays is a sample -- single calls, teacher-forced, and decode outputs of single streams -- the
rest is covered by properties that hold at any size."""
import numpy as np
import pytest
import torch

import oracle
from oracle import OracleParams
from parity_util import MARGIN, rel_l2

pytestmark = pytest.mark.gpu


def _gen(seed, B, H, n, d, recipe):
    """bf16 K, V [B, H, n, d] on the device."""
    g = torch.Generator(device="cuda").manual_seed(seed)
    z = torch.randn(B, H, n, d, device="cuda", generator=g)
    if recipe == "llama":
        hg = torch.Generator(device="cuda").manual_seed(977)          # per-head statistics, fixed across chunks
        mu = 0.5 * torch.randn(1, H, 1, d, device="cuda", generator=hg)
        s = torch.ones(1, H, 1, d, device="cuda")
        for h in range(H):
            s[0, h, 0, torch.randperm(d, device="cuda", generator=hg)[:4]] = 10.0
        K = (mu + z) * s
    else:                                                             # Student-t, 4 degrees of freedom
        chi = torch.randn(B, H, n, d, 4, device="cuda", generator=g).square_().sum(-1).div_(4.0).sqrt_()
        K = z / chi
    V = torch.randn(B, H, n, d, device="cuda", generator=g)
    return K.to(torch.bfloat16).contiguous(), V.to(torch.bfloat16).contiguous()


def _f64(x):
    return x.float().cpu().numpy().astype(np.float64)


def _check_call(ctx, P, K, V, seq, layer, head, level, ordinal, s_tol=2e-4):
    """Teacher-forced check of one call; returns the oracle's record (kept positions inside the call)."""
    e, S, p = ctx.debug_call(seq, layer, head, level, ordinal)
    e, S, p = e.cpu().numpy(), S.cpu().numpy().astype(np.float64), p.cpu().numpy().astype(np.float64)
    r = oracle.softmax_balance(P, K, V, ordinal=ordinal, level=level, forced=e)
    want = np.where(r["u"] < r["p"], 1, -1)
    diff = want != e
    assert np.all(np.abs(r["u"] - r["p"])[diff] < MARGIN) and diff.mean() <= 1e-3
    assert np.all(np.abs(S - r["S"]) <= 1e-6 + s_tol * np.maximum(1.0, np.abs(r["S"])))
    assert np.allclose(p, r["p"], atol=1e-5) and r["fails"] == 0
    return r


def _check_decode(ctx, layer, q, streams, g, tol=2e-3):
    out = ctx.decode_attn(layer, q).float().cpu().numpy()
    for (b, h) in streams:
        Kc, Vc, w, _ = ctx.cache_view(b, layer, h)
        ref = oracle.weighted_attention(_f64(Kc), _f64(Vc), _f64(w), _f64(q[b, h * g:(h + 1) * g]))
        assert rel_l2(out[b, h * g:(h + 1) * g], ref) <= tol


def test_8b_stack_shape_block_2048_chunked_prefill(cuda_lib):
    B, L, H, g, d, n, t, T, chunk = 4, 2, 8, 4, 128, 131072, 2048, 2, 8192
    ctx = cuda_lib.Context(n_seqs=B, n_layers=L, n_kv_heads=H, n_q_heads=H * g, head_dim=d, dtype="bf16", block=t,
                           levels=T, max_tokens=n, max_pending=chunk, seed=1)
    ctx.debug_enable(True)
    # sampled calls: level 0 (ordinal 0 and the last one), and a level-1 call with its two level-0 inputs
    want_rows = {(0, 0, 0): [0], (3, 1, 7): [63], (2, 1, 3): [34, 35]}          # (seq, layer, head) -> level-0 ordinals
    kept_rows = {}
    for c0 in range(0, n, chunk):
        for layer in range(L):
            K, V = _gen(3000 + 64 * layer + c0 // chunk, B, H, chunk, d, "llama")
            ctx.stream_append_layer(layer, K, V)
            ctx.compress()
            for (b, l, h), ords in want_rows.items():
                for o in ords:
                    if l == layer and c0 <= o * t < c0 + chunk:
                        sl = slice(o * t - c0, o * t - c0 + t)
                        kept_rows[(b, l, h, o)] = (_f64(K[b, h, sl]), _f64(V[b, h, sl]))
    st = ctx.stats()
    assert st["device_status"] == 0 and st["walk_fails"] == 0 and st["calls_run"] == B * L * H * (64 + 32)
    mk = lambda b, l, h: OracleParams(d=d, t=t, T=T, layer=l, head=h, max_tokens=n, seed=1 + b)
    _check_call(ctx, mk(0, 0, 0), *kept_rows[(0, 0, 0, 0)], 0, 0, 0, 0, 0)
    _check_call(ctx, mk(3, 1, 7), *kept_rows[(3, 1, 7, 63)], 3, 1, 7, 0, 63)
    P = mk(2, 1, 3)
    ra = _check_call(ctx, P, *kept_rows[(2, 1, 3, 34)], 2, 1, 3, 0, 34)
    rb = _check_call(ctx, P, *kept_rows[(2, 1, 3, 35)], 2, 1, 3, 0, 35)
    assert len(ra["kept"]) == t // 2 and len(rb["kept"]) == t // 2
    K1 = np.concatenate([kept_rows[(2, 1, 3, 34)][0][ra["kept"]], kept_rows[(2, 1, 3, 35)][0][rb["kept"]]])
    V1 = np.concatenate([kept_rows[(2, 1, 3, 34)][1][ra["kept"]], kept_rows[(2, 1, 3, 35)][1][rb["kept"]]])
    r1 = _check_call(ctx, P, K1, V1, 2, 1, 3, 1, 17)
    # its survivors are rows 17*1024 .. 18*1024 of C^2: positions, weights and stored rows, bit for bit
    pos1 = np.concatenate([34 * t + ra["kept"], 35 * t + rb["kept"]])[r1["kept"]]
    Kc, Vc, w, idx = ctx.cache_view(2, 1, 3)
    sl = slice(17 * (t // 2), 18 * (t // 2))
    assert np.array_equal(idx[sl].cpu().numpy(), pos1)
    assert np.array_equal(_f64(Kc[sl]), K1[r1["kept"]]) and np.array_equal(_f64(Vc[sl]), V1[r1["kept"]])
    # every stream: 4x compression, weight 4, increasing positions
    for b in range(B):
        for l in range(L):
            for h in range(0, H, 3):
                assert list(ctx.level_sizes(b, l, h)) == [0, 0, n >> T]
    _, _, w, idx = ctx.cache_view(1, 0, 5)
    assert torch.all(w == 4.0) and torch.all(idx[1:] > idx[:-1]) and int(idx[-1]) < n
    q = torch.randn(B, H * g, d, device="cuda", generator=torch.Generator(device="cuda").manual_seed(5)).to(torch.bfloat16)
    _check_decode(ctx, 1, q, [(2, 3), (0, 6)], g)
    ctx.close()


def test_14b_shape_three_levels_window_student_t(cuda_lib):
    B, L, H, g, d, n, t, T, W, chunk = 8, 1, 8, 5, 128, 65536, 1024, 3, 128, 8192
    ctx = cuda_lib.Context(n_seqs=B, n_layers=L, n_kv_heads=H, n_q_heads=H * g, head_dim=d, dtype="bf16", block=t,
                           levels=T, max_tokens=n, max_pending=chunk, recent_window=W, seed=1)
    ctx.debug_enable(True)
    first = None
    for c0 in range(0, n, chunk):
        K, V = _gen(4000 + c0 // chunk, B, H, chunk, d, "student_t")
        if c0 == 0:
            first = (_f64(K[5, 2, :4 * t]), _f64(V[5, 2, :4 * t]))        # the first four blocks of one stream
        ctx.stream_append_layer(0, K, V)
        ctx.compress()
    st = ctx.stats()
    assert st["device_status"] == 0 and st["calls_run"] == B * H * (63 + 31 + 15)
    # one teacher-forced chain through every level: level-0 calls 0..3 of a stream, the level-1 calls 0 and 1 on
    # their survivors, the level-2 call 0 on theirs; its survivors are the first rows of C^3
    P = OracleParams(d=d, t=t, T=T, W=W, layer=0, head=2, max_tokens=n, seed=1 + 5)
    Kl, Vl, pos = [first[0][i * t:(i + 1) * t] for i in range(4)], [first[1][i * t:(i + 1) * t] for i in range(4)], \
        [np.arange(i * t, (i + 1) * t) for i in range(4)]
    for level in range(T):
        Kn, Vn, pn = [], [], []
        for o in range(len(Kl)):
            r = _check_call(ctx, P, Kl[o], Vl[o], 5, 0, 2, level, o)
            assert len(r["kept"]) == t // 2
            Kn.append(Kl[o][r["kept"]]); Vn.append(Vl[o][r["kept"]]); pn.append(pos[o][r["kept"]])
        Kl = [np.concatenate(Kn[i:i + 2]) for i in range(0, len(Kn), 2)]
        Vl = [np.concatenate(Vn[i:i + 2]) for i in range(0, len(Vn), 2)]
        pos = [np.concatenate(pn[i:i + 2]) for i in range(0, len(pn), 2)]
    Kc, Vc, w, idx = ctx.cache_view(5, 0, 2)
    assert np.array_equal(idx[:t // 2].cpu().numpy(), pos[0]) and torch.all(w[:t // 2] == 8.0)
    assert np.array_equal(_f64(Kc[:t // 2]), Kl[0]) and np.array_equal(_f64(Vc[:t // 2]), Vl[0])
    # stored per stream: 15*512 rows at weight 8, 512 at 4, 512 at 2, 896 + the window of 128 at 1
    for b in (0, 7):
        for h in (0, 4):
            assert list(ctx.level_sizes(b, 0, h)) == [896 + W, 512, 512, 15 * 512]
            _, _, w, idx = ctx.cache_view(b, 0, h)
            assert float(w.double().sum()) == n and torch.all(idx[1:] > idx[:-1])
            assert torch.equal(idx[-W:].cpu(), torch.arange(n - W, n, dtype=torch.int32))
    q = torch.randn(B, H * g, d, device="cuda", generator=torch.Generator(device="cuda").manual_seed(6)).to(torch.bfloat16)
    _check_decode(ctx, 0, q, [(0, 0), (7, 4)], g)
    ctx.close()


@pytest.mark.parametrize("Lc,T", [(32768, 3), (2048, 1)])
def test_decode_sweep_shape_batch_32(cuda_lib, Lc, T):
    B, H, g, d = 32, 8, 5, 128
    ctx = cuda_lib.Context(n_seqs=B, n_layers=1, n_kv_heads=H, n_q_heads=H * g, head_dim=d, dtype="bf16", block=64,
                           levels=T, max_tokens=Lc << T)
    K, V = _gen(5000 + T, B, H, Lc, d, "llama")
    ctx.cache_load_level(0, T, K, V)
    q = torch.randn(B, H * g, d, device="cuda", generator=torch.Generator(device="cuda").manual_seed(7)).to(torch.bfloat16)
    out = ctx.decode_attn(0, q).float().cpu().numpy()
    assert ctx.stats()["device_status"] == 0
    for (b, h) in [(0, 0), (17, 5), (31, 7)]:
        ref = oracle.weighted_attention(_f64(K[b, h]), _f64(V[b, h]), np.full(Lc, 2.0 ** T), _f64(q[b, h * g:(h + 1) * g]))
        assert rel_l2(out[b, h * g:(h + 1) * g], ref) <= 2e-3
    ctx.close()
