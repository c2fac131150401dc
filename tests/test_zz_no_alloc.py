"""The allocation-free decode entry point against the context-based one.

balancekv_decode_attn_static serves callers that may not allocate device memory (latency
critical loops, plugins fed with framework-owned buffers, fully committed memory pools): its
scratch is a fixed array inside the library.  Here it must reproduce balancekv_decode_attn
and the CPU oracle's weighted attention, within the decode tolerance of the other GPU tests, on
two calls in a row (the second call reuses the array the first one left behind), without taking
any device memory and without tripping a bounded wait.  This file sorts last on purpose."""
import numpy as np
import pytest
import torch

from paper_2502_07861_b200 import synth

pytestmark = pytest.mark.gpu

DEC_TOL = {"fp32": 1e-5, "bf16": 2e-3}


def _dev(x, dtype):
    return torch.from_numpy(np.ascontiguousarray(x)).to(torch.bfloat16 if dtype == "bf16" else torch.float32).cuda().contiguous()


@pytest.mark.parametrize("dtype,d,g,T,n_heavy,n_tail", [("bf16", 128, 4, 2, 1500, 77), ("fp32", 64, 5, 3, 640, 0)])
def test_static_scratch_decode_matches_context_decode_twice(cuda_lib, dtype, d, g, T, n_heavy, n_tail):
    bk = cuda_lib
    B, H = 3, 2
    n = n_heavy + n_tail
    K = np.stack([np.stack([synth.stream_kv("llama", 90, b, 0, h, n, d, dtype)[0] for h in range(H)]) for b in range(B)])
    V = np.stack([np.stack([synth.stream_kv("llama", 90, b, 0, h, n, d, dtype)[1] for h in range(H)]) for b in range(B)])
    ctx = bk.Context(n_seqs=B, n_layers=1, n_kv_heads=H, n_q_heads=H * g, head_dim=d, dtype=dtype, block=64, levels=T,
                     max_tokens=max(n_heavy << T, n) + 64)
    Kd, Vd = _dev(K, dtype), _dev(V, dtype)
    ctx.cache_load_level(0, T, Kd[:, :, :n_heavy].contiguous(), Vd[:, :, :n_heavy].contiguous())
    if n_tail:
        ctx.stream_append_layer(0, Kd[:, :, n_heavy:].contiguous(), Vd[:, :, n_heavy:].contiguous())
    Ks, Vs = Kd.reshape(B * H, n, d), Vd.reshape(B * H, n, d)
    out_static = torch.empty(B * H, g, d, dtype=Kd.dtype, device="cuda")
    import oracle

    w = np.concatenate([np.full(n_heavy, float(1 << T)), np.ones(n_tail)])
    for call in range(2):                                   # two calls in a row share the built-in array
        qh = synth.queries(90, 0, call, B, H * g, d, dtype)
        q = _dev(qh, dtype)
        ref = ctx.decode_attn(0, q).float().cpu().numpy().reshape(B * H, g, d)
        out_static.fill_(float("nan"))
        qs = q.reshape(B * H, g, d)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]          # device-wide free memory, not torch's pool
        bk.decode_attn_static(Ks, Vs, n_heavy, T, qs, out_static)
        torch.cuda.synchronize()
        if call == 1:                                       # the first call on a device may load the kernel image
            assert torch.cuda.mem_get_info()[0] == free_before, "the allocation-free entry point took device memory"
        got = out_static.float().cpu().numpy()
        assert np.isfinite(got).all()
        err = np.linalg.norm(got - ref) / np.linalg.norm(ref)
        assert err <= DEC_TOL[dtype], (call, err)
        # the definition itself: Theorem 3.3's estimator over the caller's rows, by the CPU oracle
        for s in range(B * H):
            exact = oracle.weighted_attention(K.reshape(B * H, n, d)[s], V.reshape(B * H, n, d)[s], w,
                                              qh.reshape(B * H, g, d)[s])
            e2 = np.linalg.norm(got[s] - exact) / np.linalg.norm(exact)
            assert e2 <= DEC_TOL[dtype], (call, s, e2)
        assert bk.decode_attn_static_status() == 0          # no bounded wait gave up
    ctx.close()


def test_static_scratch_rejects_oversized_problems(cuda_lib):
    bk = cuda_lib
    n_streams, g, d = 4096, 8, 128                          # 4096 streams x 8 heads x 130 floats > 8 MiB
    K = torch.zeros(n_streams, 64, d, dtype=torch.bfloat16, device="cuda")
    q = torch.zeros(n_streams, g, d, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(bk.BalanceKVError) as ei:
        bk.decode_attn_static(K, K, 64, 1, q)
    assert ei.value.code == bk.binding.E_NOMEM
