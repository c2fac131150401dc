"""Seeded random scenarios against the oracle: whole-layer and per-stream appends of random sizes
(the latter take a layer's streams out of lockstep), compress calls at random points, decode steps
that append (fused when the layer is in lockstep, two launches otherwise), recent windows, several
levels.  After every scenario: teacher-forced parity of every call, bit-exact caches, decode within
tolerance, and the token count of every stream."""
import numpy as np
import pytest

from paper_2502_07861_b200 import synth
from parity_util import Harness, rel_l2, to_device

pytestmark = pytest.mark.gpu


def _rows(rng, n, d, scale, dtype="bf16"):
    K = synth.round_to((scale * rng.standard_normal((n, d))).astype(np.float32), dtype)
    V = synth.round_to(rng.standard_normal((n, d)).astype(np.float32), dtype)
    return K, V


@pytest.mark.parametrize("seed,dtype,d", [(s, "bf16", 128) for s in range(16)] + [(100 + s, "fp32", 64) for s in range(4)]
                         + [(200, "fp32", 128), (201, "bf16", 64)])
def test_random_scenario(cuda_lib, seed, dtype, d):
    """bf16 / d = 128 runs on the tensor-core kernels, the other combinations on the CUDA-core ones."""
    rng = np.random.default_rng(1000 + seed)
    s_tol, dec_tol = (2e-4, 2e-3) if dtype == "bf16" else (2e-5, 1e-5)
    B, L, H = int(rng.integers(1, 3)), int(rng.integers(1, 3)), int(rng.integers(1, 3))
    g = int(rng.choice([1, 4, 5]))
    t = int(rng.choice([64, 128]))
    T = int(rng.integers(1, 4))
    W = int(rng.choice([0, 16]))
    c = float(rng.choice([0.0, 0.6]))
    N = 12 * t
    hz = Harness(cuda_lib, B=B, L=L, H=H, g=g, d=d, dtype=dtype, t=t, T=T, N=N, W=W, seed=seed, c_override=c)
    count = np.zeros((B, L, H), np.int64)
    room = lambda: N - int(count.max())
    for _ in range(int(rng.integers(6, 12))):
        op = rng.choice(["layer", "layer", "stream", "compress", "steps"])
        if op == "layer" and room() > 1:
            n = int(rng.integers(1, min(3 * t, room()) + 1))
            l = int(rng.integers(0, L))
            KV = [[_rows(rng, n, d, 0.06, dtype) for _ in range(H)] for _ in range(B)]
            K = np.stack([np.stack([KV[b][h][0] for h in range(H)]) for b in range(B)])
            V = np.stack([np.stack([KV[b][h][1] for h in range(H)]) for b in range(B)])
            hz.append_layer(l, K, V)
            count[:, l, :] += n
        elif op == "stream" and room() > 1:
            n = int(rng.integers(1, min(t, room()) + 1))
            b, l, h = int(rng.integers(0, B)), int(rng.integers(0, L)), int(rng.integers(0, H))
            hz.append_stream(b, l, h, *_rows(rng, n, d, 0.06, dtype))
            count[b, l, h] += n
        elif op == "compress":
            hz.compress()
        elif op == "steps" and room() > 4:
            l = int(rng.integers(0, L))
            for _ in range(int(rng.integers(1, 4))):
                KV = [[_rows(rng, 1, d, 0.06, dtype) for _ in range(H)] for _ in range(B)]
                K = np.stack([np.stack([KV[b][h][0] for h in range(H)]) for b in range(B)])
                V = np.stack([np.stack([KV[b][h][1] for h in range(H)]) for b in range(B)])
                q = synth.round_to(rng.standard_normal((B, H * g, d)).astype(np.float32), dtype)
                out = hz.ctx.stream_step(0 + l, to_device(q, dtype), to_device(K, dtype), to_device(V, dtype),
                                         to_device(np.zeros_like(q), dtype)).float().cpu().numpy()
                hz.events.append(("append", l, K, V))
                count[:, l, :] += 1
                for b in range(B):
                    for h in range(H):
                        o = hz.oracle_replay(b, l, h, rec=_records(hz, b, l, h))
                        ref = o.decode(q[b, h * g:(h + 1) * g])
                        assert rel_l2(out[b, h * g:(h + 1) * g], ref) <= dec_tol
    hz.compress()
    hz.check_all(s_tol)
    for (b, l, h), o in hz.oracles.items():
        assert o.view()[2].sum() == count[b, l, h]
    for l in range(L):
        q = synth.round_to(rng.standard_normal((B, H * g, d)).astype(np.float32), dtype)
        hz.check_decode(l, q, dec_tol)
    st = hz.ctx.stats()
    assert st["device_status"] == 0 and st["tokens_appended"] == int(count.sum())


def _records(hz, b, l, h):
    """The GPU's signs of every call this stream has run so far."""
    from parity_util import gpu_call_records

    free = hz.oracle_replay(b, l, h)
    blocks = sum(1 for c in free.calls() if c["level"] == 0)
    return gpu_call_records(hz.ctx, b, l, h, blocks)
