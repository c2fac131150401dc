"""The error-against-rate sweep (shape of the paper's Fig. 1 / Fig. 2(b) on synthetic data) measures
against exact attention.  Here, for one seed of every cell of its grid -- T in 1..4, t in {64, 128, 256},
key mean shift off and on, both recipes -- the "exact" it uses (the library at T = 0) is checked against
Eq. (1) evaluated by the CPU oracle on the same bytes, and the errors of BalanceKV and of uniform
sampling are recomputed against the oracle's exact attention."""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("recipe", ["clustered", "clustered_shifted"])
@pytest.mark.parametrize("center", [0, 1])
def test_sweep_cells_measure_against_the_oracles_exact_attention(cuda_lib, recipe, center):
    from paper_2502_07861_b200 import error_sweep as es

    H, n, d, seed = 4, 8192, 128, 0
    K, V, q = es.make_kv(recipe, seed, H, n, d)
    Kh, Vh, qh = (x.float().cpu().numpy().astype(np.float64) for x in (K[0], V[0], q[0]))
    exact = np.stack([oracle.weighted_attention(Kh[h], Vh[h], None, qh[4 * h:4 * h + 4]) for h in range(H)]).reshape(H * 4, d)
    ctx = cuda_lib.Context(n_seqs=1, n_layers=1, n_kv_heads=H, n_q_heads=4 * H, head_dim=d, dtype="bf16", max_tokens=n,
                           block=64, levels=0)
    ctx.stream_append_layer(0, K, V)
    lib_exact = ctx.decode_attn(0, q).float().cpu().numpy()[0]
    ctx.close()
    assert np.linalg.norm(lib_exact - exact) / np.linalg.norm(exact) <= 2e-3
    ex_t = torch.from_numpy(exact).cuda()[None]
    for t in (64, 128, 256):
        for T in (1, 2, 3, 4):
            r = es.run_point(recipe, seed, H, n, d, t, T, 0.25, center)
            # the same cell against the oracle's exact attention
            c = cuda_lib.Context(n_seqs=1, n_layers=1, n_kv_heads=H, n_q_heads=4 * H, head_dim=d, dtype="bf16", max_tokens=n,
                                 block=t, levels=T, seed=seed, c_override=0.25, center_keys=center)
            c.stream_append_layer(0, K, V)
            c.compress()
            e_or = es.rel_err(c.decode_attn(0, q), ex_t)
            c.close()
            assert abs(e_or - r["balancekv_small_c"]) <= 4e-3, (t, T, e_or, r)
            assert 0.0 <= r["uniform"] < 1.5 and 0.0 <= r["balancekv_paper_c"] < 1.5
