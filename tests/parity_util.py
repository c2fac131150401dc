"""Shared machinery of the GPU parity tests: drive the CUDA library and the CPU oracle on the
same seeded inputs and compare them by the teacher-forced procedure.

  1. per call, the GPU's signs eta are read back (debug record);
  2. the oracle replays every call following the GPU's signs, so its S_j, p_j, u_j are those
     of the GPU's own prefix; a GPU decision must equal the oracle's (u_j < p_j), unless the
     walk margin |u_j - p_j| is below 1e-5 -- such decisions are counted (< 0.1 %);
  3. given the signs, kept indices, order, weights and the stored rows must be bit-exact;
  4. S_j must agree within the stated tolerance (this is what tests the Gram arithmetic);
  5. decode outputs must agree within 2e-3 (bf16) / 1e-5 (fp32) relative L2.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import OracleParams, OracleStream
from paper_2502_07861_b200 import synth

MARGIN = 1e-5


def to_device(x_f32: np.ndarray, dtype: str) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(x_f32))
    return t.to(torch.bfloat16 if dtype == "bf16" else torch.float32).cuda().contiguous()


def oracle_params(ctx, seq, layer, head):
    c = ctx.cfg
    return OracleParams(d=c.head_dim, t=c.block, T=c.levels, W=c.recent_window, center_keys=c.center_keys,
                        layer=layer, head=head, max_tokens=c.max_tokens, seed=c.seed + seq, delta=c.delta,
                        c_override=c.c_override, r_key=c.r_key, r_value=c.r_value)


def gpu_call_records(ctx, seq, layer, head, blocks_done):
    """{(level, ordinal): (eta, S, p)} for every call the stream has run."""
    rec = {}
    for lvl in range(ctx.cfg.levels):
        for o in range(blocks_done >> lvl):
            e, S, p = ctx.debug_call(seq, layer, head, lvl, o)
            rec[(lvl, o)] = (e.cpu().numpy(), S.cpu().numpy().astype(np.float64), p.cpu().numpy().astype(np.float64))
    return rec


def check_stream(ctx, seq, layer, head, ostream: OracleStream, rec, s_tol_rel, s_tol_abs=1e-6):
    """Steps 2-4 for one stream.  `ostream` has replayed the same appends/compresses with the
    GPU's signs forced.  Returns (decisions, decided_by_margin)."""
    calls = ostream.calls()
    assert len(calls) == len(rec), (len(calls), len(rec))
    n_dec = n_margin = 0
    for c in calls:
        eta_g, S_g, p_g = rec[(c["level"], c["ordinal"])]
        assert np.array_equal(c["eta"], eta_g)          # the oracle followed the GPU
        want = np.where(c["u"] < c["p"], 1, -1)
        diff = want != eta_g
        margin = np.abs(c["u"] - c["p"])
        assert np.all(margin[diff] < MARGIN), (c["level"], c["ordinal"], np.flatnonzero(diff)[:8], margin[diff][:8])
        n_dec += len(eta_g)
        n_margin += int(diff.sum())
        # running correlation: scale of the admissible error = sum of |G-hat| terms <= j
        tol = s_tol_abs + s_tol_rel * np.maximum(1.0, np.abs(c["S"]))
        bad = np.abs(S_g - c["S"]) > tol
        assert not bad.any(), (c["level"], c["ordinal"], np.flatnonzero(bad)[:8], S_g[bad][:4], c["S"][bad][:4])
        assert np.allclose(p_g, c["p"], atol=1e-5)
    Ko, Vo, wo, io = ostream.view()
    Kg, Vg, wg, ig = ctx.cache_view(seq, layer, head)
    assert np.array_equal(ig.cpu().numpy(), io), "kept index sets differ"
    assert np.array_equal(wg.cpu().numpy().astype(np.float64), wo), "weights differ"
    assert np.array_equal(Kg.float().cpu().numpy().astype(np.float64), Ko)
    assert np.array_equal(Vg.float().cpu().numpy().astype(np.float64), Vo)
    assert list(ctx.level_sizes(seq, layer, head)) == list(ostream.level_sizes())
    return n_dec, n_margin


def rel_l2(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


class Harness:
    """Runs a whole configuration on both sides.  K, V: float32 [B, L, H, n, d] already rounded
    to the storage dtype."""

    def __init__(self, bk, *, B, L, H, g, d, dtype, t, T, N, W=0, seed=0, **kw):
        self.bk = bk
        self.dtype = dtype
        self.B, self.L, self.H, self.g, self.d, self.t, self.T, self.W = B, L, H, g, d, t, T, W
        self.ctx = bk.Context(n_seqs=B, n_layers=L, n_kv_heads=H, n_q_heads=H * g, head_dim=d, dtype=dtype, block=t,
                              levels=T, max_tokens=N, recent_window=W, seed=seed, **kw)
        self.ctx.debug_enable(True)
        self.events = []           # ("append", layer, K[B,H,n,d], V) | ("compress",)
        self.appended = 0

    def append_layer(self, layer, K, V):
        self.ctx.stream_append_layer(layer, to_device(K, self.dtype), to_device(V, self.dtype))
        self.events.append(("append", layer, K, V))

    def append_stream(self, seq, layer, head, K, V):
        self.ctx.stream_append(seq, layer, head, to_device(K, self.dtype), to_device(V, self.dtype))
        self.events.append(("append_stream", seq, layer, head, K, V))

    def compress(self):
        self.ctx.compress()
        self.events.append(("compress",))

    def oracle_replay(self, seq, layer, head, rec=None):
        o = OracleStream(oracle_params(self.ctx, seq, layer, head))
        if rec:
            for (lvl, ordinal), (eta, _, _) in rec.items():
                o.force_eta(lvl, ordinal, eta)
        for ev in self.events:
            if ev[0] == "append":
                if ev[1] == layer:
                    o.append(ev[2][seq, head], ev[3][seq, head])
            elif ev[0] == "append_stream":          # ("append_stream", seq, layer, head, K[n,d], V[n,d])
                if ev[1:4] == (seq, layer, head):
                    o.append(ev[4], ev[5])
            else:
                o.compress()
        return o

    def check_all(self, s_tol_rel, streams=None, s_tol_abs=1e-6):
        tot = marg = 0
        self.oracles = {}
        self.recs = {}
        for seq in range(self.B):
            for layer in range(self.L):
                for head in range(self.H):
                    if streams is not None and (seq, layer, head) not in streams:
                        continue
                    free = self.oracle_replay(seq, layer, head)
                    blocks = sum(1 for c in free.calls() if c["level"] == 0)
                    rec = gpu_call_records(self.ctx, seq, layer, head, blocks)
                    forced = self.oracle_replay(seq, layer, head, rec)
                    n, m = check_stream(self.ctx, seq, layer, head, forced, rec, s_tol_rel, s_tol_abs)
                    tot += n
                    marg += m
                    self.oracles[(seq, layer, head)] = forced
                    self.recs[(seq, layer, head)] = rec
        assert marg <= 1e-3 * max(tot, 1), (marg, tot)
        return tot, marg

    def check_decode(self, layer, q_f32, tol):
        """q_f32: [B, H*g, d] rounded to dtype.  Compares with the oracle evaluated on the
        (bit-identical) cache."""
        out = self.ctx.decode_attn(layer, to_device(q_f32, self.dtype)).float().cpu().numpy()
        worst = 0.0
        for (seq, lay, head), o in self.oracles.items():
            if lay != layer:
                continue
            ref = o.decode(q_f32[seq, head * self.g:(head + 1) * self.g])
            err = rel_l2(out[seq, head * self.g:(head + 1) * self.g], ref)
            worst = max(worst, err)
            assert err <= tol, (seq, head, err)
        return worst
