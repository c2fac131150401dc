"""Attention error against compression rate on synthetic data: BalanceKV (paper constants and a
smaller walk constant c) beside uniform sampling at the same rate -- the shape of the paper's
single-layer ablations (relative error ||z - Attn|| / ||Attn|| over T and t), on seeded synthetic
keys and values instead of the paper's prompts.

    python -m paper_2502_07861_b200.error_sweep --recipe clustered --n 8192 --blocks 64,256 --levels 1,2,3 --seeds 5
    python -m paper_2502_07861_b200.error_sweep --recipe clustered_norms --buckets 4 --n 16384 --blocks 64,256 --levels 1,2 --seeds 5
    python -m paper_2502_07861_b200.error_sweep --recipe clustered_shifted --center-keys 1        (key mean shift ON; 0: OFF)

Everything runs through the library: BalanceKV = append + compress + decode; uniform sampling = a
cache loaded directly at level T with a random subset and weights 2^T; exact = a context with T = 0.
Prints one JSON line per (recipe, t, T, method) with the error averaged over seeds, heads and queries.
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as bk


def make_kv(recipe, seed, H, n, d):
    """bf16 K, V [1, H, n, d] on the device."""
    g = torch.Generator(device="cuda").manual_seed(seed)
    if recipe in ("clustered", "clustered_norms", "clustered_shifted"):
        # near-duplicate keys on a few equal-norm centres, values tied to the cluster: the case in
        # which a balanced half beats a random half
        unit = lambda a: a / a.norm(dim=-1, keepdim=True)
        centres = 6.0 * unit(torch.randn(H, 8, d, device="cuda", generator=g))
        vals = unit(torch.randn(H, 8, d, device="cuda", generator=g))
        lab = torch.randint(0, 8, (H, n), device="cuda", generator=g)
        K = torch.gather(centres, 1, lab[..., None].expand(H, n, d)) + 0.02 * torch.randn(H, n, d, device="cuda", generator=g)
        V = torch.gather(vals, 1, lab[..., None].expand(H, n, d)) + 0.02 * torch.randn(H, n, d, device="cuda", generator=g)
        if recipe == "clustered_norms":
            # value norms spread over three octaves: the case Algorithm 1's buckets are made for
            V = V * torch.exp2(-3.0 * torch.rand(H, n, 1, device="cuda", generator=g))
        Q = 0.5 * (centres[:, :4] + centres[:, 4:])                       # [H, 4, d] queries between two clusters
        if recipe == "clustered_shifted":
            # all keys share a large mean (as the paper observes for LLM keys, Appendix B.5): the case the
            # mean shift before compression is made for.  The queries stay orthogonal to the mean, so exact
            # attention is that of the unshifted keys.
            mean = 8.0 * unit(torch.randn(H, 1, d, device="cuda", generator=g))
            Q = Q - (Q * mean).sum(-1, keepdim=True) * mean / 64.0
            K = K + mean
    else:
        mu = 0.5 * torch.randn(H, 1, d, device="cuda", generator=g)
        s = torch.ones(H, 1, d, device="cuda")
        for h in range(H):
            s[h, 0, torch.randperm(d, device="cuda", generator=g)[:4]] = 10.0
        K = (mu + torch.randn(H, n, d, device="cuda", generator=g)) * s
        V = torch.randn(H, n, d, device="cuda", generator=g)
        Q = torch.randn(H, 4, d, device="cuda", generator=g)
    bf = lambda x: x.to(torch.bfloat16).contiguous()
    return bf(K[None]), bf(V[None]), bf(Q.reshape(1, H * 4, d))


def rel_err(z, ref):
    z, ref = z.float(), ref.float()
    return float(((z - ref).norm(dim=-1) / ref.norm(dim=-1).clamp_min(1e-30)).mean())


def run_point(recipe, seed, H, n, d, t, T, c_small, center, buckets=0):
    K, V, q = make_kv(recipe, seed, H, n, d)
    common = dict(n_seqs=1, n_layers=1, n_kv_heads=H, n_q_heads=4 * H, head_dim=d, dtype="bf16", max_tokens=n)
    exact_ctx = bk.Context(block=t, levels=0, **common)
    exact_ctx.stream_append_layer(0, K, V)
    exact_ctx.compress()
    exact = exact_ctx.decode_attn(0, q).clone()
    exact_ctx.close()
    out = {}
    for name, c in (("balancekv_paper_c", 0.0), ("balancekv_small_c", c_small)):
        ctx = bk.Context(block=t, levels=T, seed=seed, c_override=c, center_keys=center, **common)
        ctx.stream_append_layer(0, K, V)
        ctx.compress()
        out[name] = rel_err(ctx.decode_attn(0, q), exact)
        st = ctx.stats()
        assert st["device_status"] == 0
        out[name + "_fails"] = st["walk_fails"]
        ctx.close()
    if buckets > 0:
        # Algorithm 1 in full: one MergeAndReduce instance per value-norm bucket for the numerator
        # (||v|| <= 2 assumed by the recipes: i_top = 1), a keys-only instance for the denominator
        full = dict(common, n_layers=buckets + 1)
        for name, c in (("algorithm1_paper_c", 0.0), ("algorithm1_small_c", c_small)):
            ctx = bk.Context(block=t, levels=T, seed=seed, c_override=c, center_keys=center, **full)
            counts = ctx.stream_append_layer_bucketed(0, buckets, 1, K, V)
            ctx.stream_append_layer_keys(buckets, K)
            ctx.compress()
            out[name] = rel_err(ctx.decode_attn_merged(list(range(buckets)), [buckets], q), exact)
            st = ctx.stats()
            assert st["device_status"] == 0
            out[name + "_stored"] = st["tokens_stored"] / (H * (buckets + 1))   # rows per stream over all instances
            out[name + "_dropped"] = int(counts[:, buckets].sum())
            ctx.close()
    g = torch.Generator(device="cuda").manual_seed(10_000 + seed)
    keep = n >> T
    idx = torch.stack([torch.randperm(n, device="cuda", generator=g)[:keep].sort().values for _ in range(H)])   # [H, keep]
    ctx = bk.Context(block=t, levels=T, **common)
    gi = idx[None, :, :, None].expand(1, H, keep, d)
    ctx.cache_load_level(0, T, torch.gather(K, 2, gi).contiguous(), torch.gather(V, 2, gi).contiguous(),
                         idx[None].to(torch.int32).contiguous())
    out["uniform"] = rel_err(ctx.decode_attn(0, q), exact)
    ctx.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--recipe", default="clustered", choices=("clustered", "clustered_norms", "clustered_shifted", "llama"))
    ap.add_argument("--n", type=int, default=8192)
    ap.add_argument("--heads", type=int, default=4)
    ap.add_argument("--head-dim", type=int, default=128)
    ap.add_argument("--blocks", default="64,128,256")
    ap.add_argument("--levels", default="1,2,3,4")
    ap.add_argument("--seeds", type=int, default=10)
    ap.add_argument("--small-c", type=float, default=0.25)
    ap.add_argument("--center-keys", type=int, default=0)
    ap.add_argument("--buckets", type=int, default=0, help="> 0: also Algorithm 1 with this many value-norm buckets")
    a = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("error_sweep needs a CUDA device")
    for t in [int(x) for x in a.blocks.split(",")]:
        for T in [int(x) for x in a.levels.split(",")]:
            if a.n % (t << T):
                continue
            acc = {}
            for seed in range(a.seeds):
                for k, v in run_point(a.recipe, seed, a.heads, a.n, a.head_dim, t, T, a.small_c, a.center_keys, a.buckets).items():
                    acc[k] = acc.get(k, 0.0) + v / a.seeds
            print(json.dumps(dict(recipe=a.recipe, n=a.n, block=t, levels=T, rate=2.0 ** -T, seeds=a.seeds,
                                  center_keys=a.center_keys, small_c=a.small_c, **{k: round(v, 6) for k, v in acc.items()})))


if __name__ == "__main__":
    main()
