"""Kernel-level timing of the BalanceKV library on synthetic device data.

    python -m paper_2502_07861_b200.microbench decode   --batch 32 --cache-len 8192 --levels 2 [--two-instance]
    python -m paper_2502_07861_b200.microbench compress --streams 8 --context 32768 --block 1024 --levels 2
    python -m paper_2502_07861_b200.microbench bucket   --streams 8 --context 32768 --buckets 5

Prints one JSON line per run.  Inputs are drawn on the device (torch.randn), which is enough
for timing; parity is the tests' job.
"""
from __future__ import annotations

import argparse
import json
import os

import torch

from . import binding as bk

_ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _peaks():
    p = os.path.join(_ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return float(j["hbm_gbs"]), float(j["bf16_tflops"]), "measured"
    return 6650.0, 1590.0, "fallback"


def run_decode(a):
    print(json.dumps(decode_case(a.batch, a.kv_heads, a.group, a.head_dim, a.cache_len, a.levels, iters=a.iters,
                                 max_layers=a.max_layers, two_instance=a.two_instance, splits=a.splits, gram_path=a.gram_path)))


def decode_case(B, H, g, d, Lc, T, iters=50, max_layers=16, two_instance=False, splits=0, gram_path=0):
    """Decode attention over caches loaded directly at level T (the decode-sweep shape); returns a dict."""
    import types

    a = types.SimpleNamespace(max_layers=max_layers, two_instance=two_instance, splits=splits, iters=iters)
    esz = 2
    bytes_layer = B * H * Lc * 2 * d * esz
    # enough distinct layers that a layer is evicted from L2 (126 MB) before it is read again
    n_layers = max(2, min(a.max_layers, (512 << 20) // max(bytes_layer, 1) + 1))
    if a.two_instance:          # Algorithm 1 with a separate denominator instance: two slots (caches) per layer
        n_layers += n_layers % 2
        bytes_layer = bytes_layer * 3 // 2      # K and V of the numerator slot, K of the denominator slot
    ctx = bk.Context(n_seqs=B, n_layers=n_layers, n_kv_heads=H, n_q_heads=H * g, head_dim=d, dtype="bf16", block=64,
                     levels=T, max_tokens=Lc << T, decode_splits=a.splits, gram_path=gram_path)
    K = torch.randn(B, H, Lc, d, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    V = torch.randn(B, H, Lc, d, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    for l in range(n_layers):
        ctx.cache_load_level(l, T, K, V)
    q = torch.randn(B, H * g, d, device="cuda").to(torch.bfloat16)
    out = torch.empty_like(q)
    raw = int(torch.cuda.current_stream().cuda_stream)
    if a.two_instance:
        call = lambda i: ctx.decode_attn_two(2 * (i % (n_layers // 2)), 2 * (i % (n_layers // 2)) + 1, q, out, stream=raw)
    else:
        call = lambda i: ctx.decode_attn(i % n_layers, q, out, stream=raw)
    for i in range(3 * n_layers):
        call(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    iters = a.iters
    e0.record()
    for i in range(iters):
        call(i)
    e1.record()
    torch.cuda.synchronize()
    us = 1e3 * e0.elapsed_time(e1) / iters
    hbm, _, src = _peaks()
    gbs = bytes_layer / (us * 1e-6) / 1e9
    st = ctx.stats()
    res = dict(kernel="decode_two_instance" if a.two_instance else "decode", batch=B, kv_heads=H, group=g, head_dim=d, cache_len=Lc, levels=T,
               layers_cycled=n_layers, splits=a.splits, us_per_layer=us, algorithmic_bytes=bytes_layer, achieved_gbs=gbs,
               peak_gbs=hbm, frac=gbs / hbm, peak_source=src, device_status=st["device_status"])
    ctx.close()
    del K, V, ctx
    torch.cuda.empty_cache()
    return res


def run_compress(a):
    print(json.dumps(compress_case(a.streams, a.head_dim, a.context, a.block, a.levels, iters=a.iters, gram_path=a.gram_path,
                                   c_override=a.c_override, outliers=a.outliers, window=a.window)))


def compress_case(S, d, n, t, T, iters=10, gram_path=0, c_override=0.0, outliers=1, window=0):
    """append + compress of `S` streams (one layer), timed per kernel class; returns a dict."""
    import types

    a = types.SimpleNamespace(iters=iters, gram_path=gram_path, c_override=c_override, outliers=outliers)
    ctx = bk.Context(n_seqs=1, n_layers=1, n_kv_heads=S, n_q_heads=S, head_dim=d, dtype="bf16", block=t, levels=T,
                     max_tokens=n, gram_path=a.gram_path, c_override=a.c_override, recent_window=window)
    K = torch.randn(1, S, n, d, device="cuda", dtype=torch.float32)
    if a.outliers:
        K[..., :4] *= 10.0
    K = K.to(torch.bfloat16)
    V = torch.randn(1, S, n, d, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for _ in range(2):
        ctx.reset(); ctx.stream_append_layer(0, K, V); ctx.compress()
    ctx.profile_enable(True)
    ctx.profile_read()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    tot = 0.0
    for i in range(a.iters):
        ctx.reset()
        ctx.stream_append_layer(0, K, V)
        flush.fill_(i & 255)
        e0.record()
        ctx.compress()
        e1.record()
        torch.cuda.synchronize()
        tot += e0.elapsed_time(e1)
    prof = ctx.profile_read()
    n_calls = S * sum(((n - window) // t) >> l for l in range(T))
    flop = n_calls * 2.0 * (t * (t - 1) / 2.0) * 2.0 * d
    gw_n, gw_ms = prof["gram_walk"]
    cp_n, cp_ms = prof["compact"]
    hbm, tf, src = _peaks()
    tfl = flop * a.iters / (gw_ms * 1e-3) / 1e12 if gw_ms else 0.0
    cp_bytes = n_calls * ((t // 2) * (4 * d * 2 + 8 + 16) + t)   # rows, position, norms per survivor, sign bytes
    cp_gbs = cp_bytes * a.iters / (cp_ms * 1e-3) / 1e9 if cp_ms else 0.0
    st = ctx.stats()
    res = dict(kernel="compress", streams=S, context=n, block=t, levels=T, recent_window=window, calls=n_calls,
               compress_ms=tot / a.iters, gram_walk_ms=gw_ms / a.iters, gram_walk_launches=gw_n // a.iters,
               gram_walk_tflops=tfl, tensor_peak=tf, tensor_frac=tfl / tf,
               compact_ms=cp_ms / a.iters, compact_gbs=cp_gbs, hbm_peak=hbm, compact_frac=cp_gbs / hbm,
               radii_ms=prof["radii"][1] / a.iters, bookkeeping_ms=prof["bookkeeping"][1] / a.iters,
               token_heads_per_s=S * n / (tot / a.iters * 1e-3), walk_fails=st["walk_fails"],
               walk_kernel=st["walk_kernel"], device_status=st["device_status"], peak_source=src)
    ctx.close()
    del K, V, ctx, flush
    torch.cuda.empty_cache()
    return res


def run_bucket(a):
    """Algorithm 1's bucketing step (value norms, stable partition, scatter into the per-bucket slots),
    then compress of all slots and the merged decode over them."""
    S, d, n, t, T, nb = a.streams, a.head_dim, a.context, a.block, a.levels, a.buckets
    ctx = bk.Context(n_seqs=1, n_layers=nb + 1, n_kv_heads=S, n_q_heads=S * 4, head_dim=d, dtype="bf16", block=t,
                     levels=T, max_tokens=n)
    K = torch.randn(1, S, n, d, device="cuda", dtype=torch.float32)
    K[..., :4] *= 10.0
    K = K.to(torch.bfloat16)
    scale = torch.exp2(-float(nb) * torch.rand(1, S, n, 1, device="cuda"))     # norms spread over the nb octaves
    V = (torch.randn(1, S, n, d, device="cuda", dtype=torch.float32) * scale).to(torch.bfloat16)
    i_top = 4                                                                    # ||v|| <= 16
    q = torch.randn(1, S * 4, d, device="cuda").to(torch.bfloat16)
    out = torch.empty_like(q)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    t_route = t_comp = t_dec = 0.0
    ctx.profile_enable(True)
    for i in range(a.iters + 2):
        ctx.reset()
        flush.fill_(i & 255)
        if i == 2:
            ctx.profile_read()
        ev[0].record()
        counts = ctx.stream_append_layer_bucketed(0, nb, i_top, K, V)
        ev[1].record()
        ctx.stream_append_layer_keys(nb, K)
        ctx.compress()
        ev[2].record()
        ctx.decode_attn_merged(list(range(nb)), [nb], q, out)
        ev[3].record()
        torch.cuda.synchronize()
        if i >= 2:
            t_route += ev[0].elapsed_time(ev[1]); t_comp += ev[1].elapsed_time(ev[2]); t_dec += ev[2].elapsed_time(ev[3])
    prof = ctx.profile_read()
    hbm, _, src = _peaks()
    kept = int(counts[:, :nb].sum())
    # read V for the norms, read K and V of the kept rows, write them: 2 bytes per element
    route_bytes = S * n * d * 2 + kept * 4 * d * 2
    # class 0 also holds the keys-only append of the denominator slot: one launch per iteration, subtracted by count
    st = ctx.stats()
    print(json.dumps(dict(kernel="bucket_route", streams=S, context=n, buckets=nb, block=t, levels=T,
                          rows_kept=kept, rows_dropped=int(counts[:, nb].sum()), per_slot=counts[:, :nb].sum(0).tolist(),
                          route_call_ms=t_route / a.iters, algorithmic_bytes=route_bytes,
                          achieved_gbs=route_bytes / (t_route / a.iters * 1e-3) / 1e9, peak_gbs=hbm,
                          frac=route_bytes / (t_route / a.iters * 1e-3) / 1e9 / hbm,
                          append_class_launches=prof["append"][0] // a.iters, append_class_ms=prof["append"][1] / a.iters,
                          compress_ms=t_comp / a.iters, merged_decode_ms=t_dec / a.iters,
                          token_heads_per_s=S * n / ((t_route + t_comp) / a.iters * 1e-3),
                          device_status=st["device_status"], peak_source=src)))
    ctx.close()


def main():
    ap = argparse.ArgumentParser()
    sub = ap.add_subparsers(dest="cmd", required=True)
    d = sub.add_parser("decode")
    d.add_argument("--batch", type=int, default=32)
    d.add_argument("--kv-heads", type=int, default=8)
    d.add_argument("--group", type=int, default=5)
    d.add_argument("--head-dim", type=int, default=128)
    d.add_argument("--cache-len", type=int, default=8192)
    d.add_argument("--levels", type=int, default=2)
    d.add_argument("--iters", type=int, default=50)
    d.add_argument("--max-layers", type=int, default=16)
    d.add_argument("--two-instance", action="store_true")
    d.add_argument("--splits", type=int, default=0, help="split-K factor (0 = automatic)")
    d.add_argument("--gram-path", type=int, default=0, help="1: the CUDA-core decode kernel")
    c = sub.add_parser("compress")
    c.add_argument("--streams", type=int, default=8)
    c.add_argument("--head-dim", type=int, default=128)
    c.add_argument("--context", type=int, default=32768)
    c.add_argument("--block", type=int, default=1024)
    c.add_argument("--levels", type=int, default=2)
    c.add_argument("--iters", type=int, default=10)
    c.add_argument("--gram-path", type=int, default=0)
    c.add_argument("--c-override", type=float, default=0.0)
    c.add_argument("--outliers", type=int, default=1)
    c.add_argument("--window", type=int, default=0, help="recent window W (tokens kept out of the calls)")
    b = sub.add_parser("bucket")
    b.add_argument("--streams", type=int, default=8)
    b.add_argument("--head-dim", type=int, default=128)
    b.add_argument("--context", type=int, default=32768)
    b.add_argument("--block", type=int, default=1024)
    b.add_argument("--levels", type=int, default=2)
    b.add_argument("--buckets", type=int, default=5)
    b.add_argument("--iters", type=int, default=10)
    a = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("microbench needs a CUDA device")
    {"decode": run_decode, "compress": run_compress, "bucket": run_bucket}[a.cmd](a)


if __name__ == "__main__":
    main()
