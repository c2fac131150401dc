#!/usr/bin/env python
"""Benchmark of the BalanceKV hot path on B200.

One *step* = one pass of the whole hot path over one batch of synthetic input shaped like one
Llama-3.1-8B layer: append the 32768-token context of 8 KV heads (bf16, d=128), compress it
with blocks of 1024 and T=2, then 256 decode steps, each appending one uncompressed token per
stream and running decode attention for the 32 query heads over the weighted cache.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

prints one JSON line (rank 0).  `--impl reference` times the CPU oracle on a bounded sample.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

WORKLOAD = dict(name="llama3.1-8b-layer", n_seqs=1, n_layers=1, n_kv_heads=8, n_q_heads=32, head_dim=128, dtype="bf16",
                context=32768, block=1024, levels=2, decode_steps=256, recipe="llama", data_seed=1002, walk_seed=0)
METRIC = "compressed_kv_tokens_per_s"
UNIT = "KV token-heads/s through append+compress(T=2)+256 decode steps"


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return dict(hbm=float(j["hbm_gbs"]), tensor=float(j["bf16_tflops"]), tensor_sustained=float(j["bf16_tflops_sustained"]),
                    source="measured")
    return dict(hbm=6650.0, tensor=1590.0, tensor_sustained=1400.0, source="fallback")


def make_inputs(w, n_context, n_decode):
    """Host tensors (float32 values already rounded to bf16): context K,V, decode K,V, queries."""
    from paper_2502_07861_b200 import synth

    B, H, d = w["n_seqs"], w["n_kv_heads"], w["head_dim"]
    K = np.empty((B, H, n_context + n_decode, d), np.float32)
    V = np.empty_like(K)
    for b in range(B):
        for h in range(H):
            K[b, h], V[b, h] = synth.stream_kv(w["recipe"], w["data_seed"], b, 0, h, n_context + n_decode, d, w["dtype"])
    q = np.stack([synth.queries(w["data_seed"], 0, s, B, w["n_q_heads"], d, w["dtype"]) for s in range(n_decode)])
    return K, V, q


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for l in self.lines:
            f = [x.strip() for x in l.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


def oracle_sample(w, K, V, q, sample_tokens, decode_steps):
    """The oracle, as it stands, on the first `sample_tokens` tokens of every stream plus
    `decode_steps` decode steps; returns (seconds spent, token-heads, threads, seconds with the
    decode part scaled linearly to all of the workload's decode steps)."""
    import oracle

    B, H, d, g = w["n_seqs"], w["n_kv_heads"], w["head_dim"], w["n_q_heads"] // w["n_kv_heads"]
    t0 = time.perf_counter()
    streams = []
    for b in range(B):
        for h in range(H):
            o = oracle.OracleStream(oracle.OracleParams(d=d, t=w["block"], T=w["levels"], layer=0, head=h,
                                                        max_tokens=w["context"] + w["decode_steps"], seed=w["walk_seed"] + b))
            o.append(K[b, h, :sample_tokens], V[b, h, :sample_tokens])
            streams.append((b, h, o))
    oracle.compress_streams([s[2] for s in streams])
    t_ctx = time.perf_counter() - t0
    n_ctx = w["context"]
    for s in range(decode_steps):
        for b, h, o in streams:
            o.append(K[b, h, n_ctx + s:n_ctx + s + 1], V[b, h, n_ctx + s:n_ctx + s + 1])
            o.decode(q[s, b, h * g:(h + 1) * g])
    dt = time.perf_counter() - t0
    scaled = t_ctx + (dt - t_ctx) * (w["decode_steps"] / decode_steps if decode_steps else 0.0)
    return dt, B * H * sample_tokens, oracle.num_threads(), scaled


def run_reference(args, w):
    """CPU oracle arm on the product arm's workload: every step is the whole context of every stream
    and all decode steps.  The oracle needs several seconds per step, so at most as many of the
    requested steps run as fit in about three minutes (the line says how many)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    K, V, q = make_inputs(w, w["context"], w["decode_steps"])
    for _ in range(min(args.warmup, 1)):
        oracle_sample(w, K, V, q, w["block"] * 2, 1)
    times, budget_s = [], 180.0
    units = threads = 0
    for i in range(args.steps):
        dt, units, threads, _ = oracle_sample(w, K, V, q, w["context"], w["decode_steps"])
        times.append(dt)
        if sum(times) + dt > budget_s:
            break
    val = units * len(times) / sum(times)
    sample_txt = (f"all {w['context']} context tokens of each of the {w['n_kv_heads']} streams + all {w['decode_steps']} decode "
                  f"steps per step; {len(times)} of the {args.steps} requested steps run (time budget {budget_s:.0f} s)")
    line = dict(metric=METRIC, value=val, unit=UNIT, n_gpus=args.gpus, steps=len(times), steps_requested=args.steps,
                warmup=args.warmup, ms_per_step=1e3 * float(np.mean(times)), higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype="f64", data="synthetic", impl="reference",
                config=dict(workload=w["name"], n_kv_heads=w["n_kv_heads"], n_q_heads=w["n_q_heads"], head_dim=w["head_dim"],
                            context=w["context"], block=w["block"], levels=w["levels"], decode_steps=w["decode_steps"]),
                cpu_baseline=dict(value=val, unit=UNIT, cores=threads, kind="oracle", sample=sample_txt),
                e2e=dict(value=val, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0), gpu_launches=0)
    print(json.dumps(line))


def source_digest(*names):
    """sha256 over the named kernel sources: an ncu traffic figure is only quoted for the code it was taken from."""
    import hashlib

    h = hashlib.sha256()
    for n in names:
        with open(os.path.join(ROOT, "paper_2502_07861_b200", "csrc", n), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def measured_traffic(shape):
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the graded kernels from the
    ncu captures summarised under profiles/: entries of profiles/traffic.json that match this shape and
    whose kernel source is unchanged since the capture; anything else is reported as null."""
    path = os.path.join(ROOT, "profiles", "traffic.json")
    out = {}
    if not os.path.exists(path):
        return out
    for e in json.load(open(path)).get("entries", []):
        if e.get("shape") == shape and e.get("source_digest") == source_digest(*e.get("sources", [])):
            out[e["kernel"]] = float(e["dram_bytes_per_launch"])
    return out


def per_config(peaks):
    """The other configurations as bounded slices (each a few hundred milliseconds of GPU time): what was
    run, the figures, and how a slice relates to the whole configuration."""
    import torch

    import paper_2502_07861_b200 as bk
    from paper_2502_07861_b200 import microbench, synth

    out = {}
    # config 1: the tiny fp32 stream (CUDA-core kernels), time only
    n, t, d = 1024, 256, 64
    Kf, Vf = synth.stream_kv("outlier2", 1001, 0, 0, 0, n, d, "fp32")
    K = torch.from_numpy(Kf)[None, None].cuda().contiguous()
    V = torch.from_numpy(Vf)[None, None].cuda().contiguous()
    qs = torch.from_numpy(synth.queries(1001, 0, 0, 16, 1, d, "fp32")).cuda().contiguous()    # 16 queries
    ctx = bk.Context(n_seqs=1, n_layers=1, n_kv_heads=1, n_q_heads=1, head_dim=d, dtype="fp32", block=t, levels=1, max_tokens=n)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    tc, td = [], []
    for it in range(8):
        ctx.reset()
        ev[0].record()
        for b in range(n // t):
            ctx.stream_append_layer(0, K[:, :, b * t:(b + 1) * t].contiguous(), V[:, :, b * t:(b + 1) * t].contiguous())
            ctx.compress()
        ev[1].record()
        for i in range(16):
            ctx.decode_attn(0, qs[i:i + 1])
        ev[2].record()
        torch.cuda.synchronize()
        if it >= 3:
            tc.append(ev[0].elapsed_time(ev[1])); td.append(ev[1].elapsed_time(ev[2]))
    st = ctx.stats()
    ctx.close()
    out["config1_tiny_fp32"] = dict(
        workload="1 stream, d=64, fp32, 1024 tokens in blocks of 256, T=1, 16 decode queries", slice="whole configuration",
        append_compress_us=1e3 * float(np.mean(tc)), decode_us_per_query=1e3 * float(np.mean(td)) / 16,
        walk_kernel=int(st["walk_kernel"]), decode_kernel=int(st["decode_kernel"]),
        note="launch-latency bound (4 calls of 256 tokens): time only, no roofline claim")
    del K, V, ctx

    def compress_entry(res, workload, slice_txt, rule):
        return dict(workload=workload, slice=slice_txt, extrapolation=rule, compress_ms=res["compress_ms"],
                    compress_token_heads_per_s=res["token_heads_per_s"], calls=res["calls"],
                    gram_walk=dict(bound="tensor", achieved=res["gram_walk_tflops"], peak=peaks["tensor"], unit="TFLOP/s",
                                   frac=res["gram_walk_tflops"] / peaks["tensor"], ms=res["gram_walk_ms"]),
                    compact=dict(bound="hbm", achieved=res["compact_gbs"], peak=peaks["hbm"], unit="GB/s",
                                 frac=res["compact_gbs"] / peaks["hbm"], ms=res["compact_ms"]),
                    walk_kernel=res["walk_kernel"], device_status=res["device_status"])

    # config 3: one 8192-token prefill chunk of all 4 x 32 x 8 streams (t = 2048, T = 2)
    r3 = microbench.compress_case(4 * 32 * 8, 128, 8192, 2048, 2, iters=3)
    out["config3_8b_stack"] = compress_entry(
        r3, "4 sequences x 32 layers x 8 KV heads, d=128, bf16, t=2048, T=2",
        "one 8192-token prefill chunk of all 1024 streams (1 of 16 chunks), compress only",
        "whole configuration = 16 such chunks (work is linear in the context at fixed t); decode: see config5")
    # config 4: one chunk of 16 of the 48 layers (8 x 16 x 8 streams), t = 1024, T = 3, recent window 128
    r4 = microbench.compress_case(8 * 16 * 8, 128, 8192, 1024, 3, iters=3, window=128)
    out["config4_14b"] = compress_entry(
        r4, "8 sequences x 48 layers x 8 KV heads, d=128, bf16, t=1024, T=3, recent window 128",
        "one 8192-token prefill chunk of 16 of the 48 layers (1024 of 3072 streams), compress only",
        "whole configuration = 3 x 8 such slices (linear in streams and context)")
    # config 5: decode sweep at the 32B shape; distinct layers are cycled so that no launch re-reads L2
    sweep = []
    for Lc in (2048, 4096, 8192, 16384, 32768):
        r = microbench.decode_case(32, 8, 5, 128, Lc, 2, iters=30, max_layers=8)
        sweep.append(dict(cache_len=Lc, us_per_layer=r["us_per_layer"], us_x64_layers=64 * r["us_per_layer"],
                          achieved=r["achieved_gbs"], frac=r["frac"], layers_cycled=r["layers_cycled"],
                          device_status=r["device_status"]))
    out["config5_decode_sweep"] = dict(
        workload="batch 32 x 8 KV heads x 5 query heads each, d=128, bf16, weights 2^2, cache loaded at level T",
        slice="one layer per launch; 64 layers = 64 such launches", bound="hbm", peak=peaks["hbm"], unit="GB/s",
        points=sweep)
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="balancekv")
    ap.add_argument("--gram-path", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-config", action="store_true", help="skip the slices of the other configurations")
    ap.add_argument("--decode-splits", type=int, default=0, help="split-K factor of decode attention (0 = automatic)")
    ap.add_argument("--context", type=int, default=None, help="override the context length (profiling a small case)")
    ap.add_argument("--decode-steps", type=int, default=None)
    args = ap.parse_args()
    w = dict(WORKLOAD)
    if args.context:
        w["context"] = args.context
    if args.decode_steps is not None:
        w["decode_steps"] = args.decode_steps
    if args.impl == "reference":
        return run_reference(args, w)

    import torch
    import torch.distributed as dist

    import paper_2502_07861_b200 as bk
    from paper_2502_07861_b200 import shard

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    args.warmup = max(args.warmup, 3)

    # every rank owns an independent replica of the workload (streams shard with no exchange)
    w["data_seed"] = WORKLOAD["data_seed"] + 100 * rank
    B, H, Hq, d = w["n_seqs"], w["n_kv_heads"], w["n_q_heads"], w["head_dim"]
    n_ctx, n_dec, T, t = w["context"], w["decode_steps"], w["levels"], w["block"]
    Kf, Vf, qf = make_inputs(w, n_ctx, n_dec)
    bf = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(torch.bfloat16)
    K_ctx_h = bf(Kf[:, :, :n_ctx]).pin_memory()
    V_ctx_h = bf(Vf[:, :, :n_ctx]).pin_memory()
    K_dec_h = bf(np.moveaxis(Kf[:, :, n_ctx:], 2, 0)[:, :, :, None, :]).pin_memory()   # [steps, B, H, 1, d]
    V_dec_h = bf(np.moveaxis(Vf[:, :, n_ctx:], 2, 0)[:, :, :, None, :]).pin_memory()
    q_h = bf(qf).pin_memory()                                                          # [steps, B, Hq, d]
    out_h = torch.empty_like(q_h).pin_memory()
    K_ctx, V_ctx, K_dec, V_dec, q_d = (x.cuda() for x in (K_ctx_h, V_ctx_h, K_dec_h, V_dec_h, q_h))
    out_d = torch.empty(B, Hq, d, dtype=torch.bfloat16, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

    ctx = bk.Context(n_seqs=B, n_layers=1, n_kv_heads=H, n_q_heads=Hq, head_dim=d, dtype="bf16", block=t, levels=T,
                     max_tokens=n_ctx + n_dec, seed=shard.walk_seed(w["walk_seed"], rank * B), gram_path=args.gram_path,
                     decode_splits=args.decode_splits)

    raw_stream = int(torch.cuda.current_stream().cuda_stream)
    q_list, K_list, V_list = list(q_d.unbind(0)), list(K_dec.unbind(0)), list(V_dec.unbind(0))
    qh_list, Kh_list, Vh_list, oh_list = list(q_h.unbind(0)), list(K_dec_h.unbind(0)), list(V_dec_h.unbind(0)), list(out_h.unbind(0))

    def step_device(ev=None):
        ctx.reset()
        if ev: ev[0].record()
        ctx.stream_append_layer(0, K_ctx, V_ctx)
        ctx.compress()
        if ev: ev[1].record()
        for s in range(n_dec):
            ctx.stream_step(0, q_list[s], K_list[s], V_list[s], out_d, stream=raw_stream)
        if ev: ev[2].record()

    def step_host():
        ctx.reset()
        ctx.stream_append_layer_host(0, K_ctx_h, V_ctx_h)
        ctx.compress()
        for s in range(n_dec):
            ctx.stream_step_host(0, qh_list[s], Kh_list[s], Vh_list[s], oh_list[s], stream=raw_stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        flush.fill_(1)
        step_device()
    launches_before = ctx.stats()["kernels_launched"]
    # per-launch events around every compression-side launch and the context append.  A decode step is
    # one launch (it attends and appends the step's token), so the events that bracket the decode loop
    # give that kernel's average launch-to-launch duration; events between the launches would stop
    # consecutive launches from overlapping their launch latency and slow the loop they measure.
    ctx.profile_enable(True, classes=("append", "radii", "gram_walk", "compact", "bookkeeping"))
    ctx.profile_read()
    sampler = ClockSampler(local)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    barrier()
    sampler.start()
    for i in range(args.steps):
        flush.fill_(i & 255)       # L2 flush between timed iterations (outside the event brackets)
        step_device(evs[i])
    barrier()
    clocks = sampler.stop()
    prof = ctx.profile_read()
    ctx.profile_enable(False)
    launches = ctx.stats()["kernels_launched"] - launches_before
    t_step = np.array([e[0].elapsed_time(e[2]) for e in evs])           # ms
    t_comp = np.array([e[0].elapsed_time(e[1]) for e in evs])
    t_dec = np.array([e[1].elapsed_time(e[2]) for e in evs])
    total_ms = float(t_step.sum())
    total_ms = shard.max_over_ranks(total_ms, device="cuda")
    units_per_step = B * H * n_ctx
    value = world * units_per_step * args.steps / (total_ms * 1e-3)

    # end to end through the host-buffer entry points (pinned host memory in, host out)
    for _ in range(2):
        step_host()
    barrier()
    t0 = time.perf_counter()
    e2e_steps = max(2, min(args.steps, 5))
    for i in range(e2e_steps):
        step_host()
    barrier()
    e2e_s = time.perf_counter() - t0
    e2e_s = shard.max_over_ranks(e2e_s, device="cuda")
    esz = 2
    h2d = 2 * B * H * (n_ctx + n_dec) * d * esz + n_dec * B * Hq * d * esz
    d2h = n_dec * B * Hq * d * esz
    status = ctx.stats()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    peaks = measured_peaks()
    calls0, calls1 = n_ctx // t, (n_ctx // t) // 2
    n_calls = B * H * sum((n_ctx // t) >> l for l in range(T))
    # algorithmic work: strict lower triangle of two Gram matrices per call
    flop_per_call = 2.0 * (t * (t - 1) / 2.0) * 2.0 * d
    gw_n, gw_ms = prof["gram_walk"]
    gw_ms_per_launch = gw_ms / max(gw_n, 1)
    calls_per_launch = n_calls * args.steps / max(gw_n, 1)
    tensor_ach = flop_per_call * calls_per_launch / (gw_ms_per_launch * 1e-3) / 1e12 if gw_n else 0.0
    # compaction: per call read t/2 rows of K and V, write t/2 rows, t sign bytes, 2 index words per survivor
    cp_n, cp_ms = prof["compact"]
    cp_bytes = (t // 2) * (2 * 2 * d * esz + 8 + 16) + t      # rows, position (4+4 B), norms (8+8 B) per survivor, sign bytes
    cp_gbs = cp_bytes * n_calls * args.steps / (cp_ms * 1e-3) / 1e9 if cp_n else 0.0
    # decode: every stored row of K and V once per launch
    dc_n, dc_ms = n_dec * args.steps, float(t_dec.sum())
    stored0 = n_ctx >> T
    dec_bytes_timed = sum(B * H * (stored0 + s) * 2 * d * esz for s in range(n_dec)) * args.steps   # rows attended from the cache
    dc_gbs = dec_bytes_timed / (dc_ms * 1e-3) / 1e9 if dc_n else 0.0

    # time share of each kernel class in the timed region
    dc_launches = n_dec * args.steps
    dc_total_ms = dc_ms
    # DRAM bytes per launch from the ncu captures summarised under profiles/ (see measured_traffic); the
    # decode figure is a cold-L2 launch of the same shape, while this loop re-reads its cache from L2
    traffic = measured_traffic(dict(context=n_ctx, block=t, levels=T, streams=B * H))
    kernels = dict(
        gram_walk=dict(bound="tensor", achieved=tensor_ach, peak=peaks["tensor"], unit="TFLOP/s",
                       frac=tensor_ach / peaks["tensor"], traffic=traffic.get("gram_walk"), ms_per_launch=gw_ms_per_launch, launches=gw_n,
                       ms_total=gw_ms),
        compact=dict(bound="hbm", achieved=cp_gbs, peak=peaks["hbm"], unit="GB/s", frac=cp_gbs / peaks["hbm"],
                     traffic=traffic.get("compact"), ms_per_launch=cp_ms / max(cp_n, 1), launches=cp_n, ms_total=cp_ms),
        decode=dict(bound="hbm", achieved=dc_gbs, peak=peaks["hbm"], unit="GB/s", frac=dc_gbs / peaks["hbm"],
                    traffic=traffic.get("decode"), ms_per_launch=dc_ms / max(dc_n, 1), launches=dc_launches, launches_timed=dc_n,
                    ms_total=dc_total_ms,
                    note="the cache of this workload (35 MB) stays in L2 between decode steps; HBM-bound shapes are "
                         "timed by `python -m paper_2502_07861_b200.microbench decode`; duration = decode loop time / launches"))
    if not cp_n:
        # the tensor-core walk kernel selects and compacts at its tail: no launch of its own; the bytes it
        # moves (algorithmic, per launch of the walk kernel) are reported, its time is part of gram_walk's
        kernels["compact"] = dict(bound="hbm", fused_into="gram_walk", achieved=None, peak=peaks["hbm"], unit="GB/s", frac=None,
                                  traffic=None, algorithmic_bytes_per_walk_launch=cp_bytes * calls_per_launch, launches=0,
                                  ms_total=0.0)
        kernels["gram_walk"]["includes"] = "strict-half selection and compaction of the survivors at the tail of every call"
    for k in kernels.values():
        k["share_of_step"] = k["ms_total"] / total_ms
    dominant = max(kernels, key=lambda n: kernels[n]["ms_total"])
    roofline = dict(kernel=dominant, peak_source=peaks["source"], **kernels[dominant])
    other = dict(radii_ms=prof["radii"][1] / args.steps, append_context_ms=prof["append"][1] / max(prof["append"][0], 1),
                 bookkeeping_ms=prof["bookkeeping"][1] / args.steps)

    cpu = None
    if not args.no_cpu_baseline:
        sample, dsteps = n_ctx, (max(n_dec // 4, 1) if n_dec else 0)
        dt, units, threads, scaled = oracle_sample(w, Kf, Vf, qf, sample, dsteps)
        cpu = dict(value=units / scaled, unit=UNIT, cores=threads, kind="oracle", seconds=dt,
                   sample=f"all {n_ctx} context tokens of each of the {B * H} streams + {dsteps} of the {n_dec} decode steps "
                          f"(their time scaled to {n_dec})")
    pc = None
    if not args.no_per_config and world == 1 and (n_ctx, n_dec) == (WORKLOAD["context"], WORKLOAD["decode_steps"]):
        ctx.close()
        del K_ctx, V_ctx, flush
        torch.cuda.empty_cache()
        pc = per_config(peaks)
    line = dict(
        metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
        ms_per_step=total_ms / args.steps, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16",
        data="synthetic",
        config=dict(workload=w["name"], n_kv_heads=H, n_q_heads=Hq, head_dim=d, context=n_ctx, block=t, levels=T,
                    decode_steps=n_dec, walk_kernel={0: "none", 1: "cuda-core fp32", 2: "tcgen05"}[int(status["walk_kernel"])],
                    decode_kernel={1: "cuda-core", 2: "mma.sync + TMA"}[int(status["decode_kernel"])],
                    l2="flushed between steps (256 MB write, outside the event brackets); inputs 134 MB > L2",
                    replicas_per_gpu=1),
        compress_tokens_per_s=units_per_step / (float(t_comp.mean()) * 1e-3),
        compress_ms=float(t_comp.mean()),
        decode_us_per_step=1e3 * float(t_dec.mean()) / max(n_dec, 1),
        decode_attn_kernel_us=1e3 * dc_ms / max(dc_n, 1),
        roofline=roofline, kernels=kernels, other_kernels=other,
        e2e=dict(value=world * units_per_step * e2e_steps / e2e_s, unit=UNIT, h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h,
                 ms_per_step=1e3 * e2e_s / e2e_steps, timing="wall clock, synchronised on both sides"),
        gpu_launches=int(launches), clocks=clocks, cpu_baseline=cpu,
        device_status=int(status["device_status"]), walk_fails=int(status["walk_fails"]), per_config=pc,
    )
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
