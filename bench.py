#!/usr/bin/env python
"""Benchmark of the LCKV layer-stack decode step (one new token per sequence, all layers).

A "step" is one lckv_layer_stack_step: plan, every layer's attention over its cache (the shared
top-layer cache for condensed layers, own caches for warmup layers), the appends of the layers that
have k,v, and the length advance.  The metric is the algorithmic KV bytes the step reads
(sum over layers and sequences of 4*H_kv*d_h*visible rows) per second.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llama7b] [--batch B]
    python bench.py --impl reference ...     # times the float64 CPU checker on a bounded sample

One JSON line is printed by rank 0.  With N > 1 (torchrun) every rank runs the same per-GPU
workload on its own GPU (sequences are independent: no collective on the data path) and the
value is the sum over ranks divided by the slowest rank's time.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2405_10637_b200 import inputs as syn  # noqa: E402

METRIC = "condensed decode-attn GB/s (% of 8 TB/s HBM) and layer-stack attn µs/step vs B"
NOMINAL_HBM_GBS = 8000.0


# DRAM counters of one captured launch per kernel (ncu, small case; summaries under profiles/).  Reads grow
# with the rows read, so they are scaled by the algorithmic input bytes; the writes beyond the output rows
# (split-K partials, bounded by the worker count, and write-backs) are a per-launch constant.
NCU_CAPTURES = {
    "attn_alu_kernel": {
        "source": "profiles/attn_alu_kernel_llama7b_b8_ncu_full.md",
        "alg_in": 283.9e6 - 65536, "read": 284.00e6, "write": 3.46e6, "out": 65536,
        "applies": lambda a: a.workload in ("llama7b", "llama30b", "sweep7b") and not a.page_rows,
    },
    "attn_mma_kernel": {
        "source": "profiles/attn_mma_kernel_tinyllama_b128_ncu_full.md",
        "alg_in": 135.3e6 - 524288, "read": 143.21e6, "write": 4.6e6, "out": 524288,
        # the over-read of whole 64-row boxes depends on where the lengths sit: default context only
        "applies": lambda a: a.workload == "tinyllama" and a.context in (0, 1024) and a.batch in (0, 128)
        and not a.page_rows,
    },
}


def scaled_traffic(kernel, args, alg_bytes, out_bytes):
    """dram read + write bytes of one launch, scaled from the captured launch; None where it does not apply."""
    cap = NCU_CAPTURES[kernel]
    if not cap["applies"](args):
        return None
    reads = cap["read"] / cap["alg_in"] * (alg_bytes - out_bytes)
    return reads + out_bytes + (cap["write"] - cap["out"])


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def workload_params(args):
    wl = syn.WORKLOADS[args.workload]
    if args.workload == "llama7b":
        p = dict(batch=512, lo=256, hi=4096, t_cap=4096, sweep=[8, 16, 32, 64, 128, 256, 512])
    elif args.workload == "tinyllama":
        p = dict(batch=128, lo=1024, hi=1024, t_cap=1024, sweep=[128])
    elif args.workload == "toy":
        p = dict(batch=2, lo=128, hi=128, t_cap=128, sweep=[2])
    elif args.workload == "llama30b":
        p = dict(batch=256, lo=3072, hi=3072, t_cap=3072, sweep=[256])
    elif args.workload == "sweep7b":
        p = dict(batch=64, lo=8192, hi=8192, t_cap=8192, sweep=[64])
    elif args.workload == "gqa4":
        p = dict(batch=256, lo=4096, hi=4096, t_cap=4096, sweep=[256])
    else:
        raise SystemExit(f"unknown workload {args.workload}")
    if args.batch:
        p["batch"] = args.batch
        p["sweep"] = [b for b in p["sweep"] if b <= args.batch] or [args.batch]
        if args.batch not in p["sweep"]:
            p["sweep"].append(args.batch)
    if args.warmup_layers is not None:
        wl = wl.with_(n_warmup=args.warmup_layers)
    if args.context:
        p["lo"] = p["hi"] = args.context
        p["t_cap"] = args.context
    if args.stream_sink:
        # sink + recent-window caches of exactly t_cap rows, already full: every sequence is three
        # cache sizes long, so appends wrap around the ring and reads cover the whole cache
        p["lo"] = p["hi"] = 3 * p["t_cap"]
    else:
        # room for the tokens the run itself appends (lengths grow by one per step)
        p["t_cap"] += max(64, args.steps + args.warmup + 8)
    return wl, p


def step_kv_bytes(wl, plan_modes, lens, batch, grown=0, cap=0):
    """Algorithmic K+V bytes one step reads: every layer reads its visible rows once.
    `grown` = tokens appended to every sequence since `lens` was set."""
    per_row = 4 * wl.n_kv_heads * wl.head_dim
    ln = np.asarray(lens[:batch], np.int64) + grown
    total = 0
    for m in plan_modes:
        vis = ln + m
        if cap:
            vis = np.minimum(vis, cap)
        total += per_row * int(vis.sum())
    return total


class ClockSampler:
    """Samples nvidia-smi SM clocks and throttle reasons while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.thread.join(timeout=2)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except Exception:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons),
                "samples": len(sm)}


def oracle_sample(wl, plan, Ks, Vs, lens, rows, scale, min_seconds=10.0):
    """Times the CPU checker, as it stands, on the first `rows` sequences (all layers)."""
    from oracle import lckv_oracle as orc
    L = wl.n_layers
    q = [syn.bits(syn.randn_bf16((rows, wl.n_q_heads, wl.head_dim), 900 + l, std=wl.std))
         for l in range(L)]
    kv = [syn.bits(syn.randn_bf16((rows, wl.n_kv_heads, wl.head_dim), 950 + l, std=wl.std))
          if plan["write_slot"][l] >= 0 else None for l in range(L)]
    modes = [int(m) for m in plan["mode"]]
    nbytes = step_kv_bytes(wl, modes, lens, rows)
    t_total, n = 0.0, 0
    while t_total < min_seconds and n < 50:
        ln = np.asarray(lens[:rows], np.int32).copy()
        t0 = time.perf_counter()
        orc.stack_step(L, wl.n_warmup, q, kv, kv, Ks, Vs, ln, scale)
        t_total += time.perf_counter() - t0
        n += 1
        # undo the append so that every repetition does the same work
        # (the appended row lies beyond the restored length and is simply overwritten next time)
    return nbytes * n / t_total / 1e9, orc.num_threads(), n, t_total / n


def run_reference(args):
    """--impl reference: the float64 CPU checker on a bounded sample of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import lckv_oracle as orc
    wl, p = workload_params(args)
    rows = min(args.ref_rows, p["batch"])
    lens = syn.ragged_lengths(p["batch"], p["lo"], p["hi"], syn.seed_for(wl, syn.T_LENS)).numpy()
    plan = orc.plan(wl.n_layers, wl.n_warmup, 0)
    scale = wl.head_dim ** -0.5
    Ks = [syn.bits(syn.randn_bf16((rows, wl.n_kv_heads, p["t_cap"], wl.head_dim),
                                   syn.seed_for(wl, syn.T_K, s), std=wl.std))
          for s in range(plan["n_slots"])]
    Vs = [syn.bits(syn.randn_bf16((rows, wl.n_kv_heads, p["t_cap"], wl.head_dim),
                                   syn.seed_for(wl, syn.T_V, s), std=wl.std))
          for s in range(plan["n_slots"])]
    L = wl.n_layers
    q = [syn.bits(syn.randn_bf16((rows, wl.n_q_heads, wl.head_dim), 900 + l, std=wl.std))
         for l in range(L)]
    kv = [syn.bits(syn.randn_bf16((rows, wl.n_kv_heads, wl.head_dim), 950 + l, std=wl.std))
          if plan["write_slot"][l] >= 0 else None for l in range(L)]
    modes = [int(m) for m in plan["mode"]]
    nbytes = step_kv_bytes(wl, modes, lens, rows)

    def one():
        ln = np.asarray(lens[:rows], np.int32).copy()
        t0 = time.perf_counter()
        orc.stack_step(L, wl.n_warmup, q, kv, kv, Ks, Vs, ln, scale)
        return time.perf_counter() - t0
    for _ in range(args.warmup):
        one()
    ts = [one() for _ in range(args.steps)]
    ms = 1e3 * float(np.mean(ts))
    val = nbytes / (ms * 1e-3) / 1e9
    sample = f"first {rows} of {p['batch']} sequences, all {L} layers, one decode step per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": "GB/s", "n_gpus": 0,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(wl, p), "sample_rows": rows},
        "cpu_baseline": {"value": val, "unit": "GB/s", "cores": orc.num_threads(),
                         "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def workload_name(wl, p):
    ctx = f"ragged U[{p['lo']},{p['hi']}]" if p["lo"] != p["hi"] else f"context {p['lo']}"
    return (f"{wl.name}: L={wl.n_layers} H_q={wl.n_q_heads} H_kv={wl.n_kv_heads} d_h={wl.head_dim} "
            f"w={wl.n_warmup} {ctx} B={p['batch']} one decode step")


def time_steps(fn, steps, stream):
    """CUDA-event time of `steps` calls of fn on the current stream, in ms (total)."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        fn()
    e1.record(stream)
    e1.synchronize()
    return e0.elapsed_time(e1)


def run_ours(args):
    from paper_2405_10637_b200 import binding as lk
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus and world > 1:
        raise SystemExit("--gpus must equal WORLD_SIZE under torchrun")
    from paper_2405_10637_b200 import multi
    torch.cuda.set_device(local)
    if world > 1:
        multi.init("nccl", torch.device(f"cuda:{local}"))
    torch.cuda.set_device(local)
    dev = torch.device(f"cuda:{local}")
    torch.cuda.set_stream(torch.cuda.Stream(device=dev))  # a capturable (non-default) stream
    stream = torch.cuda.current_stream()

    wl, p = workload_params(args)
    B, T_cap = p["batch"], p["t_cap"]
    L = wl.n_layers
    # every rank draws its own sequences (different seeds): independent replicas of the workload
    lens = syn.ragged_lengths(B, p["lo"], p["hi"], syn.seed_for(wl, syn.T_LENS, rank)).numpy()
    n_pages = 0
    if args.page_rows:   # pool: what the sequences hold at the end of the longest timed run, + 2 %
        grow = max(64, args.steps + args.warmup + 8)
        n_pages = int(1.02 * sum((int(x) + grow + args.page_rows - 1) // args.page_rows for x in lens)) + 8
    cfg = lk.make_config(L, wl.n_warmup, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, B, T_cap,
                         host_staging=1, use_graph=1 if args.graph else 0, kernel_kind=args.kernel_kind,
                         top_variant=args.top_variant, stream_sink=args.stream_sink,
                         page_rows=args.page_rows, n_pages=n_pages)
    cap = T_cap if args.stream_sink else 0
    cache = lk.Cache(cfg, device=dev)
    plan = lk.lckv_plan(L, wl.n_warmup, args.top_variant)
    info = cache.info
    for s in range(info.n_slots):
        kt, vt = cache.slot_tensors(s)
        syn.fill_randn_bf16_(kt, syn.seed_for(wl, syn.T_K, s + 16 * rank), std=wl.std)
        syn.fill_randn_bf16_(vt, syn.seed_for(wl, syn.T_V, s + 16 * rank), std=wl.std)
    q = [syn.randn_bf16((B, wl.n_q_heads, wl.head_dim), 900 + l, device=dev, std=wl.std)
         for l in range(L)]
    kv = [syn.randn_bf16((B, wl.n_kv_heads, wl.head_dim), 950 + l, device=dev, std=wl.std)
          if plan["write_slot"][l] >= 0 else None for l in range(L)]
    outs = [torch.empty((B, wl.n_q_heads, wl.head_dim), dtype=torch.bfloat16, device=dev)
            for _ in range(L)]
    modes = plan["mode"]

    def reset(b):
        cache.lckv_cache_reset(lens[:b].tolist(), batch=b)

    def make_step(b):
        qs = [t[:b] for t in q]; os_ = [t[:b] for t in outs]
        kvs = [None if t is None else t[:b] for t in kv]

        def f():
            cache.lckv_layer_stack_step(qs, os_, kvs, kvs, batch=b)
        return f

    def run_timed(f, b, warm, k):
        """reset lengths, `warm` untimed steps, `k` timed steps (lengths grow by one per step).
        Returns (ms per step, mean algorithmic bytes per timed step)."""
        reset(b)
        for _ in range(warm):
            f()
        barrier()
        ms = time_steps(f, k, stream) / k
        by = sum(step_kv_bytes(wl, modes, lens, b, warm + i, cap) for i in range(k)) / k
        return ms, by

    def barrier():
        torch.cuda.synchronize()
        multi.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(ms):
        return multi.max_over_ranks(ms, dev)

    # ---- headline: K steps at the full batch --------------------------------------------------
    step = make_step(B)
    run_timed(step, B, 1, 1)  # first-touch of everything
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    ms_step, bytes_step = run_timed(step, B, args.warmup, args.steps)
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    ms_step = max_over_ranks(ms_step)
    value = world * bytes_step / (ms_step * 1e-3) / 1e9
    assert cache.lckv_cache_status() == 0, "device-side wait timed out"

    # ---- roofline of the dominant kernel: condensed attention launches on the shared cache ------
    n_launch = max(8, min(64, L))
    qd, od = q[min(1, L - 1)], outs[min(1, L - 1)]

    def attn():
        cache.lckv_decode_attention(0, lk.MODE_CONDENSED, qd, out=od, batch=B)
    reset(B)
    for _ in range(3):
        attn()
    torch.cuda.synchronize()
    ms_attn = time_steps(attn, n_launch, stream) / n_launch
    io_bytes = 2 * B * wl.n_q_heads * wl.head_dim * 2
    alg_bytes = step_kv_bytes(wl, [0], lens, B, 0, cap) + io_bytes
    peak, peak_kind = measured_peaks()
    achieved = alg_bytes / (ms_attn * 1e-3) / 1e9
    kernel_name = "attn_alu_kernel" if info.kernel_kind == 1 else "attn_mma_kernel"
    traffic = scaled_traffic(kernel_name, args, alg_bytes, io_bytes // 2)
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "traffic": traffic, "peak_kind": peak_kind,
                "kernel": kernel_name,
                "traffic_source": NCU_CAPTURES[kernel_name]["source"] if traffic else None,
                "us_per_launch": ms_attn * 1e3, "algorithmic_bytes_per_launch": alg_bytes,
                "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS}

    # ---- batch sweep (µs/step vs B) ---------------------------------------------------------
    sweep = []
    for b in p["sweep"]:
        if b > B:
            continue
        f = make_step(b)
        k = max(3, min(args.steps, 10))
        ms, by = run_timed(f, b, 3, k)
        ms = max_over_ranks(ms)
        gbs = by / (ms * 1e-3) / 1e9
        sweep.append({"B": b, "us_per_step": ms * 1e3, "kv_GBps": gbs,
                      "frac_of_measured_peak": gbs / peak, "frac_of_8TBs": gbs / NOMINAL_HBM_GBS})

    # ---- end to end through the host-buffer entry point ----------------------------------------
    # one pinned allocation per tensor kind, sliced per layer (equally spaced -> pitched copies)
    hq_all = torch.stack([t.cpu() for t in q]).pin_memory()
    hq = [hq_all[l] for l in range(L)]
    kv_layers = [l for l in range(L) if kv[l] is not None]
    hkv_all = torch.stack([kv[l].cpu() for l in kv_layers]).pin_memory()
    hkv = [None] * L
    for i, l in enumerate(kv_layers):
        hkv[l] = hkv_all[i]
    hout_all = torch.empty((L, B, wl.n_q_heads, wl.head_dim), dtype=torch.bfloat16).pin_memory()
    hout = [hout_all[l] for l in range(L)]

    def e2e_step():
        cache.lckv_layer_stack_step_host(hq, hout, hkv, hkv, batch=B)
    k = max(3, min(args.steps, 10))
    ms_e2e, by_e2e = run_timed(e2e_step, B, 3, k)
    ms_e2e = max_over_ranks(ms_e2e)
    h2d = sum(t.numel() * 2 for t in hq) + 2 * sum(t.numel() * 2 for t in hkv if t is not None)
    d2h = sum(t.numel() * 2 for t in hout)
    e2e = {"value": world * by_e2e / (ms_e2e * 1e-3) / 1e9, "unit": "GB/s",
           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e}

    # ---- CPU baseline: the checker on a bounded sample (rank 0, N = 1 only) --------------------
    cpu = None
    if rank == 0 and world == 1 and not (args.no_cpu_baseline or args.stream_sink or args.page_rows):
        rows = min(args.ref_rows, B)
        Ks = [syn.bits(cache.slot_tensors(s)[0][:rows]) for s in range(info.n_slots)]
        Vs = [syn.bits(cache.slot_tensors(s)[1][:rows]) for s in range(info.n_slots)]
        gbs, cores, n, sec = oracle_sample(wl, {k_: np.asarray(v) for k_, v in plan.items()
                                                if k_ != "n_slots"},
                                           Ks, Vs, lens, rows, wl.head_dim ** -0.5)
        cpu = {"value": gbs, "unit": "GB/s", "cores": cores, "kind": "oracle",
               "sample": f"first {rows} of {B} sequences, all {L} layers, {n} repetitions of one "
                         f"decode step ({sec:.2f} s each)"}

    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": workload_name(wl, p), "l2": "inputs larger than L2"
                       if 2 * info.slot_bytes > 2 * 126e6 else "L2-resident cache: warm",
                       "kv_bytes_per_step": bytes_step, "footprint_slots": info.n_slots,
                       "top_variant": args.top_variant, "graph": bool(args.graph),
                       "stream_sink": args.stream_sink, "page_rows": args.page_rows,
                       "cache_bytes": int(2 * info.n_slots * info.slot_bytes)},
            "frac_of_8TBs": value / world / NOMINAL_HBM_GBS,
            "clocks": clocks, "e2e": e2e, "gpu_launches": info.launches_per_step * args.steps,
            "roofline": roofline, "cpu_baseline": cpu, "sweep": sweep,
        }))
    cache.close()
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def run_prefill(args):
    """--prefill N: times the prompt-encoding attention (one layer, condensed mode, N prompt tokens
    per sequence) and reports tensor-core throughput.  Not the headline metric: a side measurement."""
    from paper_2405_10637_b200 import binding as lk
    wl, p = workload_params(args)
    n = args.prefill
    B = args.batch or 8
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    cfg = lk.make_config(2, 0, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, B, n)
    cache = lk.Cache(cfg, device=dev)
    kt, vt = cache.slot_tensors(0)
    syn.fill_randn_bf16_(kt, 1, std=wl.std); syn.fill_randn_bf16_(vt, 2, std=wl.std)
    cache.lckv_cache_reset([n] * B)
    q = syn.randn_bf16((B, n, wl.n_q_heads, wl.head_dim), 3, device=dev, std=wl.std)
    out = torch.empty_like(q)
    stream = torch.cuda.current_stream()

    def f():
        cache.lckv_prefill_attention(0, lk.MODE_CONDENSED, q, out=out)
    for _ in range(max(3, args.warmup)):
        f()
    torch.cuda.synchronize()
    ms = time_steps(f, args.steps, stream) / args.steps
    # visible (i, j) pairs with j < i: n(n-1)/2 per (sequence, head); 4*d flops per pair (QK^T and PV)
    flops = 4.0 * wl.head_dim * wl.n_q_heads * B * (n * (n - 1) / 2)
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as fh:
            peak, kind = float(json.load(fh)["bf16_tflops"]), "measured"
    except Exception:
        peak, kind = 1590.0, "fallback"
    tf = flops / (ms * 1e-3) / 1e12
    print(json.dumps({
        "metric": "prompt-encoding attention TFLOP/s (causal, useful flops only)", "value": tf,
        "unit": "TFLOP/s", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms, "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{wl.name} head layout, prompt {n}, B={B}, one layer, j<i mask"},
        "roofline": {"bound": "tensor", "achieved": tf, "peak": peak, "unit": "TFLOP/s",
                     "frac": tf / peak, "traffic": None, "peak_kind": kind,
                     "kernel": "prefill_attn_kernel" if os.environ.get("LCKV_PREFILL_KERNEL") == "mma" else "prefill_tc5_kernel"}}))
    cache.close()


def run_project(args):
    """--project D: times the fused key/value producer (x W_K^T, x W_V^T -> cache rows) for hidden width
    D at the workload's head layout.  Several weight sets are used in turn so that their bytes exceed
    the L2 (as the layers of a model would).  A side measurement, not the headline metric."""
    from paper_2405_10637_b200 import binding as lk
    wl, p = workload_params(args)
    dm = args.project
    B = args.batch or 64
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    F = wl.n_kv_heads * wl.head_dim
    T_cap = 64
    cfg = lk.make_config(2, 0, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, B, T_cap)
    cache = lk.Cache(cfg, device=dev)
    cache.lckv_cache_reset([5] * B)
    w_bytes = 2 * F * dm * 2
    n_sets = max(2, int(300e6 // w_bytes) + 1)           # > 126 MB of L2 between two uses of a set
    wk = [syn.randn_bf16((F, dm), 10 + 2 * i, device=dev, std=dm ** -0.5) for i in range(n_sets)]
    wv = [syn.randn_bf16((F, dm), 11 + 2 * i, device=dev, std=dm ** -0.5) for i in range(n_sets)]
    x = syn.randn_bf16((B, dm), 3, device=dev)
    half = wl.head_dim // 2
    ang = torch.arange(T_cap, device=dev, dtype=torch.float64)[:, None] * \
        (10000.0 ** (-2.0 * torch.arange(half, device=dev, dtype=torch.float64) / wl.head_dim))[None, :]
    cos, sin = torch.cos(ang).float().contiguous(), torch.sin(ang).float().contiguous()
    stream = torch.cuda.current_stream()
    it = [0]

    def f():
        i = it[0] % n_sets
        it[0] += 1
        cache.lckv_project_append_kv(0, x, wk[i], wv[i], cos, sin, advance_len=0)
    for _ in range(max(3, args.warmup) + n_sets):
        f()
    torch.cuda.synchronize()
    # One call is 10-50 us of device time, less than a Python call costs on the host: replay a captured
    # graph of one call per weight set so that the events see the device, not the interpreter.
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(stream)
    with torch.cuda.graph(graph, stream=side):
        for _ in range(n_sets):
            f()
    torch.cuda.synchronize()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    ms = time_steps(graph.replay, args.steps, stream) / (args.steps * n_sets)
    assert cache.lckv_cache_status() == 0, "device-side wait timed out"
    flops = 2.0 * B * 2 * F * dm
    byts = w_bytes + B * dm * 2 + 2 * B * F * 2
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as fh:
            pk = json.load(fh)
            peak_tf, peak_gb, kind = float(pk["bf16_tflops"]), float(pk["hbm_gbs"]), "measured"
    except Exception:
        peak_tf, peak_gb, kind = 1590.0, 6650.0, "fallback"
    tf = flops / (ms * 1e-3) / 1e12
    gbs = byts / (ms * 1e-3) / 1e9
    hbm_bound = byts / peak_gb / 1e9 >= flops / peak_tf / 1e12
    roof = {"bound": "hbm", "achieved": gbs, "peak": peak_gb, "unit": "GB/s", "frac": gbs / peak_gb} if hbm_bound \
        else {"bound": "tensor", "achieved": tf, "peak": peak_tf, "unit": "TFLOP/s", "frac": tf / peak_tf}
    roof.update({"traffic": None, "peak_kind": kind, "kernel": "project_kv_kernel", "tflops": tf, "GBps": gbs,
                 "algorithmic_bytes_per_launch": byts, "us_per_launch": ms * 1e3})
    print(json.dumps({
        "metric": "key/value producer (projection + rotary + append) us per call", "value": ms * 1e3,
        "unit": "us", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
        "higher_is_better": False, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{wl.name} head layout, d_model {dm}, B={B}, {n_sets} weight sets in turn",
                   "l2": "weight sets in rotation exceed L2"},
        "roofline": roof}))
    cache.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama7b", choices=sorted(syn.WORKLOADS))
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--context", type=int, default=0, help="equal context length for every sequence")
    ap.add_argument("--warmup-layers", type=int, default=None, help="override w")
    ap.add_argument("--top-variant", type=int, default=0)
    ap.add_argument("--graph", type=int, default=1)
    ap.add_argument("--kernel-kind", type=int, default=0, choices=[0, 1],
                    help="1: force the FP32-ALU attention kernel for grouped heads (0: automatic)")
    ap.add_argument("--page-rows", type=int, default=0,
                    help="P > 0: paged caches with P-row pages and a pool sized for the batch's lengths")
    ap.add_argument("--stream-sink", type=int, default=0,
                    help="s > 0: sink + recent-window caches with s sink tokens, cache size = context")
    ap.add_argument("--ref-rows", type=int, default=32)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--prefill", type=int, default=0,
                    help="N > 0: time the prompt-encoding attention on N-token prompts instead")
    ap.add_argument("--project", type=int, default=0,
                    help="D > 0: time the fused key/value producer for hidden width D instead")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device (the CUDA library has no CPU fallback)")
        if args.prefill:
            run_prefill(args)
        elif args.project:
            run_project(args)
        else:
            run_ours(args)


if __name__ == "__main__":
    main()
