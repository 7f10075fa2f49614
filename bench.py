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


# DRAM counters of one captured launch per kernel (ncu, small case): profiles/ncu_captures.json, written
# from the summaries beside it.  Reads grow with the rows read, so they are scaled by the algorithmic
# input bytes; the writes beyond the output rows (split-K partials, bounded by the worker count, and
# write-backs) are a per-launch constant.  A capture is void once the kernel's sources differ from
# the ones it was taken with (digest of the files named in the entry).
CAPTURES_FILE = os.path.join(ROOT, "profiles", "ncu_captures.json")
CSRC = os.path.join(ROOT, "paper_2405_10637_b200", "csrc")


def source_digest(files):
    """sha256 over the named kernel sources, in order."""
    import hashlib
    h = hashlib.sha256()
    for f in files:
        with open(os.path.join(CSRC, f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def load_captures():
    with open(CAPTURES_FILE) as f:
        return json.load(f)


def capture_applies(cap, args):
    """Does the captured launch's traffic scale to this run's launches?"""
    c = cap["applies"]
    if args.workload not in c["workloads"] or args.page_rows or args.stream_sink:
        return False
    if "contexts" in c and args.context not in c["contexts"]:
        return False
    if "batches" in c and args.batch not in c["batches"]:
        return False
    return True


def scaled_traffic(kernel, args, alg_bytes, out_bytes, captures=None, check_sources=True):
    """dram read + write bytes of one launch, scaled from the captured launch; None where the capture
    does not apply or the kernel has changed since."""
    cap = (captures or load_captures()).get(kernel)
    if cap is None or not capture_applies(cap, args):
        return None
    if check_sources and source_digest(cap["sources"]) != cap["sources_digest"]:
        return None
    reads = cap["dram_read_bytes"] / cap["algorithmic_input_bytes"] * (alg_bytes - out_bytes)
    return reads + out_bytes + (cap["dram_write_bytes"] - cap["output_bytes"])


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


def bf16_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as fh:
            return float(json.load(fh)["bf16_tflops"]), "measured"
    except Exception:
        return 1590.0, "fallback"


def fill_cache(cache, wl, rank=0, seqs=None):
    """Seeded N(0, std) keys and values in every slot.  seqs = (b0, b1): this cache holds sequences
    [b0, b1) of one global batch and each sequence is drawn from its own seed, so the shards of a batch
    hold the same bits however many ranks share it."""
    for s in range(cache.info.n_slots):
        kt, vt = cache.slot_tensors(s)
        if seqs is None:
            syn.fill_randn_bf16_(kt, syn.seed_for(wl, syn.T_K, s + 16 * rank), std=wl.std)
            syn.fill_randn_bf16_(vt, syn.seed_for(wl, syn.T_V, s + 16 * rank), std=wl.std)
        else:
            for i, b in enumerate(range(*seqs)):
                syn.fill_randn_bf16_(kt[i], syn.seed_for(wl, syn.T_K, 64 * (b + 1) + s), std=wl.std)
                syn.fill_randn_bf16_(vt[i], syn.seed_for(wl, syn.T_V, 64 * (b + 1) + s), std=wl.std)


def read_stream_probe(lk, buf, stream, nbytes=8 << 30):
    """Read-only stream over the first `nbytes` of a device buffer with the library's probe kernels:
    GB/s per kind (best of 5 after 2 warm-up passes) - the ceiling of a read-dominated kernel."""
    nbytes = min(nbytes, buf.numel() * buf.element_size()) // 8192 * 8192
    acc = torch.zeros(1, dtype=torch.int32, device=buf.device)
    status = torch.zeros(1, dtype=torch.int32, device=buf.device)
    out = {"bytes": nbytes}
    for kind, name in ((0, "ldg16"), (2, "ldg32"), (1, "bulk8k")):
        def f():
            lk.lckv_read_stream_probe(buf, nbytes, kind, acc, status)
        for _ in range(2):
            f()
        torch.cuda.synchronize()
        best = min(time_steps(f, 1, stream) for _ in range(5))
        out[name] = nbytes / (best * 1e-3) / 1e9
    out["best"] = max(out["ldg16"], out["ldg32"], out["bulk8k"])
    # The same kernels over a 64 MiB piece read 16 times in one launch, every line marked evict-last:
    # the passes after the first are served by the L2 - the ceiling of a layer that re-reads a cache
    # which the previous layer left there (TinyLlama shape at 512 tokens).
    small, reps = min(64 << 20, nbytes), 16
    for kind, name in ((0, "l2_ldg16"), (1, "l2_bulk8k")):
        def g():
            lk.lckv_read_stream_probe(buf, small, kind, acc, status, repeats=reps, l2_keep=1.0)
        for _ in range(2):
            g()
        torch.cuda.synchronize()
        best = min(time_steps(g, 1, stream) for _ in range(5))
        out[name] = small * reps / (best * 1e-3) / 1e9
    out["l2_resident_bytes"] = small
    assert int(status.item()) == 0, "probe wait timed out"
    return out


def time_workload(lk, dev, stream, wl, B, lens, T_cap, steps, warm=3, graph=1, top_variant=0):
    """Allocates the caches of one workload, fills them, times `steps` decode steps (after `warm`),
    frees everything.  Returns the compact record used in the `configs` array."""
    L = wl.n_layers
    cfg = lk.make_config(L, wl.n_warmup, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, B, T_cap,
                         use_graph=graph, top_variant=top_variant)
    cache = lk.Cache(cfg, device=dev)
    try:
        plan = lk.lckv_plan(L, wl.n_warmup, top_variant)
        fill_cache(cache, wl)
        q = [syn.randn_bf16((B, wl.n_q_heads, wl.head_dim), 900 + l, device=dev, std=wl.std) for l in range(L)]
        kv = [syn.randn_bf16((B, wl.n_kv_heads, wl.head_dim), 950 + l, device=dev, std=wl.std)
              if plan["write_slot"][l] >= 0 else None for l in range(L)]
        outs = [torch.empty((B, wl.n_q_heads, wl.head_dim), dtype=torch.bfloat16, device=dev) for _ in range(L)]
        cache.lckv_cache_reset(np.asarray(lens).tolist(), batch=B)

        def f():
            cache.lckv_layer_stack_step(q, outs, kv, kv, batch=B)
        for _ in range(warm):
            f()
        torch.cuda.synchronize()
        ms = time_steps(f, steps, stream) / steps
        by = sum(step_kv_bytes(wl, plan["mode"], lens, B, warm + i) for i in range(steps)) / steps
        assert cache.lckv_cache_status() == 0, "device-side wait timed out"
        info = cache.info
        gbs = by / (ms * 1e-3) / 1e9
        return {"us_per_step": ms * 1e3, "kv_GBps": gbs, "frac_of_8TBs": gbs / NOMINAL_HBM_GBS,
                "kv_bytes_per_step": by, "cache_bytes": int(2 * info.n_slots * info.slot_bytes),
                "footprint_slots": info.n_slots, "B": B, "steps": steps,
                "kernel": "attn_alu_kernel" if info.kernel_kind == 1 else "attn_mma_kernel"}
    finally:
        cache.close()
        del cache
        torch.cuda.empty_cache()


def largest_batch(wl, T_cap, n_slots, budget_bytes=180e9):
    """Largest batch whose caches (n_slots of them, T_cap rows per sequence) fit the budget."""
    return int(budget_bytes // (n_slots * 4 * wl.n_kv_heads * wl.head_dim * T_cap))


def config_matrix(lk, dev, stream):
    """The other workload shapes, each a few decode steps: toy, TinyLlama (B = 128 at three context
    lengths of the 512 + 1024 run), the 30B shape at the largest batch that fits, and the warmup-count
    sweep on the 7B shape at both long-context sizes."""
    W = syn.WORKLOADS
    rows = []

    def add(name, wl, B, T, steps, T_cap=None, **kw):
        r = time_workload(lk, dev, stream, wl, B, np.full(B, T, np.int32), T_cap or T + steps + 8, steps, **kw)
        r["workload"] = name
        rows.append(r)
    add("toy L4 MHA4 d64 w0 B2 T128", W["toy"], 2, 128, 50)
    for T in (512, 1024, 1535):   # start, middle and end of the 512 + 1024 run
        add(f"tinyllama B128 T{T}", W["tinyllama"], 128, T, 30)
    # 30B shape: 2 caches (w = 2, literal reading of "top layer"), 4096 rows per sequence
    free = torch.cuda.mem_get_info()[0]
    wl = W["llama30b"]
    B30 = min(largest_batch(wl, 4096, 2), largest_batch(wl, 4096, 2, free - 6e9))
    add(f"llama30b w2 B{B30} T2048 (largest batch whose caches fit 180 GB)", wl, B30, 2048, 3, T_cap=4096)
    for w in (0, 2, 4, 8, 32):
        wl = W["sweep7b"].with_(n_warmup=w)
        B = 64 if w < 32 else min(40, largest_batch(wl, 8192 + 16, 32, free - 6e9))   # 64 sequences x 32 caches = 275 GB: does not fit
        add(f"sweep7b w{w} B{B} T8192", wl, B, 8192, 4)
    for w in (0, 2, 32):
        add(f"sweep7b w{w} B8 T32768", W["sweep7b"].with_(n_warmup=w), 8, 32768, 4)
    return rows


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
    L = wl.n_layers
    B_job, T_cap = p["batch"], p["t_cap"]
    # Sharding.  Default: every rank runs the whole per-GPU workload on sequences of its own
    # (replicas, weak scaling).  --shard batch / heads: ONE seeded batch of B_job sequences is split
    # over the ranks by sequences or by kv heads (strong scaling); no rank needs another's data.
    b0, b1, h0, h1 = 0, B_job, 0, wl.n_kv_heads
    if args.shard == "batch":
        b0, b1 = syn.shard_batch(B_job, rank, world)
    elif args.shard == "heads":
        h0, h1 = syn.shard_heads(wl.n_kv_heads, rank, world)
    B = b1 - b0
    g = wl.n_q_heads // wl.n_kv_heads
    wl_local = wl.with_(n_q_heads=(h1 - h0) * g, n_kv_heads=h1 - h0)
    lens_seed = syn.seed_for(wl, syn.T_LENS, 0 if args.shard else rank)
    lens = syn.ragged_lengths(B_job, p["lo"], p["hi"], lens_seed).numpy()[b0:b1]
    n_pages = 0
    if args.page_rows:   # pool: what the sequences hold at the end of the longest timed run, + 2 %
        grow = max(64, args.steps + args.warmup + 8)
        n_pages = int(1.02 * sum((int(x) + grow + args.page_rows - 1) // args.page_rows for x in lens)) + 8
    cfg = lk.make_config(L, wl.n_warmup, wl_local.n_q_heads, wl_local.n_kv_heads, wl.head_dim, B, T_cap,
                         host_staging=1, use_graph=1 if args.graph else 0, kernel_kind=args.kernel_kind,
                         top_variant=args.top_variant, stream_sink=args.stream_sink,
                         page_rows=args.page_rows, n_pages=n_pages)
    cap = T_cap if args.stream_sink else 0
    cache = lk.Cache(cfg, device=dev)
    plan = lk.lckv_plan(L, wl.n_warmup, args.top_variant)
    info = cache.info
    if args.shard:
        fill_sharded(cache, wl, b0, b1, h0, h1)
    else:
        fill_cache(cache, wl, rank)
    wl = wl_local
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
    # whole-job bytes: all ranks' units over the slowest rank's time
    value = multi.sum_over_ranks(bytes_step, dev) / (ms_step * 1e-3) / 1e9
    assert cache.lckv_cache_status() == 0, "device-side wait timed out"

    # ---- spread of single steps (each bracketed by its own pair of events) -----------------------
    reset(B)
    for _ in range(3):
        step()
    torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
          for _ in range(max(5, min(args.steps, 20)))]
    for e0, e1 in ev:
        e0.record(stream)
        step()
        e1.record(stream)
    torch.cuda.synchronize()
    us = np.array([e0.elapsed_time(e1) * 1e3 for e0, e1 in ev])
    step_spread = {"n": len(us), "p10": float(np.percentile(us, 10)), "median": float(np.median(us)),
                   "p90": float(np.percentile(us, 90))}

    # ---- optional: K further steps inside one cudaProfilerStart/Stop range (for a range-based ncu
    #      capture, which counts DRAM bytes and L2 hits of whole steps without serialising the launches)
    if args.profiler_range:
        reset(B)
        for _ in range(3):
            step()
        torch.cuda.synchronize()
        torch.cuda.profiler.start()
        for _ in range(args.profiler_range):
            step()
        torch.cuda.synchronize()
        torch.cuda.profiler.stop()

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
    captures = load_captures()
    traffic = None if args.shard else scaled_traffic(kernel_name, args, alg_bytes, io_bytes // 2, captures)
    probe = read_stream_probe(lk, cache.buf, stream)
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "traffic": traffic, "peak_kind": peak_kind,
                "peak_note": "the measured peak is a read + write copy; a read-only stream on this GPU "
                             "reaches read_stream_gbs (this library's probe kernels, "
                             f"{probe['bytes'] >> 30} GiB), which is the ceiling of this read-dominated kernel",
                "read_stream_gbs": probe["best"], "read_stream": probe,
                "frac_of_read_stream": achieved / probe["best"],
                "kernel": kernel_name,
                "traffic_source": captures[kernel_name]["source"] if traffic else None,
                "us_per_launch": ms_attn * 1e3, "algorithmic_bytes_per_launch": alg_bytes,
                "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS}

    # ---- batch sweep (µs/step vs B) ---------------------------------------------------------
    sweep = []
    for b in ([] if args.shard else p["sweep"]):
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
    e2e = {"value": multi.sum_over_ranks(by_e2e, dev) / (ms_e2e * 1e-3) / 1e9, "unit": "GB/s",
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
        del Ks, Vs

    launches = info.launches_per_step * args.steps
    cache_bytes = int(2 * info.n_slots * info.slot_bytes)
    slots = info.n_slots
    cache.close()
    del cache, hq_all, hkv_all, hout_all
    torch.cuda.empty_cache()

    # ---- the other workload shapes and the kernels beside the decode path (N = 1, default run) ---
    configs = nxt = clocks_extras = None
    if world == 1 and args.extras:
        sampler = ClockSampler(local)
        sampler.start()
        configs = config_matrix(lk, dev, stream)
        nxt = {"prompt_encoding_n8192": prefill_record(lk, dev, W7B(), 8192, 8, 10),
               "kv_producer_b16": project_record(lk, dev, W7B(), 4096, 16, 20),
               "kv_producer_b512": project_record(lk, dev, W7B(), 4096, 512, 20)}
        clocks_extras = sampler.stop()

    if rank == 0:
        layer_pass_bytes = bytes_step / L
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "strong" if args.shard else "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": workload_name(syn.WORKLOADS[args.workload] if args.warmup_layers is None else
                                                 syn.WORKLOADS[args.workload].with_(n_warmup=args.warmup_layers), p),
                       "storage_dtype": "bf16 (q, K, V, outputs); fp32 scores, sums, accumulators, partials",
                       "l2": "inputs larger than L2: a layer's pass over its cache reads "
                             f"{layer_pass_bytes / 1e6:.0f} MB" if layer_pass_bytes > 2 * 126e6 else
                             f"a layer's pass reads {layer_pass_bytes / 1e6:.0f} MB, within reach of the 126 MB L2: "
                             "warm (consecutive layers re-read the shared cache)",
                       "shard": args.shard or "replicas", "sequences_this_rank": B,
                       "kv_heads_this_rank": wl.n_kv_heads,
                       "kv_bytes_per_step": bytes_step, "footprint_slots": slots,
                       "top_variant": args.top_variant, "graph": bool(args.graph),
                       "stream_sink": args.stream_sink, "page_rows": args.page_rows,
                       "cache_bytes": cache_bytes},
            "frac_of_8TBs": value / world / NOMINAL_HBM_GBS, "us_per_step_spread": step_spread,
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches,
            "roofline": roofline, "cpu_baseline": cpu, "sweep": sweep,
            "configs": configs, "next": nxt, "clocks_extras": clocks_extras,
        }))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def W7B():
    return syn.WORKLOADS["llama7b"]


def fill_sharded(cache, wl, b0, b1, h0, h1):
    """Caches of the shard [b0, b1) x kv heads [h0, h1) of one global batch: every (sequence, slot) is
    drawn from its own seed over ALL kv heads and the shard's heads are copied out, so the shards of
    any split hold the same bits as the unsplit batch."""
    for s in range(cache.info.n_slots):
        kt, vt = cache.slot_tensors(s)
        full = torch.empty((wl.n_kv_heads,) + tuple(kt.shape[2:]), dtype=torch.bfloat16, device=kt.device)
        for i, b in enumerate(range(b0, b1)):
            syn.fill_randn_bf16_(full, syn.seed_for(wl, syn.T_K, 64 * (b + 1) + s), std=wl.std)
            kt[i].copy_(full[h0:h1])
            syn.fill_randn_bf16_(full, syn.seed_for(wl, syn.T_V, 64 * (b + 1) + s), std=wl.std)
            vt[i].copy_(full[h0:h1])


def prefill_record(lk, dev, wl, n, B, steps, warm=3):
    """Prompt-encoding attention (one layer, condensed mask, n prompt tokens per sequence): useful
    causal TFLOP/s against the measured bf16 peak."""
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
    for _ in range(max(3, warm)):
        f()
    torch.cuda.synchronize()
    ms = time_steps(f, steps, stream) / steps
    assert cache.lckv_cache_status() == 0, "device-side wait timed out"
    # visible (i, j) pairs with j < i: n(n-1)/2 per (sequence, head); 4*d flops per pair (QK^T and PV)
    flops = 4.0 * wl.head_dim * wl.n_q_heads * B * (n * (n - 1) / 2)
    peak, kind = bf16_peak()
    tf = flops / (ms * 1e-3) / 1e12
    cache.close()
    del cache, q, out
    torch.cuda.empty_cache()
    return {"workload": f"{wl.name} head layout, prompt {n}, B={B}, one layer, j<i mask", "ms": ms,
            "bound": "tensor", "achieved": tf, "peak": peak, "unit": "TFLOP/s", "frac": tf / peak,
            "traffic": None, "peak_kind": kind,
            "kernel": "prefill_attn_kernel" if os.environ.get("LCKV_PREFILL_KERNEL") == "mma" else "prefill_tc5_kernel"}


def run_prefill(args):
    """--prefill N: times the prompt-encoding attention and reports tensor-core throughput.  Not the
    headline metric: a side measurement."""
    from paper_2405_10637_b200 import binding as lk
    wl, p = workload_params(args)
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    r = prefill_record(lk, dev, wl, args.prefill, args.batch or 8, args.steps, args.warmup)
    print(json.dumps({
        "metric": "prompt-encoding attention TFLOP/s (causal, useful flops only)", "value": r["achieved"],
        "unit": "TFLOP/s", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": r["ms"], "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": r["workload"]},
        "roofline": {k: r[k] for k in ("bound", "achieved", "peak", "unit", "frac", "traffic", "peak_kind", "kernel")}}))


def project_record(lk, dev, wl, dm, B, steps, warm=3):
    """The fused key/value producer (x W_K^T, x W_V^T -> cache rows) for hidden width dm at the
    workload's head layout.  Several weight sets are used in turn so that their bytes exceed the L2 (as
    the layers of a model would)."""
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
    for _ in range(max(3, warm) + n_sets):
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
    ms = time_steps(graph.replay, steps, stream) / (steps * n_sets)
    assert cache.lckv_cache_status() == 0, "device-side wait timed out"
    flops = 2.0 * B * 2 * F * dm
    byts = w_bytes + B * dm * 2 + 2 * B * F * 2
    peak_tf, kind = bf16_peak()
    peak_gb, _ = measured_peaks()
    tf = flops / (ms * 1e-3) / 1e12
    gbs = byts / (ms * 1e-3) / 1e9
    hbm_bound = byts / peak_gb / 1e9 >= flops / peak_tf / 1e12
    roof = {"bound": "hbm", "achieved": gbs, "peak": peak_gb, "unit": "GB/s", "frac": gbs / peak_gb} if hbm_bound \
        else {"bound": "tensor", "achieved": tf, "peak": peak_tf, "unit": "TFLOP/s", "frac": tf / peak_tf}
    roof.update({"traffic": None, "peak_kind": kind, "kernel": "project_kv_kernel", "tflops": tf, "GBps": gbs,
                 "algorithmic_bytes_per_launch": byts, "us_per_launch": ms * 1e3,
                 "workload": f"{wl.name} head layout, d_model {dm}, B={B}, {n_sets} weight sets in turn"})
    del graph
    cache.close()
    del cache, wk, wv
    torch.cuda.empty_cache()
    return roof


def run_project(args):
    """--project D: times the fused key/value producer.  A side measurement, not the headline metric."""
    from paper_2405_10637_b200 import binding as lk
    wl, p = workload_params(args)
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    roof = project_record(lk, dev, wl, args.project, args.batch or 64, args.steps, args.warmup)
    print(json.dumps({
        "metric": "key/value producer (projection + rotary + append) us per call", "value": roof["us_per_launch"],
        "unit": "us", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": roof["us_per_launch"] / 1e3,
        "higher_is_better": False, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": roof["workload"], "l2": "weight sets in rotation exceed L2"},
        "roofline": roof}))


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
    ap.add_argument("--shard", default="", choices=["", "batch", "heads"],
                    help="split ONE seeded batch over the ranks by sequences or by kv heads (strong scaling); "
                         "default: every rank runs its own replica of the workload (weak scaling)")
    ap.add_argument("--extras", type=int, default=-1,
                    help="1: also time the other workload shapes, prompt encoding and the key/value producer "
                         "(default: only in the plain default run)")
    ap.add_argument("--kernel-digests", action="store_true",
                    help="print the source digests profiles/ncu_captures.json compares against, and exit")
    ap.add_argument("--profiler-range", type=int, default=0,
                    help="K > 0: after the timed steps, run K more steps between cudaProfilerStart and "
                         "cudaProfilerStop (a range for ncu --replay-mode app-range)")
    ap.add_argument("--ref-rows", type=int, default=32)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--prefill", type=int, default=0,
                    help="N > 0: time the prompt-encoding attention on N-token prompts instead")
    ap.add_argument("--project", type=int, default=0,
                    help="D > 0: time the fused key/value producer for hidden width D instead")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.kernel_digests:
        for name, cap in load_captures().items():
            if isinstance(cap, dict):
                print(name, source_digest(cap["sources"]))
        return
    if args.extras < 0:   # the plain default run carries every workload shape
        args.extras = int(args.workload == "llama7b" and not (args.batch or args.context or args.page_rows or
                          args.stream_sink or args.shard or args.top_variant or args.kernel_kind or
                          args.warmup_layers is not None or args.prefill or args.project))
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
