#!/usr/bin/env python
"""Benchmark of the E-Sparse hot path on B200.

Headline: one forward pass over the seven pruned linears of a LLaMA-65B-shaped decoder layer (workload 3 of
paper_2310_15929_b200/inputs.py: q,k,v,o 8192x8192, gate,up 22016x8192, down 8192x22016) at M = 8192 tokens -- seven
esp_spgemm calls per step.  `value` is the dense-equivalent throughput 2*M*N*K / t summed over the layer (the unit the sparse
tensor-core peak is quoted in; executed flops are half of that).  The operands are produced on the device by esp_metric_prune
from seeded synthetic weights and calibration activations before the timed region.  In the same run and the same JSON line:

  decode        the six linears of an OPT-66B-shaped layer (workload 4) at M = 1 and M = 32, HBM GB/s
  llama7b       the LLaMA-7B-shaped layer (workload 1) at M = 2048 and M = 16, as earlier runs timed it
  per_config    every (workload, linear shape, M) the five workloads name: time, rate, roofline fraction, dense cuBLAS ratio
  footprint     compressed against dense bytes of the OPT-66B-shaped layer
  prune         the producer's time, beside the CPU oracle's producer on bounded samples
  cpu_baseline  the CPU oracle's fp64 product on a bounded sample of the headline workload

    python bench.py --gpus 1 --steps 20 --warmup 5
    python bench.py --impl reference          # the CPU oracle on the same bounded sample, K steps
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

HEAD_WORKLOAD, HEAD_M = 3, 8192            # llama-65b-layer, prefill
DECODE_WORKLOAD, DECODE_MS = 4, (1, 32)    # opt-66b-layer, decode
SMALL_WORKLOAD, PREFILL_M, DECODE_M = 1, 2048, 16      # llama-7b-layer (what earlier runs of this benchmark timed)
WORKLOAD = SMALL_WORKLOAD                  # the profile cases below run on this one
# dram__bytes_read.sum + dram__bytes_write.sum of the GEMM launches of one step, from the one-pass ncu captures of the
# full-size launches summarised under profiles/ (None = the kernel has changed since the counters were taken).
# Headline step: 4 x (8192 x 8192) + 2 x (22016 x 8192) + (8192 x 22016) at 8192 tokens.
PREFILL_TRAFFIC_BYTES = 4 * 0.923e9 + 2 * 2.126e9 + 2.28e9
# Decode step at one token: 4 x (9216 x 9216) + (36864 x 9216) + (9216 x 36864).
DECODE_TRAFFIC_BYTES = 4 * 99.1e6 + 388.5e6 + 387.5e6
# bounded sample of the headline workload that the CPU oracle's product is timed on
CPU_ROWS, CPU_FEATURES = 256, 1024


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_burst": p["bf16_tflops"], "bf16_sustained": p["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t_begin=0.0):
        """Summary of the samples that arrived at or after host time t_begin."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for t_arr, ln in self.lines:
            if t_arr < t_begin:
                continue
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def max_over_ranks(x, dist, device):
    """The largest of one float per rank (every rank gets it).  dist = torch.distributed or None for one rank."""
    if dist is None:
        return float(x)
    import torch
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(work_per_rank, world, ms_max):
    """Aggregate rate of `world` replicas that each did `work_per_rank` while the slowest took ms_max."""
    return world * work_per_rank / (ms_max * 1e-3)


def gemm_bytes(M, N, K):
    """Algorithmic bytes of one sparse GEMM: compressed weight + metadata, X, Y, permutation."""
    return 1.125 * N * K + 2.0 * M * K + 2.0 * M * N + 4.0 * K


def build_layer(dev, wl, alpha_of_T, lbs_max_swaps):
    """Seeded weights + calibration -> esp_metric_prune on the device for every linear of the workload."""
    import torch
    from paper_2310_15929_b200 import binding as b, inputs
    layer, prune_ms, prune_bytes, swaps = [], 0.0, 0.0, 0
    xcal_cache = {}
    for name, (N, K) in wl.linears.items():
        W = inputs.make_weight(wl, name)
        src = inputs.distinct_shapes(wl)[(N, K)]
        if K not in xcal_cache:
            xcal_cache = {}                                                            # keep only one resident
            xcal_cache[K] = torch.from_numpy(inputs.make_calibration(wl, src)).to(dev)
        Xc = xcal_cache[K]
        T = Xc.shape[0]
        o = b.esp_prune_opts_default()
        o.alpha = alpha_of_T(T)
        o.lbs_max_swaps = lbs_max_swaps
        Wd = torch.from_numpy(W).to(dev)
        del W
        ws = torch.empty(b.esp_metric_prune_workspace_bytes(N, K, T, o), dtype=torch.uint8, device=dev)
        vals = torch.empty(N, K // 2, dtype=torch.float16, device=dev)
        meta = torch.empty(N, K // 8, dtype=torch.uint8, device=dev)
        perm = torch.empty(K, dtype=torch.int32, device=dev)
        packed = torch.empty(b.esp_packed_bytes(N, K), dtype=torch.uint8, device=dev)
        stats = b.esp_prune_stats()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        b.esp_metric_prune(Wd, Xc, o, vals, meta, perm, packed, stats=stats, workspace=ws)
        e1.record()
        torch.cuda.synchronize()
        prune_ms += e0.elapsed_time(e1)
        prune_bytes += 2.0 * 2 * T * K + 2.0 * 2 * N * K + 1.125 * N * K * 2
        swaps += int(stats.lbs_swaps_total)
        layer.append(dict(name=name, N=N, K=K, W=Wd, perm=perm, packed=packed))
        del ws, vals, meta
    del xcal_cache
    torch.cuda.empty_cache()
    return layer, {"ms_layer": prune_ms, "lbs_max_swaps": lbs_max_swaps, "lbs_swaps_applied": swaps,
                   "stream_gbs_incl_shuffle": prune_bytes / (prune_ms * 1e-3) / 1e9}


def timing_weights(dev, N, K, copies):
    """Compressed weights for timing only: random kept values with legal metadata and a random channel order, made on the
    device (neither time nor traffic of the product depends on the values)."""
    import torch
    from paper_2310_15929_b200 import binding as b
    packs = []
    for _ in range(copies):
        vals = (torch.randn(N, K // 2, device=dev) * 0.02).half()
        meta = torch.full((N, K // 8), 0xE4, dtype=torch.uint8, device=dev)
        pk = torch.empty(b.esp_packed_bytes(N, K), dtype=torch.uint8, device=dev)
        b.esp_pack(vals, meta, N, K, pk)
        packs.append(pk)
        del vals, meta
    return packs, torch.randperm(K, device=dev).int()


def time_steps(fn, steps, warmup):
    import torch
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps       # ms per step


def graph_of(fn, reps=1, eager_runs=2):
    """fn() x reps recorded into one CUDA graph (after `eager_runs` plain runs for first-use set-up)."""
    import torch
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        for _ in range(eager_runs):
            fn()
        torch.cuda.synchronize()
        with torch.cuda.graph(g, stream=side):
            for _ in range(reps):
                fn()
    torch.cuda.synchronize()
    return g


def graph_time(fn, reps, rounds=5, warm=2):
    """Best time per fn() in ms over `rounds` replays of a CUDA graph of `reps` calls (CUDA events on the replaying stream)."""
    import torch
    g = graph_of(fn, reps)
    for _ in range(warm):
        g.replay()
    torch.cuda.synchronize()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    best = float("inf")
    for _ in range(rounds):
        g0.record(); g.replay(); g1.record(); torch.cuda.synchronize()
        best = min(best, g0.elapsed_time(g1) / reps)
    del g
    return best


def oracle_sample(wl, M, rows, feats):
    """The CPU oracle's fp64 product on `rows` token rows x `feats` feature rows of every linear of the workload, with the
    oracle's own selection under a seeded score and channel order (its shuffles are timed separately)."""
    from oracle import esparse_oracle as orc
    from paper_2310_15929_b200 import inputs
    g = np.random.default_rng(7)
    prepared = []
    for name, (N, K) in wl.linears.items():
        f = min(feats, N)
        W = inputs.make_weight(wl, name, No=f)
        s = 1.0 + g.random(K)
        theta = g.permutation(K).astype(np.int32)
        vals, meta, _ = orc.select_compress(W, s, theta)
        X = inputs.make_gemm_x(wl, name, rows)               # `rows` token rows drawn from the workload's activation distribution
        prepared.append((X, vals, meta, theta, f, K))

    def run():
        for X, vals, meta, theta, f, K in prepared:
            orc.product(X, vals, meta, theta)
    flops = sum(2.0 * rows * f * K for _, _, _, _, f, K in prepared)
    return run, flops, orc.oracle_threads()


def sample_text(wl, M, rows, feats):
    return (f"{rows} of {M} token rows x {feats} feature rows of each of the {len(wl.linears)} linears of {wl.name} "
            f"per step (fp64 numpy product of the decompressed weight)")


HEAD_METRIC = "2:4 sparse-GEMM dense-equivalent TFLOP/s (prefill, LLaMA-65B-shaped layer, M=8192)"


def head_config(wl, x_layout):
    return {"workload": f"{wl.name} (configs[3]): q,k,v,o 8192x8192, gate,up 22016x8192, down 8192x22016; prefill M={HEAD_M}",
            "M": HEAD_M, "x_layout": x_layout, "accumulate": "f32", "out": "f16", "static_weights": 1,
            "l2": "inputs larger than L2: 0.91 GB of distinct compressed weights + 0.9 GB of X + 1.2 GB of Y per step",
            "replicas": "one independent layer per GPU, no collective"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2310_15929_b200 import inputs
    wl = inputs.WORKLOADS[HEAD_WORKLOAD]
    rows, feats = args.cpu_rows, args.cpu_features
    run, flops, cores = oracle_sample(wl, HEAD_M, rows, feats)
    for _ in range(max(1, min(args.warmup, 2))):
        run()
    steps = max(1, args.steps)
    t0 = time.perf_counter()
    done = 0
    while done < steps and (done == 0 or time.perf_counter() - t0 < 120.0):      # bounded: a few minutes at most
        run()
        done += 1
    dt = (time.perf_counter() - t0) / done
    val = flops / dt / 1e12
    print(json.dumps({
        "impl": "reference", "metric": HEAD_METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus, "steps": done,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": dict(head_config(wl, args.x_layout), sample=sample_text(wl, HEAD_M, rows, feats),
                       note="a step of this arm is one pass of the CPU oracle over the bounded sample, not over the whole layer"),
        "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
                         "sample": sample_text(wl, HEAD_M, rows, feats)},
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def bound_of(M, N, K, ms, peaks):
    """Rate and roofline fraction of one product: HBM-bound up to 128 tokens, tensor-bound from 2048, both in between."""
    flops, nbytes = 2.0 * M * N * K, gemm_bytes(M, N, K)
    t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9) * 1e3
    t_tc = flops / (2.0 * peaks["bf16_burst"] * 1e12) * 1e3
    bound = "hbm" if M <= 128 else "tensor" if M >= 2048 else ("tensor" if t_tc > t_hbm else "hbm")
    return {"tflops": flops / ms / 1e9, "gbs": nbytes / ms / 1e6, "bound": bound,
            "frac": (t_hbm if bound == "hbm" else t_tc) / ms}


def per_config_sweep(dev, peaks, x_layout, only=None):
    """Every (workload, distinct linear shape, M) of the five workloads: esp_spgemm beside dense cuBLAS fp16 on the same shape.
    Timing-only weights; up to 256 tokens the launches rotate through more than L2 worth of weight copies."""
    import torch
    from paper_2310_15929_b200 import binding as b, inputs
    out = []
    for wl in inputs.WORKLOADS:
        if only is not None and wl.index not in only:
            continue
        for (N, K), lin in inputs.distinct_shapes(wl).items():
            small_ms = [M for M in wl.gemm_tokens if M <= 256]
            copies = max(2, int(400e6 // (1.125 * N * K)) + 1) if small_ms else 1
            packs, perm = timing_weights(dev, N, K, copies)
            Wd = [torch.randn(N, K, device=dev).half() for _ in range(min(copies, max(1, int(400e6 // (2.0 * N * K)) + 1)) if small_ms else 1)]
            for M in wl.gemm_tokens:
                o = b.esp_gemm_opts_default()
                o.x_layout = b.ESP_X_CHANNEL_MAJOR if x_layout == "channel" else b.ESP_X_TOKEN_MAJOR
                o.static_weights = 1
                ldm = (M + 7) // 8 * 8
                Xt = torch.randn(M, K, device=dev).half()
                if x_layout == "channel":
                    Xc = torch.zeros(K, ldm, dtype=torch.float16, device=dev)
                    Xc[:, :M] = Xt.t()
                    X = Xc[:, :M]
                else:
                    X = Xt
                Y = torch.empty(M, N, dtype=torch.float16, device=dev)
                nws = b.esp_spgemm_workspace_bytes(M, N, K, o)
                ws = torch.empty(nws, dtype=torch.uint8, device=dev) if nws else None
                rot = len(packs) if M <= 256 else 1
                drot = len(Wd) if M <= 256 else 1
                state = {"i": 0}

                def ours():
                    b.esp_spgemm(X, packs[state["i"] % rot], perm, Y, o, ws)
                    state["i"] += 1

                def dense():
                    torch.matmul(Xt, Wd[state["i"] % drot].t())
                    state["i"] += 1
                reps = 2 * rot if M <= 256 else (4 if M <= 2048 else 2)
                ms = graph_time(ours, reps, rounds=3)
                state["i"] = 0
                dms = graph_time(dense, 2 * drot if M <= 256 else reps, rounds=3)
                plan = b.esp_spgemm_plan(M, N, K, o, ws is not None)
                e = {"workload": wl.index, "linear": lin, "N": N, "K": K, "M": M, "ms": ms, "dense_cublas_ms": dms,
                     "speedup_vs_dense": dms / ms, "plan": [plan["kernel"], plan["token_tile"], plan["split_k"], plan["stages"]]}
                e.update(bound_of(M, N, K, ms, peaks))
                out.append(e)
                del X, Xt, Y, ws
            del packs, Wd
            torch.cuda.empty_cache()
    return out


def run_ours(args):
    import torch
    from paper_2310_15929_b200 import binding as b, inputs

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)

    peaks = measured_peaks()
    channel = args.x_layout == "channel"
    alpha_of_T = lambda T: 1.0 / math.sqrt(T)

    def make_x(wl, layer, M, keep_host=None):
        xs = []
        for lin in layer:
            H = torch.from_numpy(inputs.make_gemm_x(wl, lin["name"], M))
            X = H.to(dev)
            if channel:
                ldm = (M + 7) // 8 * 8
                Xc = torch.zeros(lin["K"], ldm, dtype=torch.float16, device=dev)
                Xc[:, :M] = X.t()
                X = Xc[:, :M]
            xs.append(X)
            if keep_host is not None:
                keep_host.append(H)
        return xs

    def make_ws(layer, M, opts, times=1):
        n = max(b.esp_spgemm_workspace_bytes(M, lin["N"], lin["K"], opts) for lin in layer)
        return torch.empty(max(16, times * n), dtype=torch.uint8, device=dev)

    def gemm_step(layer, xs, ys, opts, ws=None):
        for lin, X, Y in zip(layer, xs, ys):
            b.esp_spgemm(X, lin["packed"], lin["perm"], Y, opts, ws)

    def opts_for(static=1):
        o = b.esp_gemm_opts_default()
        o.x_layout = b.ESP_X_CHANNEL_MAJOR if channel else b.ESP_X_TOKEN_MAJOR
        o.static_weights = static             # inference: weights and permutations are never rewritten between launches
        return o

    # ================= headline: prefill on the LLaMA-65B-shaped layer =================
    wl = inputs.WORKLOADS[HEAD_WORKLOAD]
    layer, prune_info = build_layer(dev, wl, alpha_of_T, args.lbs_max_swaps)
    po = opts_for()
    host_x = []
    xs = make_x(wl, layer, HEAD_M, keep_host=host_x)
    ys = [torch.empty(HEAD_M, lin["N"], dtype=torch.float16, device=dev) for lin in layer]
    sampler = ClockSampler(local)
    sampler.start()                           # nvidia-smi needs a moment before its first sample
    pws = make_ws(layer, HEAD_M, po)
    eager_step = lambda: gemm_step(layer, xs, ys, po, pws)
    # One step = the layer's seven esp_spgemm calls (each a tiling pass over X + the GEMM), recorded once into a CUDA graph
    # and replayed: the launches then follow each other without host gaps.  --eager times the plain calls instead.
    plans = [b.esp_spgemm_plan(HEAD_M, lin["N"], lin["K"], po, True) for lin in layer]
    launches_per_step = sum(2 if p["kernel"] == b.ESP_KERNEL_PAIR_TILED else 1 for p in plans)
    if args.eager:
        step = eager_step
    else:
        step = graph_of(eager_step).replay
    for _ in range(args.warmup):
        step()
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_begin = time.time()
    e0.record()                               # on the current stream, the one every esp_spgemm call launches on
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    ms = e0.elapsed_time(e1) / args.steps
    # Keep the same load running (untimed) until at least 1.5 s of clock samples exist: nvidia-smi's period is 50 ms, so
    # the record covers the timed steps and these identical ones.
    extra_steps = 0
    while time.time() - t_begin < 1.5:
        step()
        extra_steps += 1
        if extra_steps % 8 == 0:
            torch.cuda.synchronize()
    torch.cuda.synchronize()
    clocks = sampler.stop(t_begin)
    clocks["covers"] = f"the {args.steps} timed steps and {extra_steps} further identical steps"
    if clocks.get("sm_mhz"):
        clocks["ms_per_step_x_sm_mhz"] = ms * clocks["sm_mhz"]
    ms = max_over_ranks(ms, dist, dev)
    if dist:
        dist.barrier()
    flops = sum(2.0 * HEAD_M * lin["N"] * lin["K"] for lin in layer)
    value = whole_job_rate(flops, world, ms) / 1e12
    assert b.esp_last_device_status() == b.ESP_OK

    # ---------------- end to end through the C ABI with host buffers ----------------
    hx = [(h.t().contiguous() if channel else h).pin_memory() for h in host_x]
    del host_x
    hy = [torch.empty(HEAD_M, lin["N"], dtype=torch.float16).pin_memory() for lin in layer]
    # Three streams: the upload of linear i + 1 and the download of linear i - 1 run beside the GEMM of linear i (PCIe is full
    # duplex).  A step starts after the one before it has finished on all three, and ends when its last download has.
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()

    def e2e_step():
        cur = torch.cuda.current_stream()
        start = torch.cuda.Event()
        start.record(cur)
        s_in.wait_event(start)
        s_out.wait_event(start)
        for lin, H, X, Y, HY in zip(layer, hx, xs, ys, hy):
            with torch.cuda.stream(s_in):
                X.copy_(H, non_blocking=True)
                up = torch.cuda.Event()
                up.record(s_in)
            cur.wait_event(up)
            b.esp_spgemm(X, lin["packed"], lin["perm"], Y, po, pws)
            done = torch.cuda.Event()
            done.record(cur)
            s_out.wait_event(done)
            with torch.cuda.stream(s_out):
                HY.copy_(Y, non_blocking=True)
        last = torch.cuda.Event()
        last.record(s_out)
        cur.wait_event(last)
    e2e_ms = time_steps(e2e_step, max(2, args.steps // 4), 2)
    e2e_ms = max_over_ranks(e2e_ms, dist, dev)
    e2e = {"value": whole_job_rate(flops, world, e2e_ms) / 1e12, "unit": "TFLOP/s",
           "h2d_bytes_per_step": int(sum(h.numel() * 2 for h in hx)),
           "d2h_bytes_per_step": int(sum(h.numel() * 2 for h in hy))}
    del hx, hy

    extra = {}
    if rank == 0:
        # ---------------- the same layer at M = 2048 and 4096, and dense cuBLAS fp16 on the same shapes ----------------
        def dense_step(xs_tok):
            for lin, X in zip(layer, xs_tok):
                torch.matmul(X, lin["W"].t())
        xs_tok = [x.t().contiguous() for x in xs] if channel else xs
        dense_ms = time_steps(lambda: dense_step(xs_tok), max(3, args.steps // 2), 3)
        del xs_tok
        extra["dense_cublas_f16"] = {"prefill_ms_per_step": dense_ms, "prefill_tflops": flops / (dense_ms * 1e-3) / 1e12,
                                     "speedup_prefill": dense_ms / ms}
        other = {}
        for M2 in (2048, 4096):
            xs2 = make_x(wl, layer, M2)
            ys2 = [torch.empty(M2, lin["N"], dtype=torch.float16, device=dev) for lin in layer]
            ms2 = graph_time(lambda: gemm_step(layer, xs2, ys2, po, pws), 2, rounds=3)
            f2 = sum(2.0 * M2 * lin["N"] * lin["K"] for lin in layer)
            other[f"M={M2}"] = {"ms_per_step": ms2, "tflops": f2 / (ms2 * 1e-3) / 1e12,
                                "frac": f2 / (ms2 * 1e-3) / 1e12 / (2.0 * peaks["bf16_burst"])}
            del xs2, ys2
        extra["prefill_other_token_counts"] = other
        extra["prune"] = prune_info
    del xs, ys, pws, layer
    torch.cuda.empty_cache()

    if rank == 0 and not (args.quick or world > 1):          # (with several ranks the others would wait minutes at the barrier)
        # ================= decode: the OPT-66B-shaped layer at M = 1 and 32, HBM-bound =================
        dwl = inputs.WORKLOADS[DECODE_WORKLOAD]
        dlayer, dprune = build_layer(dev, dwl, alpha_of_T, args.lbs_max_swaps)
        do = opts_for()
        dec = {"workload": f"{dwl.name} (configs[4]): q,k,v,o 9216x9216, fc1 36864x9216, fc2 9216x36864",
               "launch": "one CUDA graph of 10 layer passes (6 launches each), static_weights=1; 1.15 GB of distinct compressed "
                         "weights per pass: larger than L2", "prune": dprune}
        for M in DECODE_MS:
            dx = make_x(dwl, dlayer, M)
            dy = [torch.empty(M, lin["N"], dtype=torch.float16, device=dev) for lin in dlayer]
            dws = make_ws(dlayer, M, do)
            dms = graph_time(lambda: gemm_step(dlayer, dx, dy, do, dws), 10)
            dbytes = sum(gemm_bytes(M, lin["N"], lin["K"]) for lin in dlayer)
            dgbs = dbytes / (dms * 1e-3) / 1e9
            dxt = [x.t().contiguous() for x in dx] if channel else dx
            dense_dec_ms = graph_time(lambda: [torch.matmul(X, lin["W"].t()) for lin, X in zip(dlayer, dxt)], 10)
            # q,k,v share their input: one launch for the three (their weights and permutations stay apart)
            names = [lin["name"] for lin in dlayer]
            groups = [[names.index(n) for n in ("q", "k", "v")], [names.index("o")], [names.index("fc1")], [names.index("fc2")]]
            gws = make_ws(dlayer, M, do, times=3)

            def grouped_step():
                for idx in groups:
                    b.esp_spgemm_grouped([dx[idx[0]]] * len(idx), [dlayer[i]["packed"] for i in idx],
                                         [dlayer[i]["perm"] for i in idx], [dy[i] for i in idx], do, gws)
            gms = graph_time(grouped_step, 10)
            dec[f"M={M}"] = {"ms_per_step": dms, "value": dgbs, "unit": "GB/s",
                             "roofline": {"bound": "hbm", "achieved": dgbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                          "frac": dgbs / peaks["hbm_gbs"], "traffic": DECODE_TRAFFIC_BYTES if M == 1 else None,
                                          "frac_of_nominal_8TBs": dgbs / 8000.0, "of": peaks["source"]},
                             "dense_cublas_ms_per_step": dense_dec_ms, "speedup_vs_dense": dense_dec_ms / dms,
                             "grouped_qkv": {"launches_per_layer": 4, "ms_per_step": gms, "value": dbytes / (gms * 1e-3) / 1e9,
                                             "frac": dbytes / (gms * 1e-3) / 1e9 / peaks["hbm_gbs"]}}
            del dx, dy, dws, dxt, gws
        extra["decode"] = dec
        # ---------------- compressed against dense footprint of this layer (the paper's Table 6 quantity) ----------------
        dense_b = sum(2 * lin["N"] * lin["K"] for lin in dlayer)
        comp_b = sum(lin["N"] * lin["K"] + lin["N"] * lin["K"] // 8 for lin in dlayer)
        packed_b = sum(b.esp_packed_bytes(lin["N"], lin["K"]) for lin in dlayer)
        perm_b = sum(4 * lin["K"] for lin in dlayer)
        extra["footprint"] = {"workload": dwl.name, "dense_fp16_bytes": dense_b, "values_plus_metadata_bytes": comp_b,
                              "packed_bytes_as_stored": packed_b, "permutation_bytes": perm_b,
                              "saving_pct": 100.0 * (1.0 - (packed_b + perm_b) / dense_b),
                              "per_linear": {lin["name"]: {"dense": 2 * lin["N"] * lin["K"],
                                                           "packed": b.esp_packed_bytes(lin["N"], lin["K"])} for lin in dlayer},
                              "paper_table6_saving_pct_whole_models": [42.64, 43.01, 43.38, 43.52]}
        del dlayer
        torch.cuda.empty_cache()

        # ================= the LLaMA-7B-shaped layer as earlier runs of this benchmark timed it =================
        swl = inputs.WORKLOADS[SMALL_WORKLOAD]
        slayer, sprune = build_layer(dev, swl, alpha_of_T, args.lbs_max_swaps)
        so = opts_for()
        sx = make_x(swl, slayer, PREFILL_M)
        sy = [torch.empty(PREFILL_M, lin["N"], dtype=torch.float16, device=dev) for lin in slayer]
        sws = make_ws(slayer, PREFILL_M, so)
        sms = graph_time(lambda: gemm_step(slayer, sx, sy, so, sws), 4)
        sflops = sum(2.0 * PREFILL_M * lin["N"] * lin["K"] for lin in slayer)
        sxt = [x.t().contiguous() for x in sx] if channel else sx
        sdense = graph_time(lambda: [torch.matmul(X, lin["W"].t()) for lin, X in zip(slayer, sxt)], 4)
        del sx, sy, sws, sxt
        dx = make_x(swl, slayer, DECODE_M)
        dy = [torch.empty(DECODE_M, lin["N"], dtype=torch.float16, device=dev) for lin in slayer]
        dws = make_ws(slayer, DECODE_M, so)
        dms = graph_time(lambda: gemm_step(slayer, dx, dy, so, dws), 20)
        plain = opts_for(static=0)
        dms_plain = graph_time(lambda: gemm_step(slayer, dx, dy, plain, dws), 20)
        dms_eager = time_steps(lambda: gemm_step(slayer, dx, dy, so, dws), 40, 5)
        dbytes = sum(gemm_bytes(DECODE_M, lin["N"], lin["K"]) for lin in slayer)
        names = [lin["name"] for lin in slayer]
        groups = [[names.index(n) for n in ("q", "k", "v")], [names.index("o")], [names.index(n) for n in ("gate", "up")],
                  [names.index("down")]]
        gws = make_ws(slayer, DECODE_M, so, times=3)

        def grouped7b():
            for idx in groups:
                b.esp_spgemm_grouped([dx[idx[0]]] * len(idx), [slayer[i]["packed"] for i in idx], [slayer[i]["perm"] for i in idx],
                                     [dy[i] for i in idx], so, gws)
        gms = graph_time(grouped7b, 20)
        dxt = [x.t().contiguous() for x in dx] if channel else dx
        ddense = graph_time(lambda: [torch.matmul(X, lin["W"].t()) for lin, X in zip(slayer, dxt)], 20)
        extra["llama7b"] = {
            "workload": f"{swl.name} (configs[1])", "prune": sprune,
            "prefill": {"M": PREFILL_M, "ms_per_step": sms, "tflops": sflops / (sms * 1e-3) / 1e12,
                        "frac": sflops / (sms * 1e-3) / 1e12 / (2.0 * peaks["bf16_burst"]), "speedup_vs_dense": sdense / sms},
            "decode": {"M": DECODE_M, "ms_per_step": dms, "gbs": dbytes / (dms * 1e-3) / 1e9,
                       "frac": dbytes / (dms * 1e-3) / 1e9 / peaks["hbm_gbs"], "speedup_vs_dense": ddense / dms,
                       "plain_stream_order_in_graph_gbs": dbytes / (dms_plain * 1e-3) / 1e9,
                       "plain_calls_no_graph_gbs": dbytes / (dms_eager * 1e-3) / 1e9,
                       "grouped_4_launches_gbs": dbytes / (gms * 1e-3) / 1e9,
                       "grouped_4_launches_frac": dbytes / (gms * 1e-3) / 1e9 / peaks["hbm_gbs"]}}
        del slayer, dx, dy, dws, gws, dxt
        torch.cuda.empty_cache()

        # ================= every (workload, linear shape, M) =================
        extra["per_config"] = per_config_sweep(dev, peaks, args.x_layout)

        # ================= the producer beside the CPU oracle's producer =================
        extra["prune"]["cpu_oracle"] = producer_against_oracle(dev)

    if rank == 0:
        # ---------------- CPU oracle's product on a bounded sample of the headline workload ----------------
        rows, feats = args.cpu_rows, args.cpu_features
        run, oflops, cores = oracle_sample(wl, HEAD_M, rows, feats)
        t0 = time.perf_counter()
        passes = 0
        while passes == 0 or (time.perf_counter() - t0 < 10.0 and passes < 20):
            run()
            passes += 1
        odt = (time.perf_counter() - t0) / passes
        extra["cpu_baseline"] = {"value": oflops / odt / 1e12, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
                                 "sample": sample_text(wl, HEAD_M, rows, feats) + f"; {passes} passes of {odt:.2f} s"}
        # 2:4 sparse fp16 peak = 2 x the dense 16-bit peak (nominal ratio)
        sparse_peak = 2.0 * peaks["bf16_burst"]
        achieved = flops / (ms * 1e-3) / 1e12
        line = {
            "metric": HEAD_METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f16", "data": "synthetic", "config": head_config(wl, args.x_layout),
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
            "kernel": f"tiling pass + spgemm_pair_kernel per linear (plans {[[p['kernel'], p['token_tile']] for p in plans]}): "
                      f"{launches_per_step} launches per step, " + ("plain calls" if args.eager else "replayed from one CUDA graph per step"),
            "roofline": {"bound": "tensor", "achieved": achieved, "peak": sparse_peak, "unit": "TFLOP/s",
                         "frac": achieved / sparse_peak, "traffic": PREFILL_TRAFFIC_BYTES,
                         "note": f"dense-equivalent flops of a step (seven linears) / its CUDA-event time, tiling passes included; "
                                 f"peak = 2 x {peaks['source']} burst dense bf16 ({peaks['bf16_burst']}); against 2 x the sustained "
                                 f"figure ({peaks['bf16_sustained']}): {achieved / (2.0 * peaks['bf16_sustained']):.3f}; of nominal "
                                 f"4500: {achieved / 4500.0:.3f}"},
        }
        line.update(extra)
        print(json.dumps(line))
    if dist:
        dist.barrier()
        dist.destroy_process_group()


def producer_against_oracle(dev):
    """esp_metric_prune and the CPU oracle's whole producer on the same bounded inputs: workload 0 whole, and a slice of
    workload 1's q projection (1024 output rows, all 4096 input channels, 4096 calibration tokens, block shuffle capped at 2
    swaps per block on both sides)."""
    import torch
    from oracle import esparse_oracle as orc
    from paper_2310_15929_b200 import binding as b, inputs
    out = {}
    cases = [("workload0_whole", inputs.WORKLOADS[0], "fc", None, None, 0),
             ("workload1_q_slice_1024x4096_T4096_2swaps", inputs.WORKLOADS[1], "q", 1024, 4096, 2)]
    for label, wl, lin, No, T, cap in cases:
        W = inputs.make_weight(wl, lin, No=No)
        Xc = inputs.make_calibration(wl, lin, T=T)
        alpha = 1.0 / math.sqrt(Xc.shape[0])
        t0 = time.perf_counter()
        orc.metric_prune(W, Xc, alpha, lbs_max_swaps=cap, objectives=False)
        cpu_s = time.perf_counter() - t0
        o = b.esp_prune_opts_default()
        o.alpha, o.lbs_max_swaps = alpha, cap
        n, c = W.shape
        Wd, Xd = torch.from_numpy(W).to(dev), torch.from_numpy(Xc).to(dev)
        ws = torch.empty(b.esp_metric_prune_workspace_bytes(n, c, Xc.shape[0], o), dtype=torch.uint8, device=dev)
        vals = torch.empty(n, c // 2, dtype=torch.float16, device=dev)
        meta = torch.empty(n, c // 8, dtype=torch.uint8, device=dev)
        perm = torch.empty(c, dtype=torch.int32, device=dev)
        packed = torch.empty(b.esp_packed_bytes(n, c), dtype=torch.uint8, device=dev)
        gpu_ms = time_steps(lambda: b.esp_metric_prune(Wd, Xd, o, vals, meta, perm, packed, workspace=ws), 3, 1)
        out[label] = {"cpu_oracle_s": cpu_s, "gpu_ms": gpu_ms, "cores": orc.oracle_threads()}
    return out


def run_profile_case(args):
    """A few launches of one kernel on one LLaMA-7B-shaped linear, sized for an ncu capture (tens of MB on
    the device).  Weights are random kept values with legal metadata: traffic and timing do not depend on
    the values.  Prints the CUDA-event time of the launches it made."""
    import torch
    from paper_2310_15929_b200 import binding as b
    dev = torch.device("cuda", 0)
    torch.manual_seed(1)
    case = args.profile_case
    N, K = (4096, 4096)
    if case == "prune":
        # the producer on a slice of the LLaMA-7B-shaped q projection: all 4096 input channels and all 32768 calibration
        # tokens (268 MB of activations: larger than L2), 1024 output rows, one block-shuffle swap per block
        from paper_2310_15929_b200 import inputs
        wl = inputs.WORKLOADS[WORKLOAD]
        T = wl.calib_tokens
        W = torch.from_numpy(inputs.make_weight(wl, "q", No=1024)).to(dev)
        Xc = torch.from_numpy(inputs.make_calibration(wl, "q", T=T)).to(dev)
        o = b.esp_prune_opts_default(); o.alpha = 1.0 / math.sqrt(T); o.lbs_max_swaps = 1
        ws = torch.empty(b.esp_metric_prune_workspace_bytes(1024, K, T, o), dtype=torch.uint8, device=dev)
        vals = torch.empty(1024, K // 2, dtype=torch.float16, device=dev)
        meta = torch.empty(1024, K // 8, dtype=torch.uint8, device=dev)
        perm = torch.empty(K, dtype=torch.int32, device=dev)
        packed = torch.empty(b.esp_packed_bytes(1024, K), dtype=torch.uint8, device=dev)
        fn = lambda: b.esp_metric_prune(W, Xc, o, vals, meta, perm, packed, workspace=ws)
        ms = time_steps(fn, 2, 1)
        print(json.dumps({"case": case, "No": 1024, "C": K, "T": T, "ms": ms, "xcal_bytes": 2 * T * K}))
        return
    M = PREFILL_M if case == "prefill" else 128 if case == "mid" else DECODE_M
    if args.profile_shape:
        M, N, K = (int(v) for v in args.profile_shape.lower().split("x"))
    vals = (torch.randn(N, K // 2, device=dev) * 0.02).half()
    meta = torch.full((N, K // 8), 0xE4, dtype=torch.uint8, device=dev)
    packed = torch.empty(b.esp_packed_bytes(N, K), dtype=torch.uint8, device=dev)
    b.esp_pack(vals, meta, N, K, packed)
    perm = torch.randperm(K, device=dev).int()
    Xc = torch.zeros(K, (M + 7) // 8 * 8, dtype=torch.float16, device=dev)      # leading dimension: a multiple of 8 elements
    Xc[:, :M] = torch.randn(K, M, device=dev).half()
    X = Xc[:, :M]
    Y = torch.empty(M, N, dtype=torch.float16, device=dev)
    o = b.esp_gemm_opts_default(); o.x_layout = b.ESP_X_CHANNEL_MAJOR
    nws = b.esp_spgemm_workspace_bytes(M, N, K, o)
    ws = torch.empty(nws, dtype=torch.uint8, device=dev) if nws else None
    ms = time_steps(lambda: b.esp_spgemm(X, packed, perm, Y, o, ws), 3, 3)
    print(json.dumps({"case": case, "M": M, "N": N, "K": K, "plan": b.esp_spgemm_plan(M, N, K, o, ws is not None),
                      "ms_per_call": ms,
                      "tflops": 2.0 * M * N * K / ms / 1e9, "gbs": gemm_bytes(M, N, K) / ms / 1e6}))


# The GEMM shapes of the paper's Table 5 (context stage: 16384 tokens, decoder stage: 16 tokens); weight given as N x K.
TABLE5 = [("context Q/K/V", 16384, 5376, 14336, 8.452, 5.815), ("context Att_Out", 16384, 14336, 1792, 3.488, 2.540),
          ("context FFN-1", 16384, 7168, 14336, 11.487, 8.073), ("context FFN-2", 16384, 14336, 7168, 11.478, 8.958),
          ("decoder Q/K/V", 16, 5376, 14336, 0.122, 0.098), ("decoder Att_Out", 16, 14336, 1792, 0.046, 0.030),
          ("decoder FFN-1", 16, 7168, 14336, 0.160, 0.112), ("decoder FFN-2", 16, 14336, 7168, 0.158, 0.109)]


def run_table5(args):
    """Times esp_spgemm and dense cuBLAS fp16 on the paper's Table 5 shapes (random kept values with legal metadata and a
    random permutation: timing does not depend on the values).  One JSON line per shape; the paper's A100 times are
    printed beside ours as context."""
    import torch
    from paper_2310_15929_b200 import binding as b
    dev = torch.device("cuda", 0)
    torch.manual_seed(5)
    for name, M, N, K, paper_dense_ms, paper_sparse_ms in TABLE5:
        ncopies = 1 if M > 256 else max(2, int(300e6 // (1.125 * N * K)) + 1)      # decode: rotate weights through > L2
        packs = []
        for _ in range(ncopies):
            vals = (torch.randn(N, K // 2, device=dev) * 0.02).half()
            meta = torch.full((N, K // 8), 0xE4, dtype=torch.uint8, device=dev)
            pk = torch.empty(b.esp_packed_bytes(N, K), dtype=torch.uint8, device=dev)
            b.esp_pack(vals, meta, N, K, pk)
            packs.append(pk)
        del vals, meta
        perm = torch.randperm(K, device=dev).int()
        X = torch.randn(K, M, device=dev).half()
        Y = torch.empty(M, N, dtype=torch.float16, device=dev)
        o = b.esp_gemm_opts_default()
        o.x_layout = b.ESP_X_CHANNEL_MAJOR
        o.static_weights = 1
        nws = b.esp_spgemm_workspace_bytes(M, N, K, o)
        ws = torch.empty(nws, dtype=torch.uint8, device=dev) if nws else None
        Wd = [torch.randn(N, K, device=dev).half() for _ in range(ncopies)]
        Xt = X.t().contiguous()
        reps = 4 if M > 256 else 2 * ncopies

        def timed(fn):
            side = torch.cuda.Stream()
            g = torch.cuda.CUDAGraph()
            torch.cuda.synchronize()
            with torch.cuda.stream(side):
                for i in range(2):
                    fn(i)
                torch.cuda.synchronize()
                with torch.cuda.graph(g, stream=side):
                    for i in range(reps):
                        fn(i)
            torch.cuda.synchronize()
            g.replay()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            best = float("inf")
            for _ in range(3):
                e0.record(); g.replay(); e1.record(); torch.cuda.synchronize()
                best = min(best, e0.elapsed_time(e1) / reps)
            return best
        ms = timed(lambda i: b.esp_spgemm(X, packs[i % ncopies], perm, Y, o, ws))
        dms = timed(lambda i: torch.matmul(Xt, Wd[i % ncopies].t()))
        assert b.esp_last_device_status() == b.ESP_OK
        print(json.dumps({"table5": name, "M": M, "N": N, "K": K, "sparse_ms": ms, "dense_cublas_ms": dms,
                          "speedup_vs_dense": dms / ms, "tflops_dense_equivalent": 2.0 * M * N * K / ms / 1e9,
                          "gbs": gemm_bytes(M, N, K) / ms / 1e6, "plan": b.esp_spgemm_plan(M, N, K, o, ws is not None),
                          "paper_a100_dense_ms": paper_dense_ms, "paper_a100_sparse_ms": paper_sparse_ms,
                          "paper_speedup": paper_dense_ms / paper_sparse_ms}), flush=True)
        del packs, Wd, X, Y, Xt, ws


def spawn_replicas(args):
    """--gpus N without a launcher: start the N ranks here (one process per GPU, rendezvous on 127.0.0.1)."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--x-layout", default="channel", choices=["token", "channel"],
                    help="activation layout handed to esp_spgemm: channel = [K, M] (channels are rows)")
    ap.add_argument("--lbs-max-swaps", type=int, default=0,
                    help="cap on block-shuffle swaps per block while preparing the weights (0 = run to the end)")
    ap.add_argument("--cpu-rows", type=int, default=CPU_ROWS)
    ap.add_argument("--cpu-features", type=int, default=CPU_FEATURES)
    ap.add_argument("--eager", action="store_true", help="time plain esp_spgemm calls instead of a CUDA graph of the step")
    ap.add_argument("--quick", action="store_true", help="headline only: skip the decode, LLaMA-7B, per-config and producer sections")
    ap.add_argument("--profile-case", default=None, choices=["prefill", "decode", "mid", "prune"],
                    help="run a few launches of one small case (for ncu) instead of the benchmark")
    ap.add_argument("--profile-shape", default=None, metavar="MxNxK", help="sizes of the prefill / decode / mid profile case")
    ap.add_argument("--table5", action="store_true", help="time the GEMM shapes of the paper's Table 5 instead of the benchmark")
    ap.add_argument("--per-config", default=None, metavar="W[,W...]",
                    help="only the per-config sweep of these workloads (0..4), one JSON line per entry")
    args = ap.parse_args()
    if args.table5:
        run_table5(args)
        return
    if args.per_config is not None:
        import torch
        dev = torch.device("cuda", 0)
        for e in per_config_sweep(dev, measured_peaks(), args.x_layout, only=[int(w) for w in args.per_config.split(",")]):
            print(json.dumps(e), flush=True)
        return
    if args.profile_case:
        run_profile_case(args)
        return
    world = os.environ.get("WORLD_SIZE")
    if world is None and args.gpus > 1:
        sys.exit(spawn_replicas(args))                   # both arms: the reference arm's other ranks exit at once
    if world is not None and int(world) != args.gpus:
        sys.exit(f"bench.py: --gpus {args.gpus} but the launcher started {world} ranks")
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
