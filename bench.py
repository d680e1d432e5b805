#!/usr/bin/env python
"""Benchmark of the FusedDQP hot path on B200.

A step is one Gemma3-4B decoder layer at M = 1: the seven Q4NX projections q, k, v, o, gate, up, down
(59.1 MB of packed weights) on seeded synthetic inputs.  Projections that share their input are launched
together -- q|k|v and gate|up are concatenated along N, which in the strip-major Q4NX container is plain
concatenation of the packed bytes -- so a step is four fdqp_run calls (--fuse 0 runs the seven one by one).
Several distinct copies of the layer's weights are resident in HBM and the steps rotate through them, so every
timed step streams its weights from HBM and not from L2.  The metric is the achieved bandwidth over the algorithmic bytes of the step
(0.625*K*N + 2*M*K + 4*M*N per projection); decode tokens/s (projections only: 34 layers + LM head) is
reported beside it.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.  With --impl reference the CPU oracle is timed instead, on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import synthgen  # noqa: E402

METRIC = "fused Q4NX dequant-GEMV achieved HBM GB/s & % of peak; decode tokens/s (1 GPU)"
WORKLOAD = "Gemma3-4B decoder layer at M=1: q,k,v,o,gate,up,down Q4NX group-32 projections (seeds 1-7)"
L2_BYTES = 126e6
LAYER_COPIES = 8            # distinct weight sets resident in HBM (8 x 59 MB = 472 MB >> L2)
NOMINAL_HBM_GBS = 8000.0


def alg_bytes(M, K, N):
    return 0.625 * K * N + 2 * M * K + 4 * M * N


def layer_bytes(M=1):
    return sum(alg_bytes(M, K, N) for _, K, N, _ in synthgen.GEMMA3_4B_LAYER)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons in the background during the timed region."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) >= 7:
                self.rows.append(parts)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                smax.append(float(r[1]))
                power.append(float(r[2]))
            except ValueError:
                continue
            for name, val in zip(names, r[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------------------------- rank plumbing

def max_over_ranks(value, dist, device):
    """The slowest rank's figure: a whole-job time is the maximum over ranks (replicas do not talk otherwise)."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gbs(bytes_per_step, steps, world, ms):
    """Aggregate over all replicas: every rank moved bytes_per_step * steps in the (max-over-ranks) time ms."""
    return bytes_per_step * steps * world / (ms * 1e-3) / 1e9


# ----------------------------------------------------------------------------------------------- reference arm

def run_reference(args, rank, world):
    """Times the CPU oracle (as it stands) on the host cores: each step is one pass of the decoder layer's
    seven projections at M = 1 over the same seeded inputs, all output columns, OpenMP over columns."""
    if rank != 0:
        return
    import oracle
    cores = min(oracle.max_threads(), os.cpu_count() or 1)
    layer = [(name, K, N, synthgen.weights(seed, K, N), synthgen.activations(seed, 1, K))
             for name, K, N, seed in synthgen.GEMMA3_4B_LAYER]

    def one_pass():
        for _, K, N, w, x in layer:
            oracle.project(x, w.codes, w.scales, w.offsets, nthreads=cores)

    for _ in range(args.warmup):
        one_pass()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        one_pass()
    dt = time.perf_counter() - t0
    gbs = layer_bytes() * args.steps / dt / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "note": "CPU oracle (fp64, plain C, OpenMP over output columns)"},
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": cores, "kind": "oracle",
                         "sample": "whole layer, all 7 projections, all outputs, per step"},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------- one shape

def run_shape(args):
    """Times ONE projection shape (--shape K,N,M): the per-kernel view used for the roofline tables in profiles/.
    Weights are a seeded 4096-column matrix tiled along N (strip-major makes that byte concatenation); enough distinct
    copies are rotated to keep every launch's weights out of L2."""
    import torch

    import paper_2602_06063_b200 as fd

    K, N, M = (int(v) for v in args.shape.split(","))
    torch.cuda.set_device(0)
    peaks, peak_kind = measured_peaks()
    ctx = fd.fdqp_create(0, max(M, 8), K, N)
    for kv in args.param or []:
        key, val = kv.split("=")
        fd.fdqp_set_param(ctx, key, int(val))
    nb = min(N, 4096)
    fmt = {"q4nx": fd.FMT_Q4NX, "g64": fd.FMT_G64, "g128": fd.FMT_G128, "mxfp4": fd.FMT_MXFP4}[args.format]
    if fmt == fd.FMT_Q4NX:
        w = synthgen.weights(5, K, nb)
        tile = fd.q4nx_pack(w.codes, w.scales, w.offsets)
    else:
        w = synthgen.weights_fmt(5, K, nb, fmt)
        tile = fd.q4nx_pack_fmt(fmt, w.codes, w.scales, w.offsets)
    packed_bytes = fd.q4nx_packed_bytes_fmt(fmt, K, N)
    packed = np.tile(tile, -(-N // nb))[:packed_bytes]
    base = torch.from_numpy(np.ascontiguousarray(packed)).cuda()
    ncopies = max(1, int(np.ceil(4 * L2_BYTES / base.numel()))) if not (args.same_weights or args.l2_resident) else 1
    copies = [base] + [base.clone() for _ in range(ncopies - 1)]
    x = torch.from_numpy(synthgen.activations(1, M, K).view(np.int16)).cuda()
    epi = {"none": fd.EPI_NONE, "bf16": fd.EPI_BF16, "geglu": fd.EPI_GEGLU_BF16}[args.epilogue]
    if epi == fd.EPI_NONE:
        y = torch.empty((M, N), dtype=torch.float32, device="cuda")
    else:
        y = torch.empty((M, N // 2 if epi == fd.EPI_GEGLU_BF16 else N), dtype=torch.bfloat16, device="cuda")
    stream = torch.cuda.Stream()
    sraw = stream.cuda_stream

    gamma = torch.zeros(K, dtype=torch.int16, device="cuda")
    resid = torch.from_numpy(synthgen.activations(2, M, K).view(np.int16)).cuda()
    h_out = torch.empty((M, K), dtype=torch.int16, device="cuda")

    def launch(W):
        if fmt != fd.FMT_Q4NX:
            fd.fdqp_run_fmt(ctx, fmt, x, W, y, M, K, N, sraw)
        elif args.rmsnorm and args.residual:
            fd.fdqp_run_add_rmsnorm_epilogue(ctx, x, resid, h_out, gamma, 1e-6, W, y, epi, M, K, N, sraw)
        elif args.rmsnorm:
            fd.fdqp_run_rmsnorm_epilogue(ctx, x, gamma, 1e-6, W, y, epi, M, K, N, sraw)
        else:
            fd.fdqp_run_epilogue(ctx, x, W, y, epi, M, K, N, sraw)

    for i in range(max(3, args.warmup)):
        launch(copies[i % ncopies])
    stream.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if args.graph and not args.same_weights:
        # the timed launches replayed from one CUDA graph, so that the host's launch cost is not what is measured
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for i in range(args.steps):
                launch(copies[i % ncopies])
        with torch.cuda.stream(stream):
            g.replay()
        stream.synchronize()
        e0.record(stream)
        with torch.cuda.stream(stream):
            g.replay()
        e1.record(stream)
    else:
        e0.record(stream)
        for i in range(args.steps):
            launch(copies[i % ncopies])
        e1.record(stream)
    stream.synchronize()
    assert fd.fdqp_last_status(ctx) == 0
    us = e0.elapsed_time(e1) * 1e3 / args.steps
    gbs = (alg_bytes(M, K, N) - 0.625 * K * N + packed_bytes) / us / 1e3  # the format's own bytes per weight
    print(json.dumps({"shape": {"K": K, "N": N, "M": M}, "format": args.format, "us_per_call": us, "GBps": gbs,
                      "frac_of_measured_peak": gbs / peaks["hbm_gbs"], "frac_of_nominal_8TBps": gbs / NOMINAL_HBM_GBS,
                      "peak_kind": peak_kind, "weight_copies": ncopies, "steps": args.steps,
                      "graph": bool(args.graph and not args.same_weights), "epilogue": args.epilogue, "rmsnorm": bool(args.rmsnorm),
                      "launch": fd.fdqp_describe(ctx, M, K, N)}), flush=True)
    fd.fdqp_destroy(ctx)


# ----------------------------------------------------------------------------------------------- decode attention

def run_dequant(args):
    """Times the dequantisation engine (--dequant K,N,bf16|fp32): Q4NX -> dense matrix in HBM.  Algorithmic bytes per
    weight: 0.625 read + 2 (bf16) or 4 (fp32) written."""
    import torch

    import paper_2602_06063_b200 as fd

    parts = args.dequant.split(",")
    K, N, bf16 = int(parts[0]), int(parts[1]), parts[2] == "bf16"
    torch.cuda.set_device(0)
    peaks, peak_kind = measured_peaks()
    ctx = fd.fdqp_create(0, 8, K, N)
    fmt = {"q4nx": fd.FMT_Q4NX, "g64": fd.FMT_G64, "g128": fd.FMT_G128, "mxfp4": fd.FMT_MXFP4}[args.format]
    nb = min(N, 4096)
    w = synthgen.weights_fmt(5, K, nb, fmt) if fmt != fd.FMT_Q4NX else synthgen.weights(5, K, nb)
    tile = fd.q4nx_pack_fmt(fmt, w.codes, w.scales, w.offsets)
    nbytes = fd.q4nx_packed_bytes_fmt(fmt, K, N)
    W = torch.from_numpy(np.tile(tile, -(-N // nb))[:nbytes].copy()).cuda()
    out = torch.empty((K, N), dtype=torch.bfloat16 if bf16 else torch.float32, device="cuda")
    stream = torch.cuda.Stream()
    sraw = stream.cuda_stream
    for _ in range(3):
        fd.fdqp_dequant_fmt(ctx, fmt, W, out, bf16, K, N, sraw)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        fd.fdqp_dequant_fmt(ctx, fmt, W, out, bf16, K, N, sraw)
    e1.record(stream)
    stream.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / args.steps
    alg = nbytes + float(K) * N * (2 if bf16 else 4)
    gbs = alg / us / 1e3
    print(json.dumps({"dequant": {"K": K, "N": N, "out": parts[2], "format": args.format}, "us_per_call": us, "GBps": gbs,
                      "frac_of_measured_peak": gbs / peaks["hbm_gbs"], "peak_kind": peak_kind, "steps": args.steps}), flush=True)
    fd.fdqp_destroy(ctx)


def run_flowkv(args):
    """Times the decode attention (--flowkv H,G,d,L,window): one new token against a cache of L positions.  Enough
    distinct caches are rotated to keep every launch's keys and values out of L2.  Algorithmic bytes per call: the
    attended positions of K and V, 2 * G * n * d * 2 (q and out are negligible)."""
    import torch

    import paper_2602_06063_b200 as fd

    H, G, d, L, window = (int(v) for v in args.flowkv.split(","))
    torch.cuda.set_device(0)
    peaks, peak_kind = measured_peaks()
    ctx = fd.fdqp_create(0, 8, 256, 256)
    n = window if 0 < window < L else L
    cache_bytes = 2 * G * L * d * 2
    ncopies = max(1, int(np.ceil(4 * L2_BYTES / cache_bytes)))
    gen = torch.Generator(device="cuda").manual_seed(1)
    caches = [(torch.randn((G, L, d), device="cuda", generator=gen).to(torch.bfloat16),
               torch.randn((G, L, d), device="cuda", generator=gen).to(torch.bfloat16)) for _ in range(ncopies)]
    q = torch.randn((H, d), device="cuda", generator=gen).to(torch.bfloat16)
    out = torch.empty((H, d), dtype=torch.float32, device="cuda")
    stream = torch.cuda.Stream()
    sraw = stream.cuda_stream
    scale = d ** -0.5

    def launch(i):
        Kc, Vc = caches[i % ncopies]
        fd.fdqp_flowkv_decode(ctx, q, Kc, Vc, out, H, G, d, L, L, window, scale, sraw)

    for i in range(3):
        launch(i)
    stream.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        for i in range(args.steps):
            launch(i)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        g.replay()
        e0.record(stream)
        g.replay()
        e1.record(stream)
    stream.synchronize()
    assert fd.fdqp_last_status(ctx) == 0
    us = e0.elapsed_time(e1) * 1e3 / args.steps
    alg = 2.0 * G * n * d * 2
    gbs = alg / us / 1e3
    print(json.dumps({"flowkv": {"H": H, "G": G, "d": d, "L": L, "window": window}, "us_per_call": us, "GBps": gbs,
                      "attended_bytes": alg, "frac_of_measured_peak": gbs / peaks["hbm_gbs"],
                      "frac_of_nominal_8TBps": gbs / NOMINAL_HBM_GBS, "peak_kind": peak_kind, "cache_copies": ncopies,
                      "steps": args.steps}), flush=True)
    fd.fdqp_destroy(ctx)


# ----------------------------------------------------------------------------------------------- our arm

def run_ours(args, rank, local_rank, world):
    import torch

    import paper_2602_06063_b200 as fd

    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the FusedDQP library has no CPU path")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    peaks, peak_kind = measured_peaks()
    M = 1
    layer_shapes = synthgen.GEMMA3_4B_LAYER
    # launch groups: projections sharing their input run as one call on weights concatenated along N
    groups = [["q", "k", "v"], ["o"], ["gate", "up"], ["down"]] if args.fuse else [[n] for n, _, _, _ in layer_shapes]
    by_name = {n: (K, N, seed) for n, K, N, seed in layer_shapes}
    shapes = [("|".join(g), by_name[g[0]][0], sum(by_name[n][1] for n in g), by_name[g[0]][2]) for g in groups]
    max_K = max(K for _, K, _, _ in shapes)
    step_bytes_layer = layer_bytes(M)
    _, hk, hn, hseed = synthgen.GEMMA3_4B_LM_HEAD
    ctx = fd.fdqp_create(local_rank, 8, max(max_K, hk), max(max(N for _, _, N, _ in shapes), hn))
    if args.param:
        for kv in args.param:
            key, val = kv.split("=")
            fd.fdqp_set_param(ctx, key, int(val))

    # ---- resident inputs: LAYER_COPIES distinct weight sets, one x and one y per projection
    copies = []
    host_layer0 = None
    for c in range(LAYER_COPIES):
        layer = []
        for g in groups:
            parts = []
            for name in g:
                K, N, seed = by_name[name]
                w = synthgen.weights(seed + 1000 * c, K, N)
                parts.append(fd.q4nx_pack(w.codes, w.scales, w.offsets))
                if c == 0:
                    host_layer0 = host_layer0 or []
                    host_layer0.append((w, synthgen.activations(by_name[g[0]][2], M, K)))
            layer.append(torch.from_numpy(np.concatenate(parts)).cuda())
        copies.append(layer)
    xs_host = [synthgen.activations(seed, M, K) for _, K, _, seed in shapes]
    xs = [torch.from_numpy(x.view(np.int16)).cuda() for x in xs_host]
    ys = [torch.empty((M, N), dtype=torch.float32, device="cuda") for _, _, N, _ in shapes]
    stream = torch.cuda.Stream()
    sraw = stream.cuda_stream

    def enqueue_layer(c):
        for i, (_, K, N, _) in enumerate(shapes):
            fd.fdqp_run(ctx, xs[i], copies[c][i], ys[i], M, K, N, sraw)

    # CUDA graphs: a decode step of the real model is 34 such layers back to back, so the layers are captured
    # LAYER_COPIES at a time (one pass over all resident weight copies per graph); single-layer graphs cover the
    # remainder when the step count is not a multiple of LAYER_COPIES.
    # kernels one step launches (activation preparation and split-K sum kernels included, when the plan uses them)
    count0 = fd.fdqp_launch_count(ctx)
    enqueue_layer(0)
    torch.cuda.synchronize()
    kernels_per_step = fd.fdqp_launch_count(ctx) - count0
    graphs = None
    pass_graph = None
    if args.graph:
        graphs = []
        with torch.cuda.stream(stream):
            enqueue_layer(0)
        stream.synchronize()
        for c in range(LAYER_COPIES):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                enqueue_layer(c)
            graphs.append(g)
        pass_graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(pass_graph, stream=stream):
            for c in range(LAYER_COPIES):
                enqueue_layer(c)

    def run_steps(first, count):
        """Enqueue `count` consecutive steps starting at step index `first`."""
        i = first
        end = first + count
        while i < end:
            c = i % LAYER_COPIES
            if pass_graph is not None and c == 0 and end - i >= LAYER_COPIES:
                with torch.cuda.stream(stream):
                    pass_graph.replay()
                i += LAYER_COPIES
            elif graphs is not None:
                with torch.cuda.stream(stream):
                    graphs[c].replay()
                i += 1
            else:
                enqueue_layer(c)
                i += 1

    def step(i):
        run_steps(i, 1)

    run_steps(0, args.warmup)
    first_timed = -(-args.warmup // LAYER_COPIES) * LAYER_COPIES   # start the timed region on a pass boundary
    run_steps(args.warmup, first_timed - args.warmup)
    stream.synchronize()

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches_before = fd.fdqp_launch_count(ctx)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record(stream)
    run_steps(first_timed, args.steps)
    ev1.record(stream)
    stream.synchronize()
    barrier()
    ms = ev0.elapsed_time(ev1)
    calls_per_step = len(shapes)
    launches = kernels_per_step * args.steps
    if graphs is None:
        assert fd.fdqp_launch_count(ctx) - launches_before == launches
    clocks = sampler.stop() if rank == 0 else None
    if fd.fdqp_last_status(ctx) != 0:
        raise SystemExit("bench.py: a kernel reported " + fd.fdqp_status_string(fd.fdqp_last_status(ctx)))
    ms = max_over_ranks(ms, dist, "cuda")

    # ---- end to end: host x in, host y out, through fdqp_run_host_async (pinned buffers) + one stream sync, every step
    xs_pin = [torch.from_numpy(x.view(np.int16)).pin_memory() for x in xs_host]
    ys_pin = [torch.empty((M, N), dtype=torch.float32).pin_memory() for _, _, N, _ in shapes]
    e2e_steps = max(3, min(args.steps, 200))

    def e2e_enqueue(c):
        for j, (_, K, N, _) in enumerate(shapes):
            fd.fdqp_run_host_async(ctx, xs_pin[j], copies[c][j], ys_pin[j], M, K, N, sraw)

    e2e_enqueue(0)             # the first call allocates the context's staging buffers
    stream.synchronize()
    e2e_graphs = None
    if graphs:
        # the step's four calls recorded once per weight set and replayed: with pinned buffers used in place a step is
        # kernels only (they read x from and write y to host memory), and the host pays one launch per step
        e2e_graphs = []
        for c in range(LAYER_COPIES):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                e2e_enqueue(c)
            e2e_graphs.append(g)

    def e2e_step(i):
        c = i % LAYER_COPIES
        if e2e_graphs is not None:
            with torch.cuda.stream(stream):
                e2e_graphs[c].replay()
        else:
            e2e_enqueue(c)
        stream.synchronize()   # the step's results are in host memory from here on

    for i in range(3):
        e2e_step(i)
    barrier()
    t0 = time.perf_counter()
    for i in range(e2e_steps):
        e2e_step(3 + i)
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    e2e_s = max_over_ranks(e2e_s, dist, "cuda")

    # ---- LM head (M = 1) for the tokens/s figure: 34 layers + head, projections only
    head_ms = None
    if rank == 0 and not args.no_head:
        hw = synthgen.weights(hseed, hk, hn)
        hW = torch.from_numpy(fd.q4nx_pack(hw.codes, hw.scales, hw.offsets)).cuda()
        del hw
        hx = torch.from_numpy(synthgen.activations(hseed, 1, hk).view(np.int16)).cuda()
        hy = torch.empty((1, hn), dtype=torch.float32, device="cuda")
        for _ in range(3):
            fd.fdqp_run(ctx, hx, hW, hy, 1, hk, hn, sraw)
        h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0.record(stream)
        for _ in range(10):
            fd.fdqp_run(ctx, hx, hW, hy, 1, hk, hn, sraw)
        h1.record(stream)
        stream.synchronize()
        head_ms = h0.elapsed_time(h1) / 10

    # ---- the same projections at M = 8 (batched decode): one graph pass over the weight copies, LM head directly
    batch8 = None
    if rank == 0 and not args.no_head:
        M8 = 8
        xs8 = [torch.from_numpy(synthgen.activations(seed, M8, K).view(np.int16)).cuda() for _, K, _, seed in shapes]
        ys8 = [torch.empty((M8, N), dtype=torch.float32, device="cuda") for _, _, N, _ in shapes]

        def enqueue_layer8(c):
            for i, (_, K, N, _) in enumerate(shapes):
                fd.fdqp_run(ctx, xs8[i], copies[c][i], ys8[i], M8, K, N, sraw)

        with torch.cuda.stream(stream):
            enqueue_layer8(0)
        stream.synchronize()
        g8 = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g8, stream=stream):
            for c in range(LAYER_COPIES):
                enqueue_layer8(c)
        b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            for _ in range(3):
                g8.replay()
            b0.record(stream)
            for _ in range(20):
                g8.replay()
            b1.record(stream)
        stream.synchronize()
        layer8_ms = b0.elapsed_time(b1) / (20 * LAYER_COPIES)
        hx8 = torch.from_numpy(synthgen.activations(hseed, M8, hk).view(np.int16)).cuda()
        hy8 = torch.empty((M8, hn), dtype=torch.float32, device="cuda")
        for _ in range(3):
            fd.fdqp_run(ctx, hx8, hW, hy8, M8, hk, hn, sraw)
        b0.record(stream)
        for _ in range(10):
            fd.fdqp_run(ctx, hx8, hW, hy8, M8, hk, hn, sraw)
        b1.record(stream)
        stream.synchronize()
        head8_ms = b0.elapsed_time(b1) / 10
        batch8 = {"M": M8, "layer_ms": layer8_ms, "lm_head_ms": head8_ms,
                  "layer_gbs": layer_bytes(M8) / (layer8_ms * 1e-3) / 1e9,
                  "decode_tokens_per_s": M8 * 1e3 / (synthgen.GEMMA3_4B_LAYERS * layer8_ms + head8_ms)}
        del xs8, ys8, hx8, hy8

    # ---- LM head at a prefill chunk (M = 512, the largest baseline configuration): the tensor-core path, against the tensor roofline
    prefill = None
    if rank == 0 and not args.no_head:
        PM = 512
        pctx = fd.fdqp_create(local_rank, PM, hk, hn)
        px = torch.from_numpy(synthgen.activations(hseed, PM, hk).view(np.int16)).cuda()
        py = torch.empty((PM, hn), dtype=torch.float32, device="cuda")
        for _ in range(3):
            fd.fdqp_run(pctx, px, hW, py, PM, hk, hn, sraw)
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        p0.record(stream)
        for _ in range(6):
            fd.fdqp_run(pctx, px, hW, py, PM, hk, hn, sraw)
        p1.record(stream)
        stream.synchronize()
        if fd.fdqp_last_status(pctx) != 0:
            raise SystemExit("bench.py: the prefill kernel reported " + fd.fdqp_status_string(fd.fdqp_last_status(pctx)))
        p_ms = p0.elapsed_time(p1) / 6
        tflops = 2.0 * PM * hk * hn / (p_ms * 1e-3) / 1e12
        prefill = {"workload": f"Gemma3-4B LM head K={hk} N={hn} at M={PM}", "ms": p_ms, "tflops": tflops,
                   "bound": "tensor", "peak_burst_tflops": peaks.get("bf16_tflops"),
                   "peak_sustained_tflops": peaks.get("bf16_tflops_sustained"),
                   "frac_of_burst": tflops / peaks["bf16_tflops"] if peaks.get("bf16_tflops") else None,
                   "frac_of_sustained": (tflops / peaks["bf16_tflops_sustained"]) if peaks.get("bf16_tflops_sustained") else None,
                   "launch": fd.fdqp_describe(pctx, PM, hk, hn)}
        # smaller token counts on the same matrix (the one-SM forms of the kernel), same timing
        other = {}
        for om in (32, 128):
            for _ in range(3):
                fd.fdqp_run(pctx, px, hW, py, om, hk, hn, sraw)
            p0.record(stream)
            for _ in range(6):
                fd.fdqp_run(pctx, px, hW, py, om, hk, hn, sraw)
            p1.record(stream)
            stream.synchronize()
            if fd.fdqp_last_status(pctx) != 0:
                raise SystemExit("bench.py: the prefill kernel reported " + fd.fdqp_status_string(fd.fdqp_last_status(pctx)))
            o_ms = p0.elapsed_time(p1) / 6
            other[f"M{om}"] = {"ms": o_ms, "tflops": 2.0 * om * hk * hn / (o_ms * 1e-3) / 1e12,
                               "launch": fd.fdqp_describe(pctx, om, hk, hn)}
        prefill["other_token_counts"] = other
        fd.fdqp_destroy(pctx)
        del px, py

    # ---- next steps beside the projection: decode attention over a KV cache, and the format variants of the container
    attention = None
    formats = None
    dequant = None
    if rank == 0 and not args.no_head:
        H, G, d, L = 8, 4, 256, 32768          # Gemma3-4B heads at a 32k context
        ncache = max(1, int(np.ceil(4 * L2_BYTES / (2 * G * L * d * 2))))
        gen = torch.Generator(device="cuda").manual_seed(2)
        caches = [(torch.randn((G, L, d), device="cuda", generator=gen).to(torch.bfloat16),
                   torch.randn((G, L, d), device="cuda", generator=gen).to(torch.bfloat16)) for _ in range(ncache)]
        aq = torch.randn((H, d), device="cuda", generator=gen).to(torch.bfloat16)
        ao = torch.empty((H, d), dtype=torch.float32, device="cuda")
        attention = {"workload": f"Gemma3-4B decode attention, H={H} G={G} d={d}, L={L}", "bound": "hbm"}
        for name, window in (("global", 0), ("window_1024", 1024)):
            reps = 20
            ga = torch.cuda.CUDAGraph()
            with torch.cuda.stream(stream):
                for i in range(3):
                    fd.fdqp_flowkv_decode(ctx, aq, caches[i % ncache][0], caches[i % ncache][1], ao, H, G, d, L, L, window,
                                          d ** -0.5, sraw)
            stream.synchronize()
            with torch.cuda.graph(ga, stream=stream):
                for i in range(reps):
                    fd.fdqp_flowkv_decode(ctx, aq, caches[i % ncache][0], caches[i % ncache][1], ao, H, G, d, L, L, window,
                                          d ** -0.5, sraw)
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            with torch.cuda.stream(stream):
                ga.replay()
                a0.record(stream)
                ga.replay()
                a1.record(stream)
            stream.synchronize()
            us = a0.elapsed_time(a1) * 1e3 / reps
            n_att = window if window else L
            a_gbs = 2.0 * G * n_att * d * 2 / us / 1e3
            attention[name] = {"us": us, "gbs": a_gbs, "frac": a_gbs / peaks["hbm_gbs"]}
            del ga
        del caches
        formats = {"workload": f"LM head K={hk} N={hn} at M=1, bytes of the format's own container"}
        for name, fmt in (("g64", fd.FMT_G64), ("g128", fd.FMT_G128), ("mxfp4", fd.FMT_MXFP4)):
            fw = synthgen.weights_fmt(hseed, hk, 4096, fmt)
            tile = fd.q4nx_pack_fmt(fmt, fw.codes, fw.scales, fw.offsets)
            nbytes = fd.q4nx_packed_bytes_fmt(fmt, hk, hn)
            fW = torch.from_numpy(np.tile(tile, hn // 4096)[:nbytes].copy()).cuda()
            for _ in range(3):
                fd.fdqp_run_fmt(ctx, fmt, hx, fW, hy, 1, hk, hn, sraw)
            f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            f0.record(stream)
            for _ in range(10):
                fd.fdqp_run_fmt(ctx, fmt, hx, fW, hy, 1, hk, hn, sraw)
            f1.record(stream)
            stream.synchronize()
            f_ms = f0.elapsed_time(f1) / 10
            f_gbs = (nbytes + 2 * hk + 4 * hn) / (f_ms * 1e-3) / 1e9
            formats[name] = {"ms": f_ms, "gbs": f_gbs, "frac": f_gbs / peaks["hbm_gbs"]}
            del fW
        # the dequantisation engine on the LM head: container -> dense bf16 matrix in HBM (write-bound)
        dq_out = torch.empty((hk, hn), dtype=torch.bfloat16, device="cuda")
        for _ in range(2):
            fd.fdqp_dequant(ctx, hW, dq_out, True, hk, hn, sraw)
        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        d0.record(stream)
        for _ in range(5):
            fd.fdqp_dequant(ctx, hW, dq_out, True, hk, hn, sraw)
        d1.record(stream)
        stream.synchronize()
        dq_ms = d0.elapsed_time(d1) / 5
        dq_gbs = (0.625 + 2.0) * hk * hn / (dq_ms * 1e-3) / 1e9
        dequant = {"workload": f"LM head K={hk} N={hn} -> bf16 [K][N]", "ms": dq_ms, "gbs": dq_gbs, "bound": "hbm",
                   "frac": dq_gbs / peaks["hbm_gbs"]}
        del dq_out
        if fd.fdqp_last_status(ctx) != 0:
            raise SystemExit("bench.py: a kernel reported " + fd.fdqp_status_string(fd.fdqp_last_status(ctx)))

    # ---- CPU baseline: the oracle on the host cores, one pass over the same layer (rank 0, N = 1 only)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        import oracle
        cores = min(oracle.max_threads(), os.cpu_count() or 1)
        t0 = time.perf_counter()
        passes = 0
        while passes < 1 or time.perf_counter() - t0 < 10:   # about 10 s of oracle work
            for w, x in host_layer0:
                oracle.project(x, w.codes, w.scales, w.offsets, nthreads=cores)
            passes += 1
        dt = time.perf_counter() - t0
        cpu = {"value": layer_bytes(M) * passes / dt / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle",
               "sample": f"{passes} pass(es) of the whole layer (7 projections, all outputs), {dt:.1f} s"}

    if rank == 0:
        step_bytes = step_bytes_layer
        gbs = whole_job_gbs(step_bytes, args.steps, world, ms)
        per_launch_us = ms * 1e3 / (calls_per_step * args.steps)   # one GEMV launch incl. its preparation kernel
        achieved = (step_bytes / calls_per_step) / (per_launch_us * 1e-6) / 1e9
        layer_ms = ms / args.steps
        line = {
            "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": layer_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": WORKLOAD, "M": M, "bytes_per_step": step_bytes, "cuda_graph": (f"{LAYER_COPIES} steps per graph" if graphs else False),
                       "calls_per_step": [name for name, _, _, _ in shapes],
                       "l2": f"inputs larger than L2: steps rotate over {LAYER_COPIES} distinct weight sets "
                             f"({LAYER_COPIES * step_bytes / 1e6:.0f} MB)",
                       "multi_gpu": "independent replicas, no collective",
                       "launch": fd.fdqp_describe(ctx, 1, 2560, 10240)},
            "frac_of_nominal_8TBps": gbs / world / NOMINAL_HBM_GBS,
            "decode_tokens_per_s": (1e3 / (synthgen.GEMMA3_4B_LAYERS * layer_ms + head_ms)) if head_ms else None,
            "lm_head_ms": head_ms,
            "lm_head_gbs": (alg_bytes(1, hk, hn) / (head_ms * 1e-3) / 1e9) if head_ms else None,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": achieved / peaks["hbm_gbs"],
                         # ncu, K=2560 N=98304 M=1 (profiles/gemv_m1_k2560_n98304.md): dram read+write = 1.024 x the
                         # algorithmic bytes; traffic grows in proportion to 0.625*K*N, so scale to this call size
                         "traffic": 1.024 * step_bytes / calls_per_step, "peak_kind": peak_kind + " copy bandwidth",
                         "kernel": "fdqp_gemv_kernel", "launch_us": per_launch_us},
            "batched_decode": batch8,
            "prefill_lm_head": prefill,
            "decode_attention": attention,
            "format_variants": formats,
            "dequant_engine": dequant,
            "cpu_baseline": cpu,
            "e2e": {"value": whole_job_gbs(step_bytes, e2e_steps, world, e2e_s * 1e3), "unit": "GB/s",
                    "h2d_bytes_per_step": sum(2 * M * K for _, K, _, _ in shapes),
                    "d2h_bytes_per_step": sum(4 * M * N for _, _, N, _ in shapes), "ms_per_step": e2e_s / e2e_steps * 1e3,
                    "how": "fdqp_run_host_async per projection on pinned buffers (x read from and y written to host memory "
                           "by the kernels), " + ("the step's calls replayed from a CUDA graph, " if e2e_graphs is not None else "")
                           + "one stream synchronisation per step"},
            "gpu_launches": launches,
            "clocks": clocks,
        }
        print(json.dumps(line), flush=True)
    fd.fdqp_destroy(ctx)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=8000)
    ap.add_argument("--warmup", type=int, default=40)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--graph", type=int, default=1, help="replay each step from a CUDA graph (default 1)")
    ap.add_argument("--fuse", type=int, default=1, help="run q|k|v and gate|up as one call each (default 1)")
    ap.add_argument("--param", action="append", help="library launch parameter key=value (repeatable)")
    ap.add_argument("--shape", help="K,N,M: time this one projection shape instead of the layer workload")
    ap.add_argument("--same-weights", action="store_true", help="with --shape: reuse one weight buffer (for ncu captures)")
    ap.add_argument("--dequant", help="K,N,bf16|fp32: time the dequantisation engine (container -> dense matrix) instead")
    ap.add_argument("--flowkv", help="H,G,d,L,window: time the decode attention over a KV cache instead of a projection")
    ap.add_argument("--rmsnorm", action="store_true", help="with --shape: RMS-normalise x first (fused where possible)")
    ap.add_argument("--epilogue", default="none", choices=["none", "bf16", "geglu"],
                    help="with --shape: fused store-side epilogue (geglu: gate and up rows interleaved 16 by 16 along N)")
    ap.add_argument("--format", default="q4nx", choices=["q4nx", "g64", "g128", "mxfp4"],
                    help="with --shape: format variant of the block container (group 64 / 128, MXFP4)")
    ap.add_argument("--l2-resident", action="store_true",
                    help="with --shape: one weight copy, graph-replayed (what a call costs when its weights are already in L2)")
    ap.add_argument("--residual", action="store_true",
                    help="with --shape --rmsnorm: add a residual to x first and write the sum out (fdqp_run_add_rmsnorm_epilogue)")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--no-head", action="store_true", help="skip the LM-head timing")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        if args.steps == 8000 and args.warmup == 40:
            args.steps, args.warmup = 5, 1
        run_reference(args, rank, world)
        return
    if args.warmup < 3:
        args.warmup = 3
    if args.dequant:
        if args.steps == 8000:
            args.steps = 10
        run_dequant(args)
        return
    if args.flowkv:
        if args.steps == 8000:
            args.steps = 50
        run_flowkv(args)
        return
    if args.shape:
        if args.steps == 8000:
            args.steps = 50
        run_shape(args)
        return
    run_ours(args, rank, local_rank, world)


if __name__ == "__main__":
    main()
