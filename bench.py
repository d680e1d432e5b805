#!/usr/bin/env python
"""Benchmark of the FusedDQP hot path on B200.

A step is one pass of the hot path over the largest single-GPU configuration: the Gemma3-4B tied LM head (K = 2560,
N = 262144, 419 MB of packed Q4NX weights, seed 17) at decode M = 1 -- one fdqp_run call, one kernel launch.  The
metric is the achieved bandwidth over the algorithmic bytes of the step (0.625*K*N + 2*M*K + 4*M*N).  Beside the
headline the line carries one sub-object per BASELINE configuration and M (per-call median / min / p90 from CUDA-event
pairs, back-to-back mean from a graph replay of at least 60 ms, GB/s, fractions of the measured and the nominal peak,
the launch plan and the clock samples of its own region), the Gemma3-4B layer as single calls and as chained launches,
decode tokens/s (projections only: 34 layers + LM head), batched decode, the prefill tensor-core path, decode attention,
the format variants and the dequantisation engine.

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
WORKLOAD = "Gemma3-4B tied LM head K=2560 N=262144, Q4NX group 32, decode M=1 (seed 17): the largest single-GPU configuration"
L2_BYTES = 126e6
LAYER_COPIES = 8            # distinct weight sets resident in HBM (8 x 59 MB = 472 MB >> L2)
NOMINAL_HBM_GBS = 8000.0
# dram__bytes_read.sum + dram__bytes_write.sum of one LM-head launch (K=2560, N=262144, M=1) from an ncu capture
NCU_LM_HEAD_DRAM_BYTES = 419511296 + 3408128


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
                self.rows.append((time.time(), parts))      # host time at which the sample arrived

    @staticmethod
    def _summary(rows):
        sm, smax, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for _, r in rows:
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

    def window(self, t0, t1):
        """Samples that arrived during [t0, t1 + one period]: the clocks of one timed region."""
        if self.proc is None:
            return None
        time.sleep(0.03)                                    # let the sample that covers the end of the region arrive
        return self._summary([r for r in list(self.rows) if t0 <= r[0] <= t1 + 0.025])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        return self._summary(self.rows)


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
    """Times the CPU oracle (as it stands) on the host cores on the headline workload: each step is one pass over a
    bounded sample of the LM head's outputs at M = 1 (the first 65536 of the 262144 columns of the seeded matrix, all of
    K), OpenMP over columns; the GB/s counts the sample's own algorithmic bytes."""
    if rank != 0:
        return
    import oracle
    cores = min(oracle.max_threads(), os.cpu_count() or 1)
    _, K, N, seed = synthgen.GEMMA3_4B_LM_HEAD
    n1 = N // 4
    w = synthgen.weights(seed, K, n1)                      # the generator is column-wise: the first n1 columns of the head
    x = synthgen.activations(seed, 1, K)

    def one_pass():
        oracle.project(x, w.codes, w.scales, w.offsets, nthreads=cores)

    for _ in range(args.warmup):
        one_pass()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        one_pass()
    dt = time.perf_counter() - t0
    gbs = alg_bytes(1, K, n1) * args.steps / dt / 1e9
    sample = f"outputs 0..{n1 - 1} of the {N} of the LM head per step (a quarter of the matrix)"
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "M": 1, "K": K, "N": N, "sample": sample,
                   "note": "CPU oracle (fp64, plain C, OpenMP over output columns)"},
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
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


# ----------------------------------------------------------------------------------------------- a chained layer

def run_layer_chain(args):
    """Times the Gemma3-4B decoder layer at M = --tokens (q|k|v, o, gate|up, down on independent seeded inputs) as chained
    launches of --layer-chain layers each (fdqp_run_chain), rotating over 8 distinct weight sets."""
    import torch

    import paper_2602_06063_b200 as fd

    L, M = args.layer_chain, args.tokens
    torch.cuda.set_device(0)
    peaks, peak_kind = measured_peaks()
    by_name = {n: (K, N, seed) for n, K, N, seed in synthgen.GEMMA3_4B_LAYER}
    groups = [["q", "k", "v"], ["o"], ["gate", "up"], ["down"]]
    shapes = [("|".join(g), by_name[g[0]][0], sum(by_name[n][1] for n in g), by_name[g[0]][2]) for g in groups]
    ctx = fd.fdqp_create(0, 8, 10240, 20480)
    for kv in args.param or []:
        key, val = kv.split("=")
        fd.fdqp_set_param(ctx, key, int(val))
    copies = [[tiled_weights(fd, torch, K, N, seed + 1000 * c) for _, K, N, seed in shapes] for c in range(LAYER_COPIES)]
    xs = [torch.from_numpy(synthgen.activations(seed, M, K).view(np.int16)).cuda() for _, K, _, seed in shapes]
    ys = [torch.empty((M, N), dtype=torch.float32, device="cuda") for _, _, N, _ in shapes]
    stream = torch.cuda.Stream()
    sraw = stream.cuda_stream
    chains = [fd.make_chain([fd.chain_step(xs[j], copies[(first + l) % LAYER_COPIES][j], ys[j], K, N)
                             for l in range(L) for j, (_, K, N, _) in enumerate(shapes)]) for first in range(0, LAYER_COPIES, max(1, min(L, LAYER_COPIES)))]
    for i in range(max(3, args.warmup)):
        fd.fdqp_run_chain(ctx, chains[i % len(chains)], M, sraw)
    stream.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(args.steps):
        fd.fdqp_run_chain(ctx, chains[i % len(chains)], M, sraw)
    e1.record(stream)
    stream.synchronize()
    assert fd.fdqp_last_status(ctx) == 0
    us = e0.elapsed_time(e1) * 1e3 / (args.steps * L)
    gbs = layer_bytes(M) / us / 1e3
    print(json.dumps({"layer_chain": {"layers_per_launch": L, "M": M}, "us_per_layer": us, "GBps": gbs,
                      "frac_of_measured_peak": gbs / peaks["hbm_gbs"], "peak_kind": peak_kind, "launches": args.steps}), flush=True)
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
    for kv in args.param or []:
        k, v = kv.split("=")
        fd.fdqp_set_param(ctx, k, int(v))
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

MIN_REGION_MS = 60.0        # every timed region lasts at least this long, whatever --steps is (several clock samples)
PAIR_CALLS = 160            # per-call event pairs behind each median / min / p90


class Regions:
    """Host-time windows of the timed regions, so that each gets the clock samples that fall inside it."""

    def __init__(self, sampler):
        self.sampler = sampler

    def clocks(self, t0, t1):
        return self.sampler.window(t0, t1) if self.sampler is not None else None


def tiled_weights(fd, torch, K, N, seed, fmt=None):
    """Packed weights of a K x N matrix on the device: a seeded matrix of up to 4096 output columns tiled along N (the
    strip-major container makes that byte concatenation) -- the full recipe costs minutes of host time for the largest
    shapes and the kernels' timing does not depend on the values."""
    nb = min(N, 4096)
    if fmt is None or fmt == fd.FMT_Q4NX:
        w = synthgen.weights(seed, K, nb)
        tile = fd.q4nx_pack(w.codes, w.scales, w.offsets)
        nbytes = fd.q4nx_packed_bytes(K, N)
    else:
        w = synthgen.weights_fmt(seed, K, nb, fmt)
        tile = fd.q4nx_pack_fmt(fmt, w.codes, w.scales, w.offsets)
        nbytes = fd.q4nx_packed_bytes_fmt(fmt, K, N)
    return torch.from_numpy(np.tile(tile, -(-N // nb))[:nbytes].copy()).cuda()


def weight_copies(torch, base):
    """Enough distinct copies of a weight buffer that consecutive launches never find theirs in L2 (>= 4 x L2 in all)."""
    n = max(1, int(np.ceil(4 * L2_BYTES / base.numel())))
    return [base] + [base.clone() for _ in range(n - 1)]


def time_region(torch, stream, enqueue, ncalls_cycle, regions, min_ms=MIN_REGION_MS, pairs=PAIR_CALLS):
    """enqueue(i) puts call i (rotating inputs itself) on `stream`.  Returns per-call statistics:
    median / min / p90 of single calls bracketed by CUDA events on the launching stream (direct launches), and the mean
    of back-to-back calls replayed from a CUDA graph for at least min_ms (what a decode loop sees), with the clock
    samples taken during that region."""
    for i in range(max(3, ncalls_cycle)):
        enqueue(i)
    stream.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(pairs)]
    for i, (a, b) in enumerate(evs):
        a.record(stream)
        enqueue(i)
        b.record(stream)
    stream.synchronize()
    us = sorted(a.elapsed_time(b) * 1e3 for a, b in evs)
    per_graph = max(ncalls_cycle, 8)
    per_graph = -(-per_graph // ncalls_cycle) * ncalls_cycle
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        for i in range(per_graph):
            enqueue(i)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        for _ in range(2):
            g.replay()
        e0.record(stream)
        g.replay()
        e1.record(stream)
    stream.synchronize()
    one = max(e0.elapsed_time(e1), 1e-3)
    reps = max(1, int(np.ceil(min_ms / one)))
    t0 = time.time()
    with torch.cuda.stream(stream):
        e0.record(stream)
        for _ in range(reps):
            g.replay()
        e1.record(stream)
    stream.synchronize()
    t1 = time.time()
    ms = e0.elapsed_time(e1)
    return {"us_median": us[len(us) // 2], "us_min": us[0], "us_p90": us[int(0.9 * (len(us) - 1))],
            "us_back_to_back": ms * 1e3 / (reps * per_graph), "calls_timed": reps * per_graph, "region_ms": ms,
            "clocks": regions.clocks(t0, t1)}


def with_rates(entry, alg_bytes_per_call, peaks, flops=None):
    """GB/s over the algorithmic bytes (back-to-back mean and per-call median) against the measured and nominal peaks."""
    gbs = alg_bytes_per_call / entry["us_back_to_back"] / 1e3
    entry.update({"bytes": alg_bytes_per_call, "GBps": gbs, "frac_of_measured": gbs / peaks["hbm_gbs"],
                  "frac_of_nominal_8TBps": gbs / NOMINAL_HBM_GBS,
                  "GBps_median_call": alg_bytes_per_call / entry["us_median"] / 1e3})
    if flops is not None:
        tf = flops / entry["us_back_to_back"] / 1e6
        entry.update({"TFLOPs": tf, "frac_of_burst": tf / peaks["bf16_tflops"],
                      "frac_of_sustained": tf / peaks["bf16_tflops_sustained"]})
    return entry


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
    _, hk, hn, hseed = synthgen.GEMMA3_4B_LM_HEAD
    M = 1
    ctx = fd.fdqp_create(local_rank, 8, 21504, hn)
    for kv in args.param or []:
        key, val = kv.split("=")
        fd.fdqp_set_param(ctx, key, int(val))
    stream = torch.cuda.Stream()
    sraw = stream.cuda_stream
    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler is not None:
        sampler.start()
    regions = Regions(sampler)

    # ---- headline: the largest single-GPU configuration, the Gemma3-4B LM head at M = 1 (seed 17), one call per step
    hw = synthgen.weights(hseed, hk, hn)
    hW = torch.from_numpy(fd.q4nx_pack(hw.codes, hw.scales, hw.offsets)).cuda()
    hx_host = synthgen.activations(hseed, 1, hk)
    hx = torch.from_numpy(hx_host.view(np.int16)).cuda()
    hy = torch.empty((1, hn), dtype=torch.float32, device="cuda")
    step_bytes = alg_bytes(1, hk, hn)
    count0 = fd.fdqp_launch_count(ctx)
    fd.fdqp_run(ctx, hx, hW, hy, 1, hk, hn, sraw)
    stream.synchronize()
    kernels_per_step = fd.fdqp_launch_count(ctx) - count0
    for _ in range(args.warmup):
        fd.fdqp_run(ctx, hx, hW, hy, 1, hk, hn, sraw)
    stream.synchronize()
    # EXACTLY --steps steps per block; the block is repeated until the timed region is long enough to carry clock samples
    g_steps = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g_steps, stream=stream):
        for _ in range(args.steps):
            fd.fdqp_run(ctx, hx, hW, hy, 1, hk, hn, sraw)
    with torch.cuda.stream(stream):
        g_steps.replay()
    stream.synchronize()
    blocks = max(1, int(np.ceil(MIN_REGION_MS / (args.steps * 0.070))))
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_host0 = time.time()
    with torch.cuda.stream(stream):
        ev0.record(stream)
        for _ in range(blocks):
            g_steps.replay()
        ev1.record(stream)
    stream.synchronize()
    t_host1 = time.time()
    barrier()
    timed_steps = blocks * args.steps
    ms = max_over_ranks(ev0.elapsed_time(ev1), dist, "cuda")
    if fd.fdqp_last_status(ctx) != 0:
        raise SystemExit("bench.py: a kernel reported " + fd.fdqp_status_string(fd.fdqp_last_status(ctx)))
    head_clocks = regions.clocks(t_host0, t_host1)
    head_us = ms * 1e3 / timed_steps
    gbs = whole_job_gbs(step_bytes, timed_steps, world, ms)

    # ---- end to end: host x in, host y out through fdqp_run_host_async (pinned buffers) + one stream sync, every step
    x_pin = torch.from_numpy(hx_host.view(np.int16)).pin_memory()
    y_pin = torch.empty((1, hn), dtype=torch.float32).pin_memory()
    fd.fdqp_run_host_async(ctx, x_pin, hW, y_pin, 1, hk, hn, sraw)     # the first call allocates the staging buffers
    stream.synchronize()
    e2e_steps = max(args.steps, 200)
    for _ in range(3):
        fd.fdqp_run_host_async(ctx, x_pin, hW, y_pin, 1, hk, hn, sraw)
        stream.synchronize()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        fd.fdqp_run_host_async(ctx, x_pin, hW, y_pin, 1, hk, hn, sraw)
        stream.synchronize()                                            # the step's result is in host memory from here on
    e2e_s = max_over_ranks(time.perf_counter() - t0, dist, "cuda")

    line_extra = {}
    if rank == 0 and not args.headline_only:
        # ---- every BASELINE configuration and M: per-call statistics, GB/s, fractions, launch plan, clocks
        configs = {}

        def shape_entry(K, N, Mi, seed, W_list=None, amp=1.0):
            copies = W_list or weight_copies(torch, tiled_weights(fd, torch, K, N, seed))
            x = torch.from_numpy(synthgen.activations(seed, Mi, K, amp).view(np.int16)).cuda()
            y = torch.empty((Mi, N), dtype=torch.float32, device="cuda")
            ent = time_region(torch, stream, lambda i: fd.fdqp_run(ctx, x, copies[i % len(copies)], y, Mi, K, N, sraw),
                              len(copies), regions)
            ent["launch"] = fd.fdqp_describe(ctx, Mi, K, N)
            return with_rates(ent, alg_bytes(Mi, K, N), peaks), copies

        _, K0, N0, seed0 = synthgen.GEMMA3_1B_GATE
        configs["0: Gemma3-1B gate K=1152 N=6912 M=1"], _ = shape_entry(K0, N0, 1, seed0)
        # config 1: the Gemma3-4B decoder layer at M = 1 -- per call, as four single calls, and as chains
        by_name = {n: (K, N, seed) for n, K, N, seed in synthgen.GEMMA3_4B_LAYER}
        groups = [["q", "k", "v"], ["o"], ["gate", "up"], ["down"]]
        shapes = [("|".join(g), by_name[g[0]][0], sum(by_name[n][1] for n in g), by_name[g[0]][2]) for g in groups]
        layer_copies = []
        for c in range(LAYER_COPIES):
            layer_copies.append([tiled_weights(fd, torch, K, N, seed + 1000 * c) for _, K, N, seed in shapes])
        xs = [torch.from_numpy(synthgen.activations(seed, 1, K).view(np.int16)).cuda() for _, K, _, seed in shapes]
        ys = [torch.empty((1, N), dtype=torch.float32, device="cuda") for _, _, N, _ in shapes]
        per_call = {}
        for j, (name, K, N, seed) in enumerate(shapes):
            ent = time_region(torch, stream, lambda i, j=j, K=K, N=N: fd.fdqp_run(ctx, xs[j], layer_copies[i % LAYER_COPIES][j], ys[j], 1, K, N, sraw),
                              LAYER_COPIES, regions)
            ent["launch"] = fd.fdqp_describe(ctx, 1, K, N)
            per_call[f"{name} K={K} N={N}"] = with_rates(ent, alg_bytes(1, K, N), peaks)
        lbytes = layer_bytes(1)

        def layer_single(i):
            for j, (_, K, N, _) in enumerate(shapes):
                fd.fdqp_run(ctx, xs[j], layer_copies[i % LAYER_COPIES][j], ys[j], 1, K, N, sraw)

        def chain_of(cs):
            return fd.make_chain([fd.chain_step(xs[j], layer_copies[c][j], ys[j], K, N)
                                  for c in cs for j, (_, K, N, _) in enumerate(shapes)])

        chains1 = [chain_of([c]) for c in range(LAYER_COPIES)]
        chain8 = chain_of(range(LAYER_COPIES))
        layer = {"four_single_calls": with_rates(time_region(torch, stream, layer_single, LAYER_COPIES, regions), lbytes, peaks),
                 "one_chained_launch_per_layer": with_rates(time_region(torch, stream, lambda i: fd.fdqp_run_chain(ctx, chains1[i % LAYER_COPIES], 1, sraw), LAYER_COPIES, regions), lbytes, peaks)}
        ent8 = time_region(torch, stream, lambda i: fd.fdqp_run_chain(ctx, chain8, 1, sraw), 1, regions)
        for k in ("us_median", "us_min", "us_p90", "us_back_to_back"):
            ent8[k] /= LAYER_COPIES                                      # per layer
        layer["one_chained_launch_per_8_layers"] = with_rates(ent8, lbytes, peaks)
        configs["1: Gemma3-4B decoder layer M=1"] = {"per_call": per_call, "per_layer": layer,
                                                     "note": "the seven projections as q|k|v, o, gate|up, down (inputs sharing x are "
                                                             "concatenated along N); independent seeded inputs, so a chain cuts the "
                                                             "layer's blocks into CTA ranges as one sequence; times per layer"}
        _, K2, N2, seed2 = synthgen.GEMMA3_12B_GATE_UP
        W2 = None
        for Mi in (1, 2, 4, 8):
            configs[f"2: Gemma3-12B gate|up K={K2} N={N2} M={Mi}"], W2 = shape_entry(K2, N2, Mi, seed2, W2)
        del W2
        _, K3, N3, seed3 = synthgen.GEMMA3_27B_DOWN
        W3 = None
        for Mi in (1, 4, 8):
            configs[f"3: Gemma3-27B down K={K3} N={N3} M={Mi}"], W3 = shape_entry(K3, N3, Mi, seed3, W3, amp=K3 ** -0.5)
        del W3
        ent = time_region(torch, stream, lambda i: fd.fdqp_run(ctx, hx, hW, hy, 1, hk, hn, sraw), 1, regions)
        ent["launch"] = fd.fdqp_describe(ctx, 1, hk, hn)
        configs[f"4: Gemma3-4B LM head K={hk} N={hn} M=1"] = with_rates(ent, step_bytes, peaks)

        # ---- decode tokens/s, projections only: 34 layers + LM head (attention, norms and sampling are out of scope)
        L = synthgen.GEMMA3_4B_LAYERS
        head_steps = [fd.chain_step(hx, hW, hy, hk, hn)]
        token_chain = fd.make_chain([fd.chain_step(xs[j], layer_copies[l % LAYER_COPIES][j], ys[j], K, N)
                                     for l in range(L) for j, (_, K, N, _) in enumerate(shapes)] + head_steps)
        n_before = fd.fdqp_launch_count(ctx)
        fd.fdqp_run_chain(ctx, token_chain, 1, sraw)
        token_launches = fd.fdqp_launch_count(ctx) - n_before
        tok = time_region(torch, stream, lambda i: fd.fdqp_run_chain(ctx, token_chain, 1, sraw), 1, regions, pairs=40)
        token_bytes = L * lbytes + step_bytes

        def token_single(i):
            for l in range(L):
                layer_single(l)
            fd.fdqp_run(ctx, hx, hW, hy, 1, hk, hn, sraw)

        tok1 = time_region(torch, stream, token_single, 1, regions, pairs=40)
        decode = {"chained": dict(with_rates(tok, token_bytes, peaks), tokens_per_s=1e6 / tok["us_back_to_back"],
                                  launches_per_token=token_launches),
                  "single_calls": dict(with_rates(tok1, token_bytes, peaks), tokens_per_s=1e6 / tok1["us_back_to_back"],
                                       launches_per_token=5 * L + 1),
                  "bytes_per_token": token_bytes, "roofline_tokens_per_s": peaks["hbm_gbs"] * 1e9 / token_bytes}

        # ---- batched decode at M = 8: the layer as single calls and chained, and the LM head
        M8 = 8
        xs8 = [torch.from_numpy(synthgen.activations(seed, M8, K).view(np.int16)).cuda() for _, K, _, seed in shapes]
        ys8 = [torch.empty((M8, N), dtype=torch.float32, device="cuda") for _, _, N, _ in shapes]

        def layer8(i):
            for j, (_, K, N, _) in enumerate(shapes):
                fd.fdqp_run(ctx, xs8[j], layer_copies[i % LAYER_COPIES][j], ys8[j], M8, K, N, sraw)

        chain8_m8 = fd.make_chain([fd.chain_step(xs8[j], layer_copies[c][j], ys8[j], K, N)
                                   for c in range(LAYER_COPIES) for j, (_, K, N, _) in enumerate(shapes)])
        b_single = with_rates(time_region(torch, stream, layer8, LAYER_COPIES, regions), layer_bytes(M8), peaks)
        b_chain = time_region(torch, stream, lambda i: fd.fdqp_run_chain(ctx, chain8_m8, M8, sraw), 1, regions)
        for k in ("us_median", "us_min", "us_p90", "us_back_to_back"):
            b_chain[k] /= LAYER_COPIES
        b_chain = with_rates(b_chain, layer_bytes(M8), peaks)
        hx8 = torch.from_numpy(synthgen.activations(hseed, M8, hk).view(np.int16)).cuda()
        hy8 = torch.empty((M8, hn), dtype=torch.float32, device="cuda")
        b_head = with_rates(time_region(torch, stream, lambda i: fd.fdqp_run(ctx, hx8, hW, hy8, M8, hk, hn, sraw), 1, regions),
                            alg_bytes(M8, hk, hn), peaks)
        batch8 = {"M": M8, "layer_single_calls": b_single, "layer_chained_8_per_launch": b_chain, "lm_head": b_head,
                  "decode_tokens_per_s": M8 * 1e6 / (L * b_chain["us_back_to_back"] + b_head["us_back_to_back"])}
        del xs8, ys8, hx8, hy8

        # ---- LM head at a prefill chunk (M = 512): the tensor-core path, against the tensor roofline
        pctx = fd.fdqp_create(local_rank, 512, hk, hn)
        px = torch.from_numpy(synthgen.activations(hseed, 512, hk).view(np.int16)).cuda()
        py = torch.empty((512, hn), dtype=torch.float32, device="cuda")
        prefill = {}
        for pm in (512, 128, 32):
            ent = time_region(torch, stream, lambda i, pm=pm: fd.fdqp_run(pctx, px, hW, py, pm, hk, hn, sraw), 1, regions, pairs=24)
            ent["launch"] = fd.fdqp_describe(pctx, pm, hk, hn)
            prefill[f"M={pm}"] = with_rates(ent, alg_bytes(pm, hk, hn), peaks, flops=2.0 * pm * hk * hn)
        # the same call with bf16 outputs (what a prefill pipeline hands on): the fp32 result of M = 512 is 537 MB of stores
        py16 = torch.empty((512, hn), dtype=torch.bfloat16, device="cuda")
        ent = time_region(torch, stream, lambda i: fd.fdqp_run_epilogue(pctx, px, hW, py16, fd.EPI_BF16, 512, hk, hn, sraw), 1, regions, pairs=24)
        prefill["M=512, bf16 outputs"] = with_rates(ent, alg_bytes(512, hk, hn) - 2.0 * 512 * hn, peaks, flops=2.0 * 512 * hk * hn)
        if fd.fdqp_last_status(pctx) != 0:
            raise SystemExit("bench.py: the prefill kernel reported " + fd.fdqp_status_string(fd.fdqp_last_status(pctx)))
        fd.fdqp_destroy(pctx)
        del px, py, py16
        configs[f"4: Gemma3-4B LM head K={hk} N={hn} M=512 (tensor cores)"] = prefill["M=512"]

        # ---- next steps beside the projection: decode attention, format variants, the dequantisation engine
        H, G, d, Lc = 8, 4, 256, 32768
        ncache = max(1, int(np.ceil(4 * L2_BYTES / (2 * G * Lc * d * 2))))
        gen = torch.Generator(device="cuda").manual_seed(2)
        caches = [(torch.randn((G, Lc, d), device="cuda", generator=gen).to(torch.bfloat16),
                   torch.randn((G, Lc, d), device="cuda", generator=gen).to(torch.bfloat16)) for _ in range(ncache)]
        aq = torch.randn((H, d), device="cuda", generator=gen).to(torch.bfloat16)
        ao = torch.empty((H, d), dtype=torch.float32, device="cuda")
        attention = {"workload": f"Gemma3-4B decode attention, H={H} G={G} d={d}, L={Lc}"}
        for name, window in (("global", 0), ("window_1024", 1024)):
            ent = time_region(torch, stream, lambda i, window=window: fd.fdqp_flowkv_decode(
                ctx, aq, caches[i % ncache][0], caches[i % ncache][1], ao, H, G, d, Lc, Lc, window, d ** -0.5, sraw), ncache, regions)
            attention[name] = with_rates(ent, 2.0 * G * (window if window else Lc) * d * 2, peaks)
        del caches
        formats = {"workload": f"LM head K={hk} N={hn} at M=1, bytes of the format's own container"}
        for name, fmt in (("g64", fd.FMT_G64), ("g128", fd.FMT_G128), ("mxfp4", fd.FMT_MXFP4)):
            fW = tiled_weights(fd, torch, hk, hn, hseed, fmt)
            ent = time_region(torch, stream, lambda i, fmt=fmt, fW=fW: fd.fdqp_run_fmt(ctx, fmt, hx, fW, hy, 1, hk, hn, sraw), 1, regions, pairs=40)
            formats[name] = with_rates(ent, fW.numel() + 2 * hk + 4 * hn, peaks)
            del fW
        dq_out = torch.empty((hk, hn), dtype=torch.bfloat16, device="cuda")
        ent = time_region(torch, stream, lambda i: fd.fdqp_dequant(ctx, hW, dq_out, True, hk, hn, sraw), 1, regions, pairs=24)
        dequant = with_rates(ent, (0.625 + 2.0) * hk * hn, peaks)
        dequant["workload"] = f"LM head K={hk} N={hn} -> bf16 [K][N]"
        del dq_out
        # ---- what the weight stream could reach at most: the same bulk-copy ring with nothing behind it, over 2 GiB
        probe_bytes = 2 << 30
        probe = torch.empty(probe_bytes, dtype=torch.uint8, device="cuda")
        ent = time_region(torch, stream, lambda i: fd.fdqp_stream_read(ctx, probe, probe_bytes, sraw), 1, regions, pairs=24)
        read_ref = with_rates(ent, float(probe_bytes // 40960 * 40960), peaks)
        read_ref["workload"] = "2 GiB read once by fdqp_stream_read (bulk copies into a shared-memory ring, data dropped)"
        del probe
        if fd.fdqp_last_status(ctx) != 0:
            raise SystemExit("bench.py: a kernel reported " + fd.fdqp_status_string(fd.fdqp_last_status(ctx)))
        line_extra = {"read_stream_reference": read_ref, "configs": configs, "decode_tokens": decode, "decode_tokens_per_s": decode["chained"]["tokens_per_s"],
                      "batched_decode": batch8, "prefill_lm_head": prefill, "decode_attention": attention,
                      "format_variants": formats, "dequant_engine": dequant}

    clocks_all = sampler.stop() if sampler is not None else None

    # ---- CPU baseline: the oracle on the host cores over the same LM head (rank 0, N = 1 only): all cores, then one
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        import oracle
        cores = min(oracle.max_threads(), os.cpu_count() or 1)
        t0 = time.perf_counter()
        passes = 0
        while passes < 1 or time.perf_counter() - t0 < 8:
            oracle.project(hx_host, hw.codes, hw.scales, hw.offsets, nthreads=cores)
            passes += 1
        dt = time.perf_counter() - t0
        n1 = 8192                                                      # single thread: a 1/32 column sample
        t0 = time.perf_counter()
        oracle.project(hx_host, hw.codes, hw.scales, hw.offsets, n0=0, n1=n1, nthreads=1)
        dt1 = time.perf_counter() - t0
        cpu = {"value": step_bytes * passes / dt / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle",
               "sample": f"{passes} pass(es) over all {hn} outputs of the LM head, {dt:.1f} s",
               "single_thread": {"value": alg_bytes(1, hk, n1) / dt1 / 1e9, "unit": "GB/s", "cores": 1,
                                 "sample": f"outputs 0..{n1 - 1} of the LM head, {dt1:.1f} s"}}

    if rank == 0:
        line = {
            "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": head_us * 1e-3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": WORKLOAD, "M": M, "K": hk, "N": hn, "bytes_per_step": step_bytes,
                       "launches_per_step": kernels_per_step, "timed_steps": timed_steps,
                       "timing": f"{blocks} replays of a CUDA graph of exactly --steps = {args.steps} calls, CUDA events on the launching stream",
                       "l2": "inputs larger than L2: every step streams 419 MB of weights through a 126 MB L2",
                       "multi_gpu": "independent replicas, no collective",
                       "launch": fd.fdqp_describe(ctx, 1, hk, hn)},
            "frac_of_nominal_8TBps": gbs / world / NOMINAL_HBM_GBS,
            "roofline": {"bound": "hbm", "achieved": step_bytes / head_us / 1e3, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": step_bytes / head_us / 1e3 / peaks["hbm_gbs"],
                         # one ncu capture of this launch: dram__bytes_read.sum + dram__bytes_write.sum
                         "traffic": NCU_LM_HEAD_DRAM_BYTES, "peak_kind": peak_kind + " copy bandwidth",
                         "kernel": "fdqp_gemv_kernel<16,1,4,false,Q4NX>", "launch_us": head_us},
            "cpu_baseline": cpu,
            "e2e": {"value": whole_job_gbs(step_bytes, e2e_steps, world, e2e_s * 1e3), "unit": "GB/s",
                    "h2d_bytes_per_step": 2 * M * hk, "d2h_bytes_per_step": 4 * M * hn, "ms_per_step": e2e_s / e2e_steps * 1e3,
                    "how": "fdqp_run_host_async on pinned host buffers + one stream synchronisation per step"},
            "gpu_launches": kernels_per_step * timed_steps,
            "clocks": head_clocks or clocks_all,
        }
        line.update(line_extra)
        print(json.dumps(line), flush=True)
    fd.fdqp_destroy(ctx)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
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
    ap.add_argument("--layer-chain", type=int, default=0,
                    help="time the Gemma3-4B layer as chained launches of this many layers each (fdqp_run_chain) instead")
    ap.add_argument("--tokens", type=int, default=1, help="with --layer-chain: token rows M (1 .. 8)")
    ap.add_argument("--headline-only", action="store_true", help="only the headline workload (no per-configuration table)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        if args.steps == 200 and args.warmup == 10:
            args.steps, args.warmup = 20, 2
        run_reference(args, rank, world)
        return
    if args.warmup < 3:
        args.warmup = 3
    if args.dequant:
        if args.steps == 200:
            args.steps = 10
        run_dequant(args)
        return
    if args.flowkv:
        if args.steps == 200:
            args.steps = 50
        run_flowkv(args)
        return
    if args.layer_chain:
        if args.steps == 200:
            args.steps = 50
        run_layer_chain(args)
        return
    if args.shape:
        if args.steps == 200:
            args.steps = 50
        run_shape(args)
        return
    run_ours(args, rank, local_rank, world)


if __name__ == "__main__":
    main()
