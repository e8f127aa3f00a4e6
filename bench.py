#!/usr/bin/env python
"""Benchmark of the FBQuant decode hot path on B200.

Workload (single GPU): the seven linears of one Llama-2-7B decoder layer
(q, k, v, o: 4096->4096; gate, up: 4096->11008; down: 11008->4096) at M = 1
token, INT3 codes, group 128, rank-64 fp16 sub-branch, synthetic seeded inputs.
One "step" = one pass over the seven linears of one layer instance, each a call
of fbq_linear through the C ABI.  A pool of layer instances larger than L2 is
visited round-robin, so every step streams its weights from HBM.

The timed region replays CUDA graphs captured from the C-ABI calls (one graph
holds up to 100 steps), so that Python's launch cost does not sit between
kernels that last a few microseconds.

Prints ONE JSON line (see the keys at the bottom).  `--impl reference` times
the CPU oracle on the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

BITS, RANK, GROUP, M_TOKENS = 3, 64, 128, 1
WORKLOAD = "llama2-7b decoder-layer linears, M=1, INT3 g128, rank 64 (7 linears per step)"
GRAPH_STEPS = 100
# The seven linears of a step are independent (each has its own x).  MODE "streams" (default): a
# step issues seven fbq_linear calls round-robin over N_STREAMS CUDA streams of the bench, each with
# its decode grid bounded by its share (by size) of DECODE_CTAS CTAs; the streams are joined once
# per graph, so linears of consecutive steps overlap.  MODE "batch": a step is one fbq_linear_batch
# call (the library runs the seven launches on its side streams and joins them every step).
MODE = os.environ.get("FBQ_BENCH_MODE", "streams")
N_STREAMS = int(os.environ.get("FBQ_BENCH_STREAMS", "7"))
# main CTAs shared out among the 7 linears by size: 386 gives the 4096-wide linears 32 CTAs and the 11008-wide ones
# 86, i.e. exactly eight 16-row tiles per CTA for both (256 and 688 tiles)
DECODE_CTAS = int(os.environ.get("FBQ_BENCH_CTAS", "386"))
NVSMI_FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
                "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
                "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "fallback"


def layer_shapes():
    from workloads import LLAMA2_7B_SHAPES
    return list(LLAMA2_7B_SHAPES)


def step_bytes():
    from paper_2501_16385_b200.accounting import algorithmic_bytes
    return sum(algorithmic_bytes(M_TOKENS, N, K, BITS, RANK, GROUP) for K, N in layer_shapes())


def step_bytes_rank0():
    from paper_2501_16385_b200.accounting import algorithmic_bytes
    return sum(algorithmic_bytes(M_TOKENS, N, K, BITS, 0, GROUP) for K, N in layer_shapes())


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken during the timed region."""

    def __init__(self, gpu_index: int):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + NVSMI_FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "100"], stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.tmp.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.tmp.close()
        os.unlink(self.tmp.name)
        if sm:
            sm.sort()
            out.update(sm_mhz=sm[len(sm) // 2], sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


# --------------------------------------------------------------------------- GPU arm
class PooledLinear:
    """Device tensors of one synthetic linear (codes packed on the device by fbq_pack_int3)."""

    def __init__(self, inp, fbq, torch):
        import numpy as np

        def bits16(a):
            return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda().view(torch.float16)

        self.N = inp.N
        self.qweight = fbq.pack(torch.from_numpy(inp.codes).cuda(), inp.bits)
        self.scales, self.zeros = bits16(inp.scales), bits16(inp.zeros)
        self.x, self.A, self.B = bits16(inp.x), bits16(inp.A), bits16(inp.B)
        self.y = torch.empty((inp.M, inp.N), dtype=torch.float16, device="cuda")


def build_pool(fbq, torch, n_layers: int, seed0: int = 1000):
    """Device-resident layer instances; also returns the host inputs of instance 0."""
    from workloads import make_linear
    pool, host0 = [], []
    for li in range(n_layers):
        layer = []
        for sid, (K, N) in enumerate(layer_shapes()):
            inp = make_linear(M_TOKENS, N, K, BITS, RANK, seed=seed0 + 100 * li + sid)
            layer.append(PooledLinear(inp, fbq, torch))
            if li == 0:
                host0.append(inp)
        pool.append(layer)
    return pool, host0


_SIDE_STREAMS = []


def side_streams(torch):
    while len(_SIDE_STREAMS) < N_STREAMS - 1:
        _SIDE_STREAMS.append(torch.cuda.Stream())
    return _SIDE_STREAMS


def run_step(fbq, layer, with_branch: bool = True, streams=None):
    """One step: the seven fbq_linear calls of one layer instance.  With `streams` (the
    current stream first), call j goes to stream j % len(streams)."""
    import torch
    costs = [d.N * d.x.shape[1] for d in layer]
    for j, d in enumerate(layer):
        st = streams[j % len(streams)] if streams else None
        fbq.set_option("decode_ctas", max(8, round(DECODE_CTAS * costs[j] / sum(costs))))
        fbq.linear(d.x, d.qweight, d.scales, d.zeros, d.A if with_branch else None,
                   d.B if with_branch else None, d.N, GROUP, BITS, y=d.y, stream=st)


_BATCHES = {}


def layer_batch(fbq, layer, with_branch: bool):
    """Descriptor array of one layer instance for fbq_linear_batch (made once, reused)."""
    key = (id(layer), with_branch)
    if key not in _BATCHES:
        _BATCHES[key] = fbq.make_batch([(d.x, d.qweight, d.scales, d.zeros, d.A if with_branch else None,
                                         d.B if with_branch else None, d.y) for d in layer])
    return _BATCHES[key]


def run_steps_forked(fbq, torch, pool, n_steps: int, main, with_branch: bool):
    """n_steps steps on `main`.  Batch mode: one fbq_linear_batch per step.  Streams mode: the side
    streams are forked from / joined to `main` once around all the steps."""
    if MODE == "batch":
        for i in range(n_steps):
            fbq.linear_batch(None, GROUP, BITS, stream=main, batch=layer_batch(fbq, pool[i % len(pool)], with_branch))
        return
    sides = side_streams(torch)
    streams = [main] + sides
    for st in sides:
        st.wait_stream(main)
    for i in range(n_steps):
        run_step(fbq, pool[i % len(pool)], with_branch, streams)
    for st in sides:
        main.wait_stream(st)


def capture_graph(fbq, torch, pool, n_steps: int, stream, with_branch: bool):
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        run_steps_forked(fbq, torch, pool, n_steps, stream, with_branch)
    return g


def time_graph_steps(fbq, torch, pool, steps: int, warmup: int, barrier, with_branch: bool = True):
    """Returns elapsed milliseconds for exactly `steps` steps (CUDA events on the launching stream)."""
    L = len(pool)
    chunk = max(1, min((GRAPH_STEPS // L) * L, steps))
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        # plain launches: first-call set-up and scratch growth on every stream used later
        run_steps_forked(fbq, torch, pool, min(max(warmup, 3), 2 * L), stream, with_branch)
        stream.synchronize()
        g_main = capture_graph(fbq, torch, pool, chunk, stream, with_branch)
        rem = steps % chunk
        g_rem = capture_graph(fbq, torch, pool, rem, stream, with_branch) if rem else None
        for _ in range(max(1, (max(warmup, 3) + chunk - 1) // chunk)):
            g_main.replay()
        stream.synchronize()
        barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps // chunk):
            g_main.replay()
        if g_rem is not None:
            g_rem.replay()
        e1.record(stream)
        stream.synchronize()
        torch.cuda.synchronize()
        barrier()
        return e0.elapsed_time(e1)


def time_plain_steps(fbq, torch, pool, steps: int):
    """Plain stream launches from Python (no graph): shows the host's launch cost."""
    L = len(pool)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    main = torch.cuda.current_stream()
    for i in range(steps):
        run_steps_forked(fbq, torch, pool[i % L:i % L + 1], 1, main, True)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1)


def time_e2e(fbq, torch, pool, steps: int, warmup: int):
    """Same steps end to end through the C ABI with HOST buffers: one fbq_linear_batch_hostio call per
    step (x of the seven linears from pinned host memory, y read back to pinned host memory), then a
    stream synchronise so that the step's results are on the host.  Wall clock."""
    L = len(pool)
    xs = [[d.x.cpu().pin_memory() for d in layer] for layer in pool]
    ys = [[torch.empty((M_TOKENS, d.N), dtype=torch.float16).pin_memory() for d in layer] for layer in pool]
    batches = [fbq.make_batch([(xs[li][j], d.qweight, d.scales, d.zeros, d.A, d.B, ys[li][j]) for j, d in enumerate(layer)])
               for li, layer in enumerate(pool)]
    main = torch.cuda.current_stream()

    def one(i):
        fbq.linear_batch(None, GROUP, BITS, stream=main, batch=batches[i % L], host_io=True)
        main.synchronize()                            # the step's results are read on the host

    for i in range(max(3, warmup)):
        one(i)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for i in range(steps):
        one(i)
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    h2d = sum(K * 2 * M_TOKENS for K, _ in layer_shapes())
    d2h = sum(N * 2 * M_TOKENS for _, N in layer_shapes())
    return dt, h2d, d2h


def time_naive(fbq, torch, pool, steps: int, warmup: int):
    """The paper's unfused sub-branch layer (Section 3.2 / Fig. kernel-fusion: quantised main path
    plus two separate projections and an add) on the same inputs, as a comparator: per linear
    fbq_linear at rank 0, then t = x.A^T, u = t.B^T and y += u as three library launches (torch.mm,
    torch.mm, add_) on the same stream.  Same streams, same graph replay as the fused arm."""
    sides = side_streams(torch)
    L = len(pool)
    ts = [[torch.empty((M_TOKENS, RANK), dtype=torch.float16, device="cuda") for _ in layer] for layer in pool]
    us = [[torch.empty((M_TOKENS, d.N), dtype=torch.float16, device="cuda") for d in layer] for layer in pool]
    ats = [[d.A.t() for d in layer] for layer in pool]
    bts = [[d.B.t() for d in layer] for layer in pool]

    def run(n_steps, main):
        streams = [main] + sides
        for st in sides:
            st.wait_stream(main)
        for i in range(n_steps):
            li = i % L
            layer = pool[li]
            costs = [d.N * d.x.shape[1] for d in layer]
            for j, d in enumerate(layer):
                st = streams[j % len(streams)]
                fbq.set_option("decode_ctas", max(8, round(DECODE_CTAS * costs[j] / sum(costs))))
                fbq.linear(d.x, d.qweight, d.scales, d.zeros, None, None, d.N, GROUP, BITS, y=d.y, stream=st)
                with torch.cuda.stream(st):
                    torch.mm(d.x, ats[li][j], out=ts[li][j])
                    torch.mm(ts[li][j], bts[li][j], out=us[li][j])
                    d.y.add_(us[li][j])
        for st in sides:
            main.wait_stream(st)

    chunk = max(1, min((GRAPH_STEPS // L) * L, steps))
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        run(min(max(warmup, 3), 2 * L), stream)
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            run(chunk, stream)
        g.replay()
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        reps = max(1, steps // chunk)
        for _ in range(reps):
            g.replay()
        e1.record(stream)
        stream.synchronize()
    return e0.elapsed_time(e1) / (reps * chunk)


def time_prefill(fbq, torch, peaks, steps: int = 20, warmup: int = 3):
    """Secondary figure: the same seven linears at M = 1024, INT4, rank 64, bf16 with 1 % outlier
    channels (the prefill configuration), through fbq_linear_bf16 on one stream.  Two layer instances
    (2 x 118 MB) alternate, so operands come from HBM.  CUDA events on the launching stream."""
    from paper_2501_16385_b200.accounting import algorithmic_flops
    from paper_2501_16385_b200.microbench import make_instance
    M, bits, rank = 1024, 4, RANK
    pool = [[make_instance(M, N, K, bits, rank, "bf16", 7000 + 10 * li + sid, outlier_frac=0.01)
             for sid, (K, N) in enumerate(layer_shapes())] for li in range(2)]
    flops = sum(algorithmic_flops(M, N, K, rank) for K, N in layer_shapes())

    def step(i):
        for t in pool[i % 2]:
            fbq.linear(t["x"], t["qweight"], t["scales"], t["zeros"], t["A"], t["B"], t["y"].shape[1], GROUP, bits, y=t["y"])

    for i in range(warmup):
        step(i)
    torch.cuda.synchronize()
    before = fbq.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        step(i)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    launches = (fbq.launch_count() - before) / steps
    assert fbq.poll_status() == 0
    del pool
    torch.cuda.empty_cache()
    tf = flops / (ms * 1e-3) / 1e12
    return {"workload": "llama2-7b decoder-layer linears, M=1024, INT4 g128, rank 64, bf16, 1% outlier channels",
            "ms_per_step": ms, "tflops": tf, "steps": steps, "launches_per_step": launches,
            "roofline": {"bound": "tensor", "achieved": tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                         "frac": tf / peaks["bf16_tflops"], "kernel": "prefill_kernel<4,__nv_bfloat16,256>",
                         "algorithmic_flops_per_step": flops}}


def oracle_step_seconds(host0, reps: int):
    import oracle
    threads = oracle.max_threads()
    packed = [oracle.pack(inp.codes, inp.bits) for inp in host0]
    best = float("inf")
    for _ in range(reps):
        t0 = time.perf_counter()
        for inp, q in zip(host0, packed):
            oracle.linear_inputs(inp, qweight=q, threads=threads)
        best = min(best, time.perf_counter() - t0)
    return best, threads


def gpu_arm(args):
    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank_id = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()

    import paper_2501_16385_b200 as fbq
    if os.environ.get("FBQ_BATCH_CTAS"):
        fbq.set_option("batch_ctas", int(os.environ["FBQ_BATCH_CTAS"]))
    peaks, peak_kind = measured_peaks()
    bytes_step = step_bytes()
    pool_layers = max(2, -(-3 * 126_000_000 // bytes_step))        # pool >= 3 x L2 (126 MB)
    pool, host0 = build_pool(fbq, torch, pool_layers)

    sampler = ClockSampler(local) if rank_id == 0 else None
    ms = time_graph_steps(fbq, torch, pool, args.steps, args.warmup, barrier)
    clocks = sampler.stop() if sampler else None
    if world > 1:
        t = torch.tensor([ms], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    n_linears = len(layer_shapes())
    value = world * bytes_step * args.steps / (ms * 1e-3) / 1e9            # GB/s, whole job

    extra = {}
    if rank_id == 0:
        # sub-branch overhead: the same kernel on the same weights with rank 0
        ms0 = time_graph_steps(fbq, torch, pool, args.steps, args.warmup, lambda: None, with_branch=False)
        extra["rank0_ms_per_step"] = ms0 / args.steps
        extra["rank0_GBs"] = step_bytes_rank0() * args.steps / (ms0 * 1e-3) / 1e9
        extra["sub_branch_overhead"] = (ms / ms0 - 1.0) if world == 1 else None
        extra["byte_floor_overhead"] = bytes_step / step_bytes_rank0() - 1.0
        if world == 1 and MODE == "streams":
            naive_ms = time_naive(fbq, torch, pool, min(args.steps, 4000), args.warmup)
            fused_ms, r0_ms = ms / args.steps, ms0 / args.steps
            extra["naive_sub_branch"] = {
                "what": "rank-0 fbq_linear + torch.mm + torch.mm + add_ per linear (4 launches), same streams and graph replay",
                "ms_per_step": naive_ms, "slowdown_vs_fused": naive_ms / fused_ms,
                "overhead_vs_rank0": naive_ms / r0_ms - 1.0,
                "extra_latency_removed_by_fusion": 1.0 - (fused_ms - r0_ms) / (naive_ms - r0_ms) if naive_ms > r0_ms else None}
        plain_steps = min(args.steps, 2000)
        extra["plain_launch_ms_per_step"] = time_plain_steps(fbq, torch, pool, plain_steps) / plain_steps
        e2e_steps = min(args.steps, 500)
        dt, h2d, d2h = time_e2e(fbq, torch, pool, e2e_steps, 3)
        e2e_val = bytes_step * e2e_steps / dt / 1e9
        cpu_s, cores = oracle_step_seconds(host0, 3) if world == 1 else (None, None)
        if world == 1:
            del pool
            torch.cuda.empty_cache()
            extra["prefill"] = time_prefill(fbq, torch, peaks)
    barrier()
    if rank_id != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    line = {
        "metric": "effective HBM GB/s per linear at M=1 (algorithmic bytes / time)",
        "value": value,
        "unit": "GB/s",
        "n_gpus": world,
        "steps": args.steps,
        "warmup": args.warmup,
        "ms_per_step": ms / args.steps,
        "us_per_linear": ms * 1e3 / args.steps / n_linears,
        "pct_of_8TBs": 100.0 * value / world / 8000.0,
        "higher_is_better": True,
        "scaling": "weak",
        "vs_baseline": None,
        "dtype": "f16",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "bits": BITS, "rank": RANK, "group": GROUP, "M": M_TOKENS,
                   "linears_per_step": n_linears, "pool_layers": pool_layers,
                   "cold": "pool of %d layer instances (%.0f MB) > 3x L2, visited round-robin" %
                           (pool_layers, pool_layers * bytes_step / 1e6),
                   "launch": ("CUDA graph replay of one fbq_linear_batch call per step (7 concurrent decode launches on "
                              "the library's side streams, %d CTAs shared out by size, joined every step)"
                              % fbq.get_option("batch_ctas")) if MODE == "batch" else
                             ("CUDA graph replay of fbq_linear calls (programmatic dependent launch); the 7 "
                              "independent linears of a step go round-robin over %d streams, decode grids share %d CTAs by size"
                              % (N_STREAMS, DECODE_CTAS)),
                   "parallelism": "replicas only (no collective on the path)" if world > 1 else "1 GPU"},
        "gpu_launches": args.steps * n_linears,       # one fused decode launch per linear per step
        "roofline": {"bound": "hbm", "achieved": value / world, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": value / world / peaks["hbm_gbs"], "of": peak_kind,
                     "kernel": "decode_kernel<3,__half,1,light,int8>",
                     "algorithmic_bytes_per_step": bytes_step, "traffic": TRAFFIC_BYTES_PER_STEP},
        "clocks": clocks,
        "e2e": {"value": e2e_val, "unit": "GB/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": dt * 1e3 / e2e_steps, "steps": e2e_steps},
    }
    line.update(extra)
    if cpu_s is not None:
        line["cpu_baseline"] = {"value": bytes_step / cpu_s / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle",
                                "sample": "1 step (7 linears, all output rows), best of 3, %.3f s" % cpu_s}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# DRAM bytes (read + write) per step measured with ncu (--set full) on the seven decode
# launches of one step: 4 x 7.971 MB + 2 x 20.357 MB + 20.369 MB
# (profiles/decode_int3_r64_m1_bench.md).
TRAFFIC_BYTES_PER_STEP = 92_969_000


# ---------------------------------------------------------------------- reference arm
def reference_arm(args):
    """The CPU oracle, as it stands, on the same workload (reported baseline)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from workloads import make_linear
    import oracle
    host0 = [make_linear(M_TOKENS, N, K, BITS, RANK, seed=1000 + sid) for sid, (K, N) in enumerate(layer_shapes())]
    packed = [oracle.pack(i.codes, i.bits) for i in host0]
    threads = oracle.max_threads()
    steps = min(args.steps, 20)           # bounded: a step is ~0.1-0.5 s of host work
    warm = min(args.warmup, 2)

    def one():
        for inp, q in zip(host0, packed):
            oracle.linear_inputs(inp, qweight=q, threads=threads)

    for _ in range(warm):
        one()
    t0 = time.perf_counter()
    for _ in range(steps):
        one()
    dt = time.perf_counter() - t0
    value = step_bytes() * steps / dt / 1e9
    print(json.dumps({
        "impl": "reference", "metric": "effective HBM GB/s per linear at M=1 (algorithmic bytes / time)",
        "value": value, "unit": "GB/s", "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": steps,
        "warmup": warm, "ms_per_step": dt * 1e3 / steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "bits": BITS, "rank": RANK, "group": GROUP, "M": M_TOKENS},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": threads, "kind": "oracle",
                         "sample": "%d steps of 7 linears (all output rows)" % steps},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20000)
    ap.add_argument("--warmup", type=int, default=200)
    ap.add_argument("--impl", default="fbq", choices=["fbq", "reference"])
    args = ap.parse_args()
    if args.impl == "reference":
        reference_arm(args)
    else:
        gpu_arm(args)


if __name__ == "__main__":
    main()
