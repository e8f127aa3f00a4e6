#!/usr/bin/env python
"""Benchmark of the FBQuant inference linear on B200.

Default workload (--config 1, single GPU): the seven linears of one Llama-2-7B
decoder layer (q, k, v, o: 4096->4096; gate, up: 4096->11008; down:
11008->4096) at M = 1 token, INT3 codes, group 128, rank-64 fp16 sub-branch,
synthetic seeded inputs.  One "step" = one pass over the seven linears of one
layer instance, each a call of fbq_linear through the C ABI.  A pool of layer
instances larger than L2 is visited round-robin, so every step streams its
weights from HBM.

Launch schemes ("arms"), all timed the same way (CUDA-graph replay of the C-ABI
calls, CUDA events on the launching stream, every timed region of exactly
--steps steps repeated until at least 50 ms of GPU time have passed, median
reported):
  sequential           the seven calls of a step on ONE stream in layer order
                       (programmatic dependent launch on; also with it off).
                       This is the headline: a decoder runs its projections in
                       dependency order.
  layer_order          {q,k,v} side by side, then o, then {gate,up} side by
                       side, then down: the most overlap a decoder layer allows.
  independent_streams  the seven linears as mutually independent launches on
                       seven streams, joined once per graph (an upper bound on
                       throughput, not reachable by one decoder).
  per_shape            each of the three shapes alone, call after call on one
                       stream, with and without the sub-branch.

Prints ONE JSON line.  `--impl reference` times the CPU oracle on the same
workload instead.  --config selects the other workloads of the benchmark spec:
0 single 4096x4096 INT4 rank-32 linear, 2 the prefill layer (M = 1024, INT4,
bf16), 3 Llama-2-13B shapes (M in {1, 16}, INT3 and INT4), 4 the decode sweep
M x rank (INT4) over the 7B layer.
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

GROUP = 128
GRAPH_STEPS = 100            # steps per captured graph, at most
MIN_TIMED_MS = 50.0          # every arm repeats its timed region until this much GPU time has passed
N_STREAMS = 7
# main CTAs shared out among the 7 linears of the independent_streams arm by size
DECODE_CTAS = int(os.environ.get("FBQ_BENCH_CTAS", "386"))
NVSMI_FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
                "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
                "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
# phases of a decoder layer: linears of one phase may run side by side, phases run in order
LAYER_PHASES = [[0, 1, 2], [3], [4, 5], [6]]


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "fallback"


class Workload:
    """A decode-sized workload: the (K, N) shapes of one step in call order."""

    def __init__(self, name, shapes, bits, rank, M, phases=None, seed0=1000):
        self.name, self.shapes, self.bits, self.rank, self.M = name, list(shapes), bits, rank, M
        self.phases = phases or [[i] for i in range(len(self.shapes))]
        self.seed0 = seed0

    def step_bytes(self, rank=None):
        from paper_2501_16385_b200.accounting import algorithmic_bytes
        r = self.rank if rank is None else rank
        return sum(algorithmic_bytes(self.M, N, K, self.bits, r, GROUP) for K, N in self.shapes)


def workload_for(config: int, M=None, bits=None, rank=None) -> Workload:
    from workloads import LLAMA2_7B_SHAPES, LLAMA2_13B_SHAPES
    if config == 0:
        return Workload("single linear 4096->4096, M=1, INT4 g128, rank 32", [(4096, 4096)], 4, 32, 1, seed0=0)
    if config == 3:
        b, m = bits or 3, M or 1
        return Workload("llama2-13b decoder-layer linears, M=%d, INT%d g128, rank 64 (7 linears per step)" % (m, b),
                        LLAMA2_13B_SHAPES, b, 64, m, LAYER_PHASES, seed0=3000)
    if config == 4:
        m, r = M or 1, 64 if rank is None else rank
        return Workload("llama2-7b decoder-layer linears, M=%d, INT4 g128, rank %d (7 linears per step)" % (m, r),
                        LLAMA2_7B_SHAPES, 4, r, m, LAYER_PHASES, seed0=4000)
    return Workload("llama2-7b decoder-layer linears, M=1, INT3 g128, rank 64 (7 linears per step)",
                    LLAMA2_7B_SHAPES, 3, 64, 1, LAYER_PHASES, seed0=1000)


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken during the timed regions."""

    def __init__(self, gpu_index: int):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + NVSMI_FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"], stdout=self.tmp, stderr=subprocess.DEVNULL)
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
    """Device tensors of one synthetic linear (codes packed on the device by fbq_pack_int3/4)."""

    def __init__(self, inp, fbq, torch):
        import numpy as np

        def bits16(a):
            t = torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda()
            return t.view(torch.bfloat16 if inp.dtype == "bf16" else torch.float16)

        def f16(a):
            return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda().view(torch.float16)

        self.N, self.K = inp.N, inp.K
        self.qweight = fbq.pack(torch.from_numpy(inp.codes).cuda(), inp.bits)
        self.scales, self.zeros = f16(inp.scales), f16(inp.zeros)
        self.x = bits16(inp.x)
        self.A = bits16(inp.A) if inp.rank > 0 else None
        self.B = bits16(inp.B) if inp.rank > 0 else None
        self.y = torch.empty((inp.M, inp.N), dtype=self.x.dtype, device="cuda")


def build_pool(fbq, torch, wl: Workload, n_layers: int):
    """Device-resident layer instances; also returns the host inputs of instance 0."""
    from workloads import make_linear
    pool, host0 = [], []
    for li in range(n_layers):
        layer = []
        for sid, (K, N) in enumerate(wl.shapes):
            inp = make_linear(wl.M, N, K, wl.bits, max(wl.rank, 8), seed=wl.seed0 + 100 * li + sid)
            layer.append(PooledLinear(inp, fbq, torch))
            if li == 0:
                host0.append(inp)
        pool.append(layer)
    return pool, host0


def call_linear(fbq, wl, d, with_branch, stream=None):
    fbq.linear(d.x, d.qweight, d.scales, d.zeros, d.A if with_branch else None, d.B if with_branch else None,
               d.N, GROUP, wl.bits, y=d.y, stream=stream)


class Arms:
    """The launch schemes.  issue_*(i, main) queues step i (layer instance i % len(pool))."""

    def __init__(self, fbq, torch, wl, pool):
        self.fbq, self.torch, self.wl, self.pool = fbq, torch, wl, pool
        self.sides = [torch.cuda.Stream() for _ in range(N_STREAMS - 1)]
        self.events = [torch.cuda.Event() for _ in range(16)]

    def sequential(self, with_branch=True, only=None):
        def issue(i, main):
            for j, d in enumerate(self.pool[i % len(self.pool)]):
                if only is None or j in only:
                    call_linear(self.fbq, self.wl, d, with_branch, main)
        return issue

    def layer_order(self, with_branch=True):
        def issue(i, main):
            layer = self.pool[i % len(self.pool)]
            for phase in self.wl.phases:
                if len(phase) > 1:
                    fork = self.torch.cuda.Event()
                    fork.record(main)
                for n, j in enumerate(phase):
                    st = main if n == 0 else self.sides[n - 1]
                    if n > 0:
                        st.wait_event(fork)
                    call_linear(self.fbq, self.wl, layer[j], with_branch, st)
                for n in range(1, len(phase)):
                    main.wait_stream(self.sides[n - 1])
        return issue

    def independent(self, with_branch=True):
        costs = [K * N for K, N in self.wl.shapes]

        def issue(i, main):
            streams = [main] + self.sides
            for j, d in enumerate(self.pool[i % len(self.pool)]):
                self.fbq.set_option("decode_ctas", max(8, round(DECODE_CTAS * costs[j] / sum(costs))))
                call_linear(self.fbq, self.wl, d, with_branch, streams[j % len(streams)])
            self.fbq.set_option("decode_ctas", 0)
        return issue


def run_region(torch, issue, n_steps, main, sides, first=0):
    """n_steps steps on `main`; the side streams are forked from / joined to it around all of them."""
    for st in sides:
        st.wait_stream(main)
    for i in range(n_steps):
        issue(first + i, main)
    for st in sides:
        main.wait_stream(st)


def time_arm(torch, issue, pool_len, steps, warmup, sides, barrier=lambda: None, min_ms=MIN_TIMED_MS):
    """Median milliseconds of a region of exactly `steps` steps (CUDA events on the launching
    stream around graph replays), the region repeated until min_ms of GPU time have passed."""
    L = pool_len
    chunk = max(1, min(max(L, (GRAPH_STEPS // L) * L), steps))
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        # plain launches first: first-call set-up and scratch growth on every stream used later
        run_region(torch, issue, min(max(warmup, 3), 2 * L), stream, sides)
        stream.synchronize()

        def capture(n, first):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                run_region(torch, issue, n, stream, sides, first)
            return g

        g_main = capture(chunk, 0)
        rem = steps % chunk
        g_rem = capture(rem, 0) if rem else None

        def region():
            for _ in range(steps // chunk):
                g_main.replay()
            if g_rem is not None:
                g_rem.replay()

        for _ in range(max(1, -(-max(warmup, 3) // steps))):
            region()
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        region()
        e1.record(stream)
        stream.synchronize()
        first_ms = max(e0.elapsed_time(e1), 1e-3)
        reps = int(min(max(3, -(-min_ms // first_ms)), 5000))
        barrier()
        torch.cuda.synchronize()
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        for a, b in evs:
            a.record(stream)
            region()
            b.record(stream)
        stream.synchronize()
        torch.cuda.synchronize()
        barrier()
        times = sorted(a.elapsed_time(b) for a, b in evs)
    del g_main, g_rem
    return {"ms": times[len(times) // 2], "repeats": reps, "min_ms": times[0], "max_ms": times[-1],
            "timed_ms_total": sum(times)}


def time_plain_steps(torch, issue, steps):
    """Plain stream launches from Python (no graph): shows the host's launch cost."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    main = torch.cuda.current_stream()
    e0.record()
    for i in range(steps):
        issue(i, main)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1)


E2E_WARM_S = 0.3          # untimed end-to-end steps before the clock starts (seconds of wall time, at least `warmup` steps)


def time_e2e(fbq, torch, wl, pool, steps: int, warmup: int, batched: bool = False):
    """Same steps end to end through the C ABI with HOST buffers (x from pinned host memory, y read back to
    pinned host memory), then a stream synchronise so that the step's results are on the host.  Wall clock.
    Per linear one fbq_linear_hostio call in layer order on one stream; or, `batched`, one
    fbq_linear_batch_hostio call per step (the library runs the problems on streams of its own, so their
    small copies overlap)."""
    L = len(pool)
    xs = [[d.x.cpu().pin_memory() for d in layer] for layer in pool]
    ys = [[torch.empty((wl.M, d.N), dtype=d.x.dtype).pin_memory() for d in layer] for layer in pool]
    main = torch.cuda.current_stream()
    batches = None
    if batched:
        batches = [fbq.make_batch([(xs[li][j], d.qweight, d.scales, d.zeros, d.A, d.B, ys[li][j]) for j, d in enumerate(pool[li])])
                   for li in range(L)]

    def one(i):
        li = i % L
        if batched:
            fbq.linear_batch(None, GROUP, wl.bits, stream=main, batch=batches[li], host_io=True)
        else:
            for j, d in enumerate(pool[li]):
                fbq.linear_hostio(xs[li][j], d.qweight, d.scales, d.zeros, d.A, d.B, ys[li][j], d.N, GROUP, wl.bits, stream=main)
        main.synchronize()                            # the step's results are read on the host

    # Untimed steps until the path has settled: on this host the first tenths of a second of such steps (small copies and
    # kernel writes across the bus, a synchronise per step) run about 30 % slower than all later ones.
    tw, nw = time.perf_counter(), 0
    while nw < max(3, warmup) or time.perf_counter() - tw < E2E_WARM_S:
        one(nw)
        nw += 1
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for i in range(steps):
        one(nw + i)
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    h2d = sum(K * 2 * wl.M for K, _ in wl.shapes)
    d2h = sum(N * 2 * wl.M for _, N in wl.shapes)
    return dt, h2d, d2h


def naive_issue(fbq, torch, wl, pool):
    """The paper's unfused sub-branch layer (Section 3.2 / Fig. kernel-fusion: quantised main path plus
    two separate projections and an add) on the same inputs, as a comparator: per linear fbq_linear at
    rank 0, then the library's own unfused sub-branch launches (fbq_sub_branch_unfused: t = x.A^T, then
    y += t.B^T), on one stream in layer order."""
    def issue(i, main):
        for d in pool[i % len(pool)]:
            call_linear(fbq, wl, d, False, main)
            fbq.sub_branch_unfused(d.x, d.A, d.B, d.y, stream=main)
    return issue


def time_prefill(fbq, torch, peaks, steps: int = 20, warmup: int = 3):
    """The prefill configuration: the same seven linears at M = 1024, INT4, rank 64, bf16 with 1 % outlier
    channels, through fbq_linear_bf16 on one stream.  Two layer instances (2 x 118 MB) alternate, so
    operands come from HBM.  CUDA events on the launching stream."""
    from paper_2501_16385_b200.accounting import algorithmic_flops
    from paper_2501_16385_b200.microbench import make_instance
    from workloads import LLAMA2_7B_SHAPES
    M, bits, rank = 1024, 4, 64
    pool = [[make_instance(M, N, K, bits, rank, "bf16", 7000 + 10 * li + sid, outlier_frac=0.01)
             for sid, (K, N) in enumerate(LLAMA2_7B_SHAPES)] for li in range(2)]
    flops = sum(algorithmic_flops(M, N, K, rank) for K, N in LLAMA2_7B_SHAPES)

    def step(i):
        for t in pool[i % 2]:
            fbq.linear(t["x"], t["qweight"], t["scales"], t["zeros"], t["A"], t["B"], t["y"].shape[1], GROUP, bits, y=t["y"])

    for i in range(warmup):
        step(i)
    torch.cuda.synchronize()
    before = fbq.launch_count()
    times = []
    total = 0.0
    while total < MIN_TIMED_MS or len(times) < 3:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(steps):
            step(i)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
        total += times[-1]
    times.sort()
    ms = times[len(times) // 2] / steps
    launches = (fbq.launch_count() - before) / (steps * len(times))
    assert fbq.poll_status() == 0
    per_shape = {}
    for sid, name in ((0, "4096->4096"), (4, "4096->11008"), (6, "11008->4096")):
        K, N = LLAMA2_7B_SHAPES[sid]
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 40
        e0.record()
        for i in range(reps):
            t = pool[i % 2][sid]
            fbq.linear(t["x"], t["qweight"], t["scales"], t["zeros"], t["A"], t["B"], N, GROUP, bits, y=t["y"])
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / reps
        tfs = algorithmic_flops(M, N, K, rank) / us / 1e6
        per_shape[name] = {"us": us, "tflops": tfs, "frac": tfs / peaks["bf16_tflops"]}
    del pool
    torch.cuda.empty_cache()
    tf = flops / (ms * 1e-3) / 1e12
    return {"workload": "llama2-7b decoder-layer linears, M=1024, INT4 g128, rank 64, bf16, 1% outlier channels",
            "ms_per_step": ms, "tflops": tf, "steps": steps, "repeats": len(times), "launches_per_step": launches,
            "per_shape": per_shape,
            "roofline": {"bound": "tensor", "achieved": tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                         "frac": tf / peaks["bf16_tflops"], "kernel": "prefill_kernel<4,__nv_bfloat16,256>",
                         "algorithmic_flops_per_step": flops}}


def oracle_step_seconds(host0, reps: int, threads=None):
    import oracle
    threads = threads or oracle.max_threads()
    packed = [oracle.pack(inp.codes, inp.bits) for inp in host0]
    best = float("inf")
    for _ in range(reps):
        t0 = time.perf_counter()
        for inp, q in zip(host0, packed):
            oracle.linear_inputs(inp, qweight=q, threads=threads)
        best = min(best, time.perf_counter() - t0)
    return best, threads


def distinct_shapes(wl):
    seen, out = set(), []
    for j, s in enumerate(wl.shapes):
        if s not in seen:
            seen.add(s)
            out.append((s, [i for i, t in enumerate(wl.shapes) if t == s]))
    return out


def decode_line(args, fbq, torch, wl, peaks, peak_kind, world, rank_id, local, barrier, full=True):
    """Times one decode-sized workload with every arm; returns the JSON line (rank 0) or None."""
    import torch.distributed as dist
    bytes_step, bytes_step0 = wl.step_bytes(), wl.step_bytes(0)
    n_lin = len(wl.shapes)
    # the whole pool exceeds 3 x L2, and so does (1.2 x) every per-shape pool (the instances of one shape over all layers)
    from paper_2501_16385_b200.accounting import algorithmic_bytes as _ab
    pool_layers = max(2, -(-3 * 126_000_000 // bytes_step))
    for (K, N), idx in distinct_shapes(wl):
        pool_layers = max(pool_layers, -(-152_000_000 // (len(idx) * _ab(wl.M, N, K, wl.bits, wl.rank, GROUP))))
    pool_layers = min(pool_layers, 48)
    pool, host0 = build_pool(fbq, torch, wl, pool_layers)
    arms = Arms(fbq, torch, wl, pool)
    L = len(pool)
    has_branch = wl.rank > 0
    fbq.set_option("decode_ctas", 0)

    def T(issue, sides=(), **kw):
        return time_arm(torch, issue, L, args.steps, args.warmup, list(sides), **kw)

    sampler = ClockSampler(local) if rank_id == 0 else None
    seq = T(arms.sequential(has_branch), barrier=barrier)
    clocks = sampler.stop() if sampler else None
    ms_step = seq["ms"] / args.steps
    if world > 1:
        t = torch.tensor([ms_step], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_step = float(t.item())
    value = world * bytes_step / (ms_step * 1e-3) / 1e9            # GB/s, whole job

    def gbs(ms_per_step, nbytes=bytes_step):
        return nbytes / (ms_per_step * 1e-3) / 1e9

    extra = {}
    cpu_s = cores = None
    if rank_id == 0:
        hbm = peaks["hbm_gbs"]
        seq0 = T(arms.sequential(False))["ms"] / args.steps if has_branch else ms_step
        extra["sequential"] = {"ms_per_step": ms_step, "GBs": gbs(ms_step), "frac_of_peak": gbs(ms_step) / hbm,
                               "repeats": seq["repeats"], "timed_ms_total": seq["timed_ms_total"],
                               "min_ms_per_step": seq["min_ms"] / args.steps, "max_ms_per_step": seq["max_ms"] / args.steps,
                               "rank0_ms_per_step": seq0, "rank0_GBs": gbs(seq0, bytes_step0)}
        extra["sub_branch_overhead"] = (ms_step / seq0 - 1.0) if (world == 1 and has_branch) else None
        extra["byte_floor_overhead"] = bytes_step / bytes_step0 - 1.0
        if world == 1 and full:
            fbq.set_option("pdl", 0)
            nopdl = T(arms.sequential(has_branch))["ms"] / args.steps
            fbq.set_option("pdl", 1)
            extra["sequential"]["pdl_off_ms_per_step"] = nopdl
            extra["sequential"]["pdl_off_GBs"] = gbs(nopdl)
            if n_lin > 1:
                lo = T(arms.layer_order(has_branch), arms.sides[:2])["ms"] / args.steps
                lo0 = T(arms.layer_order(False), arms.sides[:2])["ms"] / args.steps if has_branch else lo
                extra["layer_order"] = {"ms_per_step": lo, "GBs": gbs(lo), "frac_of_peak": gbs(lo) / hbm,
                                        "rank0_ms_per_step": lo0, "sub_branch_overhead": lo / lo0 - 1.0,
                                        "what": "{q,k,v} side by side -> o -> {gate,up} side by side -> down"}
                ind = T(arms.independent(has_branch), arms.sides)["ms"] / args.steps
                ind0 = T(arms.independent(False), arms.sides)["ms"] / args.steps if has_branch else ind
                extra["independent_streams"] = {
                    "ms_per_step": ind, "GBs": gbs(ind), "frac_of_peak": gbs(ind) / hbm, "rank0_ms_per_step": ind0,
                    "rank0_GBs": gbs(ind0, bytes_step0), "sub_branch_overhead": ind / ind0 - 1.0,
                    "what": "the 7 linears as independent launches on 7 streams joined once per graph, decode grids "
                            "share %d CTAs by size; concurrent throughput, not a latency" % DECODE_CTAS}
            # each shape alone, call after call on one stream
            from paper_2501_16385_b200.accounting import algorithmic_bytes
            per_shape = {}
            for (K, N), idx in distinct_shapes(wl):
                ent = {}
                for label, wb in (("rank%d" % wl.rank, True), ("rank0", False)):
                    if not wb and not has_branch and "rank0" in ent:
                        continue
                    ms1 = T(arms.sequential(wb and has_branch, only=set(idx)))["ms"] / args.steps / len(idx)
                    by = algorithmic_bytes(wl.M, N, K, wl.bits, wl.rank if (wb and has_branch) else 0, GROUP)
                    ent[label if has_branch else "rank0"] = {"us": ms1 * 1e3, "GBs": by / ms1 / 1e6,
                                                              "frac_of_peak": by / ms1 / 1e6 / hbm}
                if has_branch:
                    ent["sub_branch_overhead"] = ent["rank%d" % wl.rank]["us"] / ent["rank0"]["us"] - 1.0
                    ent["byte_floor_overhead"] = (algorithmic_bytes(wl.M, N, K, wl.bits, wl.rank, GROUP) /
                                                  algorithmic_bytes(wl.M, N, K, wl.bits, 0, GROUP) - 1.0)
                per_shape["%d->%d" % (K, N)] = ent
            extra["per_shape_us"] = per_shape
            if has_branch and hasattr(fbq, "sub_branch_unfused"):
                naive = T(naive_issue(fbq, torch, wl, pool))["ms"] / args.steps
                extra["naive_sub_branch"] = {
                    "what": "rank-0 fbq_linear + separate down-projection and up-projection-add launches of this library "
                            "per linear (4 kernels instead of 1), one stream in layer order, same graph replay",
                    "ms_per_step": naive, "slowdown_vs_fused": naive / ms_step, "overhead_vs_rank0": naive / seq0 - 1.0,
                    "extra_latency_removed_by_fusion": 1.0 - (ms_step - seq0) / (naive - seq0) if naive > seq0 else None}
            plain_steps = min(args.steps, 500)
            extra["plain_launch_ms_per_step"] = time_plain_steps(torch, arms.sequential(has_branch), plain_steps) / plain_steps
        if world == 1:
            e2e_steps = min(max(args.steps, 50), 500)
            dt, h2d, d2h = time_e2e(fbq, torch, wl, pool, e2e_steps, 3)
            what = "fbq_linear_hostio per linear in layer order after 0.3 s of untimed steps, host buffers, synchronise per step"
            per_linear_ms = dt * 1e3 / e2e_steps
            if n_lin > 1 and hasattr(fbq, "make_batch"):
                dtb, _, _ = time_e2e(fbq, torch, wl, pool, e2e_steps, 3, batched=True)
                if dtb < dt:
                    dt = dtb
                    what = ("one fbq_linear_batch_hostio call per step after 0.3 s of untimed steps (the library's side streams overlap the problems' "
                            "small copies), host buffers, synchronise per step")
            extra["e2e"] = {"value": bytes_step * e2e_steps / dt / 1e9, "unit": "GB/s", "h2d_bytes_per_step": h2d,
                            "d2h_bytes_per_step": d2h, "ms_per_step": dt * 1e3 / e2e_steps, "steps": e2e_steps,
                            "per_linear_hostio_ms_per_step": per_linear_ms, "what": what}
            cpu_s, cores = oracle_step_seconds(host0, 3)
        status = fbq.poll_status()
        assert status == 0, "device-side status %d" % status
    del arms, pool
    torch.cuda.empty_cache()
    if rank_id != 0:
        return None
    line = {
        "metric": "effective HBM GB/s per linear at M=%d (algorithmic bytes / time)" % wl.M,
        "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "us_per_linear": ms_step * 1e3 / n_lin,
        "pct_of_8TBs": 100.0 * value / world / 8000.0,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f16", "data": "synthetic",
        "config": {"workload": wl.name, "bits": wl.bits, "rank": wl.rank, "group": GROUP, "M": wl.M,
                   "linears_per_step": n_lin, "pool_layers": pool_layers,
                   "cold": "pool of %d layer instances (%.0f MB) > 3x L2, visited round-robin" %
                           (pool_layers, pool_layers * bytes_step / 1e6),
                   "launch": "headline = `sequential`: CUDA graph replay of fbq_linear calls on ONE stream in layer order "
                             "(programmatic dependent launch); every timed region of `steps` steps repeated until >= %d ms, "
                             "median" % int(MIN_TIMED_MS),
                   "parallelism": "replicas only (no collective on the path)" if world > 1 else "1 GPU"},
        "gpu_launches": args.steps * n_lin * seq["repeats"],     # one fused launch per linear per step, all timed repeats
        "roofline": {"bound": "hbm", "achieved": value / world, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": value / world / peaks["hbm_gbs"], "of": peak_kind,
                     "kernel": "gemv_kernel<bits, T, M, ranked> (streaming decode kernel, one launch per linear)",
                     "algorithmic_bytes_per_step": bytes_step,
                     "traffic": TRAFFIC_BYTES_PER_STEP if (wl.bits, wl.rank, wl.M, n_lin) == (3, 64, 1, 7) else None},
        "clocks": clocks,
    }
    line.update(extra)
    if cpu_s is not None:
        line["cpu_baseline"] = {"value": bytes_step / cpu_s / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle",
                                "sample": "1 step (%d linears, all output rows), best of 3, %.3f s" % (n_lin, cpu_s)}
    return line


# DRAM bytes (read + write) per step measured with ncu on the three shapes of a step, one linear each
# (4 x 7.940 + 2 x 20.323 + 20.337 MB; profiles/: the streaming decode kernel's summary).
TRAFFIC_BYTES_PER_STEP = 92_743_000


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
    peaks, peak_kind = measured_peaks()
    line = None
    if args.config == 2:
        if rank_id == 0:
            sampler = ClockSampler(local)
            pf = time_prefill(fbq, torch, peaks, steps=max(3, min(args.steps, 50)), warmup=max(3, min(args.warmup, 10)))
            line = {"metric": "TFLOP/s of the prefill layer at M=1024 (algorithmic flops / time)", "value": pf["tflops"],
                    "unit": "TFLOP/s", "n_gpus": 1, "steps": pf["steps"], "warmup": max(3, min(args.warmup, 10)),
                    "ms_per_step": pf["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                    "dtype": "bf16", "data": "synthetic", "config": {"workload": pf["workload"]},
                    "gpu_launches": int(pf["launches_per_step"] * pf["steps"] * pf["repeats"]),
                    "roofline": pf["roofline"], "per_shape": pf["per_shape"], "clocks": sampler.stop()}
    elif args.config == 3:
        lines = []
        for bits in (3, 4):
            for M in (1, 16):
                ln = decode_line(args, fbq, torch, workload_for(3, M=M, bits=bits), peaks, peak_kind, world, rank_id, local,
                                 barrier, full=False)
                if ln:
                    lines.append(ln)
        if rank_id == 0:
            line = lines[0]
            line["all"] = [{"workload": l["config"]["workload"], "ms_per_step": l["ms_per_step"], "GBs": l["value"],
                            "frac_of_peak": l["roofline"]["frac"], "sub_branch_overhead": l["sub_branch_overhead"],
                            "byte_floor_overhead": l["byte_floor_overhead"]} for l in lines]
    elif args.config == 4:
        rows = []
        first = None
        for M in (1, 2, 4, 8, 16):
            base = None
            for r in (0, 16, 32, 64, 128):
                ln = decode_line(args, fbq, torch, workload_for(4, M=M, rank=r), peaks, peak_kind, world, rank_id, local,
                                 barrier, full=False)
                if not ln:
                    continue
                first = first or ln
                base = ln["ms_per_step"] if r == 0 else base
                rows.append({"M": M, "rank": r, "us_per_step": ln["ms_per_step"] * 1e3, "GBs": ln["value"],
                             "frac_of_peak": ln["roofline"]["frac"], "overhead_vs_rank0": ln["ms_per_step"] / base - 1.0,
                             "byte_floor_overhead": ln["byte_floor_overhead"]})
        if rank_id == 0:
            line = first
            line["config"]["workload"] = "llama2-7b decoder-layer linears, INT4 g128, M x rank sweep (sequential arm)"
            line["sweep"] = rows
    else:
        wl = workload_for(args.config)
        line = decode_line(args, fbq, torch, wl, peaks, peak_kind, world, rank_id, local, barrier, full=True)
        if rank_id == 0 and world == 1 and args.config == 1:
            line["prefill"] = time_prefill(fbq, torch, peaks)
    barrier()
    if rank_id == 0 and line is not None:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# ---------------------------------------------------------------------- reference arm
def reference_arm(args):
    """The CPU oracle, as it stands, on the same workload (reported baseline)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from workloads import make_linear
    import oracle
    wl = workload_for(args.config if args.config in (0, 1, 3, 4) else 1)
    host0 = [make_linear(wl.M, N, K, wl.bits, max(wl.rank, 8), seed=wl.seed0 + sid) for sid, (K, N) in enumerate(wl.shapes)]
    packed = [oracle.pack(i.codes, i.bits) for i in host0]
    threads = oracle.max_threads()
    steps = min(args.steps, 20)           # bounded: a step is ~0.1-0.5 s of host work
    warm = min(args.warmup, 2)

    def one(nthreads=threads):
        for inp, q in zip(host0, packed):
            oracle.linear_inputs(inp, qweight=q, threads=nthreads)

    for _ in range(warm):
        one()
    t0 = time.perf_counter()
    for _ in range(steps):
        one()
    dt = time.perf_counter() - t0
    value = wl.step_bytes() * steps / dt / 1e9
    single = None
    if args.config == 0:                  # the smallest configuration also single-threaded
        t1 = time.perf_counter()
        one(1)
        single = wl.step_bytes() / (time.perf_counter() - t1) / 1e9
    print(json.dumps({
        "impl": "reference", "metric": "effective HBM GB/s per linear at M=%d (algorithmic bytes / time)" % wl.M,
        "value": value, "unit": "GB/s", "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": steps,
        "warmup": warm, "ms_per_step": dt * 1e3 / steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "bits": wl.bits, "rank": wl.rank, "group": GROUP, "M": wl.M,
                   "linears_per_step": len(wl.shapes)},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": threads, "kind": "oracle",
                         "sample": "%d steps of %d linears (all output rows)" % (steps, len(wl.shapes)),
                         "single_thread_GBs": single},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="fbq", choices=["fbq", "reference"])
    ap.add_argument("--config", type=int, default=1, choices=[0, 1, 2, 3, 4])
    args = ap.parse_args()
    if args.impl == "reference":
        reference_arm(args)
    else:
        gpu_arm(args)


if __name__ == "__main__":
    main()
