"""Sub-branch overhead curve of the decode path: one Llama-2-7B decoder layer (seven linears) at
M in {1, 2, 4, 8, 16} tokens x rank in {0, 16, 32, 64, 128}, INT4 (or --bits 3), group 128.

    python -m paper_2501_16385_b200.sweep [--bits 4] [--steps 300]

Same launch scheme as bench.py's headline arm: the seven independent linears of a step go to seven
CUDA streams (joined once per graph), decode grids share 386 main CTAs by size (eight 16-row tiles per CTA for N = 4096 and 11008), CUDA-graph replay, a pool
of layer instances larger than L2, CUDA events on the launching stream.  Prints one JSON line per
(M, rank): microseconds per step, effective GB/s, and the overhead against rank 0 at the same M
beside the byte floor (extra bytes the sub-branch adds).  Inputs are random device tensors
(microbench.make_instance).
"""
import argparse
import json

import torch

from . import binding as fbq
from .accounting import algorithmic_bytes
from .microbench import make_instance

SHAPES = [(4096, 4096)] * 4 + [(4096, 11008), (4096, 11008), (11008, 4096)]       # (K, N): q k v o gate up down
TOTAL_CTAS = 386


def time_layer(M, bits, rank, steps, pool_layers=3, total_ctas=TOTAL_CTAS):
    pool = [[make_instance(M, N, K, bits, rank, "f16", 50 * li + j) for j, (K, N) in enumerate(SHAPES)]
            for li in range(pool_layers)]
    costs = [K * N for K, N in SHAPES]
    main = torch.cuda.Stream()
    sides = [torch.cuda.Stream() for _ in range(len(SHAPES) - 1)]
    streams = [main] + sides

    def run(n):
        for st in sides:
            st.wait_stream(main)
        for i in range(n):
            for j, t in enumerate(pool[i % pool_layers]):
                fbq.set_option("decode_ctas", max(8, round(total_ctas * costs[j] / sum(costs))))
                fbq.linear(t["x"], t["qweight"], t["scales"], t["zeros"], t["A"], t["B"], t["y"].shape[1], 128, bits,
                           y=t["y"], stream=streams[j])
        for st in sides:
            main.wait_stream(st)

    chunk = max(pool_layers, min(60, steps) // pool_layers * pool_layers)
    with torch.cuda.stream(main):
        run(2 * pool_layers)
        main.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=main):
            run(chunk)
        g.replay()
        main.synchronize()
        reps = max(1, steps // chunk)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(main)
        for _ in range(reps):
            g.replay()
        e1.record(main)
        main.synchronize()
    assert fbq.poll_status(main) == 0
    fbq.set_option("decode_ctas", 0)
    del pool
    torch.cuda.empty_cache()
    return e0.elapsed_time(e1) * 1e3 / (reps * chunk)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--bits", type=int, default=4)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--ctas", type=int, default=TOTAL_CTAS, help="decode CTAs shared out among the seven linears")
    ap.add_argument("--tokens", type=int, nargs="*", default=[1, 2, 4, 8, 16])
    ap.add_argument("--opt", nargs="*", default=[], help="library options as name=value (fbq_set_option)")
    a = ap.parse_args()
    for kv in a.opt:
        name, value = kv.split("=")
        fbq.set_option(name, int(value))
    for M in a.tokens:
        base = None
        for rank in (0, 16, 32, 64, 128):
            us = time_layer(M, a.bits, rank, a.steps, total_ctas=a.ctas)
            by = sum(algorithmic_bytes(M, N, K, a.bits, rank) for K, N in SHAPES)
            by0 = sum(algorithmic_bytes(M, N, K, a.bits, 0) for K, N in SHAPES)
            if rank == 0:
                base = us
            print(json.dumps({"M": M, "bits": a.bits, "rank": rank, "us_per_step": round(us, 2), "us_per_linear": round(us / 7, 2),
                              "GBs": round(by / us / 1e3, 1), "overhead_vs_rank0": round(us / base - 1.0, 3),
                              "byte_floor_overhead": round(by / by0 - 1.0, 3),
                              "kernel": fbq.select_kernel(M, 4096, 4096, 128, a.bits, rank)}), flush=True)


if __name__ == "__main__":
    main()
