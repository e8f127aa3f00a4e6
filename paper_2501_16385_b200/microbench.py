"""Time one FBQuant linear shape through the C-ABI library and print one JSON line.

    python -m paper_2501_16385_b200.microbench --M 1024 --N 4096 --K 4096 --bits 4 --rank 64 --dtype bf16

Inputs are random tensors made on the device (codes uniform, scales ~0.01, integer zero points);
the layer instance is rotated over a pool larger than L2 unless --hot is given.  Times are CUDA
events on the launching stream around `reps` back-to-back calls.  This is the command the ncu
summaries of single shapes are taken with.
"""
import argparse
import json

import torch

from . import binding as fbq
from .accounting import algorithmic_bytes, algorithmic_flops

L2_BYTES = 126e6


def make_instance(M, N, K, bits, rank, dtype, seed, outlier_frac=0.0, outlier_scale=20.0):
    """Device tensors of one synthetic linear.  outlier_frac > 0 scales that share of the input
    channels of x by outlier_scale (the activation-outlier structure of LLM prefill inputs)."""
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    G = K // 128
    act = torch.bfloat16 if dtype == "bf16" else torch.float16
    codes = torch.randint(0, 1 << bits, (N, K), dtype=torch.uint8, device="cuda", generator=g)
    inst = {
        "qweight": fbq.pack(codes, bits),
        "scales": (torch.rand((N, G), device="cuda", generator=g) * 0.015 + 0.005).half(),
        "zeros": torch.randint(2, (1 << bits) - 2, (N, G), device="cuda", generator=g).half(),
        "x": None,
        "A": (torch.randn((rank, K), device="cuda", generator=g) * 0.02).to(act) if rank else None,
        "B": (torch.randn((N, rank), device="cuda", generator=g) * 0.02).to(act) if rank else None,
        "y": torch.empty((M, N), device="cuda", dtype=act),
    }
    del codes
    x = torch.randn((M, K), device="cuda", generator=g)
    if outlier_frac > 0:
        ch = torch.randperm(K, device="cuda", generator=g)[: max(1, int(outlier_frac * K))]
        x[:, ch] *= outlier_scale
    inst["x"] = x.to(act)
    return inst


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--M", type=int, default=1024)
    ap.add_argument("--N", type=int, default=4096)
    ap.add_argument("--K", type=int, default=4096)
    ap.add_argument("--bits", type=int, default=4)
    ap.add_argument("--rank", type=int, default=64)
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "f16"])
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--hot", action="store_true", help="reuse one instance (operands stay in L2)")
    ap.add_argument("--opt", nargs="*", default=[], help="library options as name=value (fbq_set_option)")
    a = ap.parse_args()
    for kv in a.opt:
        name, value = kv.split("=")
        fbq.set_option(name, int(value))

    by = algorithmic_bytes(a.M, a.N, a.K, a.bits, a.rank)
    n_inst = 1 if a.hot else max(2, int(2 * L2_BYTES / by) + 1)
    pool = [make_instance(a.M, a.N, a.K, a.bits, a.rank, a.dtype, s) for s in range(n_inst)]

    def call(t):
        fbq.linear(t["x"], t["qweight"], t["scales"], t["zeros"], t["A"], t["B"], a.N, 128, a.bits, y=t["y"])

    for i in range(a.warmup):
        call(pool[i % n_inst])
    torch.cuda.synchronize()
    before = fbq.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(a.reps):
        call(pool[i % n_inst])
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / a.reps
    assert fbq.poll_status() == 0
    fl = algorithmic_flops(a.M, a.N, a.K, a.rank)
    print(json.dumps({
        "shape": {"M": a.M, "N": a.N, "K": a.K, "bits": a.bits, "rank": a.rank, "dtype": a.dtype},
        "kernel": fbq.select_kernel(a.M, a.N, a.K, 128, a.bits, a.rank, a.dtype == "bf16"),
        "us_per_call": round(us, 2), "tflops": round(fl / us / 1e6, 1), "gbs": round(by / us / 1e3, 1),
        "instances": n_inst, "launches_per_call": (fbq.launch_count() - before) / a.reps,
    }))


if __name__ == "__main__":
    main()
