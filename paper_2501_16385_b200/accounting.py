"""Algorithmic bytes and flops of one FBQuant linear (what the method has to
move and compute), used by the benchmark's roofline figures.

Bytes: packed codes + fp16 scales + fp16 zeros + A + B + x + y, each counted
once; the dense fp16 weight matrix is never materialised.  Flops: 2.M.N.K for
the main path and 2.M.r.(K+N) for the sub-branch (Section 3.2 of the paper
counts M0 = b.d.d and M1 = 2.b.r.d multiply-accumulates for a d x d layer).
"""
from __future__ import annotations


def algorithmic_bytes(M: int, N: int, K: int, bits: int, rank: int, group: int = 128) -> int:
    codes = N * K * bits // 8
    meta = 2 * N * (K // group) * 2
    ab = rank * (K + N) * 2
    act = 2 * M * (K + N)
    return codes + meta + ab + act


def algorithmic_flops(M: int, N: int, K: int, rank: int) -> int:
    return 2 * M * N * K + 2 * M * rank * (K + N)


def byte_floor_overhead(M: int, N: int, K: int, bits: int, rank: int, group: int = 128) -> float:
    """bytes(rank r) / bytes(rank 0) - 1: the sub-branch overhead no kernel can beat."""
    return algorithmic_bytes(M, N, K, bits, rank, group) / algorithmic_bytes(M, N, K, bits, 0, group) - 1.0
