"""ctypes front end of the CPU oracle (oracle/fbq_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA package never imports this module and
this module never imports the CUDA package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fbq_oracle.c")
_LIB = os.path.join(_HERE, "libfbq_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP over independent output rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
                               "-ffp-contract=off", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_linear.restype = ctypes.c_int
        _lib.oracle_max_threads.restype = ctypes.c_int
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _u16(a):
    a = np.ascontiguousarray(a)
    if a.dtype == np.float16:
        a = a.view(np.uint16)
    assert a.dtype == np.uint16, a.dtype
    return a


def packed_words(N: int, K: int, bits: int) -> int:
    return N * K // 8 if bits == 4 else N * K * 3 // 32


def max_threads() -> int:
    return int(_load().oracle_max_threads())


def widen(bits: np.ndarray, dtype: str = "f16") -> np.ndarray:
    bits = _u16(bits).ravel()
    out = np.zeros(bits.size, dtype=np.float64)
    _load().oracle_widen(_p(bits), _p(out), ctypes.c_int(bits.size),
                         ctypes.c_int(1 if dtype == "bf16" else 0))
    return out


def pack(codes: np.ndarray, bits: int) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    N, K = codes.shape
    assert K % (8 if bits == 4 else 32) == 0
    out = np.zeros(packed_words(N, K, bits), dtype=np.uint32)
    fn = _load().oracle_pack_int4 if bits == 4 else _load().oracle_pack_int3
    fn(_p(codes), _p(out), ctypes.c_int(N), ctypes.c_int(K))
    return out


def unpack(qweight: np.ndarray, N: int, K: int, bits: int) -> np.ndarray:
    qweight = np.ascontiguousarray(qweight, dtype=np.uint32)
    assert qweight.size == packed_words(N, K, bits)
    out = np.zeros((N, K), dtype=np.uint8)
    _load().oracle_unpack(_p(qweight), _p(out), ctypes.c_int(N), ctypes.c_int(K), ctypes.c_int(bits))
    return out


def dequant(qweight, scales, zeros, N: int, K: int, group: int, bits: int) -> np.ndarray:
    qweight = np.ascontiguousarray(qweight, dtype=np.uint32)
    s, z = _u16(scales), _u16(zeros)
    assert s.size == N * (K // group) and z.size == s.size
    W = np.zeros((N, K), dtype=np.float64)
    _load().oracle_dequant(_p(qweight), _p(s), _p(z), _p(W), ctypes.c_int(N), ctypes.c_int(K),
                           ctypes.c_int(group), ctypes.c_int(bits))
    return W


def linear(x, qweight, scales, zeros, A, B, M, N, K, group, bits, rank, *, dtype="f16",
           n_list=None, threads=1, return_t=False):
    """y (M x N, or M x len(n_list)) in float64; optionally also t = x.A^T."""
    x = _u16(x)
    qweight = np.ascontiguousarray(qweight, dtype=np.uint32)
    s, z = _u16(scales), _u16(zeros)
    assert x.size == M * K and qweight.size == packed_words(N, K, bits)
    assert s.size == N * (K // group) and z.size == s.size
    if rank > 0:
        A, B = _u16(A), _u16(B)
        assert A.size == rank * K and B.size == N * rank
    else:
        A = B = None
    if n_list is not None:
        n_list = np.ascontiguousarray(n_list, dtype=np.int32)
        assert n_list.min() >= 0 and n_list.max() < N
        cnt = int(n_list.size)
    else:
        cnt = N
    y = np.zeros((M, cnt), dtype=np.float64)
    t = np.zeros((M, max(rank, 1)), dtype=np.float64)
    rc = _load().oracle_linear(_p(x), _p(qweight), _p(s), _p(z), _p(A), _p(B), _p(y), _p(t),
                               ctypes.c_int(M), ctypes.c_int(N), ctypes.c_int(K),
                               ctypes.c_int(group), ctypes.c_int(bits), ctypes.c_int(rank),
                               ctypes.c_int(1 if dtype == "bf16" else 0), _p(n_list),
                               ctypes.c_int(cnt), ctypes.c_int(threads))
    if rc != 0:
        raise ValueError("oracle_linear rejected the request")
    if return_t:
        return y, t[:, :rank]
    return y


def linear_inputs(inp, *, n_list=None, threads=1, return_t=False, qweight=None):
    """Convenience: run the oracle on a workloads.LinearInputs record."""
    if qweight is None:
        qweight = pack(inp.codes, inp.bits)
    return linear(inp.x, qweight, inp.scales, inp.zeros, inp.A, inp.B, inp.M, inp.N, inp.K,
                  inp.group, inp.bits, inp.rank, dtype=inp.dtype, n_list=n_list,
                  threads=threads, return_t=return_t)


def float_to_half(a: np.ndarray) -> np.ndarray:
    """fp16 bit patterns (uint16) of float32 values, by the oracle's own rounding routine."""
    _load()
    a = np.ascontiguousarray(a, dtype=np.float32)
    out = np.empty(a.shape, dtype=np.uint16)
    _lib.oracle_float_to_half(_p(a), _p(out), ctypes.c_int(a.size))
    return out


def quantize_feedback(W: np.ndarray, A, B, group: int, bits: int, *, dtype: str = "f16"):
    """Feedback quantiser of Section 4.1 on W [N, K] float32 with Sigma = B.A (A [rank, K],
    B [N, rank] as 16-bit patterns, or float32 with dtype="f32", or None for rank 0).  Returns codes (uint8 [N, K]),
    scales, zeros (uint16 fp16 patterns [N, K/group]), r = W - Sigma and W_F (float32 [N, K])."""
    _load()
    W = np.ascontiguousarray(W, dtype=np.float32)
    N, K = W.shape
    rank = 0 if A is None else A.shape[0]
    if K % group != 0:
        raise ValueError("group must divide K")
    codes = np.empty((N, K), dtype=np.uint8)
    scales = np.empty((N, K // group), dtype=np.uint16)
    zeros = np.empty((N, K // group), dtype=np.uint16)
    r = np.empty((N, K), dtype=np.float32)
    wf = np.empty((N, K), dtype=np.float32)
    if dtype == "f32":
        Ab = np.ascontiguousarray(A, dtype=np.float32) if rank else None
        Bb = np.ascontiguousarray(B, dtype=np.float32) if rank else None
    else:
        Ab = _u16(A) if rank else None
        Bb = _u16(B) if rank else None
    _lib.oracle_quantize_feedback.restype = ctypes.c_int
    rc = _lib.oracle_quantize_feedback(_p(W), _p(Ab) if rank else None, _p(Bb) if rank else None, _p(codes), _p(scales),
                                       _p(zeros), _p(r), _p(wf), ctypes.c_int(N), ctypes.c_int(K), ctypes.c_int(group),
                                       ctypes.c_int(bits), ctypes.c_int(rank), ctypes.c_int({"f16": 0, "bf16": 1, "f32": 2}[dtype]))
    if rc != 0:
        raise ValueError("oracle_quantize_feedback rejected the request")
    return codes, scales, zeros, r, wf
