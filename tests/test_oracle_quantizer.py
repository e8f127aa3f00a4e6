"""Pins of the oracle's feedback quantiser (Section 4.1: W_F = Q(W - Sigma) + Sigma and the bound
|w - w_F| <= s/2) against things other than itself: hand-worked groups with ties, numpy's float16
conversion, exact recovery of weights that lie on a quantiser grid, the bound in double precision,
the feedback identity (codes depend on W - Sigma only), and the round trip through the dequantiser."""
import os

import numpy as np
import pytest

import oracle
from workloads import f32_to_bf16_bits

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _read_golden(name):
    out = {}
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                parts = line.split()
                out[parts[0]] = np.array([float(v) for v in parts[1:]])
    return out


def _half(v):
    v = np.asarray(v, dtype=np.uint16)
    return np.asarray(oracle.widen(v, "f16")).reshape(v.shape)


@pytest.mark.parametrize("tag,bits", [("int4", 4), ("int3", 3)])
def test_hand_worked_groups(tag, bits):
    g = _read_golden("quantizer_example.txt")
    r = g[tag + "_r"].astype(np.float32)[None, :]
    codes, s, z, r_out, wf = oracle.quantize_feedback(r, None, None, 8, bits)
    assert np.array_equal(codes[0], g[tag + "_q"].astype(np.uint8))
    assert _half(s)[0, 0] == g[tag + "_s"][0] and _half(z)[0, 0] == g[tag + "_z"][0]
    assert np.array_equal(r_out, r)
    assert np.array_equal(wf[0].astype(np.float64), g[tag + "_deq"])
    # the same residuals behind a rank-1 sub-branch: Sigma = B.A = 0.5 everywhere
    A = np.ones((1, 8), dtype=np.float16)
    B = np.full((1, 1), g["sigma"][0], dtype=np.float16)
    c2, s2, z2, r2, wf2 = oracle.quantize_feedback(r + np.float32(g["sigma"][0]), A, B, 8, bits)
    assert np.array_equal(c2, codes) and np.array_equal(s2, s) and np.array_equal(z2, z)
    assert np.array_equal(wf2[0].astype(np.float64), g[tag + "_deq"] + g["sigma"][0])


def test_constant_group():
    g = _read_golden("quantizer_example.txt")
    w = np.full((1, 8), g["const_c"][0], dtype=np.float32)
    codes, s, z, _, wf = oracle.quantize_feedback(w, None, None, 8, 4)
    assert _half(s)[0, 0] == g["const_s"][0] and _half(z)[0, 0] == g["const_z"][0]
    assert np.all(codes == int(g["const_q"][0])) and np.array_equal(wf, w)
    codes, s, z, _, wf = oracle.quantize_feedback(-w, None, None, 8, 4)
    assert _half(z)[0, 0] == 0 and np.all(codes == 1) and np.array_equal(wf, -w)
    codes, s, z, _, wf = oracle.quantize_feedback(0 * w, None, None, 8, 3)
    assert np.all(codes == 0) and np.all(wf == 0)


def test_half_conversion_is_numpys():
    rng = np.random.default_rng(7)
    vals = np.concatenate([rng.standard_normal(100000).astype(np.float32) * np.float32(sc)
                           for sc in (1, 1e-3, 1e-5, 3e-8, 300, 4e4)] +
                          [np.array([0, -0.0, 65504, 65519.99, 65520, 2.0 ** -24, 2.0 ** -25, 2.0 ** -25 * 1.001,
                                     2.0 ** -14, 1.5 * 2.0 ** -24, 2.5 * 2.0 ** -24], dtype=np.float32)])
    with np.errstate(over="ignore"):
        want = vals.astype(np.float16).view(np.uint16)
    assert np.array_equal(oracle.float_to_half(vals), want)


@pytest.mark.parametrize("bits", [3, 4])
def test_weights_on_a_grid_are_recovered_exactly(bits):
    # W = s0*(q0 - z0) with power-of-two s0 and every group holding code 0 and code maxq:
    # the quantiser must return exactly (q0, s0, z0) and W_F = W.
    rng = np.random.default_rng(11 + bits)
    N, K, group, maxq = 6, 256, 64, (1 << bits) - 1
    q0 = rng.integers(0, maxq + 1, size=(N, K)).astype(np.uint8)
    q0[:, ::group] = 0
    q0[:, 1::group] = maxq
    s0 = 2.0 ** rng.integers(-9, -3, size=(N, K // group))
    z0 = rng.integers(1, maxq, size=(N, K // group)).astype(np.float64)
    W = (np.repeat(s0, group, axis=1) * (q0 - np.repeat(z0, group, axis=1))).astype(np.float32)
    codes, s, z, _, wf = oracle.quantize_feedback(W, None, None, group, bits)
    assert np.array_equal(codes, q0)
    assert np.array_equal(_half(s), s0) and np.array_equal(_half(z), z0)
    assert np.array_equal(wf, W)


@pytest.mark.parametrize("bits,dtype,rank", [(4, "f16", 0), (3, "f16", 16), (4, "bf16", 8), (3, "bf16", 64)])
def test_bound_and_feedback_identity(bits, dtype, rank):
    # Eq. "diff": |w - w_F| = |(w - sigma) - Q(w - sigma)| <= s/2, whatever Sigma is; checked in
    # double precision from the stored s, z and codes, for the codes the clamp did not touch.
    rng = np.random.default_rng(100 + bits + rank)
    N, K, group, maxq = 12, 512, 128, (1 << bits) - 1
    W = (rng.standard_normal((N, K)) * 0.05).astype(np.float32)
    W[3, 5] = 0.9                                        # an outlier stretches its group's range
    if rank:
        A32 = (rng.standard_normal((rank, K)) * 0.3).astype(np.float32)
        B32 = (rng.standard_normal((N, rank)) * 0.3).astype(np.float32)
        if dtype == "bf16":
            A, B = f32_to_bf16_bits(A32), f32_to_bf16_bits(B32)
        else:
            A, B = A32.astype(np.float16).view(np.uint16), B32.astype(np.float16).view(np.uint16)
        sigma = oracle.widen(B, dtype).reshape(N, rank) @ oracle.widen(A, dtype).reshape(rank, K)   # numpy fp64 matmul
    else:
        A = B = None
        sigma = np.zeros((N, K))
    codes, s, z, r, wf = oracle.quantize_feedback(W, A, B, group, bits, dtype=dtype)
    s64, z64 = np.repeat(_half(s), group, axis=1), np.repeat(_half(z), group, axis=1)
    # residual is W - B.A (fp32 accumulation against numpy's fp64 product)
    assert np.allclose(r, W - sigma, rtol=0, atol=1e-5 * (1 + np.abs(sigma).max()))
    deq = s64 * (codes.astype(np.float64) - z64)
    unclamped = np.abs(r.astype(np.float64) / s64 + z64 - codes) <= 0.5 + 1e-6
    assert unclamped.mean() > 0.99
    err = np.abs(r.astype(np.float64) - deq)
    assert np.all(err[unclamped] <= 0.5 * s64[unclamped] * (1 + 1e-6))
    assert err.max() > 0.2 * s64.min()                   # not vacuous: errors of the order of s occur
    # reconstructed weights: W_F = Q(W - Sigma) + Sigma, so |W - W_F| obeys the same bound
    errF = np.abs(W.astype(np.float64) - wf.astype(np.float64))
    assert np.all(errF[unclamped] <= 0.5 * s64[unclamped] + 1e-5 * (1 + np.abs(sigma).max()))
    # every group uses the whole code range (min-max quantiser)
    cg = codes.reshape(N, K // group, group)
    assert np.all(cg.min(axis=2) == 0) and np.all(cg.max(axis=2) == maxq)
    # round trip through the packer and the dequantiser of the layer
    wq = oracle.dequant(oracle.pack(codes, bits), s, z, N, K, group, bits)
    assert np.array_equal(wq, deq)


def test_malformed_requests():
    W = np.zeros((2, 8), dtype=np.float32)
    with pytest.raises(ValueError):
        oracle.quantize_feedback(W, None, None, 3, 4)
    with pytest.raises(ValueError):
        oracle.quantize_feedback(W, None, None, 8, 5)
