"""GPU parity of the decode kernel's integer form (M <= 2: codes as unsigned bytes, x as three signed
base-256 digits per group scale, 8-bit integer MMAs) against the CPU oracle, next to the 16-bit form
on the same inputs, and on inputs chosen to stress the fixed-point representation of x: empty groups,
one huge element beside tiny ones, values at the ends of the format's range, fp16 subnormals."""
import dataclasses

import numpy as np
import pytest

import oracle
from gpu_utils import DeviceLinear, check_parity, torch_to_f64
from workloads import f32_to_bf16_bits, make_exact_class, make_linear

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fbq():
    import torch
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    import paper_2501_16385_b200 as lib
    lib.set_option("force_kernel", -1)
    yield lib
    lib.set_option("decode_i8", 1)
    lib.set_option("force_kernel", -1)


def _bits(xf32, dtype):
    return f32_to_bf16_bits(xf32) if dtype == "bf16" else xf32.astype(np.float16).view(np.uint16)


def _run_forced_decode(fbq, inp):
    import torch
    dev = DeviceLinear(inp, fbq)
    fbq.set_option("force_kernel", fbq.KERNEL_DECODE)
    try:
        y = dev.run(fbq)
    finally:
        fbq.set_option("force_kernel", -1)
    torch.cuda.synchronize()
    assert fbq.poll_status() == 0
    return torch_to_f64(y, inp.dtype)


@pytest.mark.parametrize("bits", [3, 4])
@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("M,N,K,rank", [(1, 272, 1024, 0), (2, 520, 2048, 16), (1, 1000, 640, 64), (2, 136, 11008, 32)])
def test_integer_and_16bit_forms_on_the_same_inputs(fbq, bits, dtype, M, N, K, rank):
    inp = make_linear(M, N, K, bits, rank, dtype=dtype, seed=7000 + N + bits, outlier_frac=0.01)
    ys = []
    for form in (1, 0):
        fbq.set_option("decode_i8", form)
        try:
            _, _, y64, y_or = check_parity(inp, fbq, expect_kernel=fbq.KERNEL_DECODE)
        finally:
            fbq.set_option("decode_i8", 1)
        ys.append(y64)
    # both forms round an fp32-accurate sum once: they agree to an ulp of the output type, and differ at all only where
    # the sum lies within its fp32 error of a rounding boundary (a per cent or two of the outputs)
    eps = 2.0 ** -10 if dtype == "f16" else 2.0 ** -7
    diff = np.abs(ys[0] - ys[1])
    assert np.mean(diff <= np.abs(y_or) * eps + 1e-6) > 0.95
    assert diff.max() <= 2 * eps * np.abs(y_or).max()


def _dequant(inp):
    s = np.repeat(inp.scales.astype(np.float64), inp.group, axis=1)
    z = np.repeat(inp.zeros.astype(np.float64), inp.group, axis=1)
    return s * (inp.codes.astype(np.float64) - z)


@pytest.mark.parametrize("bits", [3, 4])
@pytest.mark.parametrize("dtype,big,tiny", [("f16", 20000.0, 6e-5), ("f16", 3.0, 6e-8), ("bf16", 1e30, 1e-3), ("bf16", 1e-20, 1e-30)])
def test_integer_form_wide_dynamic_range(fbq, bits, dtype, big, tiny):
    # Groups of x that are empty, that hold one huge element beside tiny ones, that are all tiny.  The
    # usual bound scales with ||x||_inf and says nothing here, so the error is bounded per output from
    # the representation itself: x is exact to 2^-16 of its group's maximum, the output is rounded once.
    M, N, K, rank = 2, 264, 1536, 0
    inp = make_linear(M, N, K, bits, rank, dtype=dtype, seed=7100 + bits)
    rng = np.random.default_rng(7)
    xf = (rng.standard_normal((M, K)) * tiny).astype(np.float32)
    G = K // 128
    for m in range(M):
        for g in range(G):
            kind = (g + m) % 4
            sl = slice(g * 128, (g + 1) * 128)
            if kind == 0:
                xf[m, sl] = 0.0
            elif kind == 1:
                xf[m, g * 128 + int(rng.integers(0, 128))] = big * (-1.0 if g % 2 else 1.0)
            elif kind == 2:
                xf[m, sl] *= np.float32(big / tiny) * np.float32(0.25)
    inp = dataclasses.replace(inp, x=_bits(xf, dtype))
    y = _run_forced_decode(fbq, inp)
    assert np.all(np.isfinite(y))
    x64, w = inp.x_f64(), _dequant(inp)
    want = x64 @ w.T
    gmax = np.abs(x64).reshape(M, G, 128).max(axis=2)                       # [M][G]
    wabs = np.abs(w).reshape(N, G, 128).sum(axis=2)                          # [N][G]
    eps_out = 2.0 ** -10 if dtype == "f16" else 2.0 ** -7
    bound = (gmax @ wabs.T) * 2.0 ** -16 + np.abs(want) * eps_out + (np.abs(x64) @ np.abs(w).T) * 1e-6 + 1e-30
    if dtype == "f16":
        bound += 2.0 ** -24                                                  # the output's own subnormal spacing
    assert np.all(np.abs(y - want) <= bound)
    assert np.array_equal(np.sign(y[np.abs(want) > 4 * bound]), np.sign(want[np.abs(want) > 4 * bound]))


@pytest.mark.parametrize("bits,dtype,M", [(3, "f16", 1), (4, "f16", 2), (3, "bf16", 2), (4, "bf16", 1)])
def test_integer_form_exact_class_is_bitwise(fbq, bits, dtype, M):
    # small integers in x, powers of two in s: every product and sum is exact, so y equals the oracle bit for bit
    kw = dict(x_nnz=32, x_max=2) if dtype == "f16" else dict(x_nnz=4, x_max=1)
    exact = make_exact_class(M, 392, 1024, bits, 32, dtype=dtype, seed=7200 + bits, **kw)
    y = _run_forced_decode(fbq, exact)
    assert np.array_equal(y, oracle.linear_inputs(exact, threads=8))


def test_integer_form_rows_of_codes_at_the_ends(fbq):
    # all codes 0 and all codes 2^bits - 1 (every field of every word, the bit-sliced codes 30 and 31 included)
    for bits in (3, 4):
        inp = make_linear(1, 48, 512, bits, 0, seed=7300 + bits)
        codes = inp.codes.copy()
        codes[0::2] = 0
        codes[1::2] = (1 << bits) - 1
        inp = dataclasses.replace(inp, codes=codes)
        check_parity(inp, fbq, expect_kernel=fbq.KERNEL_DECODE)


@pytest.mark.parametrize("t_ctas", [1, 0])
@pytest.mark.parametrize("M,rank", [(1, 16), (2, 64), (3, 32), (4, 64), (4, 48), (2, 128), (1, 200)])
def test_sub_branch_paths(fbq, M, rank, t_ctas):
    # t from the CTAs at the head of the grid (t_ctas = 1) or from every CTA's epilogue warp (0); tensor-core
    # up-projection per tile (rank a multiple of 16, at most 64), the plain tile finish (rank 48) and the heavy
    # variant (rank > 64), each against the oracle; three calls in a row leave the scratch clean
    import torch
    inp = make_linear(M, 1160, 2048, 4, rank, seed=7400 + M + rank)
    fbq.set_option("decode_t_ctas", t_ctas)
    try:
        check_parity(inp, fbq, expect_kernel=fbq.KERNEL_DECODE)
        dev = DeviceLinear(inp, fbq)
        fbq.set_option("force_kernel", fbq.KERNEL_DECODE)
        ys = [dev.run(fbq).clone() for _ in range(3)]
    finally:
        fbq.set_option("force_kernel", -1)
        fbq.set_option("decode_t_ctas", 1)
    torch.cuda.synchronize()
    assert fbq.poll_status() == 0
    for y in ys[1:]:
        assert np.max(np.abs(torch_to_f64(y, "f16") - torch_to_f64(ys[0], "f16"))) <= 2e-3   # t is summed by atomics


@pytest.mark.parametrize("t_wait", [0, 1])
def test_tiles_wait_for_t_or_are_parked(fbq, t_wait):
    fbq.set_option("decode_t_wait", t_wait)
    fbq.set_option("decode_t_ctas", 0)                     # every CTA contributes to t: it is complete late
    try:
        inp = make_linear(1, 2048, 4096, 3, 64, seed=7500)
        fbq.set_option("decode_ctas", 16)                  # eight tiles per CTA: some are done before t is
        check_parity(inp, fbq, expect_kernel=fbq.KERNEL_DECODE)
    finally:
        fbq.set_option("decode_t_wait", 1)
        fbq.set_option("decode_t_ctas", 1)
        fbq.set_option("decode_ctas", 0)
