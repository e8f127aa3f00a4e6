"""GPU parity of the prefill path (M > 16: tcgen05 / tensor-memory kernel) against the CPU
oracle, through the C ABI.  Same tolerances as the decode tests: rel_F <= 5e-3 and
max-abs <= 1e-2*||x||inf*sqrt(K)/64."""
import numpy as np
import pytest

import oracle
from workloads import LLAMA2_7B_SHAPES, make_exact_class, make_linear

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fbq():
    import torch
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    import paper_2501_16385_b200 as lib
    lib.set_option("force_kernel", -1)
    return lib


from gpu_utils import DeviceLinear, check_parity, torch_to_f64  # noqa: E402


@pytest.mark.parametrize("bits", [3, 4])
@pytest.mark.parametrize("M,N,K,rank", [(17, 128, 128, 0), (128, 128, 256, 8), (130, 136, 384, 24), (64, 520, 640, 64),
                                        (300, 264, 1024, 256), (1000, 1000, 512, 16)])
def test_prefill_fp16_shapes(fbq, bits, M, N, K, rank):
    inp = make_linear(M, N, K, bits, rank, seed=900 + M + bits)
    rel, _, _, _ = check_parity(inp, fbq, expect_kernel=fbq.KERNEL_PREFILL, floor=2e-5)
    assert rel < 1e-3          # fp16 operands and output: a few 1e-4 expected


@pytest.mark.parametrize("bits", [3, 4])
def test_prefill_sub_branch_alone(fbq, bits):
    # codes == zero points: y is the low-rank product alone (t is rounded once to fp16 here)
    inp = make_linear(96, 256, 1024, bits, 64, seed=910, codes_equal_zero=True, ab_std=0.141)
    check_parity(inp, fbq, expect_kernel=fbq.KERNEL_PREFILL)
    inp = make_linear(64, 256, 512, bits, 0, seed=911)
    check_parity(inp, fbq, expect_kernel=fbq.KERNEL_PREFILL)


@pytest.mark.parametrize("bits", [3, 4])
def test_prefill_exact_class_is_bitwise(fbq, bits):
    # power-of-two scales, small-integer x, dyadic A and B: nothing rounds anywhere (the
    # dequantised weights, t and y are exactly representable in fp16)
    inp = make_exact_class(150, 392, 2048, bits, 64, seed=920, x_nnz=32, x_max=2)
    dev = DeviceLinear(inp, fbq)
    assert fbq.select_kernel(150, 392, 2048, 128, bits, 64) == fbq.KERNEL_PREFILL
    y = torch_to_f64(dev.run(fbq), "f16")
    assert fbq.poll_status() == 0
    assert np.array_equal(y, oracle.linear_inputs(inp, threads=8))


def test_prefill_zero_branches_and_literal_zero_points(fbq):
    import torch
    inp = make_linear(40, 256, 512, 3, 32, seed=930, z_values=(6, 7, 8, 9))
    check_parity(inp, fbq, expect_kernel=fbq.KERNEL_PREFILL)
    dev = DeviceLinear(inp, fbq)
    base = fbq.linear(dev.x, dev.qweight, dev.scales, dev.zeros, None, None, inp.N, 128, 3)
    for A, B in ((torch.zeros_like(dev.A), dev.B), (dev.A, torch.zeros_like(dev.B))):
        assert torch.equal(fbq.linear(dev.x, dev.qweight, dev.scales, dev.zeros, A, B, inp.N, 128, 3), base)


@pytest.mark.parametrize("shape_id", [0, 4, 6])
def test_config2_prefill_bf16_with_outliers(fbq, shape_id):
    # M = 1024, INT4, rank 64, bf16 x with 1 % of the channels scaled by 20; sampled output rows
    K, N = LLAMA2_7B_SHAPES[shape_id]
    inp = make_linear(1024, N, K, 4, 64, dtype="bf16", seed=2000 + shape_id, outlier_frac=0.01)
    rows = np.sort(np.random.default_rng(shape_id).choice(N, size=192, replace=False))
    rel, _, _, _ = check_parity(inp, fbq, expect_kernel=fbq.KERNEL_PREFILL, n_list=rows, threads=16, floor=5e-4)
    assert rel < 4e-3          # ~1.7e-3 from the bf16 output rounding, ~1.6e-3 from bf16 weights


def test_prefill_fp16_full_size(fbq):
    inp = make_linear(1024, 4096, 4096, 3, 64, seed=2100)
    rows = np.sort(np.random.default_rng(5).choice(4096, size=128, replace=False))
    rel, _, _, _ = check_parity(inp, fbq, expect_kernel=fbq.KERNEL_PREFILL, n_list=rows, threads=16, floor=2e-5)
    assert rel < 1e-3


@pytest.mark.parametrize("bits,dtype,M,N,K,rank", [(4, "bf16", 1024, 1160, 1024, 64), (3, "f16", 300, 264, 1024, 256),
                                                   (4, "f16", 513, 136, 512, 0)])
def test_prefill_cta_pair_variant(fbq, bits, dtype, M, N, K, rank):
    # the cta_group::2 kernel (two CTAs share one 256 x 256 x 16 MMA; odd tile counts get a padding CTA)
    fbq.set_option("prefill_pair", 1)
    try:
        inp = make_linear(M, N, K, bits, rank, dtype=dtype, seed=2200 + M, outlier_frac=0.01 if dtype == "bf16" else 0.0)
        check_parity(inp, fbq, expect_kernel=fbq.KERNEL_PREFILL, floor=2e-5 if dtype == "f16" else 5e-4)
        exact = make_exact_class(260, 392, 1024, bits, 64, seed=2300 + bits, x_nnz=32, x_max=2)
        dev = DeviceLinear(exact, fbq)
        assert np.array_equal(torch_to_f64(dev.run(fbq), "f16"), oracle.linear_inputs(exact, threads=8))
        assert fbq.poll_status() == 0
    finally:
        fbq.set_option("prefill_pair", 0)


@pytest.mark.parametrize("bits,dtype,M,N,K,rank", [(3, "f16", 16, 512, 4096, 64), (4, "bf16", 8, 1160, 2048, 128),
                                                   (4, "f16", 100, 384, 1408, 0), (3, "f16", 7, 136, 1024, 8)])
def test_prefill_few_tokens_split_k(fbq, bits, dtype, M, N, K, rank):
    # M <= 128: K is split over several CTAs per tile (fp32 partial tiles, the last CTA adds them up;
    # partial t per split); called three times in a row: the counters must be back at zero each time
    import torch
    inp = make_linear(M, N, K, bits, rank, dtype=dtype, seed=2400 + M, outlier_frac=0.01 if dtype == "bf16" else 0.0)
    fbq.set_option("force_kernel", fbq.KERNEL_PREFILL)
    fbq.set_option("prefill_split", 2)                                      # split whenever the tiles are few
    try:
        check_parity(inp, fbq, expect_kernel=fbq.KERNEL_PREFILL, floor=2e-5 if dtype == "f16" else 5e-4)
        dev = DeviceLinear(inp, fbq)
        ys = [dev.run(fbq).clone() for _ in range(3)]
        torch.cuda.synchronize()
        assert fbq.poll_status() == 0
        assert torch.equal(ys[0], ys[1]) and torch.equal(ys[1], ys[2])      # partials are added in split order
        for mode in (0, 1):                                                 # the unsplit kernel, and the split for deep K only
            fbq.set_option("prefill_split", mode)
            check_parity(inp, fbq, expect_kernel=fbq.KERNEL_PREFILL, floor=2e-5 if dtype == "f16" else 5e-4)
    finally:
        fbq.set_option("force_kernel", -1)
        fbq.set_option("prefill_split", 2)


def test_all_rows_full_size_prefill(fbq):
    """Every output of a 4096 x 4096 projection at M = 1024 (no row sampling), fp16."""
    inp = make_linear(1024, 4096, 4096, 4, 64, seed=90)
    check_parity(inp, fbq, expect_kernel=fbq.KERNEL_PREFILL, threads=16, floor=2e-5)
