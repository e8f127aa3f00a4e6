"""Seeded random shapes through fbq_linear against the CPU oracle: token counts on both sides of every
dispatch boundary, ragged N, K from one group to 11008, ranks from 0 to 256 (multiples of 8 and of 16),
both code widths and activation types, with and without a bound on the decode grid and a forced
number of K slices.  Whatever kernel the dispatcher picks must meet the tolerances."""
import numpy as np
import pytest

import oracle
from gpu_utils import REL_F_TOL, DeviceLinear, compare, torch_to_f64
from workloads import make_linear

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fbq():
    import torch
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    import paper_2501_16385_b200 as lib
    lib.set_option("force_kernel", -1)
    return lib


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_shapes_meet_the_tolerances(fbq, seed):
    import torch
    rng = np.random.default_rng(seed)
    kernels = set()
    for it in range(40):
        bits = int(rng.choice([3, 4]))
        dtype = str(rng.choice(["f16", "bf16"]))
        M = int(rng.choice([1, 1, 1, 2, 2, 3, 4, 5, 6, 7, 8, 16, 40, 130]))
        K = int(rng.choice([128, 256, 384, 1024, 1152, 2048, 4096, 5120, 11008]))
        N = int(rng.choice([8, 16, 24, 136, 520, 1000, 2048, 4096, 4104]))
        rank = int(rng.choice([0, 8, 16, 24, 32, 48, 64, 72, 128, 256]))
        ctas = int(rng.choice([0, 0, 0, 5, 16, 33, 89]))
        sk = int(rng.choice([0, 0, 0, 2, 3]))
        if N * K > 30e6:
            N = 1000
        inp = make_linear(M, N, K, bits, rank, dtype=dtype, seed=9000 * seed + it, outlier_frac=float(rng.choice([0.0, 0.01])))
        what = dict(bits=bits, dtype=dtype, M=M, N=N, K=K, rank=rank, ctas=ctas, sk=sk)
        fbq.set_option("decode_ctas", ctas)
        fbq.set_option("decode_sk", sk)
        try:
            dev = DeviceLinear(inp, fbq)
            y = dev.run(fbq)
            torch.cuda.synchronize()
            assert fbq.poll_status() == 0, what
        finally:
            fbq.set_option("decode_ctas", 0)
            fbq.set_option("decode_sk", 0)
        kernels.add(fbq.select_kernel(M, N, K, 128, bits, rank, dtype == "bf16"))
        y64 = torch_to_f64(y, dtype)
        y_or = oracle.linear_inputs(inp, threads=8)
        assert np.all(np.isfinite(y64)), what
        rel, mx, lim = compare(y64, y_or, inp.x_f64(), K)
        if dtype == "bf16":
            lim += 2.0 ** -8 * float(np.abs(y_or).max())          # half an ulp of the largest output (8 significant bits)
        assert rel <= REL_F_TOL, (what, rel)
        assert mx <= lim, (what, mx, lim)
    assert fbq.KERNEL_DECODE in kernels and fbq.KERNEL_PREFILL in kernels
