"""GPU parity of fbq_quantize_feedback (Section 4.1: main path Q(W - B.A)) against the CPU oracle:
codes, scales and zero points bit for bit, W_F bit for bit (both sides take every rounding decision
in single precision, in the same order), and the layer built from its output against x.W_F^T."""
import numpy as np
import pytest

import oracle
from workloads import f32_to_bf16_bits

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fbq():
    import torch
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    import paper_2501_16385_b200 as lib
    lib.set_option("force_kernel", -1)
    return lib


def _inputs(N, K, rank, dtype, seed, w_std=0.02, ab_std=0.05, outliers=True):
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((N, K)) * w_std).astype(np.float32)
    if outliers:
        idx = rng.integers(0, N * K, size=max(1, N * K // 500))
        W.ravel()[idx] *= 12.0
    if rank == 0:
        return W, None, None
    A32 = (rng.standard_normal((rank, K)) * ab_std).astype(np.float32)
    B32 = (rng.standard_normal((N, rank)) * ab_std).astype(np.float32)
    if dtype == "bf16":
        return W, f32_to_bf16_bits(A32), f32_to_bf16_bits(B32)
    return W, A32.astype(np.float16).view(np.uint16), B32.astype(np.float16).view(np.uint16)


def _dev16(bits, dtype):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda()
    return t.view(torch.bfloat16 if dtype == "bf16" else torch.float16)


def _run(fbq, W, A, B, group, bits, dtype):
    import torch
    Wd = torch.from_numpy(W).cuda()
    Ad = _dev16(A, dtype) if A is not None else None
    Bd = _dev16(B, dtype) if B is not None else None
    codes, s, z, wf = fbq.quantize_feedback(Wd, Ad, Bd, group, bits, want_wf=True)
    torch.cuda.synchronize()
    return (codes.cpu().numpy(), s.view(torch.int16).cpu().numpy().view(np.uint16),
            z.view(torch.int16).cpu().numpy().view(np.uint16), wf.cpu().numpy(), (Wd, Ad, Bd, codes, s, z))


@pytest.mark.parametrize("bits", [3, 4])
@pytest.mark.parametrize("N,K,group,rank,dtype", [(40, 512, 128, 0, "f16"), (33, 640, 128, 16, "f16"), (17, 384, 128, 64, "bf16"),
                                                 (9, 256, 32, 8, "f16"), (5, 64, 8, 24, "bf16"), (3, 2048, 1024, 4, "f16")])
def test_quantizer_matches_oracle_bit_for_bit(fbq, bits, N, K, group, rank, dtype):
    W, A, B = _inputs(N, K, rank, dtype, seed=5000 + N + bits)
    W[0, :group] = 0.0                                   # a constant group and a constant negative one
    if N > 1:
        W[1, :group] = -0.375
    codes, s, z, wf, _ = _run(fbq, W, A, B, group, bits, dtype)
    c_or, s_or, z_or, _, wf_or = oracle.quantize_feedback(W, A, B, group, bits, dtype=dtype)
    assert np.array_equal(s, s_or) and np.array_equal(z, z_or)
    assert np.array_equal(codes, c_or)
    assert np.array_equal(wf.view(np.uint32), wf_or.view(np.uint32))
    assert codes.max() == (1 << bits) - 1 and codes.min() == 0


def test_worked_example_on_the_device(fbq):
    r = np.array([[-1.75, -1, 0.125, 0.375, 0.625, 0.3, 1.9, 2]], dtype=np.float32)
    codes, s, z, wf, _ = _run(fbq, r, None, None, 8, 4, "f16")
    assert codes[0].tolist() == [0, 3, 8, 8, 10, 8, 15, 15]          # ties to even at 7.5, 8.5, 9.5
    assert s.view(np.float16)[0, 0] == 0.25 and z.view(np.float16)[0, 0] == 7
    assert wf[0].tolist() == [-1.75, -1, 0.25, 0.25, 0.75, 0.25, 2, 2]


@pytest.mark.parametrize("bits,dtype", [(3, "f16"), (4, "bf16")])
def test_full_size_rows_sampled(fbq, bits, dtype):
    # a Llama-2-7B sized projection; the oracle recomputes 96 sampled rows (rows are independent)
    N, K, rank = 4096, 4096, 64
    W, A, B = _inputs(N, K, rank, dtype, seed=5100 + bits, outliers=False)
    codes, s, z, wf, _ = _run(fbq, W, A, B, 128, bits, dtype)
    rows = np.sort(np.random.default_rng(bits).choice(N, size=96, replace=False))
    c_or, s_or, z_or, _, wf_or = oracle.quantize_feedback(W[rows], A, B[rows], 128, bits, dtype=dtype)
    assert np.array_equal(codes[rows], c_or) and np.array_equal(s[rows], s_or) and np.array_equal(z[rows], z_or)
    assert np.array_equal(wf[rows].view(np.uint32), wf_or.view(np.uint32))
    # Eq. "diff" bound on every weight the clamp left alone, in double precision
    s64 = np.repeat(s.view(np.float16).astype(np.float64), 128, axis=1)
    err = np.abs(W.astype(np.float64) - wf.astype(np.float64))
    assert np.mean(err <= 0.5 * s64 + 1e-6) > 0.999


@pytest.mark.parametrize("bits,M", [(3, 1), (4, 40)])
def test_quantise_pack_and_run_the_layer(fbq, bits, M):
    # (codes, s, z) from the quantiser, packed, run through fbq_linear with the same sub-branch:
    # y = x.dequant(Q)^T + (x.A^T).B^T = x.W_F^T, and within the quantisation bound of x.W^T.
    import torch
    N, K, rank, dtype = 264, 1024, 32, "f16"
    W, A, B = _inputs(N, K, rank, dtype, seed=5200 + bits, outliers=False)
    codes, s, z, wf, dev = _run(fbq, W, A, B, 128, bits, dtype)
    Wd, Ad, Bd, codes_d, s_d, z_d = dev
    x = (np.random.default_rng(1).standard_normal((M, K))).astype(np.float16)
    xd = torch.from_numpy(x).cuda()
    y = fbq.linear(xd, fbq.pack(codes_d, bits), s_d, z_d, Ad, Bd, N, 128, bits)
    torch.cuda.synchronize()
    y64 = y.float().cpu().numpy().astype(np.float64)
    want = x.astype(np.float64) @ wf.astype(np.float64).T
    rel = np.linalg.norm(y64 - want) / np.linalg.norm(want)
    assert rel <= 5e-3
    s64 = np.repeat(s.view(np.float16).astype(np.float64), 128, axis=1)
    bound = np.abs(x.astype(np.float64)) @ (0.5 * s64).T
    exact = x.astype(np.float64) @ W.astype(np.float64).T
    assert np.all(np.abs(want - exact) <= bound * (1 + 1e-3) + 1e-4)


def test_quantizer_rejects_bad_requests(fbq):
    import torch
    L = fbq.lib()
    W = torch.zeros((4, 64), dtype=torch.float32, device="cuda")
    c = torch.zeros((4, 64), dtype=torch.uint8, device="cuda")
    s = torch.zeros((4, 2), dtype=torch.float16, device="cuda")
    args = lambda group, bits, rank: (W.data_ptr(), None, None, c.data_ptr(), s.data_ptr(), s.data_ptr(), None, 4, 64, group, bits, rank, 0, None)
    assert L.fbq_quantize_feedback(*args(32, 4, 0)) == 0
    assert L.fbq_quantize_feedback(*args(48, 4, 0)) != 0        # group does not divide K
    assert L.fbq_quantize_feedback(*args(32, 5, 0)) != 0
    assert L.fbq_quantize_feedback(*args(32, 4, 8)) != 0        # rank > 0 without A, B
    torch.cuda.synchronize()


@pytest.mark.parametrize("bits", [3, 4])
@pytest.mark.parametrize("dtype,M", [("f16", 1), ("f16", 2), ("f16", 4), ("f16", 64), ("bf16", 64)])
def test_zero_points_outside_the_code_range_run_on_every_kernel(fbq, bits, dtype, M):
    """Groups that do not straddle zero get zero points the quantiser does not clamp: negative for an
    all-positive group, beyond 2^bits - 1 for an all-negative one.  Every kernel must take them as they are
    stored (fp16 integers of either sign): the streaming decode kernel (M <= 2), the other decode kernel
    (M = 4), the prefill kernel in fp16 and bf16 -- checked against the oracle on the quantiser's output."""
    import torch
    N, K, rank = 272, 1024, 16
    rng = np.random.default_rng(5300 + bits)
    W = (rng.standard_normal((N, K)) * 0.02).astype(np.float32)
    W[0::3] = np.abs(W[0::3]) + 0.05           # all-positive rows: z = rint(-min/s) < 0
    W[1::3] = -np.abs(W[1::3]) - 0.05          # all-negative rows: z > 2^bits - 1
    _, A, B = _inputs(N, K, rank, dtype, seed=5310 + bits)
    codes, s, z, wf, dev = _run(fbq, W, A, B, 128, bits, dtype)
    zf = z.view(np.float16).astype(np.float64)
    assert zf.min() < 0 and zf.max() > (1 << bits) - 1 and np.all(zf == np.rint(zf))
    Wd, Ad, Bd, codes_d, s_d, z_d = dev
    x32 = np.random.default_rng(2).standard_normal((M, K)).astype(np.float32)
    x_bits = f32_to_bf16_bits(x32) if dtype == "bf16" else x32.astype(np.float16).view(np.uint16)
    xd = _dev16(x_bits, dtype)
    y = fbq.linear(xd, fbq.pack(codes_d, bits), s_d, z_d, Ad, Bd, N, 128, bits)
    torch.cuda.synchronize()
    assert fbq.poll_status() == 0
    got = y.float().cpu().numpy().astype(np.float64)
    want = oracle.linear(x_bits, oracle.pack(codes, bits), s, z, A, B, M, N, K, 128, bits, rank, dtype=dtype, threads=8)
    rel = np.linalg.norm(got - want) / np.linalg.norm(want)
    assert rel <= 5e-3, rel
    xmax = float(np.max(np.abs(x32)))
    lim = 1e-2 * xmax * np.sqrt(K) / 64.0
    if dtype == "bf16":
        lim += 2.0 ** -8 * float(np.max(np.abs(want)))
    assert np.max(np.abs(got - want)) <= lim
