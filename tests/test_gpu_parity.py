"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle
on the same seeded inputs.  Bit-exact for packing, unpacking and dequantised
values; relative Frobenius error <= 5e-3 and max-abs error <= 1e-2*||x||inf*
sqrt(K)/64 for the layer output (fp16/bf16 output, fp32 accumulation)."""
import numpy as np
import pytest

import oracle
from workloads import (LLAMA2_13B_SHAPES, LLAMA2_7B_SHAPES, make_exact_class, make_linear,
                       worked_example_e1)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fbq():
    import torch
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    import paper_2501_16385_b200 as lib
    lib.set_option("force_kernel", -1)
    yield lib
    lib.set_option("force_kernel", -1)
    for name in ("decode_sk", "decode_chunk", "decode_depth", "decode_ctas", "decode_t_late"):
        lib.set_option(name, 0)


@pytest.fixture()
def torch():
    import torch as t
    return t


from gpu_utils import (DeviceLinear, REL_F_TOL, check_parity, compare, f16_to_torch,  # noqa: E402
                       torch_to_f64)


# ------------------------------------------------------------ packing / dequant
@pytest.mark.parametrize("bits", [3, 4])
@pytest.mark.parametrize("N,K", [(1, 32), (8, 128), (40, 1024), (100, 4096), (16, 11008)])
def test_pack_unpack_bit_exact(fbq, torch, bits, N, K):
    rng = np.random.default_rng(N + K + bits)
    qmax = (1 << bits) - 1
    for codes in (rng.integers(0, qmax + 1, size=(N, K), dtype=np.uint8),
                  np.full((N, K), qmax, dtype=np.uint8), np.zeros((N, K), dtype=np.uint8)):
        d = torch.from_numpy(codes).cuda()
        q = fbq.pack(d, bits)
        assert np.array_equal(q.cpu().numpy().view(np.uint32), oracle.pack(codes, bits))
        back = fbq.unpack(q, N, K, bits)
        assert np.array_equal(back.cpu().numpy(), codes)
        # unpacking words produced by the oracle's packer gives the codes as well
        q2 = torch.from_numpy(oracle.pack(codes, bits).view(np.int32)).cuda()
        assert np.array_equal(fbq.unpack(q2, N, K, bits).cpu().numpy(), codes)


def test_pack_literal_words(fbq, torch):
    c4 = torch.tensor([[0, 5, 10, 15, 4, 9, 14, 3]], dtype=torch.uint8).cuda()
    assert fbq.pack(c4, 4).cpu().numpy().view(np.uint32).tolist() == [0x3E94FA50]
    c3 = torch.tensor([[(5 * j + 3) % 8 for j in range(32)]], dtype=torch.uint8).cuda()
    assert fbq.pack(c3, 3).cpu().numpy().view(np.uint32).tolist() == [0x078CF543, 0xAA1E19D5, 0xCEA83C67]


@pytest.mark.parametrize("bits,group", [(4, 8), (4, 128), (3, 32), (3, 128)])
def test_dequant_bit_exact(fbq, torch, bits, group):
    inp = make_linear(1, 72, 1024, bits, 0, group=group, seed=3)
    q = fbq.pack(torch.from_numpy(inp.codes).cuda(), bits)
    W = fbq.dequant(q, f16_to_torch(inp.scales), f16_to_torch(inp.zeros), 72, 1024, group, bits)
    want = oracle.dequant(oracle.pack(inp.codes, bits), inp.scales, inp.zeros, 72, 1024, group, bits)
    assert np.array_equal(W.cpu().numpy().astype(np.float64), want)


# --------------------------------------------------------------- generic kernel
def test_e1_worked_example_on_gpu(fbq, torch):
    inp = worked_example_e1()
    dev = DeviceLinear(inp, fbq)
    assert fbq.select_kernel(1, 8, 8, 8, 4, 2) == fbq.KERNEL_GENERIC
    y = torch_to_f64(dev.run(fbq), "f16")
    assert y[0].tolist() == [5.75, -0.6875, 0.125, -0.0625, 2.5, -0.6875, -3.875, 0.6875]
    assert dev.qweight.cpu().numpy().view(np.uint32).tolist() == [
        0x3E94FA50, 0x61C72D83, 0x94FA50B6, 0xC72D83E9, 0xFA50B61C, 0x2D83E94F, 0x50B61C72, 0x83E94FA5]


@pytest.mark.parametrize("bits,dtype,M,N,K,group,rank", [
    (4, "f16", 1, 40, 256, 64, 8), (3, "f16", 3, 33, 512, 32, 5), (4, "bf16", 9, 17, 128, 16, 2),
    (3, "bf16", 20, 24, 256, 64, 0), (4, "f16", 5, 64, 512, 128, 12), (4, "f16", 1, 64, 1024, 128, 264)])
def test_generic_kernel_parity(fbq, bits, dtype, M, N, K, group, rank):
    inp = make_linear(M, N, K, bits, rank, group=group, dtype=dtype, seed=40 + M)
    check_parity(inp, fbq, expect_kernel=fbq.KERNEL_GENERIC)


def test_generic_forced_on_decode_shape(fbq):
    inp = make_linear(2, 256, 1024, 4, 16, seed=50)
    fbq.set_option("force_kernel", fbq.KERNEL_GENERIC)
    try:
        check_parity(inp, fbq, expect_kernel=fbq.KERNEL_GENERIC, floor=2e-5)
    finally:
        fbq.set_option("force_kernel", -1)


# ---------------------------------------------------------------- decode kernel
def test_config0_single_linear(fbq):
    # M=1, K=N=4096, INT4, group 128, rank 32 (expected error ~2e-4 from the fp16 output rounding)
    inp = make_linear(1, 4096, 4096, 4, 32, seed=0)
    rel, mx, _, _ = check_parity(inp, fbq, expect_kernel=fbq.KERNEL_DECODE, floor=2e-5)
    assert rel < 1e-3


@pytest.mark.parametrize("bits", [3, 4])
@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("M", [1, 2, 3, 8, 9, 15, 16])
def test_decode_token_counts(fbq, bits, dtype, M):
    inp = make_linear(M, 272, 1024, bits, 16, dtype=dtype, seed=100 + M)
    check_parity(inp, fbq, expect_kernel=fbq.KERNEL_DECODE, floor=1e-5)


@pytest.mark.parametrize("bits", [3, 4])
@pytest.mark.parametrize("N,K,rank", [(16, 128, 8), (8, 256, 0), (24, 384, 8), (1000, 640, 24), (4096, 128, 64),
                                      (40, 11008, 128), (5, 1280, 256)])
def test_decode_ragged_shapes(fbq, bits, N, K, rank):
    inp = make_linear(3, N, K, bits, rank, seed=7 * N + K)
    check_parity(inp, fbq, expect_kernel=fbq.KERNEL_DECODE)


@pytest.mark.parametrize("bits", [3, 4])
def test_decode_rank0_and_zero_branches_agree(fbq, torch, bits):
    inp = make_linear(2, 512, 2048, bits, 32, seed=11)
    dev = DeviceLinear(inp, fbq)
    y_full = dev.run(fbq)
    base = fbq.linear(dev.x, dev.qweight, dev.scales, dev.zeros, None, None, inp.N, 128, bits)
    for A, B in ((torch.zeros_like(dev.A), dev.B), (dev.A, torch.zeros_like(dev.B))):
        y = fbq.linear(dev.x, dev.qweight, dev.scales, dev.zeros, A, B, inp.N, 128, bits)
        assert torch.equal(y, base)            # the sub-branch only adds into the shared output
    assert not torch.equal(y_full, base)
    inp0 = make_linear(2, 512, 2048, bits, 0, seed=11)
    check_parity(inp0, fbq, expect_kernel=fbq.KERNEL_DECODE)


@pytest.mark.parametrize("M,N,K,rank", [(1, 512, 4096, 64), (2, 256, 4096, 128), (1, 256, 11008, 64), (8, 512, 4096, 64),
                                        (16, 256, 4096, 128), (4, 256, 11008, 32)])
def test_streaming_kernel_zero_t_is_not_taken_for_missing(fbq, torch, M, N, K, rank):
    # x = 0 makes every partial sum of t an exact zero.  The t slots announce themselves by being non-zero (a zero
    # is stored as -0.0), so an all-zero t must neither time out nor change y: one slot per t CTA, the slot of the
    # sum where there are many entries (K = 11008), both forms of the kernel
    inp = make_linear(M, N, K, 3, rank, seed=31 * M + rank)
    dev = DeviceLinear(inp, fbq)
    fbq.set_option("force_kernel", fbq.KERNEL_DECODE)
    try:
        for x in (torch.zeros_like(dev.x), -torch.zeros_like(dev.x)):
            y = dev.run(fbq, x=x)
            torch.cuda.synchronize()
            assert fbq.poll_status() == 0
            assert torch.count_nonzero(y).item() == 0
        check_parity(inp, fbq, expect_kernel=fbq.KERNEL_DECODE)       # and the slots are clean for the next call
    finally:
        fbq.set_option("force_kernel", -1)


@pytest.mark.parametrize("bits,dtype", [(4, "f16"), (3, "f16"), (4, "bf16"), (3, "bf16")])
def test_decode_sub_branch_alone(fbq, bits, dtype):
    # codes == zero points: the main path vanishes and y is the low-rank product alone,
    # so a sub-branch error cannot hide inside the main path's tolerance.
    # (bf16 keeps 8 significant bits: with a smaller std, y stays below 4 and half an
    # output ulp stays below the max-abs bound, so that the bound tests the kernel)
    std = 0.141 if dtype == "f16" else 0.06
    inp = make_linear(4, 512, 1024, bits, 64, dtype=dtype, seed=13, codes_equal_zero=True, ab_std=std)
    check_parity(inp, fbq, expect_kernel=fbq.KERNEL_DECODE)
    inp = make_linear(1, 4096, 4096, bits, 32, dtype=dtype, seed=14, ab_std=std)
    check_parity(inp, fbq, expect_kernel=fbq.KERNEL_DECODE)


def test_decode_int3_literal_zero_point_range(fbq):
    # zero points 6..9 lie partly outside the 3-bit code range; any integer zero point must work
    inp = make_linear(1, 512, 1024, 3, 16, seed=15, z_values=(6, 7, 8, 9))
    check_parity(inp, fbq, expect_kernel=fbq.KERNEL_DECODE)
    inp = make_linear(2, 512, 1024, 4, 16, seed=16, z_values=(0, 15, 1, 14))
    check_parity(inp, fbq, expect_kernel=fbq.KERNEL_DECODE)


@pytest.mark.parametrize("bits,dtype,M", [(4, "f16", 1), (3, "f16", 4), (4, "f16", 12), (4, "bf16", 3),
                                          (3, "bf16", 16)])
def test_decode_exact_class_is_bitwise(fbq, bits, dtype, M):
    kw = dict(x_nnz=32, x_max=2) if dtype == "f16" else dict(x_nnz=4, x_max=1)
    inp = make_exact_class(M, 528, 4096, bits, 64, dtype=dtype, seed=21 + M, **kw)
    dev = DeviceLinear(inp, fbq)
    y = torch_to_f64(dev.run(fbq), dtype)
    y_or = oracle.linear_inputs(inp, threads=8)
    assert np.array_equal(y, y_or)


def test_decode_unit_vectors_read_columns(fbq, torch):
    inp = make_linear(8, 64, 1024, 4, 8, seed=23)
    ks = [0, 7, 31, 32, 127, 128, 640, 1023]
    x = np.zeros((8, 1024), dtype=np.float16)
    for m, k in enumerate(ks):
        x[m, k] = 1.0
    inp.x = x.view(np.uint16)
    rel, mx, y, y_or = check_parity(inp, fbq, expect_kernel=fbq.KERNEL_DECODE)
    assert np.max(np.abs(y - y_or)) < 2e-4       # column entries are ~0.06: fp16 rounding only


def test_decode_linearity_and_token_independence(fbq, torch):
    inp = make_linear(3, 256, 2048, 4, 32, seed=25)
    rng = np.random.default_rng(1)
    x1 = rng.integers(-8, 9, size=2048).astype(np.float16)
    x2 = rng.integers(-8, 9, size=2048).astype(np.float16)
    x3 = (0.5 * x1.astype(np.float64) - 2.0 * x2.astype(np.float64)).astype(np.float16)
    inp.x = np.stack([x1, x2, x3]).view(np.uint16)
    rel, mx, y, _ = check_parity(inp, fbq)
    lin = 0.5 * y[0] - 2.0 * y[1]
    assert np.linalg.norm(y[2] - lin) <= 2 * REL_F_TOL * np.linalg.norm(lin)
    dev = DeviceLinear(inp, fbq)
    for m in range(3):
        ym = torch_to_f64(dev.run(fbq, x=dev.x[m:m + 1].contiguous()), "f16")
        assert np.linalg.norm(ym[0] - y[m]) <= 1e-3 * np.linalg.norm(y[m])


def test_decode_parked_tiles_path(fbq):
    # Test switch: t is contributed only after the main loop, so every tile is parked and
    # finished by the warp that completes t (the rarely taken branch of the protocol).
    fbq.set_option("decode_t_late", 1)
    try:
        for M, bits in ((1, 4), (5, 3), (16, 4)):
            check_parity(make_linear(M, 1040, 2048, bits, 32, seed=60 + M), fbq, expect_kernel=fbq.KERNEL_DECODE)
    finally:
        fbq.set_option("decode_t_late", 0)
    check_parity(make_linear(2, 1040, 2048, 4, 32, seed=66), fbq, expect_kernel=fbq.KERNEL_DECODE)


@pytest.mark.parametrize("sk,chunk,depth,ctas", [(1, 1, 1, 0), (2, 2, 2, 0), (3, 5, 3, 0), (8, 3, 2, 40), (16, 4, 4, 0),
                                                 (1, 8, 2, 7)])
def test_decode_tuning_variants(fbq, sk, chunk, depth, ctas):
    for name, v in (("decode_sk", sk), ("decode_chunk", chunk), ("decode_depth", depth), ("decode_ctas", ctas)):
        fbq.set_option(name, v)
    try:
        for bits, rank in ((4, 0), (3, 16), (4, 64)):
            check_parity(make_linear(2, 1040, 3072, bits, rank, seed=70 + sk), fbq, expect_kernel=fbq.KERNEL_DECODE)
    finally:
        for name in ("decode_sk", "decode_chunk", "decode_depth", "decode_ctas"):
            fbq.set_option(name, 0)


def test_decode_scratch_is_clean_between_calls(fbq, torch):
    # alternate shapes with different tile counts and ranks on one stream; each result must
    # still be right, and repeating a call must reproduce it bit for bit when rank == 0
    shapes = [(1, 4096, 4096, 4, 32), (16, 528, 1024, 3, 64), (1, 272, 2048, 4, 0), (4, 11008, 512, 3, 8),
              (1, 4096, 4096, 4, 32)]
    for rep in range(2):
        for i, (M, N, K, bits, rank) in enumerate(shapes):
            check_parity(make_linear(M, N, K, bits, rank, seed=80 + i), fbq, expect_kernel=fbq.KERNEL_DECODE)
    inp = make_linear(1, 4096, 4096, 4, 0, seed=90)
    dev = DeviceLinear(inp, fbq)
    y1 = dev.run(fbq).clone()
    for _ in range(5):
        assert torch.equal(dev.run(fbq), y1)


def test_decode_many_back_to_back_launches(fbq, torch):
    # programmatic dependent launch lets consecutive calls overlap; results must not change
    inps = [make_linear(1, 1024, 2048, 4, 32, seed=200 + i) for i in range(6)]
    devs = [DeviceLinear(i, fbq) for i in inps]
    ys = [None] * len(devs)
    for rep in range(4):
        for j, d in enumerate(devs):
            ys[j] = d.run(fbq)
    torch.cuda.synchronize()
    for inp, y in zip(inps, ys):
        y_or = oracle.linear_inputs(inp, threads=8)
        rel, mx, lim = compare(torch_to_f64(y, "f16"), y_or, inp.x_f64(), inp.K)
        assert rel <= REL_F_TOL and mx <= lim


def test_decode_concurrent_streams(fbq, torch):
    # Independent linears issued on several streams at once (each stream has its own scratch
    # space), with the grid limited so that launches of different streams share the SMs: the
    # launch configuration bench.py times.
    inps = [make_linear(1, N, K, 3, 64, seed=600 + i) for i, (K, N) in enumerate(LLAMA2_7B_SHAPES)]
    devs = [DeviceLinear(i, fbq) for i in inps]
    streams = [torch.cuda.Stream() for _ in range(7)]
    fbq.set_option("decode_ctas", 74)
    try:
        torch.cuda.synchronize()
        ys = [None] * len(devs)
        for rep in range(3):
            for j, d in enumerate(devs):
                i = d.inp
                ys[j] = fbq.linear(d.x, d.qweight, d.scales, d.zeros, d.A, d.B, i.N, i.group, i.bits,
                                   stream=streams[j % 7])
        torch.cuda.synchronize()
        for st in streams:
            assert fbq.poll_status(st) == 0
    finally:
        fbq.set_option("decode_ctas", 0)
    for inp, y in zip(inps, ys):
        y_or = oracle.linear_inputs(inp, threads=8)
        rel, mx, lim = compare(torch_to_f64(y, "f16"), y_or, inp.x_f64(), inp.K)
        assert rel <= REL_F_TOL and mx <= lim


# ---------------------------------------------------- workload-sized parity cases
@pytest.mark.parametrize("shape_id", [0, 4, 6])
def test_config1_llama7b_int3_rank64(fbq, shape_id):
    K, N = LLAMA2_7B_SHAPES[shape_id]
    inp = make_linear(1, N, K, 3, 64, seed=1000 + shape_id)
    rel, _, _, _ = check_parity(inp, fbq, expect_kernel=fbq.KERNEL_DECODE, floor=2e-5)
    assert rel < 1e-3
    inp = make_linear(1, N, K, 3, 64, seed=1000 + shape_id, z_values=(6, 7, 8, 9))
    check_parity(inp, fbq, expect_kernel=fbq.KERNEL_DECODE)


@pytest.mark.parametrize("shape_id", [0, 4, 6])
@pytest.mark.parametrize("M,bits", [(1, 3), (16, 4), (16, 3), (1, 4)])
def test_config3_llama13b(fbq, shape_id, M, bits):
    K, N = LLAMA2_13B_SHAPES[shape_id]
    inp = make_linear(M, N, K, bits, 64, seed=3000 + shape_id)
    rows = np.sort(np.random.default_rng(shape_id).choice(N, size=512, replace=False)) if M > 1 else None
    check_parity(inp, fbq, expect_kernel=fbq.KERNEL_DECODE, n_list=rows, floor=2e-5)


@pytest.mark.parametrize("M,rank", [(1, 0), (2, 16), (4, 32), (8, 64), (16, 128)])
def test_config4_stack_samples(fbq, M, rank):
    for shape_id in (0, 5, 6):
        K, N = LLAMA2_7B_SHAPES[shape_id]
        inp = make_linear(M, N, K, 4, rank, seed=4000 + 7 * 15 + shape_id)
        rows = np.sort(np.random.default_rng(M).choice(N, size=256, replace=False))
        check_parity(inp, fbq, expect_kernel=fbq.KERNEL_DECODE, n_list=rows, floor=2e-5)


# ------------------------------------------------------------------ other entries
def test_hostio_entry_point(fbq, torch):
    inp = make_linear(2, 512, 1024, 4, 16, seed=300)
    dev = DeviceLinear(inp, fbq)
    xh = dev.x.cpu().pin_memory()
    yh = torch.empty((2, 512), dtype=torch.float16).pin_memory()
    fbq.linear_hostio(xh, dev.qweight, dev.scales, dev.zeros, dev.A, dev.B, yh, 512, 128, 4)
    torch.cuda.synchronize()
    ref = dev.run(fbq).cpu()
    assert torch.equal(yh, ref)
    # y in pageable memory, and the direct write switched off: both go through the staging buffer and a copy
    yp = torch.zeros((2, 512), dtype=torch.float16)
    fbq.linear_hostio(xh, dev.qweight, dev.scales, dev.zeros, dev.A, dev.B, yp, 512, 128, 4)
    torch.cuda.synchronize()
    assert torch.equal(yp, ref)
    fbq.set_option("hostio_direct_y", 0)
    try:
        yh.zero_()
        fbq.linear_hostio(xh, dev.qweight, dev.scales, dev.zeros, dev.A, dev.B, yh, 512, 128, 4)
        torch.cuda.synchronize()
        assert torch.equal(yh, ref)
    finally:
        fbq.set_option("hostio_direct_y", 1)
    # a y too large to be written across the bus by the kernel (prefill-sized): staged
    big = make_linear(300, 512, 1024, 4, 16, seed=302)
    dbig = DeviceLinear(big, fbq)
    yb = torch.zeros((300, 512), dtype=torch.float16).pin_memory()
    fbq.linear_hostio(dbig.x.cpu().pin_memory(), dbig.qweight, dbig.scales, dbig.zeros, dbig.A, dbig.B, yb, 512, 128, 4)
    torch.cuda.synchronize()
    assert torch.equal(yb, dbig.run(fbq).cpu())
    assert fbq.poll_status() == 0


def test_launch_counter_counts_kernels(fbq, torch):
    inp = make_linear(1, 256, 1024, 4, 16, seed=301)
    dev = DeviceLinear(inp, fbq)
    before = fbq.launch_count()
    dev.run(fbq)
    assert fbq.launch_count() == before + 1          # decode: one fused launch
    fbq.set_option("force_kernel", fbq.KERNEL_GENERIC)
    try:
        before = fbq.launch_count()
        dev.run(fbq)
        assert fbq.launch_count() == before + 2      # generic: down-projection + main
    finally:
        fbq.set_option("force_kernel", -1)


def test_empty_and_status(fbq, torch):
    inp = make_linear(1, 64, 256, 4, 8, seed=302)
    dev = DeviceLinear(inp, fbq)
    x0 = torch.empty((0, 256), dtype=torch.float16, device="cuda")
    y0 = fbq.linear(x0, dev.qweight, dev.scales, dev.zeros, dev.A, dev.B, 64, 128, 4)
    assert y0.shape == (0, 64)
    assert fbq.poll_status() == 0


# ------------------------------------------------------------ contracts the header states
def test_non_finite_x_reaches_the_outputs(fbq, torch):
    """An Inf or a NaN in x makes every output of its token non-finite, as the definition says (every output row
    sums over every input channel) -- also in the integer form, where x passes through fixed point."""
    for bits, M, rank in ((4, 1, 0), (3, 1, 32), (4, 2, 0)):
        inp = make_linear(M, 256, 1024, bits, rank, seed=77)
        dev = DeviceLinear(inp, fbq)
        for bad in (float("inf"), float("nan")):
            x = dev.x.clone()
            x[M - 1, 300] = bad
            y = torch_to_f64(dev.run(fbq, x=x), "f16")
            assert not np.any(np.isfinite(y[M - 1])), (bits, M, rank, bad)
            if M > 1:
                assert np.all(np.isfinite(y[0]))           # the other token is untouched
        assert fbq.poll_status() == 0


def test_growing_scratch_inside_a_capture_is_refused(fbq, torch):
    """A call that would have to allocate scratch while its stream is being captured returns
    FBQ_ERR_UNSUPPORTED and queues nothing; the capture itself stays valid."""
    fbq.release_workspaces()
    inp = make_linear(1, 256, 1024, 4, 32, seed=78)
    dev = DeviceLinear(inp, fbq)
    st = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(st):
        with torch.cuda.graph(g, stream=st):
            with pytest.raises(fbq.FbqError) as err:
                fbq.linear(dev.x, dev.qweight, dev.scales, dev.zeros, dev.A, dev.B, inp.N, 128, 4, stream=st)
            assert err.value.code == -2
        st.synchronize()
        y = fbq.linear(dev.x, dev.qweight, dev.scales, dev.zeros, dev.A, dev.B, inp.N, 128, 4, stream=st)   # outside: allocates
        g2 = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g2, stream=st):
            fbq.linear(dev.x, dev.qweight, dev.scales, dev.zeros, dev.A, dev.B, inp.N, 128, 4, y=y, stream=st)
        g2.replay()
        st.synchronize()
    want = oracle.linear_inputs(inp, threads=8)
    rel, mx, lim = compare(torch_to_f64(y, "f16"), want, inp.x_f64(), inp.K)
    assert rel <= REL_F_TOL and mx <= lim


def test_all_rows_full_size_decode_m16(fbq):
    """Every output of a 13 824 x 5120 projection at M = 16 (no row sampling), through the decode kernel."""
    inp = make_linear(16, 13824, 5120, 4, 64, seed=79)
    check_parity(inp, fbq, expect_kernel=fbq.KERNEL_DECODE, threads=16, floor=2e-5)


def test_all_rows_full_size_streaming_kernel(fbq):
    """Every output of the three 7B shapes at M = 1 and of one of them at M = 2."""
    for M, (K, N), bits in ((1, (4096, 4096), 3), (1, (4096, 11008), 3), (1, (11008, 4096), 3), (2, (11008, 4096), 4)):
        inp = make_linear(M, N, K, bits, 64, seed=80 + M)
        check_parity(inp, fbq, expect_kernel=fbq.KERNEL_DECODE, threads=16, floor=2e-5)


@pytest.mark.parametrize("M,bits,rank,dtype", [(1, 3, 64, "f16"), (2, 4, 32, "f16"), (8, 4, 64, "bf16")])
def test_unfused_comparator_computes_the_same_layer(fbq, torch, M, bits, rank, dtype):
    """The paper's unfused layer (main path, then the low-rank branch as launches of its own), built from this
    library's kernels for the benchmark's comparison, against the oracle: same tolerance as the fused call (its
    extra rounding of u and of y is far inside it)."""
    inp = make_linear(M, 1024, 2048, bits, rank, dtype=dtype, seed=91)
    dev = DeviceLinear(inp, fbq)
    before = fbq.launch_count()
    y = fbq.linear(dev.x, dev.qweight, dev.scales, dev.zeros, None, None, inp.N, 128, bits)
    fbq.sub_branch_unfused(dev.x, dev.A, dev.B, y)
    torch.cuda.synchronize()
    assert fbq.launch_count() - before == 4                  # four kernels instead of one
    want = oracle.linear_inputs(inp, threads=8)
    rel, mx, lim = compare(torch_to_f64(y, dtype), want, inp.x_f64(), inp.K)
    if dtype == "bf16":
        lim += 2.0 ** -7 * float(np.max(np.abs(want)))
    assert rel <= REL_F_TOL and mx <= lim


# The streaming decode kernel's branches by shape: the straight-line look at eight t slots (up to 32 entries, up to 64,
# a ragged second half), the general look (more entries, fewer slots), the two-level t reduction, t CTAs with two
# blocks of A per warp, the up-projection's second box of B (rank above 64), and K slices of the 16-bit form.
@pytest.mark.parametrize("M,N,K,bits,rank,dtype", [
    (1, 512, 4096, 3, 16, "f16"), (1, 528, 4096, 4, 32, "bf16"), (2, 512, 4096, 3, 32, "f16"), (1, 520, 4096, 4, 48, "f16"),
    (2, 512, 4096, 3, 48, "f16"), (1, 256, 384, 3, 64, "f16"), (2, 1024, 11008, 4, 128, "f16"), (1, 512, 4096, 4, 80, "bf16"),
    (1, 1040, 11008, 3, 64, "f16"), (2, 512, 2048, 4, 128, "f16"), (4, 512, 4096, 3, 64, "f16"), (8, 520, 11008, 4, 64, "f16"),
    (16, 512, 4096, 3, 128, "bf16"), (6, 256, 13824, 4, 32, "f16")])
def test_streaming_kernel_branches(fbq, M, N, K, bits, rank, dtype):
    inp = make_linear(M, N, K, bits, rank, dtype=dtype, seed=5100 + 7 * M + rank)
    fbq.set_option("force_kernel", fbq.KERNEL_DECODE)
    try:
        check_parity(inp, fbq, expect_kernel=fbq.KERNEL_DECODE, floor=2e-5 if dtype == "f16" else 5e-4)
        assert fbq.poll_status() == 0
        # and the same call again: slots and counters were left clean
        check_parity(inp, fbq, expect_kernel=fbq.KERNEL_DECODE, floor=2e-5 if dtype == "f16" else 5e-4)
    finally:
        fbq.set_option("force_kernel", -1)


@pytest.mark.parametrize("M,K,bits,rank", [(1, 4096, 3, 32), (2, 4096, 4, 64), (1, 11008, 4, 64), (2, 2048, 3, 128)])
def test_streaming_kernel_exact_class_is_bitwise(fbq, M, K, bits, rank):
    inp = make_exact_class(M, 528, K, bits, rank, seed=5300 + M + rank, x_nnz=32, x_max=2)
    dev = DeviceLinear(inp, fbq)
    y = torch_to_f64(dev.run(fbq), "f16")
    assert np.array_equal(y, oracle.linear_inputs(inp, threads=8))
