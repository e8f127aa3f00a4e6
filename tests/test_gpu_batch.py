"""GPU parity of fbq_linear_batch (grouped decode of independent linears) against the CPU oracle
and against single fbq_linear calls, through the C ABI."""
import numpy as np
import pytest

import oracle
from workloads import make_linear

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def fbq():
    import torch
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    import paper_2501_16385_b200 as lib
    lib.set_option("force_kernel", -1)
    return lib


from gpu_utils import DeviceLinear, REL_F_TOL, compare, torch_to_f64  # noqa: E402

# a scaled-down decoder layer: q, k, v, o, gate, up, down  (K, N)
LAYER = [(512, 512)] * 4 + [(512, 1376), (512, 1376), (1408, 512)]


def _problems(fbq, M, bits, rank, dtype, seed0):
    import torch
    inps = [make_linear(M, N, K, bits, rank, dtype=dtype, seed=seed0 + i) for i, (K, N) in enumerate(LAYER)]
    devs = [DeviceLinear(inp, fbq) for inp in inps]
    probs = []
    for d, inp in zip(devs, inps):
        y = torch.empty((M, inp.N), dtype=d.x.dtype, device="cuda")
        probs.append((d.x, d.qweight, d.scales, d.zeros, d.A if rank else None, d.B if rank else None, y))
    return inps, devs, probs


@pytest.mark.parametrize("single", [1, 0])
@pytest.mark.parametrize("bits,rank,dtype,M", [(3, 64, "f16", 1), (4, 64, "bf16", 1), (3, 0, "f16", 1), (3, 16, "f16", 5),
                                              (4, 64, "f16", 2), (3, 16, "bf16", 6), (4, 8, "f16", 3), (3, 24, "f16", 4)])
def test_batch_matches_oracle_and_single_calls(fbq, bits, rank, dtype, M, single):
    import torch
    fbq.set_option("batch_single", single)       # 1: the decode kernel over a problem list; 0: one launch per problem
    inps, devs, probs = _problems(fbq, M, bits, rank, dtype, 4000 + 10 * bits + rank)
    for N, K in [(inp.N, inp.K) for inp in inps]:
        assert fbq.select_kernel(M, N, K, 128, bits, rank, dtype == "bf16") == fbq.KERNEL_DECODE
    before = fbq.launch_count()
    fbq.linear_batch(probs, 128, bits)
    torch.cuda.synchronize()
    # one launch over the problem list where the other decode kernel runs (here: ranks that are not a multiple of 16);
    # problems in the streaming kernel's domain take one launch each on the side streams
    assert fbq.launch_count() - before == (1 if (single and rank % 16 != 0) else len(probs))
    fbq.set_option("batch_single", 1)
    assert fbq.poll_status() == 0
    for inp, d, pr in zip(inps, devs, probs):
        want = oracle.linear_inputs(inp, threads=8)
        got = torch_to_f64(pr[6], dtype)
        rel, mx, lim = compare(got, want, inp.x_f64(), inp.K)
        if dtype == "bf16":                                 # half an ulp of a bf16 output alone can exceed the bound
            lim += 2.0 ** -8 * float(np.max(np.abs(want)))
        assert rel <= REL_F_TOL and mx <= lim
        assert rel >= (2e-5 if dtype == "f16" else 5e-4)    # not vacuous: the output rounding is there
        single = fbq.linear(d.x, d.qweight, d.scales, d.zeros, pr[4], pr[5], inp.N, 128, bits)
        if rank == 0:
            assert torch.equal(single, pr[6])               # fixed summation order whatever the grid size
        else:
            assert torch.allclose(single.float(), pr[6].float(), rtol=2e-2, atol=2e-3)


def test_batch_under_graph_replay(fbq):
    import torch
    inps, devs, probs = _problems(fbq, 1, 3, 64, "f16", 4500)
    batch = fbq.make_batch(probs)
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        fbq.linear_batch(None, 128, 3, stream=st, batch=batch)      # first call outside the capture
        st.synchronize()
        ref = [p[6].clone() for p in probs]
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=st):
            fbq.linear_batch(None, 128, 3, stream=st, batch=batch)
            fbq.linear_batch(None, 128, 3, stream=st, batch=batch)
        for p in probs:
            p[6].zero_()
        g.replay()
        g.replay()
        st.synchronize()
    assert fbq.poll_status(st) == 0
    for r, p in zip(ref, probs):
        assert torch.allclose(r.float(), p[6].float(), rtol=2e-2, atol=2e-3)


def test_batch_hostio_reads_and_writes_host_buffers(fbq):
    import torch
    inps, devs, probs = _problems(fbq, 1, 3, 64, "f16", 4700)
    host = [(p[0].cpu().pin_memory(), p[1], p[2], p[3], p[4], p[5], torch.zeros(p[6].shape, dtype=p[6].dtype).pin_memory())
            for p in probs]
    fbq.linear_batch(probs, 128, 3)
    fbq.linear_batch(host, 128, 3, host_io=True)
    torch.cuda.synchronize()
    assert fbq.poll_status() == 0
    for p, h in zip(probs, host):
        assert torch.allclose(p[6].cpu().float(), h[6].float(), rtol=2e-2, atol=2e-3)
        assert h[6].abs().max() > 0
    one = host[:1]                                        # a single problem goes the sequential way
    one[0][6].zero_()
    fbq.linear_batch(one, 128, 3, host_io=True)
    torch.cuda.synchronize()
    assert torch.allclose(probs[0][6].cpu().float(), one[0][6].float(), rtol=2e-2, atol=2e-3)


def test_batch_falls_back_for_prefill_sized_problems(fbq):
    import torch
    inps = [make_linear(40, 256, 256, 4, 8, seed=4600 + i) for i in range(2)]
    devs = [DeviceLinear(inp, fbq) for inp in inps]
    probs = [(d.x, d.qweight, d.scales, d.zeros, d.A, d.B, torch.empty((40, 256), dtype=torch.float16, device="cuda"))
             for d in devs]
    fbq.linear_batch(probs, 128, 4)
    torch.cuda.synchronize()
    for inp, pr in zip(inps, probs):
        rel, mx, lim = compare(torch_to_f64(pr[6], "f16"), oracle.linear_inputs(inp, threads=4), inp.x_f64(), inp.K)
        assert rel <= REL_F_TOL and mx <= lim


def test_batch_argument_checks(fbq):
    arr = (fbq.Problem * 1)()
    L = fbq.lib()
    assert L.fbq_linear_batch(arr, 0, 1, 128, 3, 0, 0, None) == 0
    assert L.fbq_linear_batch(arr, 17, 1, 128, 3, 0, 0, None) != 0
    assert L.fbq_linear_batch(None, 1, 1, 128, 3, 0, 0, None) != 0


@pytest.mark.parametrize("M", [1, 2, 4, 6])
def test_full_size_layer_in_one_batch_call(fbq, M):
    """The seven Llama-2-7B shapes (K = 4096 next to K = 11008) in one fbq_linear_batch call with the
    single-launch form switched on: whatever mix of plans the problems get, every output (sampled rows at
    these sizes) matches the oracle."""
    import torch
    from workloads import LLAMA2_7B_SHAPES
    fbq.set_option("batch_single", 1)
    bits, rank = 3, 16
    inps = [make_linear(M, N, K, bits, rank, seed=4700 + 10 * M + i) for i, (K, N) in enumerate(LLAMA2_7B_SHAPES)]
    devs = [DeviceLinear(inp, fbq) for inp in inps]
    probs = []
    for d, inp in zip(devs, inps):
        y = torch.full((M, inp.N), float("nan"), dtype=d.x.dtype, device="cuda")
        probs.append((d.x, d.qweight, d.scales, d.zeros, d.A, d.B, y))
    fbq.linear_batch(probs, 128, bits)
    torch.cuda.synchronize()
    assert fbq.poll_status() == 0
    for inp, pr in zip(inps, probs):
        rows = np.unique(np.concatenate([np.arange(0, inp.N, 37), np.arange(inp.N - 16, inp.N)]))
        want = oracle.linear_inputs(inp, n_list=rows, threads=8)
        got = torch_to_f64(pr[6], "f16")
        assert np.all(np.isfinite(got))
        rel, mx, lim = compare(got[:, rows], want, inp.x_f64(), inp.K)
        assert rel <= REL_F_TOL and mx <= lim, (inp.N, inp.K, rel, mx)
