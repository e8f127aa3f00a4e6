"""fbq_linear_noalloc: the decode layer for callers that cannot allocate device memory
(all of it already given to their own pool, or no room for the synchronisation an
allocation may imply).  Its scratch is a fixed array inside the library, so its results
must equal those of fbq_linear, whose scratch is allocated per stream -- on a first call
and again on a second one, which finds the array as the first call left it -- and, like
every other path, the CPU oracle's within the layer's tolerance.

Collected last on purpose: a failure here leaves every other test already run."""
import numpy as np
import pytest

import oracle

from workloads import make_linear

pytestmark = pytest.mark.gpu


def test_noalloc_matches_allocating_entry_point_twice():
    import torch
    assert torch.cuda.is_available()
    import paper_2501_16385_b200 as fbq
    from gpu_utils import DeviceLinear, REL_F_TOL, compare, torch_to_f64

    cases = [make_linear(1, 4096, 4096, 4, 32, seed=500), make_linear(5, 1040, 2048, 3, 64, seed=501),
             make_linear(16, 528, 1024, 4, 16, dtype="bf16", seed=502), make_linear(2, 272, 1024, 3, 0, seed=503)]
    for inp in cases:
        dev = DeviceLinear(inp, fbq)
        fbq.set_option("force_kernel", fbq.KERNEL_DECODE)     # the same kernel, whatever the dispatcher prefers at this M
        fbq.set_option("gemv", 0)                             # ... and not the streaming kernel, which the fixed array does not serve
        try:
            want = dev.run(fbq)                               # existing entry point
        finally:
            fbq.set_option("force_kernel", -1)
            fbq.set_option("gemv", 1)
        torch.cuda.synchronize()
        want64 = torch_to_f64(want, inp.dtype)
        y_or = oracle.linear_inputs(inp, threads=8)           # the definition itself
        for call in range(2):                                 # two calls in a row share the array
            y = torch.full((inp.M, inp.N), float("nan"), dtype=want.dtype, device="cuda")
            fbq.linear_noalloc(dev.x, dev.qweight, dev.scales, dev.zeros, dev.A, dev.B, inp.N, inp.group,
                               inp.bits, y)
            torch.cuda.synchronize()
            got64 = torch_to_f64(y, inp.dtype)
            assert np.all(np.isfinite(got64)), "call %d left outputs unwritten" % call
            rel, mx, lim = compare(got64, want64, inp.x_f64(), inp.K)
            assert rel <= REL_F_TOL and mx <= lim, (call, rel, mx)
            rel, mx, lim = compare(got64, y_or, inp.x_f64(), inp.K)
            if inp.dtype == "bf16":                           # half an ulp of a bf16 output alone can exceed the bound
                lim += 2.0 ** -8 * float(np.max(np.abs(y_or)))
            assert rel <= REL_F_TOL and mx <= lim, ("oracle", call, rel, mx)
            assert fbq.poll_status() == 0                     # the fixed array's own status word is clean
            if inp.rank == 0:
                assert torch.equal(y, want)                   # no atomics on this path: bit for bit


def test_noalloc_refuses_what_does_not_fit():
    import torch
    import paper_2501_16385_b200 as fbq
    L = fbq.lib()
    buf = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    p = buf.data_ptr()
    # prefill-sized M, foreign group size, N beyond the fixed array: refused, nothing runs
    assert L.fbq_linear_noalloc(p, p, p, p, None, None, p, 64, 4096, 4096, 128, 4, 0, 0, None) == -2
    assert L.fbq_linear_noalloc(p, p, p, p, None, None, p, 1, 64, 256, 64, 4, 0, 0, None) == -2
    assert L.fbq_linear_noalloc(p, p, p, p, None, None, p, 16, 65536, 4096, 128, 4, 0, 0, None) == -2
    assert L.fbq_linear_noalloc(None, p, p, p, None, None, p, 1, 64, 256, 128, 4, 0, 0, None) == -1
    torch.cuda.synchronize()
