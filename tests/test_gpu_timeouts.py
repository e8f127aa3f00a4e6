"""Failure detection on the device: a bounded wait that runs out must end the kernel, report
FBQ_ERR_TIMEOUT through fbq_poll_status, and leave the library usable.

The failure is made on purpose and on the host side of the protocol: a test switch stops the CTAs that
compute t = x.A^T from reporting it, and an option shortens the number of looks the other CTAs take at
the flag.  Nothing faults or hangs: the waiting CTAs give up after the shortened limit, the kernel
returns, the status word is read, the scratch space is reset, and the next call is checked against
the oracle."""
import numpy as np
import pytest

from workloads import make_linear

pytestmark = pytest.mark.gpu

FBQ_ERR_TIMEOUT = -5


@pytest.fixture(scope="module")
def fbq():
    import torch
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    import paper_2501_16385_b200 as lib
    yield lib
    for name in ("test_skip_t_arrive", "t_poll_limit", "test_prefill_skip_flag", "prefill_flag_polls"):
        lib.set_option(name, 0)
    lib.set_option("force_kernel", -1)


from gpu_utils import DeviceLinear, check_parity  # noqa: E402


def test_decode_wait_for_t_runs_out(fbq):
    import torch
    inp = make_linear(1, 512, 1024, 3, 32, seed=81)
    assert fbq.select_kernel(1, 512, 1024, 128, 3, 32) == fbq.KERNEL_DECODE
    check_parity(inp, fbq)                                    # first call: scratch growth, healthy path
    dev = DeviceLinear(inp, fbq)
    fbq.set_option("test_skip_t_arrive", 1)
    fbq.set_option("t_poll_limit", 2000)
    try:
        dev.run(fbq)
        torch.cuda.synchronize()                              # the kernel returned
        assert fbq.poll_status() == FBQ_ERR_TIMEOUT           # ... and said why
    finally:
        fbq.set_option("test_skip_t_arrive", 0)
        fbq.set_option("t_poll_limit", 0)
    assert fbq.poll_status() == 0                             # reading cleared the word and reset the scratch
    check_parity(inp, fbq)                                    # the next call is correct
    check_parity(make_linear(2, 512, 1024, 4, 64, seed=82), fbq)


def test_prefill_wait_for_t_runs_out(fbq):
    import torch
    inp = make_linear(64, 512, 1024, 4, 64, seed=83)
    assert fbq.select_kernel(64, 512, 1024, 128, 4, 64, False) == fbq.KERNEL_PREFILL
    check_parity(inp, fbq)
    dev = DeviceLinear(inp, fbq)
    fbq.set_option("test_prefill_skip_flag", 1)
    fbq.set_option("prefill_flag_polls", 2000)
    try:
        dev.run(fbq)
        torch.cuda.synchronize()
        assert fbq.poll_status() == FBQ_ERR_TIMEOUT
    finally:
        fbq.set_option("test_prefill_skip_flag", 0)
        fbq.set_option("prefill_flag_polls", 0)
    assert fbq.poll_status() == 0
    check_parity(inp, fbq)
