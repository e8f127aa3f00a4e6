"""Helpers shared by the GPU parity tests: move seeded inputs to the device,
call the CUDA library through its binding, compare with the CPU oracle."""
from __future__ import annotations

import numpy as np

import oracle

REL_F_TOL = 5e-3            # relative Frobenius error of y against the oracle


def max_abs_tol(x_f64: np.ndarray, K: int) -> float:
    # 1e-2 * ||x||_inf * sqrt(K) / 64  (1e-2 * ||x||_inf at K = 4096)
    return 1e-2 * float(np.max(np.abs(x_f64))) * np.sqrt(K) / 64.0


def torch_dtype(dtype: str):
    import torch
    return torch.float16 if dtype == "f16" else torch.bfloat16


def bits_to_torch(a: np.ndarray, dtype: str, device="cuda"):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(device)
    return t.view(torch_dtype(dtype))


def f16_to_torch(a: np.ndarray, device="cuda"):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(device).view(torch.float16)


def torch_to_f64(t, dtype: str) -> np.ndarray:
    import torch
    raw = t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    if dtype == "f16":
        return raw.view(np.float16).astype(np.float64)
    return (raw.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


class DeviceLinear:
    """Device-resident tensors of one workloads.LinearInputs (codes packed by the CUDA packer)."""

    def __init__(self, inp, fbq):
        import torch
        self.inp = inp
        codes = torch.from_numpy(inp.codes).cuda()
        self.qweight = fbq.pack(codes, inp.bits)
        self.scales = f16_to_torch(inp.scales)
        self.zeros = f16_to_torch(inp.zeros)
        self.x = bits_to_torch(inp.x, inp.dtype)
        self.A = bits_to_torch(inp.A, inp.dtype) if inp.rank > 0 else None
        self.B = bits_to_torch(inp.B, inp.dtype) if inp.rank > 0 else None

    def run(self, fbq, x=None):
        i = self.inp
        return fbq.linear(self.x if x is None else x, self.qweight, self.scales, self.zeros,
                          self.A, self.B, i.N, i.group, i.bits)


def compare(y_gpu_f64: np.ndarray, y_or: np.ndarray, x_f64: np.ndarray, K: int):
    """Returns (rel_F, max_abs, max_abs_limit)."""
    diff = y_gpu_f64 - y_or
    den = float(np.linalg.norm(y_or))
    rel = float(np.linalg.norm(diff)) / den if den > 0 else float(np.linalg.norm(diff))
    return rel, float(np.max(np.abs(diff))) if diff.size else 0.0, max_abs_tol(x_f64, K)


def check_parity(inp, fbq, *, expect_kernel=None, n_list=None, threads=8, floor=None):
    """Runs the CUDA path and the oracle on `inp` and asserts the tolerances."""
    import torch
    dev = DeviceLinear(inp, fbq)
    # a test that names the decode kernel means that kernel, also for token counts at which the
    # dispatcher would by now prefer the tensor-core kernel
    forced = expect_kernel == fbq.KERNEL_DECODE and fbq.get_option("force_kernel") == -1
    if forced:
        fbq.set_option("force_kernel", fbq.KERNEL_DECODE)
    try:
        if expect_kernel is not None:
            assert fbq.select_kernel(inp.M, inp.N, inp.K, inp.group, inp.bits, inp.rank,
                                     inp.dtype == "bf16") == expect_kernel
        y = dev.run(fbq)
    finally:
        if forced:
            fbq.set_option("force_kernel", -1)
    torch.cuda.synchronize()
    assert fbq.poll_status() == 0
    y64 = torch_to_f64(y, inp.dtype)
    q_or = oracle.pack(inp.codes, inp.bits)
    assert np.array_equal(dev.qweight.cpu().numpy().view(np.uint32), q_or), "packed words differ"
    y_or = oracle.linear_inputs(inp, qweight=q_or, n_list=n_list, threads=threads)
    if n_list is not None:
        y64 = y64[:, np.asarray(n_list)]
    assert np.all(np.isfinite(y64))
    rel, mx, lim = compare(y64, y_or, inp.x_f64(), inp.K)
    assert rel <= REL_F_TOL, "rel_F %.3e" % rel
    assert mx <= lim, "max abs %.3e > %.3e" % (mx, lim)
    if floor is not None:
        # an error far below the output-rounding floor means the comparison is vacuous
        assert rel >= floor, "rel_F %.3e suspiciously small" % rel
    return rel, mx, y64, y_or
