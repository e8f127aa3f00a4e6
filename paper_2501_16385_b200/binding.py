"""ctypes binding of libfbq.so.  Argument marshalling only.

Tensors are torch CUDA tensors (PyTorch supplies device memory and streams);
their data pointers and the current stream's handle are passed straight to the
C ABI declared in include/fbq.h.
"""
from __future__ import annotations

import ctypes
import os

from . import build as _build

KERNEL_NONE, KERNEL_GENERIC, KERNEL_DECODE, KERNEL_PREFILL = -1, 0, 1, 2
STATUS = {0: "FBQ_OK", -1: "FBQ_ERR_BADARG", -2: "FBQ_ERR_UNSUPPORTED", -3: "FBQ_ERR_ALIGN",
          -4: "FBQ_ERR_CUDA", -5: "FBQ_ERR_TIMEOUT"}

_lib = None


class FbqError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s failed: %s (%d)" % (where, STATUS.get(code, "?"), code))


def library_path() -> str:
    return _build.LIB


class Problem(ctypes.Structure):
    """struct fbq_problem of include/fbq.h."""
    _fields_ = [("x", ctypes.c_void_p), ("qweight", ctypes.c_void_p), ("scales", ctypes.c_void_p),
                ("zeros", ctypes.c_void_p), ("A", ctypes.c_void_p), ("B", ctypes.c_void_p), ("y", ctypes.c_void_p),
                ("N", ctypes.c_int), ("K", ctypes.c_int)]


def lib() -> ctypes.CDLL:
    """Loads libfbq.so (building it with nvcc when absent).  Raises if the
    library cannot be had: there is no other implementation to run."""
    global _lib
    if _lib is None:
        path = _build.LIB
        if not os.path.exists(path):
            path = _build.build()
        L = ctypes.CDLL(path)
        vp, i32 = ctypes.c_void_p, ctypes.c_int
        L.fbq_packed_words.restype = ctypes.c_size_t
        L.fbq_packed_words.argtypes = [i32, i32, i32]
        for name in ("fbq_pack_int4", "fbq_pack_int3"):
            getattr(L, name).argtypes = [vp, vp, i32, i32, vp]
        L.fbq_unpack.argtypes = [vp, vp, i32, i32, i32, vp]
        L.fbq_dequant.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp]
        for name in ("fbq_linear", "fbq_linear_bf16"):
            getattr(L, name).argtypes = [vp] * 7 + [i32] * 6 + [vp]
        L.fbq_linear_hostio.argtypes = [vp] * 7 + [i32] * 7 + [vp]
        L.fbq_linear_noalloc.argtypes = [vp] * 7 + [i32] * 7 + [vp]
        L.fbq_sub_branch_unfused.argtypes = [vp] * 4 + [i32] * 5 + [vp]
        L.fbq_quantize_feedback.argtypes = [vp] * 7 + [i32] * 6 + [vp]
        L.fbq_reconstruct_workspace_floats.restype = ctypes.c_size_t
        L.fbq_reconstruct_workspace_floats.argtypes = [i32, i32, i32]
        L.fbq_gram.argtypes = [vp, vp, i32, i32, vp]
        L.fbq_reconstruct_step.argtypes = [vp, vp, vp, vp, ctypes.c_float, vp, vp, i32, i32, i32, i32, i32, vp]
        L.fbq_linear_batch.argtypes = [ctypes.POINTER(Problem), i32, i32, i32, i32, i32, i32, vp]
        L.fbq_linear_batch_hostio.argtypes = [ctypes.POINTER(Problem), i32, i32, i32, i32, i32, i32, vp]
        L.fbq_select_kernel.argtypes = [i32] * 7
        L.fbq_set_option.argtypes = [ctypes.c_char_p, i32]
        L.fbq_get_option.argtypes = [ctypes.c_char_p, ctypes.POINTER(i32)]
        L.fbq_launch_count.restype = ctypes.c_longlong
        L.fbq_poll_status.argtypes = [vp]
        L.fbq_status_string.restype = ctypes.c_char_p
        L.fbq_status_string.argtypes = [i32]
        _lib = L
    return _lib


def _check(code: int, where: str) -> None:
    if code != 0:
        raise FbqError(code, where)


def _stream(stream=None):
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def packed_words(N: int, K: int, bits: int) -> int:
    return int(lib().fbq_packed_words(N, K, bits))


def pack(codes, bits: int, stream=None):
    """fbq_pack_int4 / fbq_pack_int3: codes uint8 [N, K] (cuda) -> qweight int32 words (cuda)."""
    import torch
    assert codes.is_cuda and codes.dtype == torch.uint8 and codes.is_contiguous()
    N, K = codes.shape
    nw = packed_words(N, K, bits)
    if nw == 0:
        raise FbqError(-1, "fbq_packed_words")
    q = torch.empty(nw, dtype=torch.int32, device=codes.device)
    fn = lib().fbq_pack_int4 if bits == 4 else lib().fbq_pack_int3
    _check(fn(_ptr(codes), _ptr(q), N, K, _stream(stream)), "fbq_pack_int%d" % bits)
    return q


def unpack(qweight, N: int, K: int, bits: int, stream=None):
    import torch
    codes = torch.empty((N, K), dtype=torch.uint8, device=qweight.device)
    _check(lib().fbq_unpack(_ptr(qweight), _ptr(codes), N, K, bits, _stream(stream)), "fbq_unpack")
    return codes


def dequant(qweight, scales, zeros, N: int, K: int, group: int, bits: int, stream=None):
    import torch
    W = torch.empty((N, K), dtype=torch.float32, device=qweight.device)
    _check(lib().fbq_dequant(_ptr(qweight), _ptr(scales), _ptr(zeros), _ptr(W), N, K, group, bits,
                             _stream(stream)), "fbq_dequant")
    return W


def linear(x, qweight, scales, zeros, A, B, N: int, group: int, bits: int, y=None, stream=None):
    """fbq_linear (fp16 x) or fbq_linear_bf16 (bf16 x).  x: [M, K]; A: [rank, K] or None;
    B: [N, rank] or None.  Returns y [M, N] in the dtype of x."""
    import torch
    assert x.is_cuda and x.is_contiguous() and x.dim() == 2
    M, K = x.shape
    rank = 0 if A is None else A.shape[0]
    if y is None:
        y = torch.empty((M, N), dtype=x.dtype, device=x.device)
    if x.dtype == torch.float16:
        fn, name = lib().fbq_linear, "fbq_linear"
    elif x.dtype == torch.bfloat16:
        fn, name = lib().fbq_linear_bf16, "fbq_linear_bf16"
    else:
        raise TypeError("x must be float16 or bfloat16")
    _check(fn(_ptr(x), _ptr(qweight), _ptr(scales), _ptr(zeros), _ptr(A), _ptr(B), _ptr(y),
              M, N, K, group, bits, rank, _stream(stream)), name)
    return y


def linear_hostio(x_host, qweight, scales, zeros, A, B, y_host, N: int, group: int, bits: int,
                  stream=None):
    """fbq_linear_hostio: x_host / y_host are (pinned) CPU tensors, weights stay on the device."""
    import torch
    M, K = x_host.shape
    rank = 0 if A is None else A.shape[0]
    bf16 = 1 if x_host.dtype == torch.bfloat16 else 0
    _check(lib().fbq_linear_hostio(_ptr(x_host), _ptr(qweight), _ptr(scales), _ptr(zeros), _ptr(A),
                                   _ptr(B), _ptr(y_host), M, N, K, group, bits, rank, bf16,
                                   _stream(stream)), "fbq_linear_hostio")
    return y_host


def linear_noalloc(x, qweight, scales, zeros, A, B, N: int, group: int, bits: int, y, stream=None):
    """fbq_linear_noalloc: like ``linear`` for decode shapes, but the library allocates nothing
    (its scratch lives in a fixed array inside the library).  The caller passes y.  Calls must
    not overlap on the GPU: they all share that one array."""
    import torch
    M, K = x.shape
    rank = 0 if A is None else A.shape[0]
    bf16 = 1 if x.dtype == torch.bfloat16 else 0
    _check(lib().fbq_linear_noalloc(_ptr(x), _ptr(qweight), _ptr(scales), _ptr(zeros), _ptr(A), _ptr(B),
                                    _ptr(y), M, N, K, group, bits, rank, bf16, _stream(stream)),
           "fbq_linear_noalloc")
    return y


def sub_branch_unfused(x, A, B, y, stream=None):
    """fbq_sub_branch_unfused: adds (x.A^T).B^T to y with three separate launches (the paper's unfused
    comparison layer); y must already hold the main path (fbq_linear at rank 0)."""
    import torch
    M, K = x.shape
    rank, N = A.shape[0], y.shape[1]
    bf16 = 1 if x.dtype == torch.bfloat16 else 0
    _check(lib().fbq_sub_branch_unfused(_ptr(x), _ptr(A), _ptr(B), _ptr(y), M, N, K, rank, bf16, _stream(stream)),
           "fbq_sub_branch_unfused")
    return y


def quantize_feedback(W, A, B, group: int, bits: int, want_wf: bool = False, stream=None):
    """fbq_quantize_feedback: W [N, K] float32 on the device, A [rank, K] / B [N, rank] (fp16 or
    bf16, or None).  Returns (codes uint8 [N, K], scales, zeros fp16 [N, K/group], W_F or None)."""
    import torch
    assert W.is_cuda and W.dtype == torch.float32 and W.is_contiguous()
    N, K = W.shape
    rank = 0 if A is None else A.shape[0]
    bf16 = 1 if (A is not None and A.dtype == torch.bfloat16) else 0
    codes = torch.empty((N, K), dtype=torch.uint8, device=W.device)
    scales = torch.empty((N, K // group), dtype=torch.float16, device=W.device)
    zeros = torch.empty((N, K // group), dtype=torch.float16, device=W.device)
    wf = torch.empty((N, K), dtype=torch.float32, device=W.device) if want_wf else None
    _check(lib().fbq_quantize_feedback(_ptr(W), _ptr(A), _ptr(B), _ptr(codes), _ptr(scales), _ptr(zeros), _ptr(wf),
                                       N, K, group, bits, rank, bf16, _stream(stream)), "fbq_quantize_feedback")
    return codes, scales, zeros, wf


def gram(X, stream=None):
    """fbq_gram: H = X^T X (float32 [K, K]) of calibration activations X [T, K] float32."""
    import torch
    assert X.is_cuda and X.dtype == torch.float32 and X.is_contiguous()
    T, K = X.shape
    H = torch.empty((K, K), dtype=torch.float32, device=X.device)
    _check(lib().fbq_gram(_ptr(X), _ptr(H), T, K, _stream(stream)), "fbq_gram")
    return H


def reconstruct_step(W, H, A, B, lr: float, group: int, bits: int, workspace=None, loss=None, stream=None):
    """fbq_reconstruct_step: one iteration of Algorithm 1 on float32 device tensors; A and B are
    updated in place.  Returns (loss tensor [1], workspace) so that both can be reused."""
    import torch
    N, K = W.shape
    rank = A.shape[0]
    for t in (W, H, A, B):
        assert t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()
    need = int(lib().fbq_reconstruct_workspace_floats(N, K, rank))
    if workspace is None or workspace.numel() < need:
        workspace = torch.empty(need, dtype=torch.float32, device=W.device)
    if loss is None:
        loss = torch.zeros(1, dtype=torch.float32, device=W.device)
    _check(lib().fbq_reconstruct_step(_ptr(W), _ptr(H), _ptr(A), _ptr(B), float(lr), _ptr(loss), _ptr(workspace), N, K,
                                      group, bits, rank, _stream(stream)), "fbq_reconstruct_step")
    return loss, workspace


def make_batch(problems):
    """Marshals a list of (x, qweight, scales, zeros, A, B, y) tensor tuples (A = B = None for
    rank 0; every x [M, K], y [M, N]) into the descriptor array of fbq_linear_batch.  Returns
    (array, count, M, rank, bf16); the array can be reused for as long as the tensors live."""
    import torch
    n = len(problems)
    arr = (Problem * max(n, 1))()
    M = rank = bf16 = None
    for i, (x, qw, s, z, A, B, y) in enumerate(problems):
        assert x.is_contiguous() and y.is_contiguous() and x.dtype == y.dtype and x.is_cuda == y.is_cuda
        m, r, b = x.shape[0], (0 if A is None else A.shape[0]), (1 if x.dtype == torch.bfloat16 else 0)
        if i == 0:
            M, rank, bf16 = m, r, b
        assert (m, r, b) == (M, rank, bf16), "the problems of a batch share M, rank and the activation type"
        arr[i] = Problem(_ptr(x), _ptr(qw), _ptr(s), _ptr(z), _ptr(A), _ptr(B), _ptr(y), y.shape[1], x.shape[1])
    return arr, n, M or 0, rank or 0, bf16 or 0


def linear_batch(problems, group: int, bits: int, stream=None, batch=None, host_io: bool = False):
    """fbq_linear_batch over a list of (x, qweight, scales, zeros, A, B, y) tuples, or over a
    descriptor array made earlier by make_batch (``batch``).  The y tensors are written.  With
    host_io the x and y tensors are (pinned) CPU tensors: fbq_linear_batch_hostio."""
    arr, n, M, rank, bf16 = batch if batch is not None else make_batch(problems)
    fn = lib().fbq_linear_batch_hostio if host_io else lib().fbq_linear_batch
    _check(fn(arr, n, M, group, bits, rank, bf16, _stream(stream)), "fbq_linear_batch")


def select_kernel(M, N, K, group, bits, rank, bf16=False) -> int:
    return int(lib().fbq_select_kernel(M, N, K, group, bits, rank, 1 if bf16 else 0))


def set_option(name: str, value: int) -> None:
    _check(lib().fbq_set_option(name.encode(), int(value)), "fbq_set_option(%s)" % name)


def get_option(name: str) -> int:
    v = ctypes.c_int(0)
    _check(lib().fbq_get_option(name.encode(), ctypes.byref(v)), "fbq_get_option(%s)" % name)
    return v.value


def launch_count() -> int:
    return int(lib().fbq_launch_count())


def poll_status(stream=None) -> int:
    return int(lib().fbq_poll_status(_stream(stream)))


def release_workspaces() -> None:
    _check(lib().fbq_release_workspaces(), "fbq_release_workspaces")


def status_string(code: int) -> str:
    return lib().fbq_status_string(code).decode()
