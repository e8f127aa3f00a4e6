"""B200-native FBQuant inference linear: thin Python binding of libfbq.so.

The package holds only what the hot path needs: CUDA sources and the C ABI
(csrc/, include/fbq.h at the repository root), a build helper and this ctypes
binding, whose functions carry the same names as the C entry points and only
marshal arguments.  Every step of the layer runs in the CUDA kernels; there is
no Python or CPU implementation to fall back to.
"""
from .binding import (  # noqa: F401
    FbqError,
    KERNEL_DECODE,
    KERNEL_GENERIC,
    KERNEL_NONE,
    KERNEL_PREFILL,
    Problem,
    STATUS,
    dequant,
    get_option,
    gram,
    launch_count,
    lib,
    library_path,
    make_batch,
    linear,
    linear_batch,
    linear_hostio,
    linear_noalloc,
    pack,
    packed_words,
    poll_status,
    quantize_feedback,
    reconstruct_step,
    release_workspaces,
    select_kernel,
    set_option,
    status_string,
    sub_branch_unfused,
    unpack,
)
from .accounting import algorithmic_bytes, algorithmic_flops, byte_floor_overhead  # noqa: F401
