"""Host-side checks of the C-ABI library that need no GPU: it loads, exports
every symbol the header declares, validates arguments before touching CUDA, and
its dispatch and byte/flop accounting follow the documented rules."""
import ctypes
import os
import re

import pytest

import paper_2501_16385_b200 as fbq

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "fbq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fbq_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    syms = _declared_symbols()
    assert {"fbq_pack_int3", "fbq_pack_int4", "fbq_linear", "fbq_linear_bf16", "fbq_unpack",
            "fbq_dequant", "fbq_packed_words", "fbq_select_kernel"} <= set(syms)
    L = fbq.lib()
    for s in syms:
        assert hasattr(L, s), s


def test_packed_words():
    assert fbq.packed_words(4096, 4096, 4) == 4096 * 4096 // 8
    assert fbq.packed_words(4096, 4096, 3) == 4096 * 4096 * 3 // 32
    assert fbq.packed_words(8, 36, 4) == 0 and fbq.packed_words(8, 40, 3) == 0
    assert fbq.packed_words(8, 64, 5) == 0 and fbq.packed_words(0, 64, 4) == 0


def test_dispatch_rules():
    G, D, P = fbq.KERNEL_GENERIC, fbq.KERNEL_DECODE, fbq.KERNEL_PREFILL
    sel = fbq.select_kernel
    for M in (1, 2):
        assert sel(M, 4096, 4096, 128, 4, 32) == D
        assert sel(M, 11008, 4096, 128, 3, 64, bf16=True) == D
    assert sel(6, 4096, 4096, 128, 4, 16) == D and sel(6, 4096, 4096, 128, 4, 0) == D
    assert sel(4, 4096, 4096, 128, 4, 64) == D and sel(4, 4096, 4096, 128, 4, 128) == D and sel(4, 4096, 4096, 128, 4, 256) == P
    # measured crossover where the streaming decode kernel's domain holds (N a multiple of 8, rank a multiple of 16 up
    # to 128): it takes M <= 8 for every shape, and M <= 16 while x of all K fits its shared memory
    # (M * K * 2 bytes up to 136 KB: no K slices); the tensor-core kernel the rest
    assert sel(5, 4096, 4096, 128, 4, 64) == D and sel(8, 4096, 4096, 128, 4, 128) == D and sel(8, 5120, 13824, 128, 3, 64) == D
    for M in (9, 15, 16):
        assert sel(M, 4096, 4096, 128, 4, 32) == D and sel(M, 4096, 4096, 128, 4, 64) == D and sel(M, 4096, 4096, 128, 4, 0) == D
        assert sel(M, 4096, 4096, 128, 4, 128) == D and sel(M, 4096, 4096, 128, 4, 80) == D and sel(M, 4096, 4096, 128, 4, 256) == P
        assert sel(M, 4096, 11008, 128, 4, 64) == P and sel(M, 4096, 11008, 128, 4, 128) == P and sel(M, 4096, 11008, 128, 4, 0) == P      # K too deep for one slice
    assert sel(12, 5120, 5120, 128, 4, 64) == D and sel(16, 5120, 5120, 128, 4, 64) == P and sel(16, 5120, 5120, 128, 4, 0) == P
    # outside it the other decode kernel's crossover: M * rank above 128 at M = 5, 6 goes to the tensor-core kernel
    assert sel(5, 4096, 4096, 128, 4, 24) == D and sel(6, 4096, 4096, 128, 4, 24) == P and sel(7, 4096, 4096, 128, 4, 8) == P
    assert sel(2, 4096, 4096, 128, 4, 128) == D
    for M in (7, 8, 15, 16):
        assert sel(M, 4100, 4096, 128, 4, 32) == D  # N not a multiple of 8: outside the prefill kernel's domain
    assert sel(1, 4096, 4096, 128, 4, 0) == D
    assert sel(17, 4096, 4096, 128, 4, 64) in (P, G)
    assert sel(1024, 4096, 4096, 128, 4, 64, bf16=True) in (P, G)
    assert sel(1, 8, 8, 8, 4, 2) == G               # worked example: group 8, rank 2
    assert sel(1, 64, 256, 64, 4, 8) == G           # group != 128
    assert sel(1, 64, 256, 128, 4, 12) == G         # rank not a multiple of 8
    assert sel(1, 64, 512, 128, 4, 264) == G        # rank above the fast kernels' limit
    assert sel(1, 64, 256, 128, 5, 0) == fbq.KERNEL_NONE
    assert sel(1, 64, 250, 125, 4, 0) == fbq.KERNEL_NONE
    assert sel(1, 64, 192, 48, 3, 0) == fbq.KERNEL_NONE   # 3-bit groups must hold whole 32-code runs
    assert sel(-1, 64, 256, 128, 4, 0) == fbq.KERNEL_NONE


def test_force_kernel_option_roundtrip():
    assert fbq.get_option("force_kernel") == -1
    fbq.set_option("force_kernel", fbq.KERNEL_GENERIC)
    try:
        assert fbq.select_kernel(1, 4096, 4096, 128, 4, 32) == fbq.KERNEL_GENERIC
    finally:
        fbq.set_option("force_kernel", -1)
    assert fbq.select_kernel(1, 4096, 4096, 128, 4, 32) == fbq.KERNEL_DECODE
    with pytest.raises(fbq.FbqError):
        fbq.set_option("no_such_option", 1)


def test_documented_options_exist_with_their_defaults():
    # every switch named in include/fbq.h is known to the library and starts at the documented value
    defaults = {"force_kernel": -1, "decode_sk": 0, "decode_chunk": 0, "decode_depth": 0, "decode_ctas": 0,
                "decode_i8": 1, "decode_t_ctas": 1, "decode_t_wait": 1, "batch_ctas": 400, "batch_single": 1,
                "prefill_pair": 0, "prefill_split": 2, "hostio_direct_y": 1, "pdl": 1, "decode_t_late": 0, "decode_trace": 0}
    header = open(os.path.join(os.path.dirname(__file__), "..", "include", "fbq.h")).read()
    for name, value in defaults.items():
        assert '"%s"' % name in header, name
        assert fbq.get_option(name) == value, name
        fbq.set_option(name, value)


def test_argument_validation_happens_before_any_cuda_call():
    L = fbq.lib()
    buf = (ctypes.c_char * 4096)()
    base = ctypes.addressof(buf)
    al = (base + 15) & ~15
    p = ctypes.c_void_p(al)
    odd = ctypes.c_void_p(al + 2)
    # NULL pointers, bad sizes
    assert L.fbq_linear(None, p, p, p, None, None, p, 1, 8, 128, 128, 4, 0, None) == -1
    assert L.fbq_linear(p, p, p, p, None, None, p, 1, 8, 128, 128, 4, 8, None) == -1   # rank>0, no A/B
    assert L.fbq_linear(p, p, p, p, None, None, p, 1, 8, 100, 128, 4, 0, None) == -1
    assert L.fbq_linear(p, p, p, p, None, None, p, 1, 8, 128, 128, 2, 0, None) == -1
    assert L.fbq_linear_bf16(p, p, p, p, None, None, p, -3, 8, 128, 128, 4, 0, None) == -1
    # M == 0 is a no-op
    assert L.fbq_linear(p, p, p, p, None, None, p, 0, 8, 128, 128, 4, 0, None) == 0
    # misaligned pointers
    assert L.fbq_linear(odd, p, p, p, None, None, p, 1, 8, 128, 128, 4, 0, None) == -3
    assert L.fbq_linear(p, p, p, p, None, None, odd, 1, 8, 128, 128, 4, 0, None) == -3
    assert L.fbq_pack_int4(odd, p, 8, 128, None) == -3
    assert L.fbq_pack_int3(p, p, 8, 100, None) == -1
    assert L.fbq_unpack(p, None, 8, 128, 4, None) == -1
    assert L.fbq_dequant(p, p, p, p, 8, 128, 96, 4, None) == -1
    assert fbq.status_string(-3) == "pointer not 16-byte aligned"


# ------------------------------------------------------------------ accounting
def test_sub_branch_mac_ratio_matches_section_3_2():
    # M1/M0 = 2r/d = 6.25 % at r = 128, d = 4096 (Fig. "macs-latency")
    d, r, b = 4096, 128, 1
    total = fbq.algorithmic_flops(b, d, d, r)
    main = fbq.algorithmic_flops(b, d, d, 0)
    assert main == 2 * b * d * d
    assert (total - main) / main == pytest.approx(0.0625, abs=0)


@pytest.mark.parametrize("N,K,bits,rank,mb", [
    (4096, 4096, 4, 0, 8.929), (4096, 4096, 4, 32, 9.454), (4096, 4096, 4, 64, 9.978),
    (4096, 4096, 4, 128, 11.026), (11008, 4096, 4, 0, 23.98), (4096, 11008, 4, 64, 25.92),
    (4096, 4096, 3, 0, 6.832), (4096, 4096, 3, 64, 7.881), (11008, 4096, 3, 64, 20.28),
    (5120, 5120, 4, 64, 15.26), (13824, 5120, 3, 64, 31.22)])
def test_algorithmic_bytes_table(N, K, bits, rank, mb):
    # hand-computed: codes N*K*bits/8 + scales,zeros 2*N*(K/128)*2 + A,B r*(K+N)*2 + x,y 2*(K+N)
    assert fbq.algorithmic_bytes(1, N, K, bits, rank) / 1e6 == pytest.approx(mb, abs=0.006)


def test_byte_floor_overheads():
    assert fbq.byte_floor_overhead(1, 4096, 4096, 4, 64) == pytest.approx(0.117, abs=1e-3)
    assert fbq.byte_floor_overhead(1, 4096, 4096, 3, 64) == pytest.approx(0.153, abs=1e-3)
