"""Pins of the CPU oracle against things other than itself: hand-worked values,
literal bit patterns, closed forms, library matmuls on special cases, and
invariants of the layer definition (Algorithm 1 step 6; Section 4.2)."""
import os

import numpy as np
import pytest

import oracle
from workloads import (make_exact_class, make_linear, worked_example_e1,
                       f32_to_bf16_bits, bf16_bits_to_f64)

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _read_golden(name):
    out = {}
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            parts = line.split()
            out.setdefault(parts[0], []).append(parts[1:])
    return out


def _dense_from_raw_codes(inp):
    """W[n,k] built with numpy from the *unpacked* input codes (never through
    the oracle's packer), for library cross-checks."""
    s = inp.scales.astype(np.float64).repeat(inp.group, axis=1)
    z = inp.zeros.astype(np.float64).repeat(inp.group, axis=1)
    return s * (inp.codes.astype(np.float64) - z)


# ----------------------------------------------------------------- widening
def test_widen_fp16_all_bit_patterns_matches_numpy():
    bits = np.arange(65536, dtype=np.uint16)
    got = oracle.widen(bits, "f16")
    want = bits.view(np.float16).astype(np.float64)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], want[~nan])
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(want[~nan]))


def test_widen_bf16_all_bit_patterns_matches_numpy():
    bits = np.arange(65536, dtype=np.uint16)
    got = oracle.widen(bits, "bf16")
    want = bf16_bits_to_f64(bits)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], want[~nan])


def test_bf16_rounding_helper_is_nearest_even():
    # 1 + 2^-8 is a tie between 1.0 (even) and 1 + 2^-7; 1 + 3*2^-8 ties upward to even.
    v = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20], dtype=np.float32)
    assert f32_to_bf16_bits(v).tolist() == [0x3F80, 0x3F82, 0x3F81]


# ------------------------------------------------------------------ packing
def test_pack_literal_examples():
    g = _read_golden("pack_examples.txt")
    for bits, key in ((4, "int4"), (3, "int3")):
        codes = np.array([int(v) for v in g[key][0][1:]], dtype=np.uint8)[None, :]
        words = [int(v, 16) for v in g[key][1][1:]]
        assert oracle.pack(codes, bits).tolist() == words
        assert np.array_equal(oracle.unpack(np.array(words, dtype=np.uint32), 1, codes.shape[1], bits), codes)


# (k, [(word, shift of bit 0 of the code), ...]) typed by hand from the format:
INT3_SINGLE_HOT = {
    0: [(0, 0)], 4: [(0, 12)], 5: [(0, 16)], 9: [(0, 28)], 10: [(1, 0)], 17: [(1, 22)],
    20: [(2, 0)], 29: [(2, 28)],
}


@pytest.mark.parametrize("k", sorted(INT3_SINGLE_HOT))
def test_int3_single_hot_positions(k):
    for v in (1, 2, 4, 7):
        codes = np.zeros((1, 32), dtype=np.uint8)
        codes[0, k] = v
        (word, shift), = INT3_SINGLE_HOT[k]
        want = [0, 0, 0]
        want[word] = v << shift
        assert oracle.pack(codes, 3).tolist() == want


def test_int3_codes_30_and_31_are_bit_sliced():
    for k, pos in ((30, 15), (31, 31)):
        for v in range(8):
            codes = np.zeros((1, 32), dtype=np.uint8)
            codes[0, k] = v
            want = [((v >> i) & 1) << pos for i in range(3)]
            assert oracle.pack(codes, 3).tolist() == want


def test_int4_single_hot_positions():
    for k in range(16):
        codes = np.zeros((1, 16), dtype=np.uint8)
        codes[0, k] = 0xB
        want = [0, 0]
        want[k // 8] = 0xB << (4 * (k % 8))
        assert oracle.pack(codes, 4).tolist() == want


@pytest.mark.parametrize("bits", [3, 4])
@pytest.mark.parametrize("N,K", [(1, 32), (3, 64), (8, 128), (5, 4096), (16, 11008)])
def test_pack_roundtrip_exact(bits, N, K):
    rng = np.random.default_rng(N * 1000 + K + bits)
    qmax = (1 << bits) - 1
    for codes in (rng.integers(0, qmax + 1, size=(N, K), dtype=np.uint8),
                  np.zeros((N, K), dtype=np.uint8), np.full((N, K), qmax, dtype=np.uint8)):
        q = oracle.pack(codes, bits)
        assert q.size == oracle.packed_words(N, K, bits)
        assert np.array_equal(oracle.unpack(q, N, K, bits), codes)
    # density: 8 codes per word (INT4), 32 codes per 3 words (INT3)
    assert oracle.packed_words(N, K, bits) * 32 == N * K * bits


@pytest.mark.parametrize("bits", [3, 4])
def test_pack_rows_are_independent_and_contiguous(bits):
    rng = np.random.default_rng(5)
    codes = rng.integers(0, 1 << bits, size=(4, 96 if bits == 3 else 24), dtype=np.uint8)
    q = oracle.pack(codes, bits).reshape(4, -1)
    for n in range(4):
        assert np.array_equal(q[n], oracle.pack(codes[n:n + 1], bits))


# ---------------------------------------------------------------- dequantiser
@pytest.mark.parametrize("bits", [3, 4])
def test_dequant_codes_equal_zero_points_gives_zero(bits):
    inp = make_linear(1, 16, 256, bits, 0, seed=3, codes_equal_zero=True)
    W = oracle.dequant(oracle.pack(inp.codes, bits), inp.scales, inp.zeros, 16, 256, 128, bits)
    assert np.all(W == 0.0)


@pytest.mark.parametrize("bits,group", [(4, 8), (4, 128), (3, 32), (3, 128)])
def test_dequant_matches_numpy_from_raw_codes(bits, group):
    inp = make_linear(1, 24, 512, bits, 0, group=group, seed=9)
    W = oracle.dequant(oracle.pack(inp.codes, bits), inp.scales, inp.zeros, 24, 512, group, bits)
    assert np.array_equal(W, _dense_from_raw_codes(inp))
    # s*(q-z) needs at most 11+5 significand bits: exact in fp32 as well
    assert np.array_equal(W.astype(np.float32).astype(np.float64), W)


def test_dequant_group_orientation_single_group_changed():
    # Groups are runs of `group` consecutive input channels k of ONE output row.
    inp = make_linear(1, 4, 256, 4, 0, seed=1)
    q = oracle.pack(inp.codes, 4)
    W0 = oracle.dequant(q, inp.scales, inp.zeros, 4, 256, 128, 4)
    s2 = inp.scales.copy()
    s2[2, 1] = np.float16(1.0)
    W1 = oracle.dequant(q, s2, inp.zeros, 4, 256, 128, 4)
    changed = np.argwhere(W0 != W1)
    assert set(changed[:, 0]) == {2} and changed[:, 1].min() >= 128


# ------------------------------------------------------------ the whole layer
def test_e1_hand_worked_example():
    g = {k: v[0] for k, v in _read_golden("e1_worked_example.txt").items()}
    inp = worked_example_e1()
    q = oracle.pack(inp.codes, 4)
    assert q.tolist() == [int(v, 16) for v in g["packed"]]
    y, t = oracle.linear_inputs(inp, return_t=True)
    assert t[0].tolist() == [float(v) for v in g["t"]]
    assert y[0].tolist() == [float(v) for v in g["y"]]
    main = oracle.linear(inp.x, q, inp.scales, inp.zeros, None, None, 1, 8, 8, 8, 4, 0)
    assert main[0].tolist() == [float(v) for v in g["main"]]
    assert (y - main)[0].tolist() == [float(v) for v in g["sub"]]


@pytest.mark.parametrize("bits,dtype,M,N,K,rank", [
    (4, "f16", 1, 64, 4096, 32), (3, "f16", 3, 48, 1024, 64), (4, "bf16", 5, 40, 512, 16),
    (3, "bf16", 2, 32, 2048, 8)])
def test_library_cross_check_fp64(bits, dtype, M, N, K, rank):
    inp = make_linear(M, N, K, bits, rank, dtype=dtype, seed=17, outlier_frac=0.01 if dtype == "bf16" else 0)
    y = oracle.linear_inputs(inp)
    X, A, B = inp.x_f64(), inp.A_f64(), inp.B_f64()
    want = X @ _dense_from_raw_codes(inp).T + (X @ A.T) @ B.T
    assert np.max(np.abs(y - want)) <= 1e-12 * np.max(np.abs(want))


@pytest.mark.parametrize("bits", [3, 4])
def test_rank0_is_plain_dequant_gemv(bits):
    inp = make_linear(1, 128, 1024, bits, 0, seed=4)
    y = oracle.linear_inputs(inp)
    want = inp.x_f64() @ _dense_from_raw_codes(inp).T
    assert np.max(np.abs(y - want)) <= 1e-12 * np.max(np.abs(want))


@pytest.mark.parametrize("bits", [3, 4])
def test_zero_A_or_zero_B_leaves_main_path_unchanged(bits):
    inp = make_linear(2, 32, 512, bits, 16, seed=8)
    q = oracle.pack(inp.codes, bits)
    base = oracle.linear(inp.x, q, inp.scales, inp.zeros, None, None, 2, 32, 512, 128, bits, 0)
    zA, zB = np.zeros_like(inp.A), np.zeros_like(inp.B)
    for A, B in ((zA, inp.B), (inp.A, zB)):
        y = oracle.linear(inp.x, q, inp.scales, inp.zeros, A, B, 2, 32, 512, 128, bits, 16)
        assert np.array_equal(y, base)
    full = oracle.linear_inputs(inp, qweight=q)
    assert not np.array_equal(full, base)


@pytest.mark.parametrize("bits", [3, 4])
def test_codes_equal_zero_points_leaves_textbook_low_rank_product(bits):
    inp = make_linear(3, 48, 512, bits, 32, seed=6, codes_equal_zero=True, ab_std=0.141)
    y = oracle.linear_inputs(inp)
    want = (inp.x_f64() @ inp.A_f64().T) @ inp.B_f64().T
    assert np.max(np.abs(y - want)) <= 1e-13 * np.max(np.abs(want))


def test_unit_vector_input_reads_out_a_column():
    inp = make_linear(1, 32, 256, 4, 8, seed=2)
    W = _dense_from_raw_codes(inp) + inp.B_f64() @ inp.A_f64()
    q = oracle.pack(inp.codes, 4)
    for k in (0, 7, 127, 128, 255):
        x = np.zeros((1, 256), dtype=np.float16)
        x[0, k] = 1.0
        y = oracle.linear(x, q, inp.scales, inp.zeros, inp.A, inp.B, 1, 32, 256, 128, 4, 8)
        assert np.max(np.abs(y[0] - W[:, k])) <= 1e-15


@pytest.mark.parametrize("bits", [3, 4])
def test_all_ones_input_closed_form(bits):
    # x = 1  =>  y_n = sum_g s[n,g] * (sum_{k in g} q[n,k] - group*z[n,g]) + B_n . (A 1)
    inp = make_linear(1, 24, 512, bits, 8, seed=12)
    x = np.ones((1, 512), dtype=np.float16)
    y = oracle.linear(x, oracle.pack(inp.codes, bits), inp.scales, inp.zeros, inp.A, inp.B,
                      1, 24, 512, 128, bits, 8)
    qsum = inp.codes.astype(np.int64).reshape(24, 4, 128).sum(axis=2)
    main = (inp.scales.astype(np.float64) * (qsum - 128 * inp.zeros.astype(np.float64))).sum(axis=1)
    sub = inp.B_f64() @ inp.A_f64().sum(axis=1)
    assert np.max(np.abs(y[0] - (main + sub))) <= 1e-12


def test_linearity_in_x():
    inp = make_linear(1, 32, 512, 4, 16, seed=21)
    rng = np.random.default_rng(0)
    x1 = rng.integers(-8, 9, size=(1, 512)).astype(np.float16)
    x2 = rng.integers(-8, 9, size=(1, 512)).astype(np.float16)
    a, b = 0.5, -2.0                       # exact in fp16 for these small integers
    x3 = (a * x1.astype(np.float64) + b * x2.astype(np.float64)).astype(np.float16)
    assert np.array_equal(x3.astype(np.float64), a * x1.astype(np.float64) + b * x2.astype(np.float64))
    q = oracle.pack(inp.codes, 4)
    f = lambda x: oracle.linear(x, q, inp.scales, inp.zeros, inp.A, inp.B, 1, 32, 512, 128, 4, 16)
    y1, y2, y3 = f(x1), f(x2), f(x3)
    assert np.max(np.abs(y3 - (a * y1 + b * y2))) <= 1e-12 * np.max(np.abs(y3))


def test_permuting_output_rows_permutes_y():
    inp = make_linear(2, 40, 256, 3, 8, seed=30)
    perm = np.random.default_rng(1).permutation(40)
    y = oracle.linear_inputs(inp)
    q2 = oracle.pack(inp.codes[perm], 3)
    y2 = oracle.linear(inp.x, q2, inp.scales[perm], inp.zeros[perm], inp.A, inp.B[perm],
                       2, 40, 256, 128, 3, 8)
    assert np.array_equal(y2, y[:, perm])


def test_tokens_are_independent_and_n_list_matches_full():
    inp = make_linear(4, 64, 512, 4, 16, seed=31)
    q = oracle.pack(inp.codes, 4)
    y = oracle.linear_inputs(inp, qweight=q)
    for m in range(4):
        ym = oracle.linear(inp.x[m:m + 1], q, inp.scales, inp.zeros, inp.A, inp.B, 1, 64, 512, 128, 4, 16)
        assert np.array_equal(ym[0], y[m])
    rows = np.array([63, 0, 17, 17, 32])
    ys = oracle.linear_inputs(inp, qweight=q, n_list=rows)
    assert np.array_equal(ys, y[:, rows])
    assert np.array_equal(oracle.linear_inputs(inp, qweight=q, threads=4), y)


@pytest.mark.parametrize("bits,dtype", [(4, "f16"), (3, "f16"), (4, "bf16")])
def test_exact_class_is_representable_in_the_output_type(bits, dtype):
    # The exact-class generator promises results that survive rounding to the
    # output type; the GPU parity tests rely on that to demand bit equality.
    kw = dict(x_nnz=32, x_max=2) if dtype == "f16" else dict(x_nnz=4, x_max=1)
    inp = make_exact_class(4, 64, 1024, bits, 16, dtype=dtype, seed=5, **kw)
    y = oracle.linear_inputs(inp)
    if dtype == "f16":
        back = y.astype(np.float16).astype(np.float64)
    else:
        back = bf16_bits_to_f64(f32_to_bf16_bits(y.astype(np.float32)))
    assert np.array_equal(back, y)
    assert np.any(y != 0)


def test_bad_requests_are_rejected():
    inp = make_linear(1, 8, 128, 4, 0, seed=0)
    q = oracle.pack(inp.codes, 4)
    with pytest.raises(ValueError):       # group does not divide K
        oracle.linear(inp.x, q, np.zeros((8, 1), np.float16), inp.zeros[:, :1], None, None,
                      1, 8, 128, 96, 4, 0)
    # rank > 0 without A and B: the C entry point itself refuses (returns -1)
    rc = oracle._load().oracle_linear(None, None, None, None, None, None, None, None,
                                      1, 8, 128, 128, 4, 2, 0, None, 8, 1)
    assert rc == -1
