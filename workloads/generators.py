"""Seeded synthetic tensors with the shapes and value distributions of the
paper's Llama-2 workloads (Section 5.1: group size 128, sub-branches on the
q/k/v/o/gate/up/down projections; Fig. "wallclock": batch 1).

Everything here is data preparation: draw, round once to the storage type,
hand the same bits to whoever asks.  No packing, dequantisation or contraction
lives in this module.

Storage conventions used by every consumer:
  codes   uint8  [N, K]      one quantisation code per byte, 0 .. 2**bits-1
  scales  fp16   [N, K/group]
  zeros   fp16   [N, K/group]   integer-valued
  x       uint16 [M, K]      bit patterns of fp16 or bf16 (see ``dtype``)
  A       uint16 [rank, K]   down-projection, same dtype as x
  B       uint16 [N, rank]   up-projection, same dtype as x
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

# (K, N) of the seven linears of one decoder layer, in call order
# q, k, v, o, gate, up, down.
LLAMA2_7B_SHAPES = [(4096, 4096)] * 4 + [(4096, 11008)] * 2 + [(11008, 4096)]
LLAMA2_13B_SHAPES = [(5120, 5120)] * 4 + [(5120, 13824)] * 2 + [(13824, 5120)]


# --------------------------------------------------------------------------
# storage-type conversions (exact widening, round-to-nearest-even narrowing)
# --------------------------------------------------------------------------
def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (uint16), round to nearest even."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    u = b.astype(np.uint32) << np.uint32(16)
    with np.errstate(invalid="ignore"):      # signalling-NaN patterns stay NaN
        return u.view(np.float32).astype(np.float64)


def f16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(b, dtype=np.uint16).view(np.float16).astype(np.float64)


def _to_bits(a: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "f16":
        return np.ascontiguousarray(a.astype(np.float16)).view(np.uint16).copy()
    if dtype == "bf16":
        return f32_to_bf16_bits(a.astype(np.float32))
    raise ValueError(dtype)


def bits_to_f64(b: np.ndarray, dtype: str) -> np.ndarray:
    return f16_bits_to_f64(b) if dtype == "f16" else bf16_bits_to_f64(b)


def _rng(seed: int, tensor_id: int) -> np.random.Generator:
    # Counter-based generator keyed by (seed, tensor): a tensor's values do not
    # depend on which other tensors were drawn before it.
    return np.random.Generator(np.random.Philox(key=[int(seed) & (2**64 - 1), int(tensor_id)]))


@dataclass
class LinearInputs:
    M: int
    N: int
    K: int
    group: int
    bits: int
    rank: int
    dtype: str                      # "f16" or "bf16": type of x, A, B and y
    codes: np.ndarray
    scales: np.ndarray              # np.float16
    zeros: np.ndarray               # np.float16
    x: np.ndarray                   # uint16 bit patterns
    A: np.ndarray | None
    B: np.ndarray | None
    meta: dict = field(default_factory=dict)

    def x_f64(self) -> np.ndarray:
        return bits_to_f64(self.x, self.dtype)

    def A_f64(self) -> np.ndarray:
        return bits_to_f64(self.A, self.dtype)

    def B_f64(self) -> np.ndarray:
        return bits_to_f64(self.B, self.dtype)


def make_linear(M: int, N: int, K: int, bits: int, rank: int, *, group: int = 128,
                dtype: str = "f16", seed: int = 0, z_values=None, ab_std: float = 0.02,
                outlier_frac: float = 0.0, outlier_scale: float = 20.0,
                codes_equal_zero: bool = False) -> LinearInputs:
    """One layer's inputs with the benchmark distributions.

    codes ~ U{0..2^bits-1};  scales ~ U[0.005, 0.02];  zeros ~ U(z_values)
    (default {6,7,8,9} for 4 bits and the same +-1.5 spread around mid-range,
    {2,3,4,5}, for 3 bits);  A, B ~ N(0, ab_std^2);  x ~ N(0,1) with an optional
    seeded fraction of input channels multiplied by ``outlier_scale`` for every
    token (activation outliers of the prefill workload).
    ``codes_equal_zero`` sets every code to its group's zero point, which makes
    the main path vanish and leaves the sub-branch alone in y.
    """
    assert K % group == 0
    G = K // group
    qmax = (1 << bits) - 1
    if z_values is None:
        z_values = (6, 7, 8, 9) if bits == 4 else (2, 3, 4, 5)
    z_values = np.asarray(z_values, dtype=np.int64)
    codes = _rng(seed, 1).integers(0, qmax + 1, size=(N, K), dtype=np.uint8)
    scales = _rng(seed, 2).uniform(0.005, 0.02, size=(N, G)).astype(np.float16)
    zeros_i = z_values[_rng(seed, 3).integers(0, len(z_values), size=(N, G))]
    zeros = zeros_i.astype(np.float16)
    if codes_equal_zero:
        assert zeros_i.max() <= qmax and zeros_i.min() >= 0
        codes = np.repeat(zeros_i.astype(np.uint8), group, axis=1)
    xf = _rng(seed, 4).standard_normal(size=(M, K)).astype(np.float32)
    n_out = 0
    if outlier_frac > 0.0:
        n_out = max(1, int(round(outlier_frac * K)))
        ch = _rng(seed, 5).choice(K, size=n_out, replace=False)
        xf[:, ch] *= np.float32(outlier_scale)
    x = _to_bits(xf, dtype)
    A = B = None
    if rank > 0:
        A = _to_bits((_rng(seed, 6).standard_normal(size=(rank, K)) * ab_std).astype(np.float32), dtype)
        B = _to_bits((_rng(seed, 7).standard_normal(size=(N, rank)) * ab_std).astype(np.float32), dtype)
    return LinearInputs(M, N, K, group, bits, rank, dtype, codes, scales, zeros, x, A, B,
                        meta=dict(seed=seed, z_values=z_values.tolist(), ab_std=ab_std,
                                  outlier_channels=n_out))


def make_exact_class(M: int, N: int, K: int, bits: int, rank: int, *, group: int = 128,
                     dtype: str = "f16", seed: int = 0, x_nnz: int | None = 32,
                     x_max: int = 2, b_nnz: int = 2) -> LinearInputs:
    """Inputs for which no rounding can occur anywhere in the layer.

    Scales are 2^-3 or 2^-4 (2^-3 only for bf16), x holds ``x_nnz`` non-zero
    small integers per token (all positions if None), A is in {0, +-1/4} and
    each row of B has ``b_nnz`` entries of +-1/4.  Every product and partial sum
    is then a small dyadic number: fp32 accumulation in any order and the final
    rounding to fp16 are exact, so a correct implementation must reproduce the
    plain definition bit for bit.  (With x_nnz=32, x_max=2, rank<=64:
    abs(main) <= 32*2*15/8 = 120, abs(sub) <= 2*16/4 = 8, granularity 1/16.)
    """
    G = K // group
    qmax = (1 << bits) - 1
    codes = _rng(seed, 11).integers(0, qmax + 1, size=(N, K), dtype=np.uint8)
    exps = _rng(seed, 12).integers(3, 5 if dtype == "f16" else 4, size=(N, G))
    scales = (2.0 ** (-exps.astype(np.float64))).astype(np.float16)
    zeros = _rng(seed, 13).integers(0, qmax + 1, size=(N, G)).astype(np.float16)
    r4 = _rng(seed, 14)
    xf = np.zeros((M, K), dtype=np.float32)
    vals = np.array([v for v in range(-x_max, x_max + 1) if v != 0], dtype=np.float32)
    for m in range(M):
        if x_nnz is None:
            xf[m] = r4.integers(-x_max, x_max + 1, size=K).astype(np.float32)
        else:
            pos = r4.choice(K, size=min(x_nnz, K), replace=False)
            xf[m, pos] = vals[r4.integers(0, len(vals), size=len(pos))]
    x = _to_bits(xf, dtype)
    A = B = None
    if rank > 0:
        Af = _rng(seed, 16).integers(-1, 2, size=(rank, K)).astype(np.float32) * 0.25
        Bf = np.zeros((N, rank), dtype=np.float32)
        r7 = _rng(seed, 17)
        for n in range(N):
            pos = r7.choice(rank, size=min(b_nnz, rank), replace=False)
            Bf[n, pos] = (r7.integers(0, 2, size=len(pos)).astype(np.float32) * 2 - 1) * 0.25
        A, B = _to_bits(Af, dtype), _to_bits(Bf, dtype)
    return LinearInputs(M, N, K, group, bits, rank, dtype, codes, scales, zeros, x, A, B,
                        meta=dict(seed=seed, exact=True))


def worked_example_e1() -> LinearInputs:
    """The 8x8 hand-worked layer (all values dyadic, so every correct
    implementation is bit-exact): M=1, N=K=8, group=8, 4 bits, rank 2.

      q[n][k] = (3n + 5k) mod 16      s[n] = 2^-(2 + n mod 3)    z[n] = 7 + (n mod 2)
      x[k] = k - 3
      A[0][k] = ((k mod 3) - 1)/4     A[1][k] = +1/2 for k < 4, -1/2 otherwise
      B[n] = [ (n - 4)/4 , (-1)^n / 8 ]
    The expected packed words, t, main, sub and y are stored as text fixtures
    beside the tests; they were worked out by hand from the layer definition.
    """
    N = K = 8
    n = np.arange(N)[:, None]
    k = np.arange(K)[None, :]
    codes = ((3 * n + 5 * k) % 16).astype(np.uint8)
    scales = (2.0 ** -(2 + (np.arange(N) % 3))).astype(np.float16).reshape(N, 1)
    zeros = (7 + (np.arange(N) % 2)).astype(np.float16).reshape(N, 1)
    xf = (np.arange(K) - 3).astype(np.float32).reshape(1, K)
    Af = np.stack([((np.arange(K) % 3) - 1) / 4.0,
                   np.where(np.arange(K) < 4, 0.5, -0.5)]).astype(np.float32)
    Bf = np.stack([(np.arange(N) - 4) / 4.0, ((-1.0) ** np.arange(N)) / 8.0], axis=1).astype(np.float32)
    return LinearInputs(1, N, K, 8, 4, 2, "f16", codes, scales, zeros,
                        _to_bits(xf, "f16"), _to_bits(Af, "f16"), _to_bits(Bf, "f16"),
                        meta=dict(name="E1"))
