"""Pins of the oracle's reconstruction step (Algorithm 1 lines 5-9, Section 4.2) against the
mathematics: the trace form equals the squared output error computed from X itself, the printed
gradient matches finite differences of the DETACHED objective, the chain rule through Sigma = B A
matches finite differences in A and B, zero gradient for A while B = 0 (Algorithm 1's initialisation),
and gradient descent on synthetic activations lowers the loss."""
import numpy as np
import pytest

import oracle
from oracle import reconstruct as rec


def _problem(N=24, K=256, T=96, rank=8, seed=0, b_zero=False):
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((N, K)) * 0.05).astype(np.float32)
    X = rng.standard_normal((T, K)) * (1.0 + 4.0 * (rng.random(K) < 0.05))      # a few loud channels
    A = (rng.standard_normal((rank, K)) * 0.05).astype(np.float32)
    B = np.zeros((N, rank), np.float32) if b_zero else (rng.standard_normal((N, rank)) * 0.05).astype(np.float32)
    return W, X, A, B


@pytest.mark.parametrize("bits", [3, 4])
def test_trace_form_is_the_squared_output_error(bits):
    W, X, A, B = _problem(seed=bits)
    H = rec.gram(X)
    loss, G, gA, gB, D, codes = rec.loss_and_grads(W, H, A, B, 128, bits)
    # Z = W X^T and Z' = Q(W - BA) X^T + B A X^T computed the long way, from X, not from H
    s64 = W.astype(np.float64) - D                       # W_F
    Z = W.astype(np.float64) @ X.T
    Zp = (s64 - B.astype(np.float64) @ A.astype(np.float64)) @ X.T + B.astype(np.float64) @ (A.astype(np.float64) @ X.T)
    assert np.isclose(loss, np.linalg.norm(Z - Zp) ** 2, rtol=1e-10)
    assert loss > 0


def test_printed_gradient_is_that_of_the_detached_objective():
    W, X, A, B = _problem(seed=5)
    H = rec.gram(X)
    loss, G, gA, gB, D, _ = rec.loss_and_grads(W, H, A, B, 128, 4)
    Qc = W.astype(np.float64) - D - B.astype(np.float64) @ A.astype(np.float64)      # Q(W - Sigma), held fixed
    def f(Sigma):
        Dl = W.astype(np.float64) - Qc - Sigma
        return np.sum((Dl @ H) * Dl)
    S0 = B.astype(np.float64) @ A.astype(np.float64)
    rng = np.random.default_rng(1)
    for _ in range(5):
        V = rng.standard_normal(S0.shape)
        eps = 1e-6
        num = (f(S0 + eps * V) - f(S0 - eps * V)) / (2 * eps)
        assert np.isclose(num, np.sum(G * V), rtol=1e-6)
    # with the straight-through surrogate Q(w) = w and nothing detached, Delta_F = W - (W - Sigma) - Sigma
    # vanishes identically, hence its gradient too: the reason the paper detaches the feedback signal
    assert np.abs(W.astype(np.float64) - (W.astype(np.float64) - S0) - S0).max() < 1e-15


def test_chain_rule_through_the_low_rank_factors():
    W, X, A, B = _problem(N=12, K=128, T=64, rank=4, seed=6)
    H = rec.gram(X)
    loss, G, gA, gB, D, _ = rec.loss_and_grads(W, H, A, B, 128, 4)
    Qc = W.astype(np.float64) - D - B.astype(np.float64) @ A.astype(np.float64)
    def f(Bv, Av):
        Dl = W.astype(np.float64) - Qc - Bv @ Av
        return np.sum((Dl @ H) * Dl)
    A64, B64 = A.astype(np.float64), B.astype(np.float64)
    rng = np.random.default_rng(2)
    eps = 1e-6
    for _ in range(6):
        i, j = rng.integers(0, B.shape[0]), rng.integers(0, B.shape[1])
        E = np.zeros_like(B64); E[i, j] = eps
        assert np.isclose((f(B64 + E, A64) - f(B64 - E, A64)) / (2 * eps), gB[i, j], rtol=1e-5, atol=1e-9)
        i, j = rng.integers(0, A.shape[0]), rng.integers(0, A.shape[1])
        E = np.zeros_like(A64); E[i, j] = eps
        assert np.isclose((f(B64, A64 + E) - f(B64, A64 - E)) / (2 * eps), gA[i, j], rtol=1e-5, atol=1e-9)


def test_initialisation_of_algorithm_1_moves_b_first():
    # A ~ N(0, sigma^2), B = 0: dL/dA = B^T G = 0 and dL/dB = G A^T != 0, and Sigma = 0 means the
    # quantiser sees W itself
    W, X, A, B = _problem(seed=7, b_zero=True)
    H = rec.gram(X)
    loss, G, gA, gB, D, codes = rec.loss_and_grads(W, H, A, B, 128, 3)
    assert np.all(gA == 0) and np.abs(gB).max() > 0
    c0, *_ = oracle.quantize_feedback(W, None, None, 128, 3)
    assert np.array_equal(codes, c0)


@pytest.mark.parametrize("bits", [3, 4])
def test_gradient_descent_lowers_the_reconstruction_loss(bits):
    W, X, A, B = _problem(N=32, K=256, T=128, rank=16, seed=8 + bits, b_zero=True)
    H = rec.gram(X)
    lr = 0.2 / (np.linalg.eigvalsh(H)[-1] * np.linalg.norm(A.astype(np.float64), 2) ** 2)
    losses = []
    A64, B64 = A.astype(np.float64), B.astype(np.float64)
    for _ in range(20):                                  # the paper trains 20 epochs (Section 5.1)
        loss, A64, B64 = rec.step(W, H, A64.astype(np.float32), B64.astype(np.float32), lr, 128, bits)
        losses.append(loss)
    assert losses[-1] < 0.9 * losses[0]
    assert min(losses) == losses[-1] or losses[-1] < 1.02 * min(losses)       # no blow-up at the end
