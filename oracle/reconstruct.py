"""CPU oracle of one iteration of layer-wise reconstruction (Algorithm 1, lines 5-9; Section 4.2)
-- TEST INFRASTRUCTURE ONLY, like the rest of this package.

With W [N, K] the layer's weights, X [T, K] calibration activations (rows are tokens), H = X^T X,
Sigma = B.A (A [r, K], B [N, r]) and Q the group-wise quantiser of Section 4.1:

    Z  = W X^T                                   (line 5)
    Z' = Q(W - B A) X^T + B A X^T                (line 6)
    Delta_F = W - Q(W - Sigma) - Sigma           (so that Z - Z' = Delta_F X^T)
    L  = tr(Delta_F H Delta_F^T) = ||Z - Z'||_F^2   (line 7; see the reading below)
    dL/dSigma = -2 Delta_F H                     (line 8: W and Q(W - Sigma) detached, Eq. after
                                                  "This modification yields")
    dL/dB = (dL/dSigma) A^T,  dL/dA = B^T (dL/dSigma)      (chain rule through Sigma = B A)
    A <- A - lr dL/dA,  B <- B - lr dL/dB        (line 9, plain gradient descent)

Reading: the paper prints L_F both as the Frobenius norm and as the trace, which is its square;
the printed gradient -2 Delta_F X^T X is that of the trace form, which is taken here.  The
optimiser is not named beyond "gradient descent": fixed-step descent.  Both gradients use the
A and B from before the step.

The quantiser call is the oracle's single-precision one (its codes are rounding decisions); all
matrix products here are numpy float64.
"""
import numpy as np

from . import quantize_feedback


def gram(X: np.ndarray) -> np.ndarray:
    X = np.asarray(X, dtype=np.float64)
    return X.T @ X


def delta_f(W, A, B, group: int, bits: int):
    """Delta_F = W - W_F for float32 master copies A, B; also returns the codes."""
    codes, s, z, r, wf = quantize_feedback(np.asarray(W, np.float32), np.asarray(A, np.float32),
                                           np.asarray(B, np.float32), group, bits, dtype="f32")
    return np.asarray(W, np.float64) - wf.astype(np.float64), codes


def loss_and_grads(W, H, A, B, group: int, bits: int):
    """L, dL/dSigma, dL/dA, dL/dB at (A, B), with W and Q(W - B A) detached."""
    D, codes = delta_f(W, A, B, group, bits)
    H = np.asarray(H, np.float64)
    DH = D @ H
    loss = float(np.sum(DH * D))
    G = -2.0 * DH
    gB = G @ np.asarray(A, np.float64).T
    gA = np.asarray(B, np.float64).T @ G
    return loss, G, gA, gB, D, codes


def step(W, H, A, B, lr: float, group: int, bits: int):
    """One iteration: returns (loss before the update, A', B') with A', B' float64."""
    loss, G, gA, gB, _, _ = loss_and_grads(W, H, A, B, group, bits)
    return loss, np.asarray(A, np.float64) - lr * gA, np.asarray(B, np.float64) - lr * gB
