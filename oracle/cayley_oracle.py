"""Plain float64 oracle of Cayley SGD with momentum (Algorithm 3), the orthogonal
optimiser the paper compares QR-Orth with (Sec. 5.3, Table 4).

TEST INFRASTRUCTURE: slow, obviously-correct numpy in float64; never imported by
the product path and never tuned for speed.  The steps are taken in the order
and notation of Algorithm 3.  Pinned by tests that do not reuse these formulas:
the exact Cayley transform solved with a linear solver (the limit of the inner
iteration), the closed form of W for an orthonormal iterate, the planar rotation
by 2 atan(alpha w / 2), skew-symmetry, the step-size rule on both sides of the
clip and first-order descent of the loss.  No function here is "parity unpinned".

Notation of Algorithm 3: X_k = the orthonormal iterate (here the rotation R
itself, there is no latent), M_k = the momentum, G(X_k) = dL/dR, l = learning
rate, beta = momentum coefficient, q = 0.5, s = 2, eps = 1e-8.

Readings taken where Algorithm 3 is garbled or silent (also listed in the
design notes of the repository):
  * The skew-symmetrisation step is printed with W_k on both sides; it is read as
    W_k = What_k - What_k^T (the only reading that makes W_k skew-symmetric, which
    the Cayley transform needs to stay on the orthogonal group).
  * The norm in the step-size rule is not named; the Frobenius norm is taken.  It
    bounds the spectral norm from above, so the inner iteration still contracts
    with factor <= q.
  * Y^0 = X_k + alpha M_{k+1} (the printed X without an index is X_k).
  * The loop runs exactly n_steps times; the loss reported for step k is the loss
    of X_k before the update (same convention as the QR-Orth loop).
  * X_1 is the orthogonal factor (positive-diagonal QR) of the initial latent the
    QR-Orth loop would start from, so both optimisers start from one rotation.
"""
from __future__ import annotations

import numpy as np

from . import calib_oracle as co

F64 = np.float64


def cayley_sgd_step(X: np.ndarray, M: np.ndarray, G: np.ndarray, lr: float, beta: float,
                    q: float = 0.5, s: int = 2, eps: float = 1e-8):
    """One iteration of the loop body of Algorithm 3.

    X: iterate (d x d), M: momentum, G: Euclidean gradient dL/dX at X.
    Returns a dict with every intermediate: M_half (momentum after the gradient
    is folded in), W_hat, W, M_new, alpha, Y (list Y^0..Y^s), X_new.
    """
    X = np.asarray(X, dtype=F64)
    M = np.asarray(M, dtype=F64)
    G = np.asarray(G, dtype=F64)
    # momentum accumulates the negative gradient
    M_half = beta * M - G
    # auxiliary matrix: M X^T - 1/2 X (X^T M X^T)
    W_hat = M_half @ X.T - 0.5 * (X @ (X.T @ M_half @ X.T))
    # skew-symmetric part (times two)
    W = W_hat - W_hat.T
    # momentum projected to the tangent space at X
    M_new = W @ X
    # step size: the learning rate, clipped so that the inner iteration contracts
    alpha = min(lr, 2.0 * q / (np.linalg.norm(W, "fro") + eps))
    # fixed-point iteration for the Cayley transform Y = X + alpha/2 W (X + Y)
    Y = [X + alpha * M_new]
    for _ in range(s):
        Y.append(X + 0.5 * alpha * (W @ (X + Y[-1])))
    return {"M_half": M_half, "W_hat": W_hat, "W": W, "M_new": M_new, "alpha": float(alpha),
            "Y": Y, "X_new": Y[-1]}


def cayley_calib_step(X_tokens: np.ndarray, R: np.ndarray, M: np.ndarray, lr: float, beta: float,
                      reduction: str = "mean", q: float = 0.5, s: int = 2, eps: float = 1e-8,
                      sign_decider=None):
    """One calibration iteration with Cayley SGD in place of QR-Orth: rotate, Whip
    loss (Eq. 4) and its gradient with respect to the rotation, then Algorithm 3's
    update of the rotation.  sign_decider as in calib_oracle.calib_step."""
    O = co.rotate(X_tokens, R)
    loss = co.whip_loss(O, reduction)
    G = co.whip_grad_wrt_output(O, reduction, None if sign_decider is None else sign_decider(O))
    Gq = co.grad_wrt_rotation(X_tokens, G)
    out = cayley_sgd_step(R, M, Gq, lr, beta, q, s, eps)
    out.update({"O": O, "loss": loss, "G": G, "Gq": Gq, "R_new": out["X_new"]})
    return out


def cayley_calib_run(X_tokens: np.ndarray, Z0: np.ndarray, lr: float, beta: float, n_steps: int,
                     reduction: str = "mean", q: float = 0.5, s: int = 2, eps: float = 1e-8):
    """Algorithm 3's loop for exactly n_steps iterations from X_1 = the orthogonal
    factor of Z0.  Returns (losses[n_steps], R_final, M_final)."""
    R, _ = co.qr_pos(np.asarray(Z0, dtype=F64))
    M = np.zeros_like(R)
    losses = np.empty(n_steps, dtype=F64)
    for k in range(n_steps):
        out = cayley_calib_step(X_tokens, R, M, lr, beta, reduction, q, s, eps)
        losses[k] = out["loss"]
        R, M = out["R_new"], out["M_new"]
    return losses, R, M
