"""Plain float64 oracle of one calibration iteration (Algorithm 1 body).

TEST INFRASTRUCTURE: slow, obviously-correct numpy in float64; never imported by
the product path and never tuned for speed.  Every function cites the passage
of the paper it restates.  All parts are pinned by tests that do not depend on
this file's own formulas (closed forms, finite differences, LAPACK, invariants);
no function here is "parity unpinned".

Notation (the paper overloads R): X = activations, N tokens x d channels, one
token per row.  Z = latent d x d.  R = the rotation = orthogonal factor of
Z = R U, U upper triangular (Sec. 4.3 names the factors R and U; Algorithm 2
calls them Q and R).  O = X R.  G = dL/dO.  Gq = dL/dR.  Gz = dL/dZ.

Readings taken where the paper is silent (each is also listed in the design
notes of the repository):
  * Whip of a matrix (Algorithm 1, the loss of the rotated activations) = mean over tokens of Eq. 4 applied
    to each token row; "sum" keeps the plain sum over tokens.
  * d|o|/do at o = 0 is taken as 0.
  * The rotation reported is the unique factor with diag(U) > 0; Algorithm 2's
    own sign rule yields the same R up to column signs, which change neither
    the loss nor dL/dZ.
  * Algorithm 2's update of Q as printed touches only Q[k:n, k:n]; the accumulated
    product of reflectors needs the full rows k:n, which is what is done here.
  * Plain SGD: no momentum, no weight decay, constant learning rate.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


def widen_input(x) -> np.ndarray:
    """Stored inputs (fp32, or bf16 already widened to fp32) -> float64, exactly."""
    return np.asarray(x, dtype=F64)


# ----------------------------------------------------------------------------
# Whip loss (Eq. 4) and its derivative
# ----------------------------------------------------------------------------
def whip_per_token(O: np.ndarray) -> np.ndarray:
    """Eq. 4 for each token row: sum over channels of exp(-|o_i|)."""
    O = np.asarray(O, dtype=F64)
    return np.exp(-np.abs(O)).sum(axis=-1)


def whip_loss(O: np.ndarray, reduction: str = "mean") -> float:
    """Algorithm 1 (loss step): Whip of the rotated activation matrix."""
    per_tok = whip_per_token(O)
    if reduction == "mean":
        return float(per_tok.sum() / per_tok.shape[0])
    if reduction == "sum":
        return float(per_tok.sum())
    raise ValueError(reduction)


def whip_grad_wrt_output(O: np.ndarray, reduction: str = "mean", sign_of_O=None) -> np.ndarray:
    """G = dL/dO.  d/do exp(-|o|) = -sign(o) exp(-|o|), sign(0) = 0 (Eq. 4).

    Eq. 4 has a kink at o = 0, so sign(o) is a discrete decision taken on a
    floating-point value.  A caller comparing against an implementation in lower
    precision may pass sign_of_O (entries in {-1, 0, +1}) to take that decision
    in the other implementation's precision for outputs that are zero to within
    its rounding error; everything else is unchanged.
    """
    O = np.asarray(O, dtype=F64)
    scale = 1.0 / O.shape[0] if reduction == "mean" else 1.0
    sgn = np.sign(O) if sign_of_O is None else np.asarray(sign_of_O, dtype=F64)
    return -sgn * np.exp(-np.abs(O)) * scale


# ----------------------------------------------------------------------------
# QR-Orth forward: Householder QR (Algorithm 2), then the positive-diagonal gauge
# ----------------------------------------------------------------------------
def householder_qr_alg2(Z: np.ndarray):
    """Algorithm 2 with its own sign rule v = x + sign(x_1)||x|| e_1.

    Returns (Q, U) with Z = Q U, Q orthogonal, U upper triangular, in the raw
    gauge of the algorithm: U_kk = -sign(x_1)||x|| for k < n, last diagonal
    entry untouched.  sign(0) is taken as +1 (the paper leaves it undefined).
    """
    Z = np.asarray(Z, dtype=F64)
    n = Z.shape[0]
    assert Z.shape == (n, n)
    U = Z.copy()
    Qt = np.eye(n, dtype=F64)            # accumulates H_{n-1} ... H_1 = Q^T
    for k in range(n - 1):
        x = U[k:, k]
        normx = np.sqrt(np.dot(x, x))
        if normx == 0.0:
            continue                      # column already zero: H_k = I
        v = x.copy()
        v[0] += (1.0 if x[0] >= 0.0 else -1.0) * normx
        v /= np.sqrt(np.dot(v, v))
        U[k:, k:] -= 2.0 * np.outer(v, v @ U[k:, k:])
        Qt[k:, :] -= 2.0 * np.outer(v, v @ Qt[k:, :])
        U[k + 1:, k] = 0.0                # exact zeros below the diagonal
    return Qt.T.copy(), U


def _fix_gauge(Q: np.ndarray, U: np.ndarray):
    """R = Q diag(s), U <- diag(s) U with s_j = sign(U_jj) (+1 when zero)."""
    s = np.where(np.diag(U) < 0.0, -1.0, 1.0)
    return Q * s[None, :], U * s[:, None]


def qr_pos(Z: np.ndarray):
    """Sec. 4.3: Z = R U with R orthogonal; gauge fixed to diag(U) > 0."""
    Q, U = householder_qr_alg2(Z)
    return _fix_gauge(Q, U)


def qr_pos_lapack(Z: np.ndarray):
    """The same unique factorisation obtained from the library QR.

    Used by tests to pin qr_pos, and at sizes where the literal Algorithm 2
    loop above would take minutes.
    """
    Q, U = np.linalg.qr(np.asarray(Z, dtype=F64), mode="complete")
    return _fix_gauge(Q, np.triu(U))


# ----------------------------------------------------------------------------
# Rotation, back-propagation, optimiser
# ----------------------------------------------------------------------------
def rotate(X: np.ndarray, R: np.ndarray) -> np.ndarray:
    """Algorithm 1 (rotation step): O = X @ R (tokens are rows)."""
    return widen_input(X) @ np.asarray(R, dtype=F64)


def grad_wrt_rotation(X: np.ndarray, G: np.ndarray) -> np.ndarray:
    """Chain rule through O = X R:  Gq = X^T G."""
    return widen_input(X).T @ np.asarray(G, dtype=F64)


def qr_backward(R: np.ndarray, U: np.ndarray, Gq: np.ndarray) -> np.ndarray:
    """dL/dZ given dL/dR, for Z = R U (Algorithm 1, update step, by the chain rule).

    dZ = dR U + R dU.  With A = R^T dZ U^-1 = Omega + dU U^-1, Omega = R^T dR
    skew and dU U^-1 upper triangular, Omega is fixed by the strictly lower part
    of A.  Hence dL = <R^T Gq, Omega> = <tril(B - B^T, -1), A> with B = R^T Gq,
    i.e.  Gz = R tril(B - B^T, -1) U^-T.
    """
    R = np.asarray(R, dtype=F64)
    U = np.asarray(U, dtype=F64)
    B = R.T @ np.asarray(Gq, dtype=F64)
    S = np.tril(B - B.T, -1)
    M = R @ S
    # Gz U^T = M  <=>  U Gz^T = M^T
    return np.linalg.solve(U, M.T).T


def sgd_step(Z: np.ndarray, Gz: np.ndarray, lr: float) -> np.ndarray:
    """Algorithm 1 (update step): Z <- Z - eta dL/dZ."""
    return np.asarray(Z, dtype=F64) - lr * np.asarray(Gz, dtype=F64)


def momentum_step(Z: np.ndarray, Gz: np.ndarray, velocity: np.ndarray, lr: float, momentum: float):
    """SGD with (heavy-ball) momentum on the latent: the paper optimises Z with a standard
    optimiser (Sec. 4.3, "SGD or Adam").  v <- mu v + g;  Z <- Z - eta v.  Returns (Z, v)."""
    v = momentum * np.asarray(velocity, dtype=F64) + np.asarray(Gz, dtype=F64)
    return np.asarray(Z, dtype=F64) - lr * v, v


def adam_step(Z: np.ndarray, Gz: np.ndarray, m: np.ndarray, v: np.ndarray, t: int, lr: float,
              beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8):
    """Adam on the latent (Sec. 4.3 / the optimiser comparison table use it unchanged), in its
    published form: m <- b1 m + (1 - b1) g;  v <- b2 v + (1 - b2) g^2;  bias-corrected
    mhat = m / (1 - b1^t), vhat = v / (1 - b2^t);  Z <- Z - eta mhat / (sqrt(vhat) + eps).
    t is the 1-based index of this step.  Returns (Z, m, v)."""
    g = np.asarray(Gz, dtype=F64)
    m = beta1 * np.asarray(m, dtype=F64) + (1.0 - beta1) * g
    v = beta2 * np.asarray(v, dtype=F64) + (1.0 - beta2) * g * g
    mhat = m / (1.0 - beta1 ** t)
    vhat = v / (1.0 - beta2 ** t)
    return np.asarray(Z, dtype=F64) - lr * mhat / (np.sqrt(vhat) + eps), m, v


def calib_step(X: np.ndarray, Z: np.ndarray, lr: float, reduction: str = "mean",
               qr=qr_pos, sign_decider=None):
    """One pass of the loop body of Algorithm 1.

    Returns a dict with every intermediate so that tests can compare each stage.
    The loss is L(Z) before the update.  sign_decider(O) -> sign array lets a
    test take the sign decision at the kink of Eq. 4 in the precision of the
    implementation under test (see whip_grad_wrt_output).
    """
    R, U = qr(Z)
    O = rotate(X, R)
    loss = whip_loss(O, reduction)
    G = whip_grad_wrt_output(O, reduction, None if sign_decider is None else sign_decider(O))
    Gq = grad_wrt_rotation(X, G)
    Gz = qr_backward(R, U, Gq)
    Z_new = sgd_step(Z, Gz, lr)
    return {"R": R, "U": U, "O": O, "loss": loss, "G": G, "Gq": Gq, "Gz": Gz,
            "Z_new": Z_new}


def calib_run(X: np.ndarray, Z0: np.ndarray, lr: float, n_steps: int,
              reduction: str = "mean", qr=qr_pos):
    """Algorithm 1's loop for exactly n_steps iterations.

    Returns (losses[n_steps], Z_final, R_final) with R_final the rotation of the
    final latent (one more QR, not the rotation used by the last step).
    """
    Z = np.asarray(Z0, dtype=F64).copy()
    losses = np.empty(n_steps, dtype=F64)
    for k in range(n_steps):
        out = calib_step(X, Z, lr, reduction, qr)
        losses[k] = out["loss"]
        Z = out["Z_new"]
    R, _ = qr(Z)
    return losses, Z, R
