"""Pins of the Cayley-SGD oracle (Algorithm 3) against facts it does not itself
define: the exact Cayley transform from a linear solve, the closed form of W at
an orthonormal iterate, the planar rotation angle, skew-symmetry, the step-size
clip and first-order descent of the Whip loss.  Each is chosen so that a dropped
term, a wrong sign or factor, or a transposed operand in the oracle fails it."""
import math

import numpy as np
import pytest

import oracle as orc

RNG = np.random.default_rng(4321)


def rand_orth(d, rng=RNG):
    q, r = np.linalg.qr(rng.standard_normal((d, d)))
    return q * np.sign(np.diag(r))


@pytest.mark.parametrize("d,beta", [(5, 0.0), (12, 0.9), (33, 0.5)])
def test_w_is_skew_and_momentum_is_tangent(d, beta):
    X, M, G = rand_orth(d), RNG.standard_normal((d, d)), RNG.standard_normal((d, d))
    out = orc.cayley_sgd_step(X, M, G, lr=0.1, beta=beta)
    W = out["W"]
    assert np.abs(W + W.T).max() == 0.0                      # exactly skew-symmetric
    # M_new = W X lies in the tangent space at X: X^T M_new is skew-symmetric
    A = X.T @ out["M_new"]
    assert np.abs(A + A.T).max() < 1e-13


@pytest.mark.parametrize("d", [4, 9, 24])
def test_w_closed_form_at_orthonormal_iterate(d):
    # X X^T = I  =>  What = B - B/2 with B = M X^T, so W = (B - B^T) / 2 with M = beta M0 - G.
    X, M0, G = rand_orth(d), RNG.standard_normal((d, d)), RNG.standard_normal((d, d))
    beta = 0.7
    out = orc.cayley_sgd_step(X, M0, G, lr=0.01, beta=beta)
    B = (beta * M0 - G) @ X.T
    assert np.abs(out["W"] - 0.5 * (B - B.T)).max() < 1e-13
    # without momentum the projected momentum is minus the Riemannian gradient (G - X G^T X) / 2
    out0 = orc.cayley_sgd_step(X, np.zeros((d, d)), G, lr=0.01, beta=0.0)
    assert np.abs(out0["M_new"] + 0.5 * (G - X @ G.T @ X)).max() < 1e-13


def test_w_hat_uses_the_half_weighted_correction_for_non_orthonormal_x():
    # For X = c Q (Q orthonormal) the correction term scales like c^4 and the first like c^2 (per
    # factor of M X^T): What = c B - c^3 B / 2 with B = M Q^T.  Fails if the 1/2, a transpose or a
    # factor of X is lost.
    d, c = 7, 1.3
    Q, G = rand_orth(d), RNG.standard_normal((d, d))
    out = orc.cayley_sgd_step(c * Q, np.zeros((d, d)), G, lr=0.01, beta=0.0)
    B = -G @ Q.T
    assert np.abs(out["W_hat"] - (c * B - 0.5 * c ** 3 * B)).max() < 1e-12


@pytest.mark.parametrize("d,lr", [(6, 0.05), (20, 0.2)])
def test_inner_iteration_converges_to_exact_cayley_transform(d, lr):
    # The fixed point of Y = X + a/2 W (X + Y) is Y = (I - a/2 W)^-1 (I + a/2 W) X, which is orthogonal.
    X, G = rand_orth(d), RNG.standard_normal((d, d))
    out = orc.cayley_sgd_step(X, np.zeros((d, d)), G, lr=lr, beta=0.0, s=80)
    a, W = out["alpha"], out["W"]
    Y_exact = np.linalg.solve(np.eye(d) - 0.5 * a * W, (np.eye(d) + 0.5 * a * W) @ X)
    assert np.abs(out["X_new"] - Y_exact).max() < 1e-12
    assert np.abs(Y_exact.T @ Y_exact - np.eye(d)).max() < 1e-12
    # each sweep shrinks the distance to the fixed point by at least the contraction factor a |W| / 2 <= q
    errs = [np.linalg.norm(y - Y_exact) for y in out["Y"][:8]]
    rho = 0.5 * a * np.linalg.norm(W, 2)
    assert rho <= 0.5 + 1e-12
    for e0, e1 in zip(errs, errs[1:]):
        assert e1 <= rho * e0 * (1 + 1e-6) + 1e-15


def test_two_sweeps_are_the_default_and_nearly_orthogonal():
    d = 16
    X, G = rand_orth(d), 0.1 * RNG.standard_normal((d, d))
    out = orc.cayley_sgd_step(X, np.zeros((d, d)), G, lr=0.05, beta=0.0)
    assert len(out["Y"]) == 3                                   # Y^0, Y^1, Y^2
    a, W = out["alpha"], out["W"]
    Y_exact = np.linalg.solve(np.eye(d) - 0.5 * a * W, (np.eye(d) + 0.5 * a * W) @ X)
    rho = 0.5 * a * np.linalg.norm(W, 2)
    e0 = np.linalg.norm(out["Y"][0] - Y_exact, 2)
    assert np.linalg.norm(out["X_new"] - Y_exact, 2) <= rho ** 2 * e0 * (1 + 1e-6)
    assert np.abs(out["X_new"].T @ out["X_new"] - np.eye(d)).max() < 1e-3


def test_planar_rotation_angle():
    # d = 2: W = [[0, -w], [w, 0]]; the exact Cayley transform rotates by 2 atan(a w / 2).
    th = 0.4
    X = np.array([[math.cos(th), -math.sin(th)], [math.sin(th), math.cos(th)]])
    G = np.array([[0.3, -1.1], [0.8, 0.2]])
    out = orc.cayley_sgd_step(X, np.zeros((2, 2)), G, lr=0.3, beta=0.0, s=200)
    w = out["W"][1, 0]
    phi = 2.0 * math.atan(0.5 * out["alpha"] * w)
    Rphi = np.array([[math.cos(phi), -math.sin(phi)], [math.sin(phi), math.cos(phi)]])
    assert np.abs(out["X_new"] - Rphi @ X).max() < 1e-13


def test_step_size_rule_both_sides_of_the_clip():
    d = 8
    X, G = rand_orth(d), RNG.standard_normal((d, d))
    small = orc.cayley_sgd_step(X, np.zeros((d, d)), 1e-3 * G, lr=0.5, beta=0.0)
    assert small["alpha"] == 0.5                                 # 2q / |W| is far above the learning rate
    big = orc.cayley_sgd_step(X, np.zeros((d, d)), 1e3 * G, lr=0.5, beta=0.0)
    B = -1e3 * G @ X.T
    wn = math.sqrt(((0.5 * (B - B.T)) ** 2).sum())
    assert big["alpha"] == pytest.approx(1.0 / (wn + 1e-8), rel=1e-12)    # 2 q = 1
    assert big["alpha"] < 0.5


def test_first_order_descent_of_the_whip_loss():
    # d/da L(Cayley(a W) X) at a = 0 equals <Gq, W X> = -|Gq X^T - X Gq^T|_F^2 / 4 < 0 (no momentum).
    d, n = 12, 40
    Xt = RNG.laplace(size=(n, d))
    R = rand_orth(d)
    h = 1e-5
    out = orc.cayley_calib_step(Xt, R, np.zeros((d, d)), lr=h, beta=0.0, s=40)
    Gq = out["Gq"]
    slope = -0.25 * ((Gq @ R.T - R @ Gq.T) ** 2).sum()
    assert slope < 0
    assert float((Gq * out["M_new"]).sum()) == pytest.approx(slope, rel=1e-10)
    l1 = orc.whip_loss(orc.rotate(Xt, out["R_new"]))
    assert (l1 - out["loss"]) / h == pytest.approx(slope, rel=1e-3)


def test_run_keeps_orthogonality_and_decreases_loss():
    d, n = 16, 256
    Xt = RNG.laplace(size=(n, d))
    Xt[:, 3] *= 20.0
    Z0 = np.eye(d) + 0.01 * RNG.standard_normal((d, d))
    losses, R, M = orc.cayley_calib_run(Xt, Z0, lr=0.005, beta=0.9, n_steps=30)
    # two sweeps leave an error of order (alpha |W| / 2)^3 per step, so the iterate drifts off the
    # orthogonal group slowly; with this step size it stays within 1e-3
    assert np.abs(R.T @ R - np.eye(d)).max() < 1e-3
    assert losses[-1] < losses[0]
    # step 0 starts from the positive-diagonal orthogonal factor of Z0
    R0, _ = orc.qr_pos(Z0)
    assert losses[0] == pytest.approx(orc.whip_loss(orc.rotate(Xt, R0)), rel=1e-14)
