"""Pins of the float64 oracle against facts it does not itself define:
closed forms of Eq. 4, finite differences, LAPACK, algebraic invariants.
Each test is built so that one plausible slip in the oracle (a dropped term,
a sign, a transposed operand, a wrong index) makes it fail."""
import math

import numpy as np
import pytest

import oracle as orc
from paper_2511_04063_b200 import inputs as gen

RNG = np.random.default_rng(1234)


def hadamard(n):
    return gen.sylvester_hadamard(n).astype(np.float64)


# ---------------------------------------------------------------- Whip (Eq. 4)
@pytest.mark.parametrize("d,n", [(4, 3), (16, 7), (64, 5)])
def test_whip_zero_input_gives_d(d, n):
    # exp(-|0|) = 1 per channel -> every token contributes d; mean = d, sum = n d
    O = np.zeros((n, d))
    assert orc.whip_loss(O) == pytest.approx(d, abs=1e-14)
    assert orc.whip_loss(O, "sum") == pytest.approx(n * d, abs=1e-12)


@pytest.mark.parametrize("d,a,j", [(8, 2.5, 3), (16, 0.75, 0), (32, 11.0, 31)])
def test_whip_one_hot_closed_forms(d, a, j):
    X = np.zeros((1, d))
    X[0, j] = a
    # identity rotation: d-1 zero channels and one channel a
    assert orc.whip_loss(orc.rotate(X, np.eye(d))) == pytest.approx((d - 1) + math.exp(-a), rel=1e-14)
    # normalised Hadamard: every channel has magnitude a / sqrt(d)
    Rh = hadamard(d) / math.sqrt(d)
    assert orc.whip_loss(orc.rotate(X, Rh)) == pytest.approx(d * math.exp(-a / math.sqrt(d)), rel=1e-14)
    # negative entry: |.| makes the value identical
    assert orc.whip_loss(orc.rotate(-X, Rh)) == pytest.approx(d * math.exp(-a / math.sqrt(d)), rel=1e-14)


def test_whip_hand_computed_2x2():
    O = np.array([[1.0, -2.0], [0.5, 0.0]])
    per_tok = [math.exp(-1) + math.exp(-2), math.exp(-0.5) + 1.0]
    assert np.allclose(orc.whip_per_token(O), per_tok, rtol=1e-15)
    assert orc.whip_loss(O) == pytest.approx(sum(per_tok) / 2, rel=1e-15)
    G = orc.whip_grad_wrt_output(O)
    expect = np.array([[-math.exp(-1), math.exp(-2)], [-math.exp(-0.5), 0.0]]) / 2
    assert np.allclose(G, expect, rtol=1e-15, atol=0)


def test_whip_token_permutation_and_column_symmetries():
    X = RNG.standard_normal((40, 12))
    R, _ = orc.qr_pos(RNG.standard_normal((12, 12)))
    L = orc.whip_loss(orc.rotate(X, R))
    perm = RNG.permutation(40)
    assert orc.whip_loss(orc.rotate(X[perm], R)) == pytest.approx(L, rel=1e-13)
    signs = RNG.integers(0, 2, 12) * 2.0 - 1.0
    assert orc.whip_loss(orc.rotate(X, R * signs[None, :])) == pytest.approx(L, rel=1e-13)
    cperm = RNG.permutation(12)
    assert orc.whip_loss(orc.rotate(X, R[:, cperm])) == pytest.approx(L, rel=1e-13)


@pytest.mark.parametrize("d", [3, 8, 16])
@pytest.mark.parametrize("reduction", ["mean", "sum"])
def test_whip_gradient_central_differences(d, reduction):
    O = RNG.standard_normal((5, d)) * 2.0
    G = orc.whip_grad_wrt_output(O, reduction)
    h = 1e-5
    for t in range(5):
        for j in range(d):
            Op, Om = O.copy(), O.copy()
            Op[t, j] += h
            Om[t, j] -= h
            fd = (orc.whip_loss(Op, reduction) - orc.whip_loss(Om, reduction)) / (2 * h)
            assert fd == pytest.approx(G[t, j], rel=1e-7, abs=2e-9)


def test_gradient_wrt_rotation_central_differences():
    d, n = 6, 9
    X = RNG.standard_normal((n, d))
    R = RNG.standard_normal((d, d))          # the chain rule holds for any matrix
    G = orc.whip_grad_wrt_output(orc.rotate(X, R))
    Gq = orc.grad_wrt_rotation(X, G)
    h = 1e-6
    for i in range(d):
        for j in range(d):
            Rp, Rm = R.copy(), R.copy()
            Rp[i, j] += h
            Rm[i, j] -= h
            fd = (orc.whip_loss(orc.rotate(X, Rp)) - orc.whip_loss(orc.rotate(X, Rm))) / (2 * h)
            assert fd == pytest.approx(Gq[i, j], rel=1e-6, abs=1e-10)


def test_sign_override_only_changes_the_overridden_entries():
    O = np.array([[1e-9, -2.0, 0.5], [-1e-9, 3.0, 0.0]])
    G0 = orc.whip_grad_wrt_output(O)
    S = np.sign(O)
    S[0, 0] = -1.0                      # the other implementation saw a tiny negative value
    G1 = orc.whip_grad_wrt_output(O, sign_of_O=S)
    assert G1[0, 0] == -G0[0, 0] and abs(G1[0, 0]) == pytest.approx(0.5, rel=1e-8)
    mask = np.ones_like(O, bool)
    mask[0, 0] = False
    assert np.array_equal(G0[mask], G1[mask])


# ------------------------------------------------------------- QR (Algorithm 2)
@pytest.mark.parametrize("n", [1, 2, 5, 33, 128])
def test_qr_factorisation_properties(n):
    Z = RNG.standard_normal((n, n))
    R, U = orc.qr_pos(Z)
    assert np.abs(R.T @ R - np.eye(n)).max() <= 1e-12
    assert np.abs(R @ U - Z).max() <= 1e-12
    assert np.abs(np.tril(U, -1)).max() == 0.0
    assert (np.diag(U) > 0).all()


@pytest.mark.parametrize("n", [4, 17, 64, 200])
def test_qr_matches_lapack_after_gauge_fix(n):
    Z = RNG.standard_normal((n, n))
    R, U = orc.qr_pos(Z)
    Rl, Ul = orc.qr_pos_lapack(Z)
    assert np.abs(R - Rl).max() <= 1e-12
    assert np.abs(U - Ul).max() <= 1e-11


def test_qr_raw_alg2_sign_rule():
    # v = x + sign(x1)||x|| e1 maps x to -sign(x1)||x|| e1: the raw diagonal of U
    # has the opposite sign of the leading entry of each reduced column, and the
    # last diagonal entry is not reflected.
    Z = RNG.standard_normal((7, 7))
    Q, U = orc.householder_qr_alg2(Z)
    assert np.abs(Q @ U - Z).max() <= 1e-13
    assert np.abs(Q.T @ Q - np.eye(7)).max() <= 1e-13
    assert np.sign(U[0, 0]) == -np.sign(Z[0, 0])
    assert abs(U[0, 0]) == pytest.approx(np.linalg.norm(Z[:, 0]), rel=1e-14)
    # 2 x 2 by hand: x = (3, 4) -> ||x|| = 5, U00 = -5, first column of Q = -(3,4)/5
    Q2, U2 = orc.householder_qr_alg2(np.array([[3.0, 1.0], [4.0, 2.0]]))
    assert U2[0, 0] == pytest.approx(-5.0, rel=1e-15)
    assert np.allclose(Q2[:, 0], [-0.6, -0.8], rtol=1e-14)
    assert U2[0, 1] == pytest.approx(-(3 * 1 + 4 * 2) / 5.0, rel=1e-14)


def test_qr_of_orthogonal_matrix_is_itself():
    H = hadamard(32) / math.sqrt(32)
    signs = RNG.integers(0, 2, 32) * 2.0 - 1.0
    Z = H * signs[None, :]
    R, U = orc.qr_pos(Z)
    assert np.abs(R - Z).max() <= 1e-13
    assert np.abs(U - np.eye(32)).max() <= 1e-13


def test_qr_right_multiplication_by_upper_triangular_keeps_R():
    Z = RNG.standard_normal((10, 10))
    T = np.triu(RNG.standard_normal((10, 10)))
    T[np.diag_indices(10)] = np.abs(np.diag(T)) + 0.5
    R1, _ = orc.qr_pos(Z)
    R2, _ = orc.qr_pos(Z @ T)
    assert np.abs(R1 - R2).max() <= 1e-11


# ---------------------------------------------------------------- QR backward
def _fd_jacobian_R(Z, h=1e-6):
    n = Z.shape[0]
    J = np.zeros((n, n, n, n))
    for k in range(n):
        for l in range(n):
            Zp, Zm = Z.copy(), Z.copy()
            Zp[k, l] += h
            Zm[k, l] -= h
            J[:, :, k, l] = (orc.qr_pos_lapack(Zp)[0] - orc.qr_pos_lapack(Zm)[0]) / (2 * h)
    return J


def test_qr_backward_against_bruteforce_jacobian_d4():
    for trial in range(3):
        Z = RNG.standard_normal((4, 4)) + 2.0 * np.eye(4)
        R, U = orc.qr_pos(Z)
        Gq = RNG.standard_normal((4, 4))
        J = _fd_jacobian_R(Z)
        Gz_fd = np.einsum("ij,ijkl->kl", Gq, J)
        Gz = orc.qr_backward(R, U, Gq)
        assert np.abs(Gz - Gz_fd).max() <= 1e-7


@pytest.mark.parametrize("d", [3, 8, 16])
def test_composed_loss_gradient_central_differences(d):
    n = 3 * d
    X = RNG.standard_normal((n, d)) * 1.5
    Z = RNG.standard_normal((d, d)) + 3.0 * np.eye(d)
    out = orc.calib_step(X, Z, lr=0.0)

    def L(Zm):
        return orc.whip_loss(orc.rotate(X, orc.qr_pos_lapack(Zm)[0]))

    h = 1e-6
    Gz_fd = np.zeros_like(Z)
    for k in range(d):
        for l in range(d):
            Zp, Zm = Z.copy(), Z.copy()
            Zp[k, l] += h
            Zm[k, l] -= h
            Gz_fd[k, l] = (L(Zp) - L(Zm)) / (2 * h)
    assert np.abs(out["Gz"] - Gz_fd).max() <= 5e-8 * max(1.0, np.abs(Gz_fd).max())


def test_qr_backward_invariants():
    d = 12
    Z = RNG.standard_normal((d, d)) + 2.0 * np.eye(d)
    R, U = orc.qr_pos(Z)
    Gq = RNG.standard_normal((d, d))
    Gz = orc.qr_backward(R, U, Gq)
    # R does not change when Z is multiplied on the right by an upper-triangular
    # matrix, so dL/dZ has no component along Z T: triu(Z^T Gz) = 0.
    assert np.abs(np.triu(Z.T @ Gz)).max() <= 1e-12
    # gauge: flipping column signs of R (and rows of U, and columns of Gq) leaves Gz
    s = RNG.integers(0, 2, d) * 2.0 - 1.0
    Gz2 = orc.qr_backward(R * s[None, :], U * s[:, None], Gq * s[None, :])
    assert np.abs(Gz - Gz2).max() <= 1e-12
    # the raw Algorithm-2 gauge gives the same latent gradient for the Whip loss
    X = RNG.standard_normal((30, d))
    a = orc.calib_step(X, Z, 0.1, qr=orc.qr_pos)
    b = orc.calib_step(X, Z, 0.1, qr=orc.householder_qr_alg2)
    assert a["loss"] == pytest.approx(b["loss"], rel=1e-13)
    assert np.abs(a["Gz"] - b["Gz"]).max() <= 1e-12
    assert np.abs(a["Z_new"] - b["Z_new"]).max() <= 1e-12


# ------------------------------------------------------------ optimiser / step
def test_sgd_step_definition():
    Z = RNG.standard_normal((5, 5))
    Gz = RNG.standard_normal((5, 5))
    Zn = orc.sgd_step(Z, Gz, 0.25)
    assert np.array_equal(Zn, Z - 0.25 * Gz)
    assert np.array_equal(orc.sgd_step(Z, Gz, 0.0), Z)


def test_rotation_preserves_token_norms():
    w = gen.scaled(gen.WORKLOADS["c1_tiny"], d=32, n_tokens=64)
    X = gen.gen_activations(w)[0].astype(np.float64)
    Z0 = gen.gen_latent_init(w)[0].astype(np.float64)
    out = orc.calib_step(X, Z0, w.lr)
    assert np.allclose(np.linalg.norm(out["O"], axis=1), np.linalg.norm(X, axis=1), rtol=1e-12)


def test_small_run_decreases_loss_and_is_deterministic():
    w = gen.scaled(gen.WORKLOADS["c1_tiny"], d=32, n_tokens=256, n_outlier_channels=2)
    X = gen.gen_activations(w)[0]
    Z0 = gen.gen_latent_init(w)[0]
    l1, Z1, R1 = orc.calib_run(X, Z0, w.lr, 10)
    l2, Z2, R2 = orc.calib_run(X, Z0, w.lr, 10)
    assert np.array_equal(l1, l2) and np.array_equal(Z1, Z2) and np.array_equal(R1, R2)
    assert (np.diff(l1) < 0).all()
    assert np.abs(R1.T @ R1 - np.eye(32)).max() <= 1e-12
    # loss reported for step k is L(Z_k) before the update
    assert l1[0] == pytest.approx(orc.whip_loss(orc.rotate(X, orc.qr_pos(Z0)[0])), rel=1e-14)


def test_c1_trajectory_matches_stored_fixture():
    """The stored trajectory was written by tests/golden/write_c1_trajectory.py,
    which calls only the oracle; this guards the oracle against silent edits."""
    import json, os
    path = os.path.join(os.path.dirname(__file__), "golden", "c1_tiny_trajectory.json")
    ref = json.load(open(path))
    w = gen.WORKLOADS["c1_tiny"]
    X = gen.gen_activations(w)[0]
    Z0 = gen.gen_latent_init(w)[0]
    losses, Z, R = orc.calib_run(X, Z0, w.lr, 3, qr=orc.qr_pos)
    assert np.allclose(losses, ref["losses"][:3], rtol=1e-12)


# --------------------------------------------------------------------- optimisers on the latent
def test_momentum_zero_is_plain_sgd_and_constant_gradient_gives_geometric_series():
    rng = np.random.default_rng(1)
    Z, g = rng.standard_normal((5, 5)), rng.standard_normal((5, 5))
    Z1, v1 = orc.momentum_step(Z, g, np.zeros_like(Z), 0.1, 0.0)
    assert np.array_equal(Z1, orc.sgd_step(Z, g, 0.1)) and np.array_equal(v1, g)
    mu, lr, Zk, v = 0.9, 0.05, Z.copy(), np.zeros_like(Z)
    for k in range(1, 8):
        Zk, v = orc.momentum_step(Zk, g, v, lr, mu)
        assert np.allclose(v, g * (1 - mu ** k) / (1 - mu), rtol=1e-13)          # closed form of the velocity
    total = sum((1 - mu ** k) / (1 - mu) for k in range(1, 8))
    assert np.allclose(Zk, Z - lr * total * g, rtol=1e-12, atol=1e-14)


def test_adam_first_step_is_lr_times_sign_and_is_scale_free():
    rng = np.random.default_rng(2)
    Z, g = rng.standard_normal((6, 6)), rng.standard_normal((6, 6))
    zeros = np.zeros_like(Z)
    Z1, m1, v1 = orc.adam_step(Z, g, zeros, zeros, 1, 1e-2, eps=0.0)
    assert np.allclose(Z1, Z - 1e-2 * np.sign(g), rtol=0, atol=1e-15)            # mhat / sqrt(vhat) = g / |g|
    assert np.allclose(m1, 0.1 * g) and np.allclose(v1, 1e-3 * g * g)
    Za, _, _ = orc.adam_step(Z, 1000.0 * g, zeros, zeros, 1, 1e-2, eps=0.0)
    assert np.allclose(Za, Z1, atol=1e-14)                                       # invariant to gradient scale
    # a constant gradient keeps every step at exactly lr: bias correction cancels the warm-up
    Zk, m, v = Z.copy(), zeros, zeros
    for t in range(1, 6):
        Zn, m, v = orc.adam_step(Zk, g, m, v, t, 1e-2, eps=0.0)
        assert np.allclose(Zn - Zk, -1e-2 * np.sign(g), atol=1e-14)
        Zk = Zn


def test_adam_epsilon_bounds_the_step_for_tiny_gradients():
    Z, g = np.zeros((2, 2)), np.full((2, 2), 1e-12)
    Z1, _, _ = orc.adam_step(Z, g, np.zeros_like(Z), np.zeros_like(Z), 1, 1.0, eps=1e-8)
    assert np.allclose(Z1, -1e-12 / (1e-12 + 1e-8))                              # |step| = lr g / (|g| + eps)


# --------------------------------------------------------------------- evaluation metrics (Eq. 1, quantisation error)
def test_outlier_count_matches_brute_force_and_is_rotation_sensitive():
    rng = np.random.default_rng(4)
    O = rng.standard_normal((7, 9)) * 3
    brute = sum(1 for t in range(7) for j in range(9) if abs(O[t, j]) > 2.5)
    assert orc.outlier_count(O, 2.5) == brute
    # one massive channel: d outliers-free values after a Hadamard rotation spreads it (norm invariance)
    d = 16
    x = np.zeros((1, d)); x[0, 3] = 8.0
    H = np.array([[(-1) ** bin(i & j).count("1") for j in range(d)] for i in range(d)]) / np.sqrt(d)
    assert orc.outlier_count(x, 4.0) == 1 and orc.outlier_count(x @ H, 4.0) == 0


def test_asymmetric_quantiser_closed_forms():
    # values already on the grid of the row are reproduced exactly
    row = np.array([[-1.0, -0.5, 0.0, 0.5, 1.0, 6.5]])            # range 7.5, 4 bits: step 0.5
    assert np.allclose(orc.quantize_per_token_asymmetric(row, 4), row, atol=1e-12)
    assert orc.quantization_mse(row, 4) < 1e-24
    # the error of any entry is at most half a step (plus the shift of the rounded zero point)
    rng = np.random.default_rng(5)
    O = rng.standard_normal((50, 33)) * rng.uniform(0.1, 20, size=(50, 1))
    for bits in (2, 4, 8):
        Q = orc.quantize_per_token_asymmetric(O, bits)
        step = (O.max(1) - O.min(1)) / (2 ** bits - 1)
        assert (np.abs(Q - O).max(axis=1) <= step * (1.0 + 1e-9)).all()
        assert len(np.unique(np.round(Q[0] / step[0], 6))) <= 2 ** bits
    # uniform data on [0, 1): mean squared error of a uniform quantiser is step^2 / 12
    U = rng.uniform(0, 1, size=(20, 20000))
    mse = orc.quantization_mse(U, 4)
    assert abs(mse - (1.0 / 15) ** 2 / 12) < 0.05 * (1.0 / 15) ** 2 / 12
    # constant rows carry no error; per-token scaling makes the relative error scale-free
    assert orc.quantization_mse(np.full((3, 5), 2.5), 4) == 0.0
    assert np.isclose(orc.quantization_mse(O * 8.0, 4), 64.0 * orc.quantization_mse(O, 4), rtol=1e-12)
