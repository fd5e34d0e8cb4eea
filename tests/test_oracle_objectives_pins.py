"""Pins of the alternative-objective oracle (variance, kurtosis, quantisation loss; the ablation of
Sec. 5.3) against closed forms, a library routine, invariances and finite differences."""
import numpy as np
import pytest
import scipy.stats

import oracle as orc
from oracle import objectives as obj

RNG = np.random.default_rng(777)


@pytest.mark.parametrize("d", [2, 5, 16, 101])
def test_variance_and_kurtosis_of_an_arithmetic_progression(d):
    # values a + h * (0 .. d-1): variance h^2 (d^2 - 1) / 12, excess kurtosis -(6/5)(d^2 + 1)/(d^2 - 1)
    a, h = 3.5, 0.7
    O = (a + h * np.arange(d))[None, :]
    assert obj.per_token(O, "variance")[0] == pytest.approx(h * h * (d * d - 1) / 12.0, rel=1e-12)
    assert obj.per_token(O, "kurtosis")[0] == pytest.approx(-1.2 * (d * d + 1) / (d * d - 1), rel=1e-11)


def test_two_point_row_has_kurtosis_minus_two_and_variance_a_squared():
    O = np.array([[2.5, -2.5, 2.5, -2.5, -2.5, 2.5]])
    assert obj.per_token(O, "variance")[0] == pytest.approx(6.25, rel=1e-14)
    assert obj.per_token(O, "kurtosis")[0] == pytest.approx(-2.0, abs=1e-13)


def test_kurtosis_matches_library_routine_and_is_near_zero_for_gaussian_rows():
    O = RNG.standard_normal((7, 4001))
    k = obj.per_token(O, "kurtosis")
    assert np.allclose(k, scipy.stats.kurtosis(O, axis=1, fisher=True, bias=True), rtol=1e-12, atol=1e-12)
    assert np.abs(k).max() < 0.3
    heavy = RNG.laplace(size=(3, 20001))
    assert np.all(np.abs(obj.per_token(heavy, "kurtosis") - 3.0) < 0.5)       # Laplace: excess kurtosis 3


@pytest.mark.parametrize("name", ["variance", "kurtosis"])
def test_shift_and_scale_behaviour(name):
    O = RNG.laplace(size=(5, 33))
    base = obj.per_token(O, name)
    assert np.allclose(obj.per_token(O + 4.2, name), base, rtol=1e-11)         # shift invariant
    factor = 9.0 if name == "variance" else 1.0                                  # degree 2 / degree 0
    assert np.allclose(obj.per_token(3.0 * O, name), factor * base, rtol=1e-11)
    G = obj.grad_wrt_output(O, name, "sum")
    assert np.abs(G.sum(axis=1)).max() < 1e-12                                   # shift invariance
    euler = (G * O).sum(axis=1)                                                  # Euler: degree * value
    assert np.allclose(euler, (2.0 if name == "variance" else 0.0) * base, atol=1e-11)


@pytest.mark.parametrize("name", ["variance", "kurtosis"])
@pytest.mark.parametrize("reduction", ["mean", "sum"])
def test_gradient_by_central_differences(name, reduction):
    O = RNG.laplace(size=(4, 9))
    G = obj.grad_wrt_output(O, name, reduction)
    h = 1e-6
    for t in range(O.shape[0]):
        for j in range(O.shape[1]):
            P, M = O.copy(), O.copy()
            P[t, j] += h
            M[t, j] -= h
            fd = (obj.loss(P, name, reduction) - obj.loss(M, name, reduction)) / (2 * h)
            assert G[t, j] == pytest.approx(fd, rel=2e-6, abs=1e-9)


def test_variance_is_rotation_invariant_up_to_the_mean_term():
    # |o|^2 is preserved by a rotation, so d * variance = |x|^2 - d * mean(o)^2: the remark of Sec. 4.1
    # that variance is a poor objective under norm invariance
    d = 12
    x = RNG.laplace(size=(6, d))
    Q, _ = np.linalg.qr(RNG.standard_normal((d, d)))
    O = x @ Q
    lhs = d * obj.per_token(O, "variance")
    assert np.allclose(lhs, (x ** 2).sum(axis=1) - d * O.mean(axis=1) ** 2, rtol=1e-12)


def test_quant_loss_equals_the_evaluation_metric_and_is_zero_on_grid_rows():
    O = RNG.laplace(size=(8, 40))
    assert obj.loss(O, "quant", "mean", 4) == pytest.approx(orc.quantization_mse(O, 4), rel=1e-14)
    grid = np.arange(16.0)[None, :] * 0.25 - 1.0         # 16 levels of a 4-bit grid: reproduced exactly
    assert obj.loss(grid, "quant", "mean", 4) == pytest.approx(0.0, abs=1e-28)
    assert np.abs(obj.grad_wrt_output(grid, "quant", "sum", 4)).max() < 1e-13


def test_quant_gradient_by_finite_differences_on_interior_entries():
    # moving an entry that is neither the row's min nor its max, by less than its distance to a rounding
    # boundary, leaves the grid and every code unchanged: the loss is then exactly quadratic in it
    bits = 4
    O = RNG.laplace(size=(5, 24))
    G = obj.grad_wrt_output(O, "quant", "mean", bits)
    lo, hi = O.min(axis=1, keepdims=True), O.max(axis=1, keepdims=True)
    scale = (hi - lo) / 15.0
    frac = np.abs(O / scale - np.rint(O / scale))
    h = 1e-7
    checked = 0
    for t in range(O.shape[0]):
        for j in range(O.shape[1]):
            if O[t, j] in (lo[t, 0], hi[t, 0]) or frac[t, j] > 0.49:
                continue
            P, M = O.copy(), O.copy()
            P[t, j] += h
            M[t, j] -= h
            fd = (obj.loss(P, "quant", "mean", bits) - obj.loss(M, "quant", "mean", bits)) / (2 * h)
            assert G[t, j] == pytest.approx(fd, rel=1e-5, abs=1e-10)
            checked += 1
    assert checked > 80
    # residuals never exceed half a step
    assert (np.abs(G) * O.shape[0] * O.shape[1] / 2.0 <= 0.5 * scale + 1e-12).all()


@pytest.mark.parametrize("name", ["variance", "kurtosis"])
def test_objective_step_gradient_through_rotation_and_qr(name):
    # FD of the composed loss with respect to the latent, as for the Whip loss
    d, n = 5, 11
    X = RNG.laplace(size=(n, d))
    Z = np.eye(d) + 0.1 * RNG.standard_normal((d, d))
    out = obj.objective_step(X, Z, 0.1, name)
    h = 1e-6
    for (i, j) in [(0, 0), (1, 3), (4, 2), (3, 3)]:
        P, M = Z.copy(), Z.copy()
        P[i, j] += h
        M[i, j] -= h
        fd = (obj.objective_step(X, P, 0.1, name)["loss"] - obj.objective_step(X, M, 0.1, name)["loss"]) / (2 * h)
        assert out["Gz"][i, j] == pytest.approx(fd, rel=1e-5, abs=1e-9)
    assert np.allclose(out["Z_new"], Z - 0.1 * out["Gz"])


def test_quant_grid_reproduces_the_quantiser_and_a_decider_changes_only_what_it_decides():
    O = RNG.laplace(size=(6, 30))
    O[2, :] = 1.25                                               # constant row
    scale, zero, codes = obj.quant_grid(O, 4)
    deq = np.where(scale == 0.0, O, scale * (codes - zero))
    assert np.array_equal(deq, orc.quantize_per_token_asymmetric(O, 4))
    same = obj.grad_wrt_output(O, "quant", "sum", 4, code_decider=lambda O_, s_, z_, c_: c_)
    assert np.array_equal(same, obj.grad_wrt_output(O, "quant", "sum", 4))
    # bumping one code by one moves that entry's derivative by exactly -(2/d) scale
    def bump(O_, s_, z_, c_):
        c = c_.copy()
        c[0, 3] += 1.0
        return c
    moved = obj.grad_wrt_output(O, "quant", "sum", 4, code_decider=bump) - same
    assert moved[0, 3] == pytest.approx(-2.0 / 30 * scale[0, 0], rel=1e-12)
    moved[0, 3] = 0.0
    assert np.abs(moved).max() == 0.0
