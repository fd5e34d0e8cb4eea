"""Plain float64 oracle of the three alternative calibration objectives of the ablation in
Sec. 5.3 ("Optimization objectives": quantisation loss, variance, kurtosis, against the Whip loss).

TEST INFRASTRUCTURE: never imported by the product path.

The paper names the objectives but prints no formula for them.  Readings (also listed in the design
notes of the repository), chosen to mirror Eq. 4, which is a per-token function of the rotated
activation vector o = x R in R^d, averaged over tokens:
  * variance:  v(o) = (1/d) sum_j (o_j - mu)^2,  mu = (1/d) sum_j o_j   (population variance over
    the channels of a token);
  * kurtosis:  k(o) = m4 / m2^2 - 3 with m_p = (1/d) sum_j (o_j - mu)^p  (excess kurtosis: the
    paper's appendix on activation statistics says a Gaussian has kurtosis 0);
  * quantisation loss:  e(o) = (1/d) sum_j (o_j - Q(o)_j)^2 with Q the per-token asymmetric uniform
    quantiser of oracle/eval_metrics.py; its derivative is taken with the grid (scale, zero point)
    held fixed and rounding piecewise constant: de/do_j = (2/d) (o_j - Q(o)_j)  (the derivative
    almost everywhere of the error on a fixed grid).
Each loss is the mean over tokens ("sum" keeps the plain sum), as for the Whip loss.

Pins (tests/test_oracle_objectives_pins.py): closed forms on arithmetic progressions and two-point
rows, a library routine for the kurtosis, shift / scale invariances and their consequences for the
gradients, finite differences.
"""
from __future__ import annotations

import numpy as np

from . import calib_oracle as co
from .eval_metrics import quantize_per_token_asymmetric

F64 = np.float64
OBJECTIVES = ("variance", "kurtosis", "quant")


def _central(O):
    O = np.asarray(O, dtype=F64)
    return O - O.mean(axis=1, keepdims=True)


def per_token(O: np.ndarray, objective: str, bits: int = 4) -> np.ndarray:
    """The objective of each token row of O."""
    O = np.asarray(O, dtype=F64)
    if objective == "variance":
        return (_central(O) ** 2).mean(axis=1)
    if objective == "kurtosis":
        C = _central(O)
        m2 = (C ** 2).mean(axis=1)
        m4 = (C ** 4).mean(axis=1)
        return m4 / m2 ** 2 - 3.0
    if objective == "quant":
        return ((O - quantize_per_token_asymmetric(O, bits)) ** 2).mean(axis=1)
    raise ValueError(objective)


def loss(O: np.ndarray, objective: str, reduction: str = "mean", bits: int = 4) -> float:
    pt = per_token(O, objective, bits)
    if reduction == "mean":
        return float(pt.sum() / pt.shape[0])
    if reduction == "sum":
        return float(pt.sum())
    raise ValueError(reduction)


def quant_grid(O: np.ndarray, bits: int):
    """Per-token grid of the asymmetric uniform quantiser: (scale, zero, codes), scale = 0 on a
    constant row (which is reproduced exactly)."""
    O = np.asarray(O, dtype=F64)
    maxq = float(2 ** bits - 1)
    lo = O.min(axis=1, keepdims=True)
    hi = O.max(axis=1, keepdims=True)
    scale = (hi - lo) / maxq
    safe = np.where(scale == 0.0, 1.0, scale)
    zero = np.rint(-lo / safe)
    codes = np.clip(np.rint(O / safe) + zero, 0.0, maxq)
    return scale, zero, codes


def grad_wrt_output(O: np.ndarray, objective: str, reduction: str = "mean", bits: int = 4,
                    code_decider=None) -> np.ndarray:
    """G = dL/dO (N x d).

    The quantiser's code rint(o / scale) + zero is a discrete decision taken on a floating-point
    value: an implementation in lower precision may legitimately take the neighbouring code for an
    entry that sits on a rounding boundary.  code_decider(O, scale, zero, codes) -> codes lets a test
    take that decision in the precision of the implementation under test (as sign_decider does for
    the kink of Eq. 4); the derivative formula itself is unchanged."""
    O = np.asarray(O, dtype=F64)
    n, d = O.shape
    if objective == "variance":
        # d/do_j (1/d) sum_i c_i^2 with c_i = o_i - mu:  (2/d) c_j   (sum_i c_i = 0)
        G = 2.0 * _central(O) / d
    elif objective == "kurtosis":
        C = _central(O)
        m2 = (C ** 2).mean(axis=1, keepdims=True)
        m3 = (C ** 3).mean(axis=1, keepdims=True)
        m4 = (C ** 4).mean(axis=1, keepdims=True)
        # dm4/do_j = (4/d)(c_j^3 - m3), dm2/do_j = (2/d) c_j
        G = (4.0 / d) * ((C ** 3 - m3) / m2 ** 2 - m4 * C / m2 ** 3)
    elif objective == "quant":
        if code_decider is None:
            G = 2.0 * (O - quantize_per_token_asymmetric(O, bits)) / d
        else:
            scale, zero, codes = quant_grid(O, bits)
            codes = code_decider(O, scale, zero, codes)
            G = np.where(scale == 0.0, 0.0, 2.0 * (O - scale * (codes - zero)) / d)
    else:
        raise ValueError(objective)
    return G / n if reduction == "mean" else G


def objective_step(X: np.ndarray, Z: np.ndarray, lr: float, objective: str, reduction: str = "mean",
                   bits: int = 4, qr=co.qr_pos, code_decider=None):
    """One pass of the loop body of Algorithm 1 with the Whip loss replaced by `objective`."""
    R, U = qr(Z)
    O = co.rotate(X, R)
    L = loss(O, objective, reduction, bits)
    G = grad_wrt_output(O, objective, reduction, bits, code_decider)
    Gq = co.grad_wrt_rotation(X, G)
    Gz = co.qr_backward(R, U, Gq)
    return {"R": R, "U": U, "O": O, "loss": L, "G": G, "Gq": Gq, "Gz": Gz, "Z_new": co.sgd_step(Z, Gz, lr)}
