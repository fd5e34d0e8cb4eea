"""Plain oracle of the two quantities the paper uses to judge a rotation (Sec. 4.1, Eq. 1; the
appendix on outliers and quantisation errors): the number of outliers of the rotated activations
and their activation-quantisation error.

TEST INFRASTRUCTURE: never imported by the product path.

Readings (the paper gives neither tau nor the quantiser's formula beyond "per-token asymmetric"):
  * outliers: Eq. 1 summed over tokens, count of |o_tj| > tau, tau supplied by the caller;
  * quantisation: for each token row, scale = (max - min) / (2^bits - 1), zero = round(-min / scale),
    q = clip(round(o / scale) + zero, 0, 2^bits - 1), dequantised value scale * (q - zero)
    (round half to even); a constant row is reproduced exactly; the error is the mean squared
    difference over all entries.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


def outlier_count(O: np.ndarray, tau: float) -> int:
    """Eq. 1, summed over the token rows of O."""
    return int((np.abs(np.asarray(O, dtype=F64)) > tau).sum())


def quantize_per_token_asymmetric(O: np.ndarray, bits: int) -> np.ndarray:
    """Fake-quantised copy of O: per-token (row) asymmetric uniform quantisation to `bits` bits."""
    O = np.asarray(O, dtype=F64)
    maxq = float(2 ** bits - 1)
    lo = O.min(axis=1, keepdims=True)
    hi = O.max(axis=1, keepdims=True)
    scale = (hi - lo) / maxq
    flat = scale == 0.0
    scale = np.where(flat, 1.0, scale)
    zero = np.rint(-lo / scale)
    q = np.clip(np.rint(O / scale) + zero, 0.0, maxq)
    deq = scale * (q - zero)
    return np.where(flat, O, deq)


def quantization_mse(O: np.ndarray, bits: int) -> float:
    O = np.asarray(O, dtype=F64)
    return float(np.mean((quantize_per_token_asymmetric(O, bits) - O) ** 2))
