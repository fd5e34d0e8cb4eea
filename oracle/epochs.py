"""Plain oracle of Algorithm 1's loop around the step: seeded token sampling and mini-batch epochs.

TEST INFRASTRUCTURE: never imported by the product path.

Readings (the paper gives a sampling ratio, a batch size and an epoch count in its hyper-parameter
appendix but not how tokens are drawn or batched):
  * epoch e uses the seeded permutation of oracle/token_sampling.py with seed + e and keeps its
    first floor(ratio * n_pool) rows (uniform sampling without replacement), the product taken in
    double precision on the float32 value of the ratio (the interface passes a float);
  * an optimiser step consumes accum * n_tokens consecutive sampled rows and takes one step of
    Algorithm 1's body on all of them together (gradient accumulation over accum micro-batches of
    n_tokens rows is, by linearity, the same as one batch of accum * n_tokens rows);
  * an incomplete last step of an epoch is dropped.
"""
from __future__ import annotations

import numpy as np

from . import calib_oracle as co
from .token_sampling import gather_tokens


def steps_per_epoch(n_pool: int, n_tokens: int, sample_ratio: float, accum: int) -> int:
    n_sampled = int(np.floor(np.float64(np.float32(sample_ratio)) * np.float64(n_pool)))
    return n_sampled // (n_tokens * accum)


def epoch_batches(pool: np.ndarray, n_tokens: int, sample_ratio: float, accum: int, seed: int):
    """The token batches (accum * n_tokens rows each) of one epoch, in order."""
    k = steps_per_epoch(pool.shape[0], n_tokens, sample_ratio, accum)
    m = n_tokens * accum
    return [gather_tokens(pool, seed, s * m, m) for s in range(k)]


def calib_run_epochs(pool: np.ndarray, Z0: np.ndarray, lr: float, n_tokens: int, sample_ratio: float,
                     accum: int, n_epochs: int, seed: int, reduction: str = "mean", qr=co.qr_pos):
    """Returns (losses[n_epochs * steps_per_epoch], Z_final, R_final)."""
    Z = np.asarray(Z0, dtype=co.F64).copy()
    losses = []
    for e in range(n_epochs):
        for Xb in epoch_batches(pool, n_tokens, sample_ratio, accum, seed + e):
            out = co.calib_step(co.widen_input(Xb), Z, lr, reduction, qr)
            losses.append(out["loss"])
            Z = out["Z_new"]
    R, _ = qr(Z)
    return np.asarray(losses, dtype=co.F64), Z, R
