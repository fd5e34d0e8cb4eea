"""Pins of the epoch / mini-batch oracle: what it must do follows from the sampler's pinned
permutation and from invariances of the step, not from its own code."""
import numpy as np
import pytest

import oracle as orc
from oracle import epochs as ep

RNG = np.random.default_rng(99)


def test_one_full_batch_per_epoch_equals_the_plain_loop():
    # ratio 1, one step per epoch of all tokens: every epoch sees a permutation of the pool, and the step is
    # invariant to the order of tokens, so the run equals Algorithm 1's plain loop on the pool
    d, n = 6, 37
    pool = RNG.laplace(size=(n, d))
    Z0 = np.eye(d) + 0.05 * RNG.standard_normal((d, d))
    losses, Z, R = ep.calib_run_epochs(pool, Z0, 0.05, n, 1.0, 1, 4, seed=7)
    ref_losses, Z_ref, R_ref = orc.calib_run(pool, Z0, 0.05, 4)
    assert np.allclose(losses, ref_losses, rtol=1e-12)
    assert np.allclose(Z, Z_ref, atol=1e-12) and np.allclose(R, R_ref, atol=1e-12)


@pytest.mark.parametrize("n_pool,n_tokens,ratio,accum,expect", [(1000, 100, 0.5, 2, 2), (1000, 100, 0.1, 1, 1),
                                                                (2048, 256, 0.5, 2, 2), (999, 10, 0.1, 3, 3),
                                                                (50, 100, 1.0, 1, 0)])
def test_steps_per_epoch(n_pool, n_tokens, ratio, accum, expect):
    assert ep.steps_per_epoch(n_pool, n_tokens, ratio, accum) == expect


def test_batches_of_an_epoch_are_disjoint_rows_of_the_pool_and_differ_between_epochs():
    n, d = 300, 3
    pool = np.arange(n * d, dtype=np.float64).reshape(n, d)       # row i starts with 3 i: rows identify themselves
    b0 = ep.epoch_batches(pool, 20, 0.5, 2, seed=11)
    assert len(b0) == 3 and all(b.shape == (40, d) for b in b0)
    rows = np.concatenate(b0)[:, 0] / d
    assert len(set(rows.tolist())) == 120                         # no row twice within an epoch
    first150 = orc.gather_tokens(pool, 11, 0, 150)[:, 0] / d      # the sampled set is the head of the permutation
    assert set(rows.tolist()) <= set(first150.tolist())
    b1 = ep.epoch_batches(pool, 20, 0.5, 2, seed=12)
    assert not np.array_equal(np.concatenate(b1), np.concatenate(b0))


def test_accumulation_is_a_mean_over_micro_batches():
    # the gradient of the mean loss over a batch is the mean of the micro-batch gradients (linearity):
    # checked from the stage functions, independently of the epoch driver
    d, m = 5, 12
    X = RNG.laplace(size=(2 * m, d))
    Z = np.eye(d) + 0.05 * RNG.standard_normal((d, d))
    big = orc.calib_step(X, Z, 0.1)
    a, b = orc.calib_step(X[:m], Z, 0.1), orc.calib_step(X[m:], Z, 0.1)
    assert np.allclose(big["Gz"], 0.5 * (a["Gz"] + b["Gz"]), atol=1e-13)
    assert big["loss"] == pytest.approx(0.5 * (a["loss"] + b["loss"]), rel=1e-13)
