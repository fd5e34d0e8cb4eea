"""Momentum SGD and Adam on the latent (Sec. 4.3: QR-Orth works with any standard optimiser; the
paper reports SGD and Adam) against the float64 oracle, free-running for a few steps on the fp32
path, and eager-vs-graph consistency on the tensor-core path."""
import numpy as np
import pytest
import torch

import oracle as orc
import paper_2511_04063_b200 as dq
from paper_2511_04063_b200 import inputs as gen
from gpu_util import Calib, x_f64

pytestmark = pytest.mark.gpu

STEPS = 3


def _oracle_run(X, Z0, lr, kind, b1, b2, eps):
    Z = Z0.astype(np.float64)
    m, v = np.zeros_like(Z), np.zeros_like(Z)
    grads = []
    for t in range(1, STEPS + 1):
        g = orc.calib_step(X, Z, lr)["Gz"]
        grads.append(g)
        if kind == "momentum":
            Z, m = orc.momentum_step(Z, g, m, lr, b1)
        else:
            Z, m, v = orc.adam_step(Z, g, m, v, t, lr, b1, b2, eps)
    return Z, grads


@pytest.mark.parametrize("d,n", [(128, 512), (192, 416)])       # shared-memory 128 x 128 kernels / general path
def test_momentum_matches_oracle(d, n):
    w = gen.scaled(gen.WORKLOADS["c1_tiny"], d=d, n_tokens=n, n_outlier_channels=2)
    c = Calib(w)
    dq.dq_calib_set_optimizer(c.h, dq.DQ_SGD_MOMENTUM, w.lr, 0.9)
    c.step(STEPS)
    assert c.status() == dq.DQ_OK
    Z_ref, _ = _oracle_run(x_f64(w, c.X_host), c.Z0_host[0], w.lr, "momentum", 0.9, 0.0, 0.0)
    Z = c.latent()[0].astype(np.float64)
    # linear in the gradient: fp32 rounding of dL/dZ (about 1e-3 relative) carries over
    assert np.linalg.norm(Z - Z_ref) <= 5e-3 * np.linalg.norm(Z_ref - c.Z0_host[0])
    c.close()


@pytest.mark.parametrize("d,n", [(128, 512), (192, 416)])
def test_adam_matches_oracle_where_the_gradient_sign_is_decided(d, n):
    w = gen.scaled(gen.WORKLOADS["c1_tiny"], d=d, n_tokens=n, n_outlier_channels=2)
    lr, b1, b2, eps = 1e-3, 0.9, 0.999, 1e-8
    c = Calib(w)
    dq.dq_calib_set_optimizer(c.h, dq.DQ_ADAM, lr, b1, b2, eps)
    c.step(STEPS)
    assert c.status() == dq.DQ_OK
    Z_ref, grads = _oracle_run(x_f64(w, c.X_host), c.Z0_host[0], lr, "adam", b1, b2, eps)
    Z = c.latent()[0].astype(np.float64)
    # Adam divides by |g|-like quantities: an entry whose gradient is within fp32 rounding of zero may
    # step the other way.  Compare where every step's gradient is clear of that band (the sign is a
    # discrete decision taken on a floating-point value); there the error of a step is ~1e-3 lr.
    clear = np.ones_like(Z, dtype=bool)
    for g in grads:
        clear &= np.abs(g) >= 0.05 * np.median(np.abs(g))
    assert clear.mean() > 0.8
    print("adam: clear %.3f, max err / lr %.3e" % (clear.mean(), np.abs(Z - Z_ref)[clear].max() / lr))
    assert np.abs(Z - Z_ref)[clear].max() <= 5e-2 * lr * STEPS
    # every entry moved by about lr per step (the first step is exactly lr in magnitude)
    moved = np.abs(Z - c.Z0_host[0])[clear]
    assert moved.max() <= 1.05 * lr * STEPS and np.median(moved) >= 0.5 * lr
    M = c.buf(dq.DQ_BUF_OPT_M).cpu().numpy()[0]
    assert np.isfinite(M).all() and np.abs(M).max() > 0
    c.close()


@pytest.mark.parametrize("opt", ["momentum", "adam"])
def test_tensor_core_path_optimiser_state_advances_identically_eager_and_replayed(opt):
    """The step count of Adam lives on the device, so a replayed CUDA graph and step-by-step calls
    with per-phase timing (never replayed) must give bit-identical latents."""
    w = gen.scaled(gen.WORKLOADS["c2_7b"], d=256, n_tokens=1024, n_outlier_channels=3)
    outs = []
    for eager in (False, True):
        c = Calib(w)
        if opt == "adam":
            dq.dq_calib_set_optimizer(c.h, dq.DQ_ADAM, 1e-3, 0.9, 0.999, 1e-8)
        else:
            dq.dq_calib_set_optimizer(c.h, dq.DQ_SGD_MOMENTUM, w.lr, 0.9)
        if eager:
            dq.dq_calib_set_timing(c.h, True)
        losses = c.step(5)
        assert c.status() == dq.DQ_OK
        outs.append((losses.copy(), c.latent().copy()))
        c.close()
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])
    assert outs[0][0][-1, 0] < outs[0][0][0, 0]


def test_set_optimizer_rejects_bad_arguments():
    w = gen.scaled(gen.WORKLOADS["c1_tiny"], d=128, n_tokens=256)
    c = Calib(w)
    lib = dq.load_library()
    assert lib.dq_calib_set_optimizer(c.h, 7, 0.1, 0.9, 0.999, 1e-8) == dq.DQ_ERR_INVALID_ARG
    assert lib.dq_calib_set_optimizer(c.h, dq.DQ_ADAM, 0.1, 1.0, 0.999, 1e-8) == dq.DQ_ERR_INVALID_ARG
    assert lib.dq_calib_set_optimizer(c.h, dq.DQ_ADAM, 0.1, 0.9, 0.999, -1.0) == dq.DQ_ERR_INVALID_ARG
    assert lib.dq_calib_set_optimizer(None, dq.DQ_SGD, 0.1, 0.0, 0.0, 0.0) == dq.DQ_ERR_INVALID_ARG
    c.close()


@pytest.mark.parametrize("opt", ["momentum", "adam"])
def test_tensor_core_path_optimiser_update_matches_oracle_rule_on_its_own_gradients(opt):
    """Teacher-forced on the gradient: after every step on the tensor-core path the latent must be what the
    oracle's update rule makes of the previous latent, the previous optimiser state and the dL/dZ the kernels
    just produced (the gradient itself is compared with the oracle by the stage tests).  Steps after the first
    are replayed from a CUDA graph, so Adam's step count must advance on the device."""
    w = gen.scaled(gen.WORKLOADS["c2_7b"], d=256, n_tokens=1024, n_outlier_channels=3)
    lr, b1, b2, eps = (1e-3, 0.9, 0.999, 1e-8) if opt == "adam" else (w.lr, 0.9, 0.0, 0.0)
    c = Calib(w)
    dq.dq_calib_set_optimizer(c.h, dq.DQ_ADAM if opt == "adam" else dq.DQ_SGD_MOMENTUM, lr, b1, b2, eps)
    Z = c.latent()[0].astype(np.float64)
    m, v = np.zeros_like(Z), np.zeros_like(Z)
    for t in range(1, 5):
        c.step(1)
        assert c.status() == dq.DQ_OK
        g = c.buf(dq.DQ_BUF_GZ).cpu().numpy()[0].astype(np.float64)
        if opt == "adam":
            Z_ref, m, v = orc.adam_step(Z, g, m, v, t, lr, b1, b2, eps)
        else:
            Z_ref, m = orc.momentum_step(Z, g, m, lr, b1)
        Zg = c.latent()[0].astype(np.float64)
        moved = np.abs(Z_ref - Z).max()
        # fp32 arithmetic of the update: a few ulp of the latent plus 1e-5 of the step
        assert np.abs(Zg - Z_ref).max() <= 4 * 6e-8 * np.abs(Z).max() + 2e-5 * moved, (opt, t)
        assert moved > 0
        M = c.buf(dq.DQ_BUF_OPT_M).cpu().numpy()[0].astype(np.float64)
        assert np.abs(M - m).max() <= 1e-5 * np.abs(m).max() + 1e-12
        Z = Zg                                                      # the next step starts from the kernel's latent
        m = M
        if opt == "adam":
            v = c.buf(dq.DQ_BUF_OPT_V).cpu().numpy()[0].astype(np.float64)
    c.close()
