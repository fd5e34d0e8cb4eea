"""Cayley SGD with momentum (Algorithm 3; the optimiser Sec. 5.3 / Table 4 compare QR-Orth with) on
the tensor-core path against the float64 oracle: every stage of one update fed with the kernel's
own gradient (so the six split-bf16 products are checked at their own precision), one whole
teacher-forced step, a free run replayed as a CUDA graph, and argument checking."""
import numpy as np
import pytest
import torch

import oracle as orc
import paper_2511_04063_b200 as dq
from paper_2511_04063_b200 import inputs as gen
from gpu_util import Calib, x_f64, bf16_sign_decider

pytestmark = pytest.mark.gpu

LOSS_TOL_BF16 = 2e-2
R_TOL = 1e-3


def small(name, **kw):
    return gen.scaled(gen.WORKLOADS[name], **kw)


def _state(c):
    R = c.rotation()
    M = c.buf(dq.DQ_BUF_CAYLEY_M).cpu().numpy().astype(np.float64)
    return R, M


CASES = [
    (small("c2_7b", d=256, n_tokens=1024, n_outlier_channels=3), 1e-3, 0.9, 2),
    (small("c2_7b", d=256, n_tokens=1024, n_outlier_channels=3), 1e4, 0.5, 3),     # step size clipped by 2 q / |W|
    (small("c4_13b", d=640, n_tokens=512, batch=2, n_outlier_channels=4), 1e-2, 0.9, 2),
]


@pytest.mark.parametrize("w,lr,beta,s", CASES, ids=lambda v: getattr(v, "name", str(v)))
def test_cayley_update_every_stage(w, lr, beta, s):
    c = Calib(w, lr=lr)
    dq.dq_calib_set_orth_method(c.h, dq.DQ_ORTH_CAYLEY, beta, 0.0, s)
    n, d, batch = w.n_tokens, w.d, w.batch
    branches = set()
    for step in range(2):     # step 0: zero momentum from the QR factor; step 1: momentum in play
        R0, M0 = _state(c)
        if step == 0:
            for b in range(batch):    # X_1 = orthogonal factor of the latent
                assert np.abs(R0[b] - orc.qr_pos_lapack(c.Z0_host[b])[0]).max() <= 5e-5
                assert np.abs(M0[b]).max() == 0.0
        loss = c.step(1)[0]
        assert c.status() == dq.DQ_OK
        Gq = c.buf(dq.DQ_BUF_GQ).cpu().numpy().astype(np.float64)
        Gt = c.buf(dq.DQ_BUF_G, dtype=torch.bfloat16, shape=(batch, d, n)).float().cpu().numpy().astype(np.float64)
        alpha = c.buf(dq.DQ_BUF_CAYLEY_ALPHA, shape=(batch,)).cpu().numpy().astype(np.float64)
        R1, M1 = _state(c)
        for b in range(batch):
            X = x_f64(w, c.X_host, b)
            # (i) Algorithm 3's update alone, from the kernel's own gradient: three split-bf16 MMAs
            # per product give ~2^-17 relative error per product; a few products deep: 1e-4 relative.
            upd = orc.cayley_sgd_step(R0[b], M0[b], Gq[b], lr, beta, s=s)
            branches.add(upd["alpha"] == lr)
            assert abs(alpha[b] - upd["alpha"]) <= 1e-5 * upd["alpha"]
            assert np.abs(M1[b] - upd["M_new"]).max() <= 1e-4 * np.abs(upd["M_new"]).max()
            assert np.abs(R1[b] - upd["X_new"]).max() <= 2e-5
            # (ii) the whole iteration from the same rotation and momentum: loss and dL/dR carry the
            # bf16 rounding of R in the Whip contraction (see the QR-Orth parity test for the bounds)
            # the sign of dL/dO is the kernel's only where the rounding of R to bf16 moved o across the kink
            stats = {}
            ref = orc.cayley_calib_step(X, R0[b], M0[b], lr, beta, s=s,
                                        sign_decider=bf16_sign_decider(X, R0[b], R0[b], Gt[b].T, stats))
            assert abs(loss[b] - ref["loss"]) <= LOSS_TOL_BF16 * ref["loss"]
            # dL/dR inherits e^-|o| dO from the bf16 rotation, with dO up to a few 1e-2 on outlier-heavy
            # tokens: up to 1e-1 relative once the rotation is no longer a Hadamard-like matrix
            rel_gq = np.linalg.norm(Gq[b] - ref["Gq"]) / np.linalg.norm(ref["Gq"])
            rel_m = np.linalg.norm(M1[b] - ref["M_new"]) / np.linalg.norm(ref["M_new"])
            print("step %d problem %d: overridden %.4f%%, rel err dL/dR %.3e, M %.3e, max |dR| %.3e" %
                  (step, b, 100 * stats["overridden"], rel_gq, rel_m, np.abs(R1[b] - ref["R_new"]).max()))
            assert rel_gq <= 1e-1 and rel_m <= 1e-1
            # the update is (to first order) alpha M_new, so its error is the relative error of M_new
            # times the step; the 1e-3 per-step bound on the rotation is meaningful for steps up to 1e-2
            step_max = np.abs(ref["R_new"] - R0[b]).max()
            assert np.linalg.norm(R1[b] - ref["R_new"]) <= 1.5e-1 * np.linalg.norm(ref["R_new"] - R0[b]) + 1e-5 * d
            if step_max <= 1e-2:
                assert np.abs(R1[b] - ref["R_new"]).max() <= R_TOL
            else:
                assert np.abs(R1[b] - ref["R_new"]).max() <= 2e-1 * step_max
            # W is skew-symmetric, so M_new = W R is tangent at R: R^T M_new is skew-symmetric
            A = R0[b].T @ M1[b]
            assert np.abs(A + A.T).max() <= 1e-4 * max(1.0, np.abs(A).max())
    print("alpha == lr branch seen:", branches)
    c.close()


def test_both_sides_of_the_step_size_clip_are_covered():
    # recomputed from the oracle on the two d = 256 cases above: one keeps lr, the other is clipped
    w = CASES[0][0]
    X = x_f64(w, gen.gen_activations(w))
    R, _ = orc.qr_pos_lapack(gen.gen_latent_init(w)[0])
    a_small = orc.cayley_calib_step(X, R, np.zeros_like(R), CASES[0][1], 0.9)["alpha"]
    a_big = orc.cayley_calib_step(X, R, np.zeros_like(R), CASES[1][1], 0.5)["alpha"]
    assert a_small == CASES[0][1] and a_big < CASES[1][1]


def test_cayley_free_run_replayed_matches_oracle_and_timed_run():
    w = small("c2_7b", d=512, n_tokens=1024, n_outlier_channels=3)
    lr, beta, steps = 2e-3, 0.9, 5
    runs = []
    for timed in (False, True):
        c = Calib(w, lr=lr)
        dq.dq_calib_set_orth_method(c.h, dq.DQ_ORTH_CAYLEY, beta)
        if timed:
            dq.dq_calib_set_timing(c.h, True)      # never replays a captured graph
        losses = c.step(steps)[:, 0]
        assert c.status() == dq.DQ_OK
        runs.append((losses, c.rotation()[0], c.buf(dq.DQ_BUF_CAYLEY_M).cpu().numpy()[0].copy()))
        launches = dq.dq_calib_launch_count(c.h)
        c.close()
    assert np.array_equal(runs[0][0], runs[1][0])
    assert np.array_equal(runs[0][1], runs[1][1]) and np.array_equal(runs[0][2], runs[1][2])
    assert launches > 0
    ref_losses, R_ref, _ = orc.cayley_calib_run(x_f64(w, gen.gen_activations(w)), gen.gen_latent_init(w)[0], lr, beta, steps)
    losses, R, _ = runs[0]
    assert np.abs(losses - ref_losses).max() <= LOSS_TOL_BF16 * ref_losses.max()
    assert losses[-1] < losses[0]
    # free-running: every step's dL/dR carries a few per cent of error from the bf16 rotation (and sign
    # decisions at the kink differ), so the iterates drift apart by a fraction of the distance moved
    R0, _ = orc.qr_pos_lapack(gen.gen_latent_init(w)[0])
    moved = np.linalg.norm(R_ref - R0)
    print("free run: moved %.3e, drift %.3e, max |dR| %.3e" % (moved, np.linalg.norm(R - R_ref), np.abs(R - R_ref).max()))
    assert np.linalg.norm(R - R_ref) <= 0.25 * moved
    # the iterate leaves the orthogonal group only as far as the oracle's does (two sweeps are inexact)
    off = np.abs(R.T @ R - np.eye(w.d)).max()
    off_ref = np.abs(R_ref.T @ R_ref - np.eye(w.d)).max()
    assert off <= 2.0 * off_ref + 1e-4


def test_switching_back_to_qr_orth_restarts_from_the_latent():
    w = small("c2_7b", d=256, n_tokens=1024, n_outlier_channels=3)
    c = Calib(w)
    R0 = c.rotation()[0]
    dq.dq_calib_set_orth_method(c.h, dq.DQ_ORTH_CAYLEY, 0.9)
    c.step(2)
    assert np.abs(c.rotation()[0] - R0).max() > 0        # the iterate moved
    assert np.array_equal(c.latent(), c.Z0_host)           # the latent is not touched by Cayley SGD
    dq.dq_calib_set_orth_method(c.h, dq.DQ_ORTH_QR)
    # the same rotation again (the first came from the start at W = I of an orthogonal latent, this one from a
    # Householder factorisation: the unique factor either way, to the accuracy of the split-bf16 products)
    assert np.abs(c.rotation()[0] - R0).max() <= 5e-6
    c.close()


def test_set_orth_method_rejects_bad_arguments():
    w = small("c2_7b", d=256, n_tokens=1024, n_outlier_channels=3)
    c = Calib(w)
    for args in [(7, 0.0, 0.0, 0), (dq.DQ_ORTH_CAYLEY, 1.0, 0.0, 0), (dq.DQ_ORTH_CAYLEY, -0.1, 0.0, 0),
                 (dq.DQ_ORTH_CAYLEY, 0.5, 1.5, 0), (dq.DQ_ORTH_CAYLEY, 0.5, 0.5, 17)]:
        with pytest.raises(dq.DartQuantError) as e:
            dq.dq_calib_set_orth_method(c.h, *args)
        assert e.value.status == dq.DQ_ERR_INVALID_ARG
    c.close()
    w32 = gen.scaled(gen.WORKLOADS["c1_tiny"], d=128, n_tokens=256)
    c = Calib(w32)
    with pytest.raises(dq.DartQuantError) as e:
        dq.dq_calib_set_orth_method(c.h, dq.DQ_ORTH_CAYLEY, 0.9)
    assert e.value.status == dq.DQ_ERR_UNSUPPORTED
    c.close()
