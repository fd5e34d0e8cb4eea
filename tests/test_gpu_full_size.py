"""Parity at the full sizes of the five benchmark workloads, in the launch configuration the
benchmark times (same handle, same kernels, same split factors): one teacher-forced
calibration step from a seeded latent near the workload's initialisation, against the float64
oracle run on all tokens.  Contract tolerances: loss relative error <= 2e-2 (bf16 tensor-core
path) / <= 1e-4 (fp32 path); max|R_gpu - R_ref| <= 1e-3 for the rotation used by the step (the
rotation of the same latent: no sign decision enters it) and for the rotation of the updated
latent; max|R^T R - I| <= 1e-4.  On the bf16 path dL/dR, dL/dZ and the update are checked against
the first-order error model of the one rounding the path commits (R to bf16), and the numbers
without the sign hook are printed beside the hooked ones."""
import numpy as np
import pytest
import torch

import oracle as orc
import paper_2511_04063_b200 as dq
from paper_2511_04063_b200 import inputs as gen
from gpu_util import Calib, x_f64, bf16_step_reference, check_bf16_gradients, perturbed_latent, MAX_OVERRIDDEN

pytestmark = pytest.mark.gpu

R_TOL, ORTHO_TOL = 1e-3, 1e-4


@pytest.mark.parametrize("name,qr", [("c1_tiny", "householder"), ("c1_tiny", "iterative"), ("c2_7b", "householder"), ("c2_7b", "iterative"),
                                     ("c3_heads", "householder"), ("c3_heads", "iterative"), ("c4_13b", "householder"), ("c4_13b", "iterative"),
                                     ("c5_70b", "householder"), ("c5_70b", "iterative")])
def test_one_step_at_full_size(name, qr):
    w = gen.WORKLOADS[name]
    c = Calib(w)
    dq.dq_calib_set_qr_method(c.h, dq.DQ_QR_ITERATIVE if qr == "iterative" else dq.DQ_QR_HOUSEHOLDER, 0)
    Z = perturbed_latent(w, c.Z0_host, w.seed)
    c.set_latent(Z)
    if qr == "iterative":
        # the first step after set_latent factors with Householder; the step under test is the next
        # one, which uses the incremental factorisation
        c.step(1)
        assert c.status() == dq.DQ_OK
        Z = c.latent()
    loss = c.step(1)[0]
    assert c.status() == dq.DQ_OK
    R_used = c.buf(dq.DQ_BUF_R).cpu().numpy().astype(np.float64)
    G_dev = Gq_all = Gz_all = None
    if w.path != "fp32":
        G_dev = c.buf(dq.DQ_BUF_G, dtype=torch.bfloat16, shape=(w.batch, w.d, w.n_tokens)).clone()
        Gq_all = c.buf(dq.DQ_BUF_GQ).cpu().numpy()
        Gz_all = c.buf(dq.DQ_BUF_GZ).cpu().numpy()
    Z1_all = c.latent()
    R_next = c.rotation()
    assert c.status() == dq.DQ_OK
    tol_loss = 1e-4 if w.path == "fp32" else 2e-2
    heads = range(w.batch) if w.batch <= 4 else (0, w.batch // 2, w.batch - 1)   # sampled problems
    # dL/dR, dL/dZ and the update are checked against the error model in the default configuration (the one the
    # benchmark times); the Householder variant differs only in how R is obtained, which the checks on R cover
    extended = qr == "iterative"
    for b in heads:
        X = x_f64(w, c.X_host, b)
        tag = "%s/%s[%d]" % (name, qr, b)
        if w.path == "fp32":
            ref = orc.calib_step(X, Z[b], w.lr, qr=orc.qr_pos_lapack)
            st = None
        else:
            # Eq. 4 has a kink at o = 0: where the rounding of R to bf16 moved the kernel's o across it, the
            # sign of dL/dO is the kernel's decision (read from its stored dL/dO); everywhere else the signs
            # must agree (checked inside), and the fraction of entries handed over is bounded
            G_tok = G_dev[b].t().float().cpu().numpy()
            st = bf16_step_reference(X, Z[b], w.lr, R_used[b], G_tok, extended=extended)
            del G_tok
            ref = st["ref"]
            assert st["overridden"] <= MAX_OVERRIDDEN, (tag, st["overridden"])
        assert abs(loss[b] - ref["loss"]) <= tol_loss * ref["loss"], (name, b, loss[b], ref["loss"])
        assert np.abs(R_used[b] - ref["R"]).max() <= R_TOL
        assert np.abs(R_used[b].T @ R_used[b] - np.eye(w.d)).max() <= ORTHO_TOL
        Rn_ref, _ = orc.qr_pos_lapack(ref["Z_new"])
        err_next = np.abs(R_next[b] - Rn_ref).max()
        print("%s: loss %.6f ref %.6f, |R-Rref| %.2e, |Rnext-ref| %.2e%s" %
              (tag, loss[b], ref["loss"], np.abs(R_used[b] - ref["R"]).max(), err_next,
               "" if st is None else ", overridden %.4f%%" % (100 * st["overridden"])))
        assert err_next <= R_TOL
        assert np.abs(R_next[b].T @ R_next[b] - np.eye(w.d)).max() <= ORTHO_TOL
        Z1 = Z1_all[b].astype(np.float64)
        if w.path == "fp32":
            # the update itself, relative to the size of the step
            step_ref = ref["Z_new"] - Z[b].astype(np.float64)
            assert np.linalg.norm(Z1 - ref["Z_new"]) <= 1e-3 * np.linalg.norm(step_ref) + 1e-6 * np.linalg.norm(Z[b])
        elif extended:
            check_bf16_gradients(tag, Gq_all[b].astype(np.float64), Gz_all[b].astype(np.float64), Z1,
                                 Z[b].astype(np.float64), w.lr, st)
            Rn_free, _ = orc.qr_pos_lapack(st["free"]["Z_new"])
            print("%s: max|R_next - ref| hook-free %.2e, rotation moved %.2e" %
                  (tag, np.abs(R_next[b] - Rn_free).max(), np.abs(Rn_ref - ref["R"]).max()))
        del X, ref, st
    c.close()
