"""Helpers shared by the GPU parity tests (marshalling between numpy and torch)."""
import numpy as np
import torch

import oracle as orc
import paper_2511_04063_b200 as dq
from paper_2511_04063_b200 import inputs as gen


def to_device_x(w, X):
    """Stored activations (float32 or bf16 bit patterns) -> CUDA tensor [batch, N, d]."""
    if w.x_dtype == "fp32":
        return torch.from_numpy(X).cuda()
    return torch.from_numpy(X.view(np.int16)).cuda().view(torch.bfloat16)


def path_of(w):
    return dq.DQ_PATH_FP32 if w.path == "fp32" else dq.DQ_PATH_BF16_TC


class Calib:
    """Owns a handle plus the tensors it borrows."""

    def __init__(self, w, X=None, Z0=None, lr=None, reduction=dq.DQ_MEAN_TOKENS):
        self.w = w
        self.X_host = gen.gen_activations(w) if X is None else X
        self.Z0_host = gen.gen_latent_init(w) if Z0 is None else Z0
        self.X = to_device_x(w, self.X_host)
        self.Z0 = torch.from_numpy(self.Z0_host).cuda()
        self.h = dq.dq_calib_init(self.X, self.Z0, lr=w.lr if lr is None else lr, path=path_of(w),
                                  reduction=reduction)
        self.dd = (w.batch, w.d, w.d)
        dq.dq_calib_set_keep_gradient(self.h, True)    # the tests read dL/dO (DQ_BUF_G) at every shape

    def step(self, n=1):
        loss = torch.empty((n, self.w.batch), dtype=torch.float32, device="cuda")
        dq.dq_calib_step(self.h, n, loss)
        return loss.cpu().numpy().astype(np.float64)

    def rotation(self):
        R = torch.empty(self.dd, dtype=torch.float32, device="cuda")
        dq.dq_calib_get_rotation(self.h, R)
        return R.cpu().numpy().astype(np.float64)

    def latent(self):
        Z = torch.empty(self.dd, dtype=torch.float32, device="cuda")
        dq.dq_calib_get_latent(self.h, Z)
        return Z.cpu().numpy()

    def set_latent(self, Z):
        dq.dq_calib_set_latent(self.h, torch.from_numpy(np.ascontiguousarray(Z, dtype=np.float32)).cuda())

    def buf(self, which, dtype=torch.float32, shape=None):
        shape = self.dd if shape is None else shape
        return dq.dq_calib_debug_buffer(self.h, which, dtype, shape)

    def status(self):
        return dq.dq_calib_status(self.h)

    def close(self):
        if self.h is not None:
            dq.dq_calib_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def x_f64(w, X, b=0):
    return gen.activations_as_f32(w, X)[b].astype(np.float64)


def sign_decider_from_gpu(G_gpu_token_major, band):
    """Eq. 4 has a kink at o = 0: where the oracle's |O| is within `band` (the rounding
    error of the GPU arithmetic; scalar or per-token column vector) the sign decision is
    taken in the kernel's precision, i.e. from the stored dL/dO.  Elsewhere the signs must agree."""
    sg = -np.sign(G_gpu_token_major)

    def decide(O):
        s = np.sign(O)
        near = np.abs(O) <= band
        # beyond |o| ~ 87 exp(-|o|) underflows in fp32 and the stored derivative is an exact 0
        chk = ~near & (np.abs(O) < 60.0)
        assert np.array_equal(s[chk], sg[chk]), "sign of dL/dO differs away from the kink"
        return np.where(near, sg, s)
    return decide
