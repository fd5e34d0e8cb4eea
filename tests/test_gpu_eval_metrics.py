"""Outlier count (Eq. 1) and per-token asymmetric quantisation error of O = X R against the float64
oracle.  The count is a discrete decision on a floating-point value: entries within the rounding
band of the kernel's O around tau may fall on either side, so the kernel's count must lie between
the oracle's counts at tau -+ band.  The quantisation error is continuous in O."""
import numpy as np
import pytest
import torch

import oracle as orc
import paper_2511_04063_b200 as dq
from paper_2511_04063_b200 import inputs as gen

pytestmark = pytest.mark.gpu


def _rotation(d, seed):
    R, _ = orc.qr_pos_lapack(np.random.default_rng(seed).standard_normal((d, d)))
    return R.astype(np.float32)


@pytest.mark.parametrize("name,d,n,bits", [("c2_7b", 256, 1024, 4), ("c5_70b", 512, 2048, 4), ("c4_13b", 640, 384, 8),
                                           ("c1_tiny", 96, 300, 4), ("c1_tiny", 128, 256, 2)])
def test_outliers_and_quantisation_error(name, d, n, bits):
    w = gen.scaled(gen.WORKLOADS[name], d=d, n_tokens=n, n_outlier_channels=3)
    Xh = gen.gen_activations(w)[0]
    X64 = gen.activations_as_f32(w, Xh[None])[0].astype(np.float64)
    R = _rotation(d, d + bits)
    if w.x_dtype == "fp32":
        Xd, rel = torch.from_numpy(Xh).cuda(), 2.0 ** -20
    else:
        Xd, rel = torch.from_numpy(Xh.view(np.int16)).cuda().view(torch.bfloat16), 2.0 ** -8   # bf16(R)
    for rot, Rm in (("identity", np.eye(d, dtype=np.float32)), ("random", R)):
        O = X64 @ Rm.astype(np.float64)
        tau = float(3.0 * np.std(O))
        cnt, mse = dq.dq_eval_rotation(Xd, torch.from_numpy(Rm).cuda(), tau, bits)
        band = rel * np.linalg.norm(X64, axis=1)[:, None] * np.ones((1, d)) * 4.0 / np.sqrt(d) + rel * np.abs(O)
        lo = int((np.abs(O) > tau + band).sum())
        hi = int((np.abs(O) > tau - band).sum())
        assert lo <= cnt <= hi, (rot, lo, cnt, hi)
        assert hi - lo <= max(8, 0.10 * max(hi, 1))               # the band is narrow: the check has teeth
        ref = orc.quantization_mse(O, bits)
        assert abs(mse - ref) <= (2e-2 if w.x_dtype == "bf16" else 1e-4) * ref, (rot, mse, ref)

def test_eval_rotation_rejects_bad_arguments():
    import ctypes as C
    lib = dq.load_library()
    X = torch.zeros((128, 128), device="cuda")
    R = torch.eye(128, device="cuda")
    out = torch.zeros(2, dtype=torch.float64, device="cuda")
    p = lambda t: C.c_void_p(t.data_ptr())
    assert lib.dq_eval_rotation(p(X), dq.DQ_FP32, 128, 128, 128, p(R), 1.0, 0, p(out), None) == dq.DQ_ERR_INVALID_ARG
    assert lib.dq_eval_rotation(p(X), dq.DQ_FP32, 128, 128, 128, p(R), -1.0, 4, p(out), None) == dq.DQ_ERR_INVALID_ARG
    assert lib.dq_eval_rotation(None, dq.DQ_FP32, 128, 128, 128, p(R), 1.0, 4, p(out), None) == dq.DQ_ERR_INVALID_ARG
    Xb = torch.zeros((100, 128), dtype=torch.bfloat16, device="cuda")
    assert lib.dq_eval_rotation(p(Xb), dq.DQ_BF16, 100, 128, 128, p(R), 1.0, 4, p(out), None) == dq.DQ_ERR_UNSUPPORTED
