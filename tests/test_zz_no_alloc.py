"""dq_rotate_apply_static: the rotation Y = X R for callers that cannot allocate device memory
(all of HBM already belongs to their own arena, or a cudaFree-induced device synchronisation is
not acceptable on their path).  Its scratch is a fixed array inside the library, so the check is
simply that it gives what dq_rotate_apply gives -- on two calls in a row with different rotations,
because the array keeps the previous call's contents and a stale read would show up on the second.

Collected last on purpose (file name): a run that stops at the first failure has then already
run every other test."""
import ctypes as C

import numpy as np
import pytest
import torch

import paper_2511_04063_b200 as dq
from paper_2511_04063_b200 import inputs as gen

pytestmark = pytest.mark.gpu


def _orthogonal(d, seed):
    q, r = np.linalg.qr(np.random.default_rng(seed).standard_normal((d, d)))
    return (q * np.sign(np.diag(r))[None, :]).astype(np.float32)


def test_static_scratch_rotation_matches_allocating_entry_point_twice_in_a_row():
    n = 512
    for call, (d, seed) in enumerate([(640, 11), (256, 12)]):      # second call uses a smaller part of the array
        X = torch.from_numpy(gen.f32_to_bf16_bits(
            np.random.default_rng(seed).standard_normal((n, d)).astype(np.float32)).view(np.int16)).cuda().view(torch.bfloat16)
        R = torch.from_numpy(_orthogonal(d, seed)).cuda()
        Y_ref = torch.empty((n, d), dtype=torch.bfloat16, device="cuda")
        Y_new = torch.full((n, d), float("nan"), dtype=torch.bfloat16, device="cuda")
        dq.dq_rotate_apply(X, R, Y_ref)
        dq.dq_rotate_apply_static(X, R, Y_new)
        torch.cuda.synchronize()
        a, b = Y_ref.float().cpu().numpy(), Y_new.float().cpu().numpy()
        assert np.isfinite(b).all(), call
        # same tolerance as the bf16 rotate_apply parity test (bf16 operands and output)
        assert np.abs(a - b).max() <= 6e-2, call
        assert np.linalg.norm(a - b) <= 1e-2 * np.linalg.norm(a), call


def test_static_scratch_rotation_rejects_sizes_beyond_its_array():
    lib = dq.load_library()
    d, n = 2176, 128                                               # 17 * 128 > 2048
    X = torch.zeros((n, d), dtype=torch.bfloat16, device="cuda")
    Y = torch.zeros((n, d), dtype=torch.bfloat16, device="cuda")
    R = torch.zeros((d, d), dtype=torch.float32, device="cuda")
    p = lambda t: C.c_void_p(t.data_ptr())
    st = lib.dq_rotate_apply_static(p(X), n, d, d, p(R), p(Y), d, None)
    assert st == dq.DQ_ERR_UNSUPPORTED
    with pytest.raises(dq.DartQuantError):
        dq.dq_rotate_apply_static(X, R, Y)
    assert lib.dq_rotate_apply_static(None, n, d, d, p(R), p(Y), d, None) == dq.DQ_ERR_INVALID_ARG
