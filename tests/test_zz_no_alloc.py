"""dq_rotate_apply_static: the rotation Y = X R for callers that cannot allocate device memory
(all of HBM already belongs to their own arena, or a cudaFree-induced device synchronisation is
not acceptable on their path).  Its scratch is a fixed array inside the library, so the check is
that it gives exactly what dq_rotate_apply gives (and what the float64 oracle gives, within bf16
rounding) -- on calls in a row with different rotations and sizes, because the array keeps the
previous call's contents and a stale read would show up on the later ones -- and that it takes no
device memory.

Collected last on purpose (file name): a run that stops at the first failure has then already
run every other test."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle as orc
import paper_2511_04063_b200 as dq
from paper_2511_04063_b200 import inputs as gen

pytestmark = pytest.mark.gpu


def _orthogonal(d, seed):
    q, r = np.linalg.qr(np.random.default_rng(seed).standard_normal((d, d)))
    return (q * np.sign(np.diag(r))[None, :]).astype(np.float32)


def test_static_scratch_rotation_matches_allocating_entry_point_twice_in_a_row():
    n = 512
    # the second call uses a smaller part of the array than the first, the third all of it (d = 2048)
    for call, (d, seed) in enumerate([(640, 11), (256, 12), (2048, 13)]):
        Xb = gen.f32_to_bf16_bits(np.random.default_rng(seed).standard_normal((n, d)).astype(np.float32))
        X = torch.from_numpy(Xb.view(np.int16)).cuda().view(torch.bfloat16)
        Rh = _orthogonal(d, seed)
        R = torch.from_numpy(Rh).cuda()
        Y_ref = torch.empty((n, d), dtype=torch.bfloat16, device="cuda")
        Y_new = torch.full((n, d), float("nan"), dtype=torch.bfloat16, device="cuda")
        dq.dq_rotate_apply(X, R, Y_ref)
        dq.dq_rotate_apply_static(X, R, Y_new)
        torch.cuda.synchronize()
        a, b = Y_ref.float().cpu().numpy(), Y_new.float().cpu().numpy()
        assert np.isfinite(b).all(), call
        # both entry points run the same kernels on the same operands: the outputs are identical
        assert np.array_equal(a, b), call
        # and both are the rotation: against the float64 oracle, with the tolerance of the bf16 rotate_apply
        # parity test (bf16 operand R and bf16 output, 2^-9 each)
        ref = orc.rotate(gen.bf16_bits_to_f32(Xb).reshape(n, d), Rh)
        assert np.abs(b - ref).max() <= 6e-2, call
        assert np.linalg.norm(b - ref) <= 1e-2 * np.linalg.norm(ref), call


def test_static_scratch_rotation_takes_no_device_memory():
    """After one warm-up call (the first call on a device resolves the array's address and may load the
    library's kernels), further calls leave the amount of free device memory unchanged."""
    n, d = 256, 512
    X = torch.zeros((n, d), dtype=torch.bfloat16, device="cuda")
    Y = torch.empty((n, d), dtype=torch.bfloat16, device="cuda")
    R = torch.eye(d, dtype=torch.float32, device="cuda")
    dq.dq_rotate_apply_static(X, R, Y)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(20):
        dq.dq_rotate_apply_static(X, R, Y)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0


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
