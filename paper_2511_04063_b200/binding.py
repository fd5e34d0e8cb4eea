"""ctypes binding of the C ABI declared in include/dartquant.h.

Argument marshalling only: every step of the calibration path runs in the CUDA
kernels of libdartquant.so.  PyTorch supplies device memory and streams.  There
is no fallback: if the library is missing, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libdartquant.so")

DQ_OK, DQ_ERR_INVALID_ARG, DQ_ERR_UNSUPPORTED, DQ_ERR_ALLOC, DQ_ERR_CUDA = 0, 1, 2, 3, 4
DQ_ERR_SINGULAR, DQ_ERR_NONFINITE, DQ_ERR_TIMEOUT, DQ_ERR_NOT_CONVERGED = 5, 6, 7, 8
DQ_QR_HOUSEHOLDER, DQ_QR_ITERATIVE = 0, 1
DQ_ORTH_QR, DQ_ORTH_CAYLEY = 0, 1
DQ_OBJ_WHIP, DQ_OBJ_VARIANCE, DQ_OBJ_KURTOSIS, DQ_OBJ_QUANT = 0, 1, 2, 3
DQ_FP32, DQ_BF16 = 0, 1
DQ_PATH_FP32, DQ_PATH_BF16_TC = 0, 1
DQ_MEAN_TOKENS, DQ_SUM_TOKENS = 0, 1
DQ_SGD, DQ_SGD_MOMENTUM, DQ_ADAM = 0, 1, 2
DQ_PHASE_NAMES = ("qr_forward", "rotate_whip", "grad_rotation", "qr_backward", "update")
DQ_BUF_R, DQ_BUF_U, DQ_BUF_GQ, DQ_BUF_GZ, DQ_BUF_G, DQ_BUF_PARTIALS, DQ_BUF_Z, DQ_BUF_OPT_M, DQ_BUF_OPT_V = range(9)
DQ_BUF_CAYLEY_M, DQ_BUF_CAYLEY_ALPHA = 9, 10

EXPORTED_SYMBOLS = (
    "dq_calib_init", "dq_calib_step", "dq_calib_get_rotation", "dq_rotate_apply",
    "dq_calib_get_latent", "dq_calib_set_latent", "dq_calib_refresh_inputs", "dq_calib_status",
    "dq_calib_get_timings", "dq_calib_set_timing", "dq_calib_debug_buffer", "dq_calib_launch_count", "dq_status_string",
    "dq_calib_destroy", "dq_version", "dq_rotate_apply_static", "dq_calib_set_qr_method", "dq_calib_set_optimizer", "dq_gather_tokens", "dq_eval_rotation",
    "dq_calib_set_orth_method", "dq_calib_set_objective", "dq_calib_run_epochs", "dq_calib_mma_flops", "dq_calib_set_keep_gradient",
    "dq_calib_set_backward_precision", "dq_calib_selftest_bounded_wait", "dq_calib_time_product",
)


class dq_calib_config(C.Structure):
    _fields_ = [("d", C.c_int32), ("n_tokens", C.c_int64), ("batch", C.c_int32), ("x_dtype", C.c_int32),
                ("path", C.c_int32), ("reduction", C.c_int32), ("optimizer", C.c_int32), ("lr", C.c_float),
                ("ldx", C.c_int64)]


class DartQuantError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (dq_status %d)" % (where, status_string(status), status))


_lib = None


def load_library(path: str = LIB_PATH) -> C.CDLL:
    """Loads libdartquant.so.  Raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(path):
        raise ImportError("libdartquant.so is not built: run `python -m paper_2511_04063_b200.build` "
                          "(the calibration path has no non-CUDA implementation)")
    lib = C.CDLL(path)
    vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
    lib.dq_calib_init.argtypes = [C.POINTER(vp), C.POINTER(dq_calib_config), vp, vp, vp]
    lib.dq_calib_step.argtypes = [vp, i32, vp]
    lib.dq_calib_get_rotation.argtypes = [vp, vp]
    lib.dq_rotate_apply.argtypes = [vp, i32, i64, i32, i64, vp, vp, i64, vp]
    lib.dq_rotate_apply_static.argtypes = [vp, i64, i32, i64, vp, vp, i64, vp]
    lib.dq_rotate_apply_static.restype = i32
    lib.dq_calib_set_optimizer.argtypes = [vp, i32, C.c_float, C.c_float, C.c_float, C.c_float]
    lib.dq_calib_set_optimizer.restype = i32
    lib.dq_calib_set_qr_method.argtypes = [vp, i32, i32]
    lib.dq_calib_set_qr_method.restype = i32
    lib.dq_calib_run_epochs.argtypes = [vp, vp, i64, i64, C.c_float, i32, i32, C.c_uint64, vp, C.POINTER(i64)]
    lib.dq_calib_run_epochs.restype = i32
    lib.dq_calib_set_objective.argtypes = [vp, i32, i32]
    lib.dq_calib_set_objective.restype = i32
    lib.dq_calib_set_orth_method.argtypes = [vp, i32, C.c_float, C.c_float, i32]
    lib.dq_calib_set_orth_method.restype = i32
    lib.dq_gather_tokens.argtypes = [vp, i32, i64, i32, i64, C.c_uint64, i64, i64, vp, i64, vp]
    lib.dq_gather_tokens.restype = i32
    lib.dq_eval_rotation.argtypes = [vp, i32, i64, i32, i64, vp, C.c_float, i32, vp, vp]
    lib.dq_eval_rotation.restype = i32
    lib.dq_calib_get_latent.argtypes = [vp, vp]
    lib.dq_calib_set_latent.argtypes = [vp, vp]
    lib.dq_calib_status.argtypes = [vp]
    lib.dq_calib_refresh_inputs.argtypes = [vp]
    lib.dq_calib_get_timings.argtypes = [vp, C.POINTER(C.c_float), i32]
    lib.dq_calib_set_timing.argtypes = [vp, i32]
    lib.dq_calib_debug_buffer.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(i64)]
    lib.dq_calib_set_keep_gradient.argtypes = [vp, i32]
    lib.dq_calib_set_keep_gradient.restype = i32
    lib.dq_calib_selftest_bounded_wait.argtypes = [vp, C.c_uint64, vp]
    lib.dq_calib_selftest_bounded_wait.restype = i32
    lib.dq_calib_time_product.argtypes = [vp, i32, i32, C.POINTER(C.c_float)]
    lib.dq_calib_time_product.restype = i32
    lib.dq_calib_set_backward_precision.argtypes = [vp, i32]
    lib.dq_calib_set_backward_precision.restype = i32
    lib.dq_calib_launch_count.argtypes = [vp]
    lib.dq_calib_mma_flops.argtypes = [vp]
    lib.dq_calib_mma_flops.restype = C.c_double
    lib.dq_calib_launch_count.restype = i64
    lib.dq_status_string.argtypes = [i32]
    lib.dq_status_string.restype = C.c_char_p
    lib.dq_calib_destroy.argtypes = [vp]
    lib.dq_calib_destroy.restype = None
    lib.dq_version.restype = C.c_char_p
    for name in ("dq_calib_init", "dq_calib_step", "dq_calib_get_rotation", "dq_rotate_apply",
                 "dq_calib_get_latent", "dq_calib_set_latent", "dq_calib_status", "dq_calib_get_timings",
                 "dq_calib_set_timing", "dq_calib_debug_buffer", "dq_calib_refresh_inputs"):
        getattr(lib, name).restype = i32
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().dq_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != DQ_OK:
        raise DartQuantError(status, where)


def _ptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else C.c_void_p(0)


def _stream_ptr(stream=None):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


# ---------------------------------------------------------------------------
# Same-name wrappers (torch tensors in, raw pointers out)
# ---------------------------------------------------------------------------
def dq_calib_init(X, Z0, *, lr: float, path: int, reduction: int = DQ_MEAN_TOKENS, stream=None):
    """X: CUDA tensor [batch, N, d] or [N, d], float32 or bfloat16, contiguous rows (borrowed:
    keep it alive).  Z0: CUDA float32 [batch, d, d] or [d, d] (copied).  Returns an opaque handle."""
    import torch
    assert X.is_cuda and Z0.is_cuda and Z0.dtype == torch.float32 and Z0.is_contiguous()
    if X.dim() == 2:
        X = X.unsqueeze(0)
    batch, n, d = X.shape
    assert X.stride(2) == 1 and X.stride(0) == n * X.stride(1)
    cfg = dq_calib_config(d=d, n_tokens=n, batch=batch,
                          x_dtype=DQ_FP32 if X.dtype == torch.float32 else DQ_BF16, path=path,
                          reduction=reduction, optimizer=DQ_SGD, lr=lr, ldx=X.stride(1))
    h = C.c_void_p(0)
    _check(load_library().dq_calib_init(C.byref(h), C.byref(cfg), _ptr(X), _ptr(Z0), _stream_ptr(stream)),
           "dq_calib_init")
    return h


def dq_calib_step(h, n_steps: int, loss_out=None):
    _check(load_library().dq_calib_step(h, n_steps, _ptr(loss_out)), "dq_calib_step")


def dq_calib_get_rotation(h, R_out):
    _check(load_library().dq_calib_get_rotation(h, _ptr(R_out)), "dq_calib_get_rotation")


def dq_calib_get_latent(h, Z_out):
    _check(load_library().dq_calib_get_latent(h, _ptr(Z_out)), "dq_calib_get_latent")


def dq_calib_set_latent(h, Z):
    _check(load_library().dq_calib_set_latent(h, _ptr(Z)), "dq_calib_set_latent")


def dq_calib_refresh_inputs(h):
    _check(load_library().dq_calib_refresh_inputs(h), "dq_calib_refresh_inputs")


def dq_calib_status(h) -> int:
    return int(load_library().dq_calib_status(h))


def dq_calib_set_timing(h, enabled: bool):
    _check(load_library().dq_calib_set_timing(h, int(enabled)), "dq_calib_set_timing")


def dq_calib_set_optimizer(h, optimizer: int, lr: float, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8):
    _check(load_library().dq_calib_set_optimizer(h, optimizer, lr, beta1, beta2, eps), "dq_calib_set_optimizer")


def dq_calib_set_qr_method(h, method: int, n_iters: int = 0):
    _check(load_library().dq_calib_set_qr_method(h, method, n_iters), "dq_calib_set_qr_method")


def dq_calib_run_epochs(h, pool, sample_ratio: float, accum: int, n_epochs: int, seed: int, loss_out=None) -> int:
    """pool: CUDA tensor [n_pool, d] (row stride = pool.stride(0)).  Returns the number of optimiser steps."""
    steps = C.c_int64(0)
    _check(load_library().dq_calib_run_epochs(h, pool.data_ptr(), pool.shape[0], pool.stride(0), sample_ratio, accum,
                                              n_epochs, seed, loss_out.data_ptr() if loss_out is not None else None,
                                              C.byref(steps)), "dq_calib_run_epochs")
    return int(steps.value)


def dq_calib_set_keep_gradient(h, keep: bool = True):
    _check(load_library().dq_calib_set_keep_gradient(h, 1 if keep else 0), "dq_calib_set_keep_gradient")


def dq_calib_set_backward_precision(h, split: bool):
    """QR-Orth backward on split-bf16 operands (True) or plain bf16 operands (False, the default)."""
    _check(load_library().dq_calib_set_backward_precision(h, 1 if split else 0), "dq_calib_set_backward_precision")


def dq_calib_selftest_bounded_wait(h, limit_ns: int) -> int:
    """Runs the library's bounded in-kernel wait on a barrier nothing arrives at; returns the nanoseconds it
    waited before giving up (synchronises).  Leaves DQ_ERR_TIMEOUT in the handle's status word."""
    import torch
    waited = torch.zeros(1, dtype=torch.int64, device="cuda")
    _check(load_library().dq_calib_selftest_bounded_wait(h, limit_ns, waited.data_ptr()), "dq_calib_selftest_bounded_wait")
    return int(waited.cpu()[0])


def dq_calib_time_product(h, nterms: int, reps: int = 10) -> float:
    """Mean milliseconds of one dense d^3 QR-Orth product (nterms 3: split-bf16, 1: plain bf16); measurement."""
    ms = C.c_float(0.0)
    _check(load_library().dq_calib_time_product(h, nterms, reps, C.byref(ms)), "dq_calib_time_product")
    return float(ms.value)


def dq_calib_mma_flops(h) -> float:
    return float(load_library().dq_calib_mma_flops(h))


def dq_calib_set_objective(h, objective: int, bits: int = 0):
    _check(load_library().dq_calib_set_objective(h, objective, bits), "dq_calib_set_objective")


def dq_calib_set_orth_method(h, method: int, beta: float = 0.0, q: float = 0.0, s: int = 0):
    _check(load_library().dq_calib_set_orth_method(h, method, beta, q, s), "dq_calib_set_orth_method")


def dq_calib_get_timings(h) -> dict:
    arr = (C.c_float * len(DQ_PHASE_NAMES))()
    _check(load_library().dq_calib_get_timings(h, arr, len(DQ_PHASE_NAMES)), "dq_calib_get_timings")
    return {k: float(arr[i]) for i, k in enumerate(DQ_PHASE_NAMES)}


def dq_calib_debug_buffer(h, which: int, dtype, shape):
    """A torch view (no copy) of one of the handle's device workspaces."""
    import torch
    p, n = C.c_void_p(0), C.c_int64(0)
    _check(load_library().dq_calib_debug_buffer(h, which, C.byref(p), C.byref(n)), "dq_calib_debug_buffer")
    numel = 1
    for s in shape:
        numel *= s
    assert numel <= n.value, (numel, n.value)
    itemsize = torch.empty((), dtype=dtype).element_size()
    buf = (C.c_byte * (numel * itemsize)).from_address(p.value)
    # wrap device memory through the CUDA array interface
    class _Wrap:
        pass
    w = _Wrap()
    typestr = {torch.float32: "<f4", torch.bfloat16: "<i2"}[dtype]
    w.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": typestr, "data": (p.value, False),
                                  "version": 2}
    del buf
    t = torch.as_tensor(w, device="cuda")
    return t.view(torch.bfloat16) if dtype == torch.bfloat16 else t


def dq_calib_launch_count(h) -> int:
    return int(load_library().dq_calib_launch_count(h))


def dq_calib_destroy(h):
    load_library().dq_calib_destroy(h)


def dq_rotate_apply(X, R, Y, stream=None):
    """Y = X R.  X, Y: CUDA [n, d] float32 or bfloat16 (same dtype); R: CUDA float32 [d, d]."""
    import torch
    assert X.is_cuda and R.is_cuda and Y.is_cuda and X.dtype == Y.dtype and R.dtype == torch.float32
    assert X.stride(1) == 1 and Y.stride(1) == 1 and R.is_contiguous()
    n, d = X.shape
    _check(load_library().dq_rotate_apply(_ptr(X), DQ_FP32 if X.dtype == torch.float32 else DQ_BF16, n, d,
                                          X.stride(0), _ptr(R), _ptr(Y), Y.stride(0), _stream_ptr(stream)),
           "dq_rotate_apply")


def dq_rotate_apply_static(X, R, Y, stream=None):
    """Y = X R for bfloat16 X, Y ([n, d]) and float32 R ([d, d]) without any device allocation:
    for callers whose memory is all spoken for (see include/dartquant.h).  d <= 2048."""
    import torch
    assert X.is_cuda and R.is_cuda and Y.is_cuda and R.dtype == torch.float32
    assert X.dtype == torch.bfloat16 and Y.dtype == torch.bfloat16
    assert X.stride(1) == 1 and Y.stride(1) == 1 and R.is_contiguous()
    n, d = X.shape
    _check(load_library().dq_rotate_apply_static(_ptr(X), n, d, X.stride(0), _ptr(R), _ptr(Y), Y.stride(0),
                                                 _stream_ptr(stream)), "dq_rotate_apply_static")


def dq_gather_tokens(X, seed: int, first: int, count: int, out, stream=None):
    """out[i] = X[pi_seed(first + i)]: seeded sampling of token rows without replacement.
    X: CUDA [n, d] float32 or bfloat16; out: CUDA [count, d] of the same dtype."""
    import torch
    assert X.is_cuda and out.is_cuda and X.dtype == out.dtype and X.dim() == 2 and out.dim() == 2
    n, d = X.shape
    _check(load_library().dq_gather_tokens(_ptr(X), DQ_FP32 if X.dtype == torch.float32 else DQ_BF16, n, d,
                                           X.stride(0), seed, first, count, _ptr(out), out.stride(0),
                                           _stream_ptr(stream)), "dq_gather_tokens")


def dq_eval_rotation(X, R, tau: float, bits: int, stream=None):
    """(number of outliers |o| > tau, mean squared per-token asymmetric quantisation error) of O = X R.
    X: CUDA [n, d] float32 or bfloat16; R: CUDA float32 [d, d].  Synchronises to read the result."""
    import torch
    assert X.is_cuda and R.is_cuda and R.dtype == torch.float32 and X.dim() == 2
    assert X.stride(1) == 1 and R.is_contiguous()
    n, d = X.shape
    out = torch.zeros(2, dtype=torch.float64, device=X.device)
    _check(load_library().dq_eval_rotation(_ptr(X), DQ_FP32 if X.dtype == torch.float32 else DQ_BF16, n, d,
                                           X.stride(0), _ptr(R), tau, bits, _ptr(out), _stream_ptr(stream)),
           "dq_eval_rotation")
    res = out.cpu()
    return int(round(float(res[0]))), float(res[1])


def dq_version() -> str:
    return load_library().dq_version().decode()
