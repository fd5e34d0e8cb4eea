"""Seeded synthetic calibration inputs (shared by the CUDA path and the tests).

This module holds none of the method's arithmetic: it only draws random numbers
with a counter-based generator (numpy's Philox), shapes them like the LLM
activations the paper calibrates on (zero mean, heavy tails, a few massive
outlier channels: Sec. 4.2 and the activation-statistics appendix) and rounds
them once to the storage type.  The five workloads are the ones the benchmark
contract names; real calibration activations are not available offline, so
these stand in for them.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np


# --------------------------------------------------------------------------
# bf16 storage helpers (numpy has no bfloat16): round-to-nearest-even on the
# top 16 bits of an IEEE float32.
# --------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounding = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + rounding) >> 16).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


@dataclass(frozen=True)
class CalibWorkload:
    name: str
    d: int                    # channels (size of the rotation)
    n_tokens: int             # tokens per problem
    batch: int                # independent problems (heads)
    x_dtype: str              # "fp32" | "bf16"
    dist: str                 # "normal" | "student_t" | "laplace"
    nu: float                 # degrees of freedom for student_t
    n_outlier_channels: int   # per problem
    outlier_scale: tuple      # (lo, hi): uniform in [lo, hi]; lo == hi -> constant
    token_lognormal_sigma: float
    z0: str                   # "eye_noise" | "hadamard" | "hadamard_kron5"
    lr: float
    steps: int
    seed: int = 0
    path: str = "bf16_tc"     # "fp32" | "bf16_tc"


# The benchmark's five workloads.  Learning rates of 2-5 follow the paper's
# hyper-parameter table (R1 of the 7B / 13B / 70B models, R2 for per-head).
WORKLOADS = {
    "c1_tiny": CalibWorkload("c1_tiny", 256, 2048, 1, "fp32", "normal", 0.0, 4, (50.0, 50.0),
                             0.0, "eye_noise", 1e-2, 20, 0, "fp32"),
    "c2_7b": CalibWorkload("c2_7b", 4096, 16384, 1, "bf16", "student_t", 3.0, 41, (20.0, 100.0),
                           0.0, "hadamard", 2e-3, 100, 0),
    "c3_heads": CalibWorkload("c3_heads", 128, 16384, 32, "bf16", "laplace", 0.0, 2, (30.0, 30.0),
                              0.0, "hadamard", 1e-3, 200, 0),
    "c4_13b": CalibWorkload("c4_13b", 5120, 32768, 1, "bf16", "student_t", 3.0, 26, (50.0, 50.0),
                            0.0, "hadamard_kron5", 1e-2, 100, 0),
    "c5_70b": CalibWorkload("c5_70b", 8192, 65536, 1, "bf16", "student_t", 2.5, 25, (100.0, 100.0),
                            0.5, "hadamard", 1e-3, 100, 0),
}


def scaled(w: CalibWorkload, **kw) -> CalibWorkload:
    """A smaller / altered copy of a workload (same recipe, other sizes)."""
    from dataclasses import replace
    return replace(w, **kw)


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed, stream]))


def _draw(rng, dist, nu, shape):
    if dist == "normal":
        return rng.standard_normal(shape, dtype=np.float32)
    if dist == "student_t":
        return rng.standard_t(nu, size=shape).astype(np.float32)
    if dist == "laplace":
        return rng.laplace(0.0, 1.0, size=shape).astype(np.float32)
    raise ValueError(dist)


def outlier_channels(w: CalibWorkload, problem: int = 0):
    """(channel indices, scales) of the seeded outlier channels of one problem."""
    rng = _rng(w.seed, 1000 + problem)
    idx = np.sort(rng.choice(w.d, size=w.n_outlier_channels, replace=False))
    lo, hi = w.outlier_scale
    sc = rng.uniform(lo, hi, size=w.n_outlier_channels) if hi > lo else np.full(w.n_outlier_channels, lo)
    return idx, sc.astype(np.float32)


def gen_activations(w: CalibWorkload, chunk_rows: int = 8192) -> np.ndarray:
    """X as stored: float32 [batch, N, d] for fp32 workloads, bf16 bit patterns
    (uint16) [batch, N, d] for bf16 workloads.  batch == 1 keeps the axis."""
    out_dtype = np.float32 if w.x_dtype == "fp32" else np.uint16
    X = np.empty((w.batch, w.n_tokens, w.d), dtype=out_dtype)
    for b in range(w.batch):
        idx, sc = outlier_channels(w, b)
        rng = _rng(w.seed, 1 + b)
        rng_tok = _rng(w.seed, 500000 + b)
        for r0 in range(0, w.n_tokens, chunk_rows):
            r1 = min(w.n_tokens, r0 + chunk_rows)
            blk = _draw(rng, w.dist, w.nu, (r1 - r0, w.d))
            blk[:, idx] *= sc[None, :]
            if w.token_lognormal_sigma > 0.0:
                s = rng_tok.lognormal(0.0, w.token_lognormal_sigma, size=r1 - r0).astype(np.float32)
                blk *= s[:, None]
            X[b, r0:r1] = blk if w.x_dtype == "fp32" else f32_to_bf16_bits(blk)
    return X


def activations_as_f32(w: CalibWorkload, X: np.ndarray) -> np.ndarray:
    """Exact float32 values of the stored activations."""
    return X if w.x_dtype == "fp32" else bf16_bits_to_f32(X).reshape(X.shape)


def sylvester_hadamard(n: int) -> np.ndarray:
    """+-1 Sylvester matrix of order n = 2^k (float32)."""
    assert n > 0 and (n & (n - 1)) == 0, "Sylvester construction needs a power of two"
    H = np.ones((1, 1), dtype=np.float32)
    while H.shape[0] < n:
        H = np.block([[H, H], [H, -H]])
    return H


def _givens_orthogonal(k: int, rng) -> np.ndarray:
    """A seeded k x k orthogonal matrix as a product of plane rotations."""
    Q = np.eye(k, dtype=np.float64)
    for i in range(k):
        for j in range(i + 1, k):
            th = rng.uniform(0.0, 2.0 * np.pi)
            Gm = np.eye(k)
            Gm[i, i] = Gm[j, j] = np.cos(th)
            Gm[i, j] = -np.sin(th)
            Gm[j, i] = np.sin(th)
            Q = Q @ Gm
    return Q


def gen_latent_init(w: CalibWorkload) -> np.ndarray:
    """Z0, float32 [batch, d, d].

    "hadamard": a random Hadamard matrix H diag(+-1) / sqrt(d) (the paper's
    initialisation).  "hadamard_kron5" (d = 5 * 2^k has no Sylvester form):
    (H_{d/5}/sqrt(d/5) kron O5) diag(+-1) with O5 a seeded 5x5 orthogonal.
    "eye_noise": I + 0.01 N(0,1)  (1e-2 read as the standard deviation).
    """
    Z = np.empty((w.batch, w.d, w.d), dtype=np.float32)
    for b in range(w.batch):
        rng = _rng(w.seed, 2000000 + b)
        if w.z0 == "eye_noise":
            Z[b] = np.eye(w.d, dtype=np.float32) + np.float32(0.01) * rng.standard_normal((w.d, w.d), dtype=np.float32)
        elif w.z0 == "hadamard":
            signs = rng.integers(0, 2, size=w.d).astype(np.float32) * 2.0 - 1.0
            Z[b] = sylvester_hadamard(w.d) * (signs[None, :] / np.float32(np.sqrt(w.d)))
        elif w.z0 == "hadamard_kron5":
            assert w.d % 5 == 0
            m = w.d // 5
            O5 = _givens_orthogonal(5, rng)
            signs = rng.integers(0, 2, size=w.d).astype(np.float64) * 2.0 - 1.0
            base = np.kron(sylvester_hadamard(m).astype(np.float64) / np.sqrt(m), O5)
            Z[b] = (base * signs[None, :]).astype(np.float32)
        else:
            raise ValueError(w.z0)
    return Z
