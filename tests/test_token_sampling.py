"""Seeded token sampling / mini-batch selection (Algorithm 1: X <- token_sampling(X)).
CPU: pins of the oracle (published known-answer vectors of the generator, bijection, uniformity).
GPU: the gather kernel is bit-exact against the oracle."""
import os

import numpy as np
import pytest

import oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def test_philox_known_answer_vectors():
    rows = [l.split() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        w = [int(v, 16) for v in r]
        assert list(orc.philox4x32_10(w[0:4], w[4:6])) == w[6:10]


@pytest.mark.parametrize("n", [1, 2, 3, 16, 17, 100, 1000, 4097])
def test_permutation_is_a_bijection_and_depends_on_the_seed(n):
    p = [orc.permute_index(i, n, 12345) for i in range(n)]
    assert sorted(p) == list(range(n))
    if n >= 100:
        q = [orc.permute_index(i, n, 12346) for i in range(n)]
        assert p != q and sum(a == b for a, b in zip(p, q)) < n // 10


def test_samples_are_uniform_over_rows():
    # every row should be the first sample about equally often over many seeds (n = 20, 4000 seeds:
    # expected 200 per row, standard deviation ~14)
    n, counts = 20, np.zeros(20)
    for seed in range(4000):
        counts[orc.permute_index(0, n, seed)] += 1
    assert counts.min() > 140 and counts.max() < 260


def test_minibatch_windows_partition_the_tokens():
    X = np.arange(50, dtype=np.float32)[:, None] * np.ones((1, 4), dtype=np.float32)
    batches = [orc.gather_tokens(X, 9, first, 10) for first in range(0, 50, 10)]
    seen = np.concatenate([b[:, 0] for b in batches])
    assert sorted(seen.tolist()) == list(range(50))


# --------------------------------------------------------------------------------------------- GPU
@pytest.mark.gpu
@pytest.mark.parametrize("n,d,dtype,pad", [(1000, 64, "fp32", 0), (4097, 128, "bf16", 8), (300, 256, "bf16", 0),
                                           (65536, 128, "bf16", 0)])
def test_gather_kernel_is_bit_exact(n, d, dtype, pad):
    import torch
    import paper_2511_04063_b200 as dq
    rng = np.random.default_rng(n)
    ld = d + pad
    if dtype == "fp32":
        host = rng.standard_normal((n, ld)).astype(np.float32)
        X = torch.from_numpy(host).cuda()[:, :d]
    else:
        host = rng.integers(0, 2 ** 15, size=(n, ld)).astype(np.int16)          # any bit patterns
        X = torch.from_numpy(host).cuda().view(torch.bfloat16)[:, :d]
    for seed, first, count in [(7, 0, min(n, 257)), (2 ** 40 + 3, n - 100, 100), (5, 13, 0)]:
        out = torch.zeros((max(count, 1), d + pad), dtype=X.dtype, device="cuda")[:, :d]
        dq.dq_gather_tokens(X, seed, first, count, out)          # count == 0: a no-op
        torch.cuda.synchronize()
        if count == 0:
            continue
        ref = orc.gather_tokens(host[:, :d], seed, first, count)
        got = out[:count].contiguous().view(torch.int16 if dtype == "bf16" else torch.float32).cpu().numpy()
        assert np.array_equal(got, ref)


@pytest.mark.gpu
def test_gather_rejects_bad_arguments():
    import ctypes as C
    import torch
    import paper_2511_04063_b200 as dq
    lib = dq.load_library()
    X = torch.zeros((64, 64), device="cuda")
    out = torch.zeros((8, 64), device="cuda")
    p = lambda t: C.c_void_p(t.data_ptr())
    assert lib.dq_gather_tokens(p(X), dq.DQ_FP32, 64, 64, 64, 1, 60, 8, p(out), 64, None) == dq.DQ_ERR_INVALID_ARG
    assert lib.dq_gather_tokens(None, dq.DQ_FP32, 64, 64, 64, 1, 0, 8, p(out), 64, None) == dq.DQ_ERR_INVALID_ARG
    assert lib.dq_gather_tokens(p(X), dq.DQ_FP32, 64, 62, 64, 1, 0, 8, p(out), 64, None) == dq.DQ_ERR_UNSUPPORTED


@pytest.mark.gpu
def test_minibatch_step_equals_step_on_the_gathered_batch():
    """Gather a mini-batch into the buffer the handle borrows, refresh, step: same loss as a handle
    created on that batch."""
    import torch
    import paper_2511_04063_b200 as dq
    from paper_2511_04063_b200 import inputs as gen
    w = gen.scaled(gen.WORKLOADS["c2_7b"], d=256, n_tokens=4096, n_outlier_channels=3)
    Xfull = torch.from_numpy(gen.gen_activations(w)[0].view(np.int16)).cuda().view(torch.bfloat16)
    Z0 = torch.from_numpy(gen.gen_latent_init(w)).cuda()
    nb = 1024
    batch = torch.empty((nb, w.d), dtype=torch.bfloat16, device="cuda")
    dq.dq_gather_tokens(Xfull, 3, 0, nb, batch)
    h = dq.dq_calib_init(batch, Z0, lr=w.lr, path=dq.DQ_PATH_BF16_TC)
    l0 = torch.empty((1, 1), device="cuda")
    dq.dq_calib_step(h, 1, l0)
    dq.dq_calib_set_latent(h, Z0)
    dq.dq_gather_tokens(Xfull, 3, nb, nb, batch)                  # next window, in place
    dq.dq_calib_refresh_inputs(h)
    l1 = torch.empty((1, 1), device="cuda")
    dq.dq_calib_step(h, 1, l1)
    batch2 = batch.clone()
    h2 = dq.dq_calib_init(batch2, Z0, lr=w.lr, path=dq.DQ_PATH_BF16_TC)
    l2 = torch.empty((1, 1), device="cuda")
    dq.dq_calib_step(h2, 1, l2)
    assert dq.dq_calib_status(h) == dq.DQ_OK and dq.dq_calib_status(h2) == dq.DQ_OK
    assert float(l1) == float(l2) and float(l0) != float(l1)
    dq.dq_calib_destroy(h); dq.dq_calib_destroy(h2)
