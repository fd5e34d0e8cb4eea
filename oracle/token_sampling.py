"""Plain oracle of seeded token sampling / mini-batch selection (Algorithm 1: X <- token_sampling(X);
the appendix on hyper-parameters: a fraction of the tokens, mini-batches over several epochs).

TEST INFRASTRUCTURE: never imported by the product path.

Reading (the paper does not say how tokens are drawn): uniform sampling WITHOUT replacement, given
by a seeded pseudo-random permutation pi of the token indices [0, n): the sample of size k is
X[pi(0)], ..., X[pi(k-1)]; mini-batches are consecutive windows of pi; another epoch uses another
seed.  pi is a balanced Feistel network on 2w bits (2^(2w) >= n) with cycle walking (apply the
network again while the result is >= n: a bijection of [0, n)), whose round function is the
counter-based generator Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as
easy as 1, 2, 3", SC 2011), written here from its published definition.
"""
from __future__ import annotations

import numpy as np

M0, M1 = 0xD2511F53, 0xCD9E8D57          # Philox4x32 multipliers
W0, W1 = 0x9E3779B9, 0xBB67AE85          # Weyl key increments
MASK = 0xFFFFFFFF
FEISTEL_ROUNDS = 4


def philox4x32_10(counter, key):
    """counter: 4 uint32, key: 2 uint32 -> 4 uint32 (ten rounds)."""
    c0, c1, c2, c3 = (int(v) & MASK for v in counter)
    k0, k1 = (int(v) & MASK for v in key)
    for _ in range(10):
        p0, p1 = M0 * c0, M1 * c2
        hi0, lo0, hi1, lo1 = p0 >> 32, p0 & MASK, p1 >> 32, p1 & MASK
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0) & MASK, lo1, (hi0 ^ c3 ^ k1) & MASK, lo0
        k0, k1 = (k0 + W0) & MASK, (k1 + W1) & MASK
    return c0, c1, c2, c3


def _half_bits(n: int) -> int:
    w = 1
    while (1 << (2 * w)) < n:
        w += 1
    return w


def permute_index(i: int, n: int, seed: int) -> int:
    """pi_seed(i) for 0 <= i < n."""
    w = _half_bits(n)
    mask = (1 << w) - 1
    x = i
    while True:
        left, right = x >> w, x & mask
        for r in range(FEISTEL_ROUNDS):
            f = philox4x32_10((right, r, 0, 0), (seed & MASK, (seed >> 32) & MASK))[0] & mask
            left, right = right, left ^ f
        x = (left << w) | right
        if x < n:
            return x


def gather_tokens(X: np.ndarray, seed: int, first: int, count: int) -> np.ndarray:
    """Rows X[pi_seed(first)], ..., X[pi_seed(first + count - 1)]."""
    n = X.shape[0]
    idx = [permute_index(first + i, n, seed) for i in range(count)]
    return X[np.asarray(idx, dtype=np.int64)]
