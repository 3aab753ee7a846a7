"""Randomized permuted block-Hadamard rotation -- oracle (test infrastructure).

Eq. 9 of the paper:  Pi_d = blkdiag(H_h D_1, ..., H_h D_{d/h}) * P_pi, with
H_h the h x h Walsh-Hadamard matrix scaled so its entries are +-1/sqrt(h)
(supplement A, "Setup"), D_j Rademacher sign diagonals and P_pi the matrix of
a uniform random permutation.  The permutation acts first (Sec. 4.4).

Readings where the paper is silent:
  * P_pi is a gather: (P_pi x)_k = x[pi(k)].
  * the signs are indexed by the position AFTER the permutation.
  * H_h is in natural (Sylvester) order: H[l, i] = (-1)^popcount(l & i).
  * the random draw is specified here: SplitMix64 seeded from
    (seed, dim, block), Fisher-Yates with rejection sampling for pi, then one
    64-bit word per 64 signs.

Everything is the dense definition: no fast transform is used.
"""
import numpy as np

_M64 = (1 << 64) - 1


class SplitMix64:
    """Steele/Lea/Flood SplitMix64; state advances by the golden-ratio odd constant."""

    def __init__(self, state):
        self.state = state & _M64

    def next(self):
        self.state = (self.state + 0x9E3779B97F4A7C15) & _M64
        z = self.state
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
        return z ^ (z >> 31)

    def bounded(self, n):
        """Uniform integer in [0, n) by rejection (no modulo bias)."""
        thr = ((1 << 64) - n) % n
        while True:
            r = self.next()
            if r >= thr:
                return r % n


def make_rpbh(dim, block, seed):
    """Draw (pi, sigma) for Pi_d.  Returns (perm int32[dim], signs int8[dim] in {+1,-1})."""
    if block <= 0 or block & (block - 1) or dim % block:
        raise ValueError("block must be a power of two dividing dim")
    g = SplitMix64(seed ^ ((dim & 0xFFFFFFFF) << 32) ^ block)
    p = list(range(dim))
    for i in range(dim - 1, 0, -1):
        j = g.bounded(i + 1)
        p[i], p[j] = p[j], p[i]
    words = [g.next() for _ in range((dim + 63) // 64)]
    signs = np.empty(dim, dtype=np.int8)
    for k in range(dim):
        signs[k] = -1 if (words[k // 64] >> (k % 64)) & 1 else 1
    return np.asarray(p, dtype=np.int32), signs


def hadamard(h):
    """Unnormalised Sylvester Walsh-Hadamard matrix, entries +-1 (int64)."""
    idx = np.arange(h)
    anded = idx[:, None] & idx[None, :]
    pop = np.zeros_like(anded)
    v = anded.copy()
    while v.any():
        pop += v & 1
        v >>= 1
    return 1 - 2 * (pop & 1)


def dense_pi(dim, block, perm, signs):
    """The d x d matrix of Eq. 9 (float64).  Pi[j*h + l, pi(j*h + i)] = H[l,i] * sigma_{jh+i} / sqrt(h)."""
    H = hadamard(block).astype(np.float64) / np.sqrt(float(block))
    P = np.zeros((dim, dim), dtype=np.float64)
    for j in range(dim // block):
        for i in range(block):
            k = j * block + i
            P[j * block:(j + 1) * block, perm[k]] = H[:, i] * float(signs[k])
    return P


def rotate_rows(X, block, perm, signs):
    """x' = Pi_d x for every row of X (float64 [N, d]) -> float64 [N, d].

    Steps of Eq. 9 in order: permutation gather, sign flip, per-block dense
    Hadamard product with the 1/sqrt(h) scale.
    """
    X = np.asarray(X, dtype=np.float64)
    n, d = X.shape
    y = X[:, perm] * signs.astype(np.float64)[None, :]
    H = hadamard(block).astype(np.float64)
    yb = y.reshape(n, d // block, block)
    zb = np.einsum("li,nji->njl", H, yb) / np.sqrt(float(block))
    return zb.reshape(n, d)
