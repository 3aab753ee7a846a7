"""Row-wise rotate -> norm -> nearest level -- oracle (test infrastructure, CPU, fp64).

Online activation path (Eq. 7-8, Algorithm 1 "Online"):
    x' = Pi_d x,   s = ||x'||_2,   x~' = x' / (s + eps),   eps = 1e-10,
    idx_k = index of the codebook level nearest to x~'_k.
Offline weight path (Eq. 4-6, Algorithm 1 "Offline"): the same steps on every
row w_i of W (W' = W Pi^T means w'_i = Pi w_i), with the row norm r'_i stored
in bf16 (Sec. 4.2).

Readings where the paper is silent: inputs are bf16 bit patterns taken as
exact reals; nearest level is evaluated as "number of cell boundaries strictly
below the value", so an exact tie goes to the lower index; the stored
activation norm is s itself (not s + eps); a zero weight row uses the same eps
guard as Eq. 7; the bf16 weight norm is RNE(fp32(r')).
"""
import numpy as np

from . import bf16 as _bf16
from . import rpbh as _rpbh

EPS = 1e-10


def nearest_level_bruteforce(t, centroids):
    """Eq. 3 literally: argmin_c |t - c| (first minimum on ties). t: any shape."""
    t = np.asarray(t, dtype=np.float64)
    dist = np.abs(t[..., None] - np.asarray(centroids, dtype=np.float64))
    return np.argmin(dist, axis=-1).astype(np.uint8)


def count_boundaries(t, boundaries):
    """#{ j : beta_j < t } for sorted cell boundaries (midpoints of adjacent levels)."""
    return np.searchsorted(np.asarray(boundaries, dtype=np.float64), np.asarray(t, dtype=np.float64),
                           side="left").astype(np.uint8)


def quantize_rows(x_bf16_bits, block, perm, signs, boundaries):
    """Algorithm 1 "Online" on every row.

    x_bf16_bits : uint16 [N, d] bf16 bit patterns
    Returns dict with
      idx      uint8  [N, d]  level index per rotated coordinate
      norm     float64 [N]    s = ||Pi x||
      rotated  float64 [N, d] x' = Pi x
      unit     float64 [N, d] x' / (s + eps)
    """
    X = _bf16.bf16_bits_to_f64(x_bf16_bits)
    Z = _rpbh.rotate_rows(X, block, perm, signs)
    s = np.sqrt(np.sum(Z * Z, axis=1))
    T = Z / (s + EPS)[:, None]
    return {"idx": count_boundaries(T, boundaries), "norm": s, "rotated": Z, "unit": T}


def quantize_weight_rows(w_bf16_bits, block, perm, signs, boundaries):
    """Algorithm 1 "Offline" on every row of W; adds the bf16-stored row norm."""
    out = quantize_rows(w_bf16_bits, block, perm, signs, boundaries)
    out["norm_bf16_bits"] = _bf16.f64_to_bf16_bits(out["norm"])
    return out
