"""Lloyd-Max scalar codebook for the sphere-coordinate marginal -- oracle
(test infrastructure, CPU only, arbitrary precision via mpmath).

Eq. 2: a coordinate of a uniformly random unit vector in R^d has density
    f_d(t) = Gamma(d/2) / (sqrt(pi) Gamma((d-1)/2)) * (1 - t^2)^((d-3)/2),  t in [-1, 1].
Eq. 3 / Sec. 4.5: the codebook C^(d,b) is the MSE-optimal (Lloyd-Max) set of
2^b levels for f_d; quantisation maps t to the nearest level.

The Lloyd-Max conditions are
    boundary  beta_j = (c_j + c_{j+1}) / 2                    (nearest-level rule)
    centroid  c_j    = int t f_d dt / int f_d dt over its cell (conditional mean)
and the plain Lloyd iteration alternates the two until it stops moving.
f_d is even, so the optimal codebook is antisymmetric; the iteration is
carried on the positive half (cells [0, beta_1], ..., [beta_{M-1}, 1], M = 2^b/2)
and mirrored.  f_d is log-concave for d >= 3, so the fixed point is unique and
the starting point does not matter.

Closed forms used for the two integrals (the normalising constant cancels in c_j):
    int_0^t f_d = 1/2 * I_{t^2}(1/2, (d-1)/2)        (regularised incomplete beta)
    int_a^b t (1-t^2)^((d-3)/2) dt = [(1-a^2)^((d-1)/2) - (1-b^2)^((d-1)/2)] / (d-1)

Readings where the paper is silent: the codebook is fit to the exact f_d (not
its Gaussian approximation); levels are numbered in ascending order; the fp32
boundary table is the fp64 value rounded once, the bf16 level table is rounded
fp64 -> fp32 -> bf16.
"""
import numpy as np
from mpmath import mp, mpf

from . import bf16 as _bf16

_DPS = 40


def lloyd_iterate(mass, moment, upper, start, tol=mpf(10) ** -24, max_iter=20000):
    """Plain Lloyd iteration on the positive half of an even density.

    mass(a, b)   -> int_a^b f        (any common positive factor allowed)
    moment(a, b) -> int_a^b t f(t)   (same factor)
    upper        -> right end of the support (mp.inf allowed if mass/moment accept it)
    start        -> increasing positive initial levels
    Returns (levels, inner boundaries) as lists of mpf; boundary 0 (at t = 0) is implied.
    """
    c = [mpf(v) for v in start]
    m = len(c)
    for _ in range(max_iter):
        edges = [mpf(0)] + [(c[j] + c[j + 1]) / 2 for j in range(m - 1)] + [upper]
        new = [moment(edges[j], edges[j + 1]) / mass(edges[j], edges[j + 1]) for j in range(m)]
        step = max(abs(new[j] - c[j]) for j in range(m))
        c = new
        if step <= tol * c[-1]:
            break
    else:
        raise RuntimeError("Lloyd iteration did not converge")
    return c, [(c[j] + c[j + 1]) / 2 for j in range(m - 1)]


def _fd_mass(d):
    b = (mpf(d) - 1) / 2

    def half_cdf(t):          # int_0^t f_d
        if t >= 1:
            return mpf(1) / 2
        if t <= 0:
            return mpf(0)
        return mp.betainc(mpf(1) / 2, b, 0, t * t, regularized=True) / 2

    return lambda lo, hi: half_cdf(hi) - half_cdf(lo)


def _fd_moment(d):
    # int_a^b t f_d(t) dt with the same normalisation as _fd_mass
    logk = mp.loggamma(mpf(d) / 2) - mp.loggamma((mpf(d) - 1) / 2) - mp.log(mp.pi) / 2
    k = mp.e ** logk
    p = (mpf(d) - 1) / 2

    def prim(t):
        return (1 - t * t) ** p if t < 1 else mpf(0)

    return lambda lo, hi: k * (prim(lo) - prim(hi)) / (d - 1)


class Codebook:
    """Result of lloyd_max(d, bits): all tables a quantiser or a decoder needs."""

    def __init__(self, dim, bits, levels_mp, bounds_mp, probs_mp):
        self.dim, self.bits = dim, bits
        self.levels_mp, self.bounds_mp, self.probs_mp = levels_mp, bounds_mp, probs_mp
        self.centroids = np.array([float(v) for v in levels_mp], dtype=np.float64)
        self.boundaries = np.array([float(v) for v in bounds_mp], dtype=np.float64)
        self.probs = np.array([float(v) for v in probs_mp], dtype=np.float64)
        self.boundaries_f32 = self.boundaries.astype(np.float32)
        self.centroids_bf16_bits = _bf16.f64_to_bf16_bits(self.centroids)
        self.centroids_decoded = _bf16.bf16_bits_to_f64(self.centroids_bf16_bits)
        # d * MSE = d * (E t^2 - sum p c^2), with E t^2 = 1/d on the unit sphere
        self.distortion = float(1 - dim * sum(p * c * c for p, c in zip(probs_mp, levels_mp)))


_CACHE = {}


def lloyd_max(dim, bits):
    """Lloyd-Max codebook C^(dim,bits) of Eq. 3 for the density f_dim of Eq. 2."""
    key = (dim, bits)
    if key in _CACHE:
        return _CACHE[key]
    if dim < 3 or bits < 1 or bits > 8:
        raise ValueError("need dim >= 3 and 1 <= bits <= 8")
    old = mp.dps
    mp.dps = _DPS
    try:
        m = (1 << bits) // 2
        sigma = 1 / mp.sqrt(dim)
        span = min(3 * sigma, mpf(1))                      # start inside the support
        start = [span * (2 * j + 1) / (2 * m) for j in range(m)]
        mass, moment = _fd_mass(dim), _fd_moment(dim)
        pos, inner = lloyd_iterate(mass, moment, mpf(1), start)
        edges = [mpf(0)] + inner + [mpf(1)]
        ppos = [mass(edges[j], edges[j + 1]) for j in range(m)]
        levels = [-v for v in reversed(pos)] + pos
        bounds = [-v for v in reversed(inner)] + [mpf(0)] + inner
        probs = list(reversed(ppos)) + ppos
        cb = Codebook(dim, bits, levels, bounds, probs)
    finally:
        mp.dps = old
    _CACHE[key] = cb
    return cb
