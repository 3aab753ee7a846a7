"""Pins for oracle/codebook.py (Eq. 2-3, Sec. 4.5)."""
import math
import os

import numpy as np
import pytest
import scipy.integrate
import torch
from mpmath import mp, mpf

from oracle import bf16, codebook

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    for line in open(os.path.join(GOLD, name)):
        if line.startswith("#") or not line.strip():
            continue
        yield [s.strip() for s in line.split("|")]


def _fd(d):
    """Eq. 2 typed out directly, in float64 (independent of the oracle's closed-form integrals)."""
    lk = math.lgamma(d / 2) - math.lgamma((d - 1) / 2) - 0.5 * math.log(math.pi)
    return lambda t: math.exp(lk + (d - 3) / 2 * math.log1p(-t * t)) if abs(t) < 1 else 0.0


def test_generic_iteration_reproduces_classical_gaussian_tables():
    # Same Lloyd iteration, Gaussian density plugged in: must give Max's 1960 tables.
    mp.dps = 30
    phi = lambda t: mp.exp(-t * t / 2) / mp.sqrt(2 * mp.pi)
    mass = lambda a, b: (mp.erf(b / mp.sqrt(2)) - mp.erf(a / mp.sqrt(2))) / 2
    moment = lambda a, b: phi(a) - phi(b)
    for f in _rows("max1960_gaussian.txt"):
        bits = int(f[0])
        want_c = [float(v) for v in f[1].split()]
        want_b = [float(v) for v in f[2].split()]
        m = len(want_c)
        c, b = codebook.lloyd_iterate(mass, moment, mp.inf, [mpf(3) * (2 * j + 1) / (2 * m) for j in range(m)])
        for got, want in zip(c, want_c):
            assert abs(float(got) - want) <= 6e-4 * want          # 4 printed digits
        for got, want in zip(b, want_b):
            assert abs(float(got) - want) <= 6e-4 * want
        edges = [mpf(0)] + b + [mp.inf]
        mse = 1 - 2 * sum(mass(edges[j], edges[j + 1]) * c[j] ** 2 for j in range(m))
        assert abs(float(mse) - float(f[3])) <= 6e-4 * float(f[3])
        assert bits == int(math.log2(2 * m))


@pytest.mark.parametrize("d", [3, 4, 64, 1024, 12288])
def test_one_bit_closed_form(d):
    # 1 bit: the two levels are +-E|t| = +-Gamma(d/2) / (sqrt(pi) Gamma((d+1)/2))
    cb = codebook.lloyd_max(d, 1)
    want = math.exp(math.lgamma(d / 2) - math.lgamma((d + 1) / 2)) / math.sqrt(math.pi)
    assert cb.centroids.tolist() == pytest.approx([-want, want], rel=1e-13)
    assert cb.boundaries.tolist() == [0.0]


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_d3_marginal_is_uniform_so_codebook_is_uniform(bits):
    # f_3 is constant on [-1, 1]: the optimal quantiser is the uniform one.
    cb = codebook.lloyd_max(3, bits)
    L = 1 << bits
    assert np.allclose(cb.centroids, (2 * np.arange(L) + 1) / L - 1, rtol=0, atol=1e-14)
    assert np.allclose(cb.probs, 1.0 / L, atol=1e-15)
    assert cb.distortion == pytest.approx(1 - 3 * np.mean(((2 * np.arange(L) + 1) / L - 1) ** 2), rel=1e-12)


@pytest.mark.parametrize("d,bits", [(64, 3), (1024, 4), (3072, 2), (5120, 3)])
def test_lloyd_max_conditions_by_independent_quadrature(d, bits):
    cb = codebook.lloyd_max(d, bits)
    L = 1 << bits
    c, b = cb.centroids, cb.boundaries
    assert len(c) == L and len(b) == L - 1
    assert np.all(np.diff(c) > 0) and np.all(np.diff(b) > 0)
    assert np.array_equal(c, -c[::-1]) and np.array_equal(b, -b[::-1]) and b[L // 2 - 1] == 0.0
    assert np.allclose(b, (c[:-1] + c[1:]) / 2, rtol=1e-15, atol=1e-18)        # nearest-level boundaries
    f = _fd(d)
    edges = np.concatenate([[-1.0], b, [1.0]])
    sig = 1 / math.sqrt(d)
    tot_p = tot_e = 0.0
    for j in range(L):
        lo, hi = max(edges[j], -14 * sig), min(edges[j + 1], 14 * sig)       # tails beyond 14 sigma are < 1e-40
        p = scipy.integrate.quad(f, lo, hi, epsabs=0, epsrel=1e-13, limit=200)[0]
        m1 = scipy.integrate.quad(lambda t: t * f(t), lo, hi, epsabs=0, epsrel=1e-13, limit=200)[0]
        e2 = scipy.integrate.quad(lambda t: (t - c[j]) ** 2 * f(t), lo, hi, epsabs=0, epsrel=1e-13, limit=200)[0]
        assert m1 / p == pytest.approx(c[j], rel=2e-10)                        # centroid = conditional mean
        assert p == pytest.approx(cb.probs[j], rel=2e-10)
        tot_p += p; tot_e += e2
    assert tot_p == pytest.approx(1.0, abs=1e-10)
    assert d * tot_e == pytest.approx(cb.distortion, rel=1e-8)
    assert float(np.dot(cb.probs, c)) == pytest.approx(0.0, abs=1e-17)


def test_converges_to_gaussian_tables_from_below_as_d_grows():
    want = [float(v) for v in next(f for f in _rows("max1960_gaussian.txt") if f[0] == "4")[1].split()]
    prev_gap = None
    for d in (256, 1024, 13824):
        cb = codebook.lloyd_max(d, 4)
        got = math.sqrt(d) * cb.centroids[8:]
        assert np.all(np.abs(got / want - 1) < 3.0 / d + 5e-4)
        gap = 2.732589570995 - got[-1]                       # outer level approaches from below
        assert gap > 0 and (prev_gap is None or gap < prev_gap)
        prev_gap = gap


def test_against_independent_40_digit_values():
    for f in _rows("fd_codebooks_40digit.txt"):
        d, bits = map(int, f[0].split())
        cb = codebook.lloyd_max(d, bits)
        want = np.array([float(v) for v in f[1].split()])
        got = math.sqrt(d) * cb.centroids[(1 << bits) // 2:]
        assert np.abs(got / want - 1).max() < 2e-12
        assert cb.distortion == pytest.approx(float(f[2]), rel=2e-9)


def test_bf16_rounding_matches_an_independent_converter():
    g = np.random.default_rng(0)
    x = np.concatenate([g.standard_normal(20000) * 10.0 ** g.uniform(-6, 6, 20000),
                        codebook.lloyd_max(1024, 4).centroids, [0.0, -0.0, 1.0, 1.00390625, 1.01171875]])
    ours = bf16.f64_to_bf16_bits(x)
    ref = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ours, ref)
    back = bf16.bf16_bits_to_f64(ours)
    assert np.array_equal(back, torch.from_numpy(ref.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy())
    # ties go to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert bf16.f64_to_bf16_bits(np.array([1.00390625]))[0] == 0x3F80
    assert bf16.f64_to_bf16_bits(np.array([1.01171875]))[0] == 0x3F82


def test_decode_tables():
    cb = codebook.lloyd_max(1024, 4)
    assert cb.boundaries_f32.dtype == np.float32 and cb.centroids_bf16_bits.dtype == np.uint16
    assert np.abs(cb.centroids_decoded / cb.centroids - 1).max() <= 2.0 ** -8
    assert np.array_equal(cb.centroids_decoded, -cb.centroids_decoded[::-1])


@pytest.mark.parametrize("d", [3072, 5120])
def test_stored_6bit_codebook_satisfies_the_lloyd_max_conditions(d):
    """The 64-level codebooks under tests/golden/ (minutes of oracle time each, hence stored) are checked against the
    defining conditions of Eq. 3's codebook with an independent quadrature: every centroid is the conditional mean of
    f_d (Eq. 2) over its cell, whose edges are the midpoints of neighbouring centroids; the table is antisymmetric."""
    import os
    from scipy import integrate
    path = os.path.join(os.path.dirname(__file__), "golden", f"lloyd_max_d{d}_b6.txt")
    c = np.array([float(x) for x in open(path).read().split("\n") if x and not x.startswith("#")])
    assert c.shape == (64,) and np.all(np.diff(c) > 0)
    assert np.allclose(c, -c[::-1], rtol=1e-12, atol=0)
    edges = np.concatenate([[-1.0], 0.5 * (c[:-1] + c[1:]), [1.0]])
    e = 0.5 * (d - 3)
    sig = d ** -0.5

    def f(t):
        return np.exp(e * np.log1p(-t * t))
    for j in range(32, 64):
        lo, hi = edges[j], min(edges[j + 1], 12 * sig)
        mass = integrate.quad(f, lo, hi, epsabs=0, epsrel=1e-12)[0]
        mom = integrate.quad(lambda t: t * f(t), lo, hi, epsabs=0, epsrel=1e-12)[0]
        assert abs(mom / mass - c[j]) <= 1e-8 * c[-1]
