"""Pins for oracle/rpbh.py (Eq. 9 and supplement A of the paper)."""
import itertools
import os
import zlib

import numpy as np
import pytest
import scipy.linalg

from oracle import rpbh

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_splitmix64_published_vector():
    # first outputs of SplitMix64 from state 0 (widely published test vector)
    g = rpbh.SplitMix64(0)
    assert g.next() == 0xE220A8397B1DCDAF
    assert g.next() == 0x6E789E6AA1B965F4


@pytest.mark.parametrize("h", [1, 2, 4, 8, 64, 128, 256])
def test_hadamard_is_sylvester_and_orthogonal(h):
    H = rpbh.hadamard(h)
    assert set(np.unique(H)) <= {-1, 1}
    assert np.array_equal(H @ H.T, h * np.eye(h, dtype=H.dtype))       # H H^T = h I exactly
    assert np.array_equal(H, scipy.linalg.hadamard(h))                   # library Sylvester construction
    R = np.array([[1]])
    while R.shape[0] < h:                                                # recursive definition
        R = np.block([[R, R], [R, -R]])
    assert np.array_equal(H, R)


def test_generator_pins_from_spec():
    for line in open(os.path.join(GOLD, "rpbh_generator_pins.txt")):
        if line.startswith("#") or not line.strip():
            continue
        f = [s.strip() for s in line.split("|")]
        dim, block, seed = map(int, f[0].split())
        perm, signs = rpbh.make_rpbh(dim, block, seed)
        assert perm[:8].tolist() == list(map(int, f[1].split()))
        assert perm[-4:].tolist() == list(map(int, f[2].split()))
        word = sum(int(signs[k] == -1) << k for k in range(min(64, dim)))
        assert word == int(f[3], 16) & ((1 << min(64, dim)) - 1)
        assert zlib.crc32(perm.astype("<i4").tobytes()) == int(f[4], 16)
        assert zlib.crc32(signs.astype(np.int8).tobytes()) == int(f[5], 16)
        assert int((signs == -1).sum()) == int(f[6])


@pytest.mark.parametrize("dim,block,seed", [(8, 4, 0), (64, 16, 3), (256, 64, 1), (384, 128, 7), (768, 256, 2)])
def test_pi_is_orthogonal_and_matches_rowwise_transform(dim, block, seed):
    perm, signs = rpbh.make_rpbh(dim, block, seed)
    assert sorted(perm.tolist()) == list(range(dim))                     # bijection
    P = rpbh.dense_pi(dim, block, perm, signs)
    assert np.abs(P @ P.T - np.eye(dim)).max() < 1e-14                   # Pi Pi^T = I
    g = np.random.default_rng(seed)
    X = g.standard_normal((5, dim)) * 10.0 ** g.uniform(-3, 3, size=(5, 1))
    Z = rpbh.rotate_rows(X, block, perm, signs)
    assert np.allclose(Z, X @ P.T, rtol=0, atol=1e-12 * np.abs(X).max())
    nx, nz = np.linalg.norm(X, axis=1), np.linalg.norm(Z, axis=1)
    assert np.abs(nz / nx - 1).max() < 1e-13                             # ||Pi x|| = ||x||


def test_block_transform_is_an_involution():
    h = 64
    Hn = rpbh.hadamard(h) / np.sqrt(h)
    assert np.abs(Hn @ Hn - np.eye(h)).max() < 1e-14


def test_identity_permutation_unit_vector():
    dim, h = 32, 8
    perm = np.arange(dim, dtype=np.int32)
    signs = np.ones(dim, dtype=np.int8)
    x = np.zeros((1, dim)); x[0, 0] = 1.0
    z = rpbh.rotate_rows(x, h, perm, signs)[0]
    assert np.allclose(z[:h], 1 / np.sqrt(h), atol=1e-16) and np.all(z[h:] == 0)


def test_permutation_is_a_gather_and_signs_follow_it():
    # x = e_i must land in the block holding the position k with pi(k) = i, carrying sigma_k (P_pi acts first).
    dim, h = 64, 16
    perm, signs = rpbh.make_rpbh(dim, h, 5)
    H = rpbh.hadamard(h)
    for i in [0, 7, 33, 63]:
        x = np.zeros((1, dim)); x[0, i] = 2.0
        z = rpbh.rotate_rows(x, h, perm, signs)[0]
        k = int(np.where(perm == i)[0][0])
        j, col = divmod(k, h)
        expect = np.zeros(dim)
        expect[j * h:(j + 1) * h] = 2.0 * signs[k] * H[:, col] / np.sqrt(h)
        assert np.allclose(z, expect, atol=1e-15)


@pytest.mark.parametrize("h", [4, 8])
def test_conditional_variance_is_block_mass_over_h(h):
    # Lemma 1's proof: for a fixed permutation, Var over the signs of z^{(j)}_l equals M_j / h.
    dim = 2 * h
    g = np.random.default_rng(11)
    x = g.standard_normal(dim); x /= np.linalg.norm(x)
    perm = g.permutation(dim).astype(np.int32)
    y = x[perm]
    sums = np.zeros(dim); sq = np.zeros(dim)
    pats = list(itertools.product([1, -1], repeat=h))
    for pa in pats:
        s = np.array(pa + pa, dtype=np.int8)
        z = rpbh.rotate_rows(x[None, :], h, perm, s)[0]
        sums += z; sq += z * z
    mean, var = sums / len(pats), sq / len(pats)
    assert np.abs(mean).max() < 1e-14
    for j in range(2):
        Mj = np.sum(y[j * h:(j + 1) * h] ** 2)
        assert np.allclose(var[j * h:(j + 1) * h], Mj / h, atol=1e-14)


def test_mass_balancing_bound_of_lemma_2():
    # |M_j - 1/k| <= mu_inf sqrt((h/2) log(4k/delta)) for all j, w.p. >= 1 - delta/2 over pi (Eq. 12).
    dim, h, delta = 512, 64, 0.1
    k = dim // h
    g = np.random.default_rng(3)
    x = g.standard_normal(dim); x[::50] *= 4.0; x /= np.linalg.norm(x)
    mu = np.max(x * x)
    bound = mu * np.sqrt(h / 2 * np.log(4 * k / delta))
    bad = 0
    trials = 300
    for seed in range(trials):
        perm, _ = rpbh.make_rpbh(dim, h, seed)
        M = np.sum((x[perm] ** 2).reshape(k, h), axis=1)
        bad += bool(np.any(np.abs(M - 1 / k) > bound))
    assert bad <= delta / 2 * trials + 3 * np.sqrt(trials * delta / 2)


def test_fisher_yates_is_uniform_on_s4_and_signs_are_balanced():
    counts = {}
    minus = 0
    trials = 12000
    for seed in range(trials):
        perm, signs = rpbh.make_rpbh(4, 4, seed)
        counts[tuple(perm.tolist())] = counts.get(tuple(perm.tolist()), 0) + 1
        minus += int((signs == -1).sum())
    assert len(counts) == 24
    exp = trials / 24
    chi2 = sum((c - exp) ** 2 / exp for c in counts.values())
    assert chi2 < 60.0                       # 23 d.o.f.: P(chi2 > 60) ~ 4e-5
    assert abs(minus / (4 * trials) - 0.5) < 0.01
