"""Pins for oracle/quantize.py and oracle/qlinear.py (Eq. 4-8, Algorithm 1)."""
import math

import numpy as np
import pytest

from oracle import bf16, codebook, qlinear, quantize, rpbh
from paper_2607_02461_b200 import synth


def test_boundary_count_equals_bruteforce_nearest_level():
    cb = codebook.lloyd_max(256, 4)
    g = np.random.default_rng(1)
    t = np.concatenate([g.standard_normal(20000) / 16, [0.0, -0.0, 1.0, -1.0],
                        cb.centroids, cb.boundaries + 1e-12, cb.boundaries - 1e-12])   # |t-c| itself rounds at ~1e-17
    assert np.array_equal(quantize.count_boundaries(t, cb.boundaries),
                          quantize.nearest_level_bruteforce(t, cb.centroids))
    # exactly on a boundary both neighbours are nearest; the oracle's rule picks the lower index.
    # (The midpoint is compared in float arithmetic, so only assert where |t-c| ties exactly.)
    on = quantize.count_boundaries(cb.boundaries, cb.boundaries)
    assert quantize.count_boundaries(np.array([5e-324, -5e-324, 0.0, -0.0]), cb.boundaries).tolist() == [8, 7, 7, 7]
    assert np.array_equal(on, np.arange(15))


@pytest.mark.parametrize("dim,block,bits", [(256, 64, 4), (384, 128, 3), (512, 256, 2)])
def test_rowwise_quantiser_invariants(dim, block, bits):
    perm, signs = rpbh.make_rpbh(dim, block, 0)
    cb = codebook.lloyd_max(dim, bits)
    xb = synth.activations(12, dim, seed=5)
    out = quantize.quantize_rows(xb, block, perm, signs, cb.boundaries)
    X = bf16.bf16_bits_to_f64(xb)
    assert np.allclose(out["norm"], np.linalg.norm(X, axis=1), rtol=1e-13)            # s = ||Pi x|| = ||x||
    assert np.allclose(np.sum(out["rotated"] ** 2, axis=1), out["norm"] ** 2, rtol=1e-13)
    P = rpbh.dense_pi(dim, block, perm, signs)                                         # dense route of Eq. 7
    Zd = X @ P.T
    sd = np.linalg.norm(Zd, axis=1)
    Td = Zd / (sd + 1e-10)[:, None]
    idx_d = quantize.nearest_level_bruteforce(Td, cb.centroids)
    diff = idx_d != out["idx"]
    # the two routes may only disagree where a coordinate sits on a boundary to rounding
    if diff.any():
        gap = np.min(np.abs(out["unit"][diff][:, None] - cb.boundaries[None, :]), axis=1)
        assert gap.max() < 1e-14
    assert diff.mean() < 1e-4
    assert out["idx"].max() < (1 << bits)


def test_degenerate_tokens():
    dim, block = 256, 64
    perm, signs = rpbh.make_rpbh(dim, block, 2)
    cb = codebook.lloyd_max(dim, 4)
    x = np.zeros((3, dim), dtype=np.float32)
    x[1, 37] = 30000.0                       # one huge outlier
    x[2, :] = 1.5                            # constant token
    out = quantize.quantize_rows(synth.to_bf16_bits(x), block, perm, signs, cb.boundaries)
    assert out["norm"][0] == 0.0 and np.all(out["idx"][0] == 7)                        # padding token: t = 0 -> lower middle bin
    k = int(np.where(perm == 37)[0][0]); j = k // block
    z = out["rotated"][1]
    s = out["norm"][1]
    assert s == pytest.approx(float(bf16.bf16_bits_to_f64(synth.to_bf16_bits(np.float32([30000.0])))[0]))
    assert np.allclose(np.abs(z[j * block:(j + 1) * block]), s / math.sqrt(block), rtol=1e-14)
    mask = np.ones(dim, bool); mask[j * block:(j + 1) * block] = False
    assert np.all(z[mask] == 0) and np.all(out["idx"][1][mask] == 7)
    hi = int(np.sum(cb.boundaries < 1 / math.sqrt(block)))                           # |t| = 1/sqrt(h) on the whole block
    assert set(np.unique(out["idx"][1][~mask])) == {15 - hi, hi} and hi == 14
    assert np.all(np.isfinite(out["unit"]))


def test_gaussian_rows_reach_the_codebook_distortion():
    dim, block = 1024, 128
    perm, signs = rpbh.make_rpbh(dim, block, 0)
    g = np.random.default_rng(4)
    xb = synth.to_bf16_bits(g.standard_normal((64, dim)).astype(np.float32))
    for bits in (2, 3, 4):
        cb = codebook.lloyd_max(dim, bits)
        out = quantize.quantize_rows(xb, block, perm, signs, cb.boundaries)
        mse = dim * np.mean((out["unit"] - cb.centroids[out["idx"]]) ** 2)
        assert mse == pytest.approx(cb.distortion, rel=0.03)


def test_rotation_cancels_in_the_product():
    # W' x' = W Pi^T Pi x = W x (Sec. 4.3) to 1e-10 relative in fp64
    dim, block, m, n = 384, 128, 40, 9
    perm, signs = rpbh.make_rpbh(dim, block, 9)
    W = bf16.bf16_bits_to_f64(synth.weights(m, dim, seed=1))
    X = bf16.bf16_bits_to_f64(synth.activations(n, dim, seed=2))
    Wr = rpbh.rotate_rows(W, block, perm, signs)          # rows of W' = W Pi^T
    Xr = rpbh.rotate_rows(X, block, perm, signs)
    ref = X @ W.T
    assert np.linalg.norm(Xr @ Wr.T - ref) <= 1e-10 * np.linalg.norm(ref)
    assert np.abs(Xr @ Wr.T - ref).max() <= 1e-10 * np.abs(ref).max()


def test_weight_rows_norm_storage():
    dim, block, m = 256, 128, 16
    perm, signs = rpbh.make_rpbh(dim, block, 0)
    cb = codebook.lloyd_max(dim, 3)
    wb = synth.weights(m, dim, seed=3)
    wb[5, :] = 0                                            # a zero row must not divide by zero
    out = quantize.quantize_weight_rows(wb, block, perm, signs, cb.boundaries)
    r = bf16.bf16_bits_to_f64(out["norm_bf16_bits"])
    assert r[5] == 0.0 and np.all(out["idx"][5] == 3)
    good = np.arange(m) != 5
    assert np.abs(r[good] / out["norm"][good] - 1).max() <= 2.0 ** -8
    assert np.allclose(out["norm"], np.linalg.norm(bf16.bf16_bits_to_f64(wb), axis=1), rtol=1e-13)


def test_qlinear_matches_triple_loop_and_closed_forms():
    g = np.random.default_rng(0)
    n, m, d = 5, 7, 16
    ca, cw = codebook.lloyd_max(16, 4).centroids_decoded, codebook.lloyd_max(16, 2).centroids_decoded
    ia = g.integers(0, 16, (n, d)).astype(np.uint8)
    iw = g.integers(0, 4, (m, d)).astype(np.uint8)
    s, r = g.uniform(0.5, 2, n), g.uniform(0.5, 2, m)
    Y = qlinear.qlinear(ia, s, ca, iw, r, cw)
    assert np.allclose(Y, qlinear.qlinear_bruteforce(ia, s, ca, iw, r, cw), rtol=1e-13, atol=1e-15)
    ia[:] = 13; iw[:] = 2                                    # all indices equal: Y = s r d c_a c_w
    Y = qlinear.qlinear(ia, s, ca, iw, r, cw)
    assert np.allclose(Y, np.outer(s, r) * d * ca[13] * cw[2], rtol=1e-13)
    # transposition guard: non-square, distinguishable operands
    ia = np.zeros((2, d), np.uint8); ia[1, :] = 15
    iw = np.zeros((3, d), np.uint8); iw[2, :] = 3
    Y = qlinear.qlinear(ia, np.ones(2), ca, iw, np.array([1.0, 2.0, 3.0]), cw)
    assert Y.shape == (2, 3) and Y[1, 2] == pytest.approx(3 * d * ca[15] * cw[3]) and Y[0, 1] == pytest.approx(2 * d * ca[0] * cw[0])


@pytest.mark.parametrize("bw,ba,lo,hi", [(4, 4, 0.10, 0.19), (3, 3, 0.21, 0.33), (2, 4, 0.30, 0.42)])
def test_end_to_end_error_tracks_the_two_distortions(bw, ba, lo, hi):
    # ||Y - X W^T|| / ||X W^T|| ~ sqrt(D_a + D_w): a dropped norm, a wrong table or a transposed
    # operand gives O(1) error instead.
    dim, block, n, m = 1024, 128, 48, 96
    perm, signs = rpbh.make_rpbh(dim, block, 0)
    cba, cbw = codebook.lloyd_max(dim, ba), codebook.lloyd_max(dim, bw)
    xb, wb = synth.activations(n, dim, seed=1000), synth.weights(m, dim, seed=2000)
    qa = quantize.quantize_rows(xb, block, perm, signs, cba.boundaries)
    qw = quantize.quantize_weight_rows(wb, block, perm, signs, cbw.boundaries)
    Y = qlinear.qlinear(qa["idx"], qa["norm"].astype(np.float32), cba.centroids_decoded,
                        qw["idx"], bf16.bf16_bits_to_f64(qw["norm_bf16_bits"]), cbw.centroids_decoded)
    ref = bf16.bf16_bits_to_f64(xb) @ bf16.bf16_bits_to_f64(wb).T
    err = np.linalg.norm(Y - ref) / np.linalg.norm(ref)
    assert lo < err < hi
    assert err == pytest.approx(math.sqrt(cba.distortion + cbw.distortion), rel=0.35)
