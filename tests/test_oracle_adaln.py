"""Pins of the AdaLN weight-only INT4 oracle (groups of 64, round to nearest) against things it does not compute
itself: a hand-worked group, the round-to-nearest error bound, exhaustive search over the 16 grid points,
exact symmetries, and a triple loop for the product."""
import numpy as np
import pytest

from oracle import adaln as oad
from oracle import bf16 as obf
from paper_2607_02461_b200 import synth


def _bits(x):
    return obf.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def test_hand_worked_group_is_reproduced_exactly():
    # one group: the 15 multiples of 0.5 from -3.5 to 3.5, padded with zeros: scale = 3.5 / 7 = 0.5, q = w / 0.5
    w = np.zeros((1, 64), np.float32)
    w[0, :15] = 0.5 * np.arange(-7, 8)
    q, sb = oad.rtn_int4(_bits(w))
    assert obf.bf16_bits_to_f64(sb)[0, 0] == 0.5
    assert q[0, :15].tolist() == list(range(-7, 8)) and not q[0, 15:].any()
    assert np.array_equal(oad.dequantize(q, sb), w.astype(np.float64))
    # a second group with another magnitude does not disturb the first (groups are independent)
    w2 = np.concatenate([w, 1024.0 * w], axis=1)
    q2, sb2 = oad.rtn_int4(_bits(w2))
    assert np.array_equal(q2[:, :64], q) and np.array_equal(q2[:, 64:], q)
    assert obf.bf16_bits_to_f64(sb2).tolist() == [[0.5, 512.0]]


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_round_to_nearest_error_bound_and_extremes(seed):
    wb = synth.weights(48, 512, seed=seed)
    w = obf.bf16_bits_to_f64(wb)
    q, sb = oad.rtn_int4(wb)
    s = np.repeat(obf.bf16_bits_to_f64(sb), 64, axis=1)
    assert q.min() >= -8 and q.max() <= 7
    # nearest grid point: at most half a step away (the bf16 rounding of the scale moves the largest element of a
    # group at most 7 * 2^-8 steps past +-7)
    assert np.all(np.abs(w - q * s) <= 0.5 * s * (1 + 1e-6) + 1e-300)
    # the largest element of every group sits on +-7
    g = np.abs(w).reshape(48, 8, 64)
    qa = np.abs(q.astype(np.int32)).reshape(48, 8, 64)
    top = np.take_along_axis(qa, g.argmax(axis=2)[:, :, None], axis=2)
    assert np.all(top == 7)


def test_exhaustive_search_over_the_grid_agrees():
    wb = synth.weights(16, 256, seed=5)
    w = obf.bf16_bits_to_f64(wb)
    q, sb = oad.rtn_int4(wb)
    s = np.repeat(obf.bf16_bits_to_f64(sb), 64, axis=1)
    grid = np.arange(-8, 8, dtype=np.float64)
    err = np.abs(w[:, :, None] - grid[None, None, :] * s[:, :, None])      # [m, d, 16]
    best = err.min(axis=2)
    mine = np.abs(w - q * s)
    # the chosen point is a minimiser (ties and fp32-division rounding: within 1e-6 of a step of the minimum)
    assert np.all(mine <= best + 1e-6 * s)
    assert np.mean(grid[err.argmin(axis=2)] == q) > 0.999


def test_exact_symmetries():
    wb = synth.weights(8, 192, seed=9)
    q, sb = oad.rtn_int4(wb)
    # sign flip (bit 15 of every bf16): q changes sign, scales stay
    qn, sbn = oad.rtn_int4(wb ^ np.uint16(0x8000))
    assert np.array_equal(qn, -q) and np.array_equal(sbn, sb)
    # multiplying by a power of two: scales move by that power, q stays
    w4 = _bits(obf.bf16_bits_to_f64(wb).astype(np.float32) * np.float32(4.0))
    q4, sb4 = oad.rtn_int4(w4)
    assert np.array_equal(q4, q)
    assert np.array_equal(obf.bf16_bits_to_f64(sb4), 4.0 * obf.bf16_bits_to_f64(sb))
    # permuting the coordinates inside a group permutes q the same way and keeps the scale
    perm = np.random.default_rng(0).permutation(64)
    wp = wb.copy()
    wp[:, 64:128] = wb[:, 64:128][:, perm]
    qp, sbp = oad.rtn_int4(wp)
    assert np.array_equal(qp[:, 64:128], q[:, 64:128][:, perm]) and np.array_equal(sbp, sb)


def test_zero_group_and_zero_row():
    w = np.zeros((2, 128), np.float32)
    w[1, 64:] = np.linspace(-1, 1, 64)
    q, sb = oad.rtn_int4(_bits(w))
    assert not q[0].any() and not sb[0].any() and not q[1, :64].any() and sb[1, 0] == 0
    x = _bits(np.ones((1, 128), np.float32))
    y = oad.adaln_linear(x, q, sb)
    assert y[0, 0] == 0.0 and np.isfinite(y).all()


def test_product_equals_triple_loop_and_plain_matmul_on_grid_weights():
    rng = np.random.default_rng(3)
    m, d, n = 5, 128, 3
    wb = synth.weights(m, d, seed=4)
    xb = _bits(rng.standard_normal((n, d)))
    q, sb = oad.rtn_int4(wb)
    s = obf.bf16_bits_to_f64(sb)
    x = obf.bf16_bits_to_f64(xb)
    want = np.zeros((n, m))
    for a in range(n):
        for r in range(m):
            for i in range(d):
                want[a, r] += x[a, i] * float(q[r, i]) * s[r, i // 64]
    got = oad.adaln_linear(xb, q, sb)
    assert np.allclose(got, want, rtol=1e-13, atol=1e-300)
    # weights that already sit on a grid (integers -7..7 times a power of two) are reproduced, so the layer is x W^T
    wi = rng.integers(-7, 8, size=(m, d)).astype(np.float32)
    wi[:, 0] = 7
    wi[:, 64] = -7
    wgrid = wi * np.float32(2.0 ** -6)
    qg, sg = oad.rtn_int4(_bits(wgrid))
    assert np.array_equal(qg, wi.astype(np.int8))
    assert np.allclose(oad.adaln_linear(xb, qg, sg), x @ wgrid.astype(np.float64).T, rtol=1e-13)
