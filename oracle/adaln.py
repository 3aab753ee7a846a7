"""AdaLN modulation projection: weight-only INT4 round-to-nearest, groups of 64 -- oracle (test infrastructure, CPU).

The supplementary section on quantized layers keeps the AdaLN modulation projections outside the rotated
codebook path: only their weights are quantized, "INT4 RTN at group size 64", and the activation (one
conditioning token per step) stays in bf16 (also Sec. 5.1 and the AdaLN bit-width ablation).  The paper gives
no formula for the grid, so this file fixes the plainest reading and says so:

    for every weight row and every group G of 64 consecutive input coordinates
        scale_G = bf16( max_{i in G} |w_i| / 7 )            (symmetric grid, no zero point; fp32 division)
        q_i     = clamp( rint( w_i / scale_G ), -8, 7 )     (fp32 division, ties to even; q = 0 when scale_G = 0)
    y_n[row] = sum_G scale_G * sum_{i in G} q_i * x_n[i]

The integer decision is taken in fp32, the precision the device kernel uses, so both sides can be compared
bit for bit; the product itself is fp64 here.
"""
import numpy as np

from . import bf16 as obf

GROUP = 64


def rtn_int4(w_bits):
    """w_bits: uint16 bf16 bit patterns [m, d], d a multiple of 64.
    Returns (q int8 [m, d] in -8..7, scale_bits uint16 [m, d/64])."""
    w = obf.bf16_bits_to_f64(w_bits).astype(np.float32)          # exact
    m, d = w.shape
    if d % GROUP:
        raise ValueError("d must be a multiple of 64")
    g = w.reshape(m, d // GROUP, GROUP)
    amax = np.abs(g).max(axis=2)
    scale_bits = obf.f32_to_bf16_bits(amax / np.float32(7.0))
    scale = obf.bf16_bits_to_f64(scale_bits).astype(np.float32)
    safe = np.where(scale > 0, scale, np.float32(1.0))
    ratio = (g / safe[:, :, None]).astype(np.float32)            # IEEE fp32 division
    q = np.clip(np.rint(ratio), -8, 7)
    q = np.where(scale[:, :, None] > 0, q, 0.0)
    return q.reshape(m, d).astype(np.int8), scale_bits


def dequantize(q, scale_bits):
    """The weights the layer actually applies: q * scale per group, exact in fp64."""
    m, d = q.shape
    s = obf.bf16_bits_to_f64(scale_bits)
    return (q.astype(np.float64).reshape(m, d // GROUP, GROUP) * s[:, :, None]).reshape(m, d)


def adaln_linear(x_bits, q, scale_bits):
    """x_bits: uint16 bf16 bit patterns [n, d].  Returns the fp64 product [n, m]."""
    x = obf.bf16_bits_to_f64(x_bits)
    return x @ dequantize(q, scale_bits).T
