"""bfloat16 bit helpers for the oracle (test infrastructure, CPU only).

bfloat16 is the upper 16 bits of an IEEE-754 binary32.  Conversions to bf16
round to nearest, ties to even; a float64 is first rounded to float32 and then
to bf16 (two roundings), which is what a device-side
float -> bfloat16 conversion of a value held in fp32 does.
"""
import numpy as np


def bf16_bits_to_f64(bits):
    """uint16 bf16 bit patterns -> exact float64 values."""
    b = np.asarray(bits, dtype=np.uint16)
    f32 = (b.astype(np.uint32) << np.uint32(16)).view(np.float32)
    return f32.astype(np.float64)


def f32_to_bf16_bits(x):
    """float32 -> bf16 bit patterns, round-to-nearest-even (finite inputs)."""
    u = np.ascontiguousarray(np.asarray(x, dtype=np.float32)).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    rounded = u + np.uint32(0x7FFF) + lsb
    return (rounded >> np.uint32(16)).astype(np.uint16)


def f64_to_bf16_bits(x):
    """float64 -> float32 (RNE) -> bf16 (RNE)."""
    return f32_to_bf16_bits(np.asarray(x, dtype=np.float64).astype(np.float32))


def round_to_bf16(x):
    """float64 values rounded through float32 to bf16, returned as float64."""
    return bf16_bits_to_f64(f64_to_bf16_bits(x))
