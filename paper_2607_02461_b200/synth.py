"""Seeded synthetic inputs shaped like the paper's DiT workloads.

This module only draws random tensors (numpy PCG64) and rounds them to bf16
bit patterns.  It contains none of the method's arithmetic, so that both the
CUDA path and the independent CPU oracle can consume identical bits.

Recipe (stands in for real DiT activations / weights, which need checkpoints):
  activations  Z ~ N(0,1) [N, d]; each token scaled by exp(U(ln 0.1, ln 10));
               round(0.01 d) seeded channels multiplied by 30 (channel outliers)
  weights      N(0, 0.02^2) [m, d]
  drift        per call c the outlier channel set and per-channel multipliers
               (log-uniform on [10, 100]) are re-drawn
"""
import numpy as np


def to_bf16_bits(x):
    """float32 array -> uint16 bf16 bit patterns (round to nearest even)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    return ((u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(np.uint16)


def activations(n_tokens, dim, seed, outlier_frac=0.01, outlier_gain=30.0):
    """uint16 [n_tokens, dim] bf16 bits."""
    g = np.random.Generator(np.random.PCG64(seed))
    z = g.standard_normal((n_tokens, dim), dtype=np.float32)
    scale = np.exp(g.uniform(np.log(0.1), np.log(10.0), size=n_tokens)).astype(np.float32)
    z *= scale[:, None]
    n_out = int(round(outlier_frac * dim))
    if n_out:
        ch = g.choice(dim, n_out, replace=False)
        z[:, ch] *= np.float32(outlier_gain)
    return to_bf16_bits(z)


def activations_drift(n_tokens, dim, seed, call, outlier_frac=0.01):
    """Timestep-drift variant: outlier channels and gains (10-100x) re-drawn per call."""
    g = np.random.Generator(np.random.PCG64(seed))
    z = g.standard_normal((n_tokens, dim), dtype=np.float32)
    scale = np.exp(g.uniform(np.log(0.1), np.log(10.0), size=n_tokens)).astype(np.float32)
    z *= scale[:, None]
    gc = np.random.Generator(np.random.PCG64(3000 + call))
    n_out = int(round(outlier_frac * dim))
    ch = gc.choice(dim, n_out, replace=False)
    gain = np.exp(gc.uniform(np.log(10.0), np.log(100.0), size=n_out)).astype(np.float32)
    z[:, ch] *= gain[None, :]
    return to_bf16_bits(z)


def weights(m, dim, seed, std=0.02):
    """uint16 [m, dim] bf16 bits."""
    g = np.random.Generator(np.random.PCG64(seed))
    w = g.standard_normal((m, dim), dtype=np.float32) * np.float32(std)
    return to_bf16_bits(w)


# Named workloads: (tokens, [(name, d_in, d_out), ...])
FLUX_TOKENS = 4608
FLUX_LAYERS = [("qkv", 3072, 9216), ("proj", 3072, 3072), ("mlp_up", 3072, 12288), ("mlp_down", 12288, 3072)]
WAN_TOKENS = 32760
WAN_LAYERS = [("qkv", 5120, 15360), ("proj", 5120, 5120), ("ffn_up", 5120, 13824), ("ffn_down", 13824, 5120)]
