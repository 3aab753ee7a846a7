"""Quantized linear layer on decoded operands -- oracle (test infrastructure, CPU, fp64).

The quantized layer computes W^' x^' (Sec. 4.3, after Eq. 8) with
    W^' = diag(r') Q_bw(W~')          (Eq. 6)
    x^' = s * Q_ba(x~')               (Eq. 8)
so  Y[n, i] = s_n * r'_i * sum_k C_a[idxA[n, k]] * C_w[idxW[i, k]].

The level tables C_a, C_w and the row norms r' are taken AS DECODED by a
bf16 tensor-core path (levels rounded to bf16, r' stored in bf16, s in fp32);
the arithmetic itself is fp64.
"""
import numpy as np


def qlinear(idx_a, s, levels_a, idx_w, r, levels_w):
    """idx_a uint8 [N, d], s float [N], idx_w uint8 [m, d], r float [m]; tables are float64 arrays."""
    A = np.asarray(levels_a, dtype=np.float64)[np.asarray(idx_a)]
    B = np.asarray(levels_w, dtype=np.float64)[np.asarray(idx_w)]
    core = A @ B.T
    return core * np.asarray(s, dtype=np.float64)[:, None] * np.asarray(r, dtype=np.float64)[None, :]


def qlinear_bruteforce(idx_a, s, levels_a, idx_w, r, levels_w):
    """Triple loop, for tiny shapes only."""
    n, d = idx_a.shape
    m = idx_w.shape[0]
    out = np.zeros((n, m), dtype=np.float64)
    for a in range(n):
        for i in range(m):
            acc = 0.0
            for k in range(d):
                acc += float(levels_a[idx_a[a, k]]) * float(levels_w[idx_w[i, k]])
            out[a, i] = float(s[a]) * float(r[i]) * acc
    return out
