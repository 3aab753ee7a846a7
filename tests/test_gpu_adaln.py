"""GPU parity of the AdaLN modulation projection (weight-only INT4 RTN, groups of 64, bf16 activations) against the
CPU oracle, through the C ABI."""
import numpy as np
import pytest

from oracle import adaln as oad
from oracle import bf16 as obf
from paper_2607_02461_b200 import binding as B
from paper_2607_02461_b200 import synth

pytestmark = pytest.mark.gpu

F32_TOL = 2e-6      # fp32 output, relative Frobenius: fp32 accumulation of <= 14k exact 12-bit products per output
BF16_TOL = 3e-3     # bf16 output: one rounding to 8 bits (2^-9 relative per element at worst)


def _dev(bits_u16):
    import torch
    return torch.from_numpy(bits_u16.view(np.int16)).cuda().view(torch.bfloat16)


def _bits(t):
    import torch
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def _cond_tokens(n, d, seed):
    """Conditioning vectors after SiLU: mostly small, a few large channels."""
    rng = np.random.default_rng(seed)
    v = rng.standard_normal((n, d)).astype(np.float32) * 0.7
    v[:, rng.choice(d, max(1, d // 100), replace=False)] *= 12.0
    v = v / (1.0 + np.exp(-v))
    return synth.to_bf16_bits(v)


@pytest.mark.parametrize("m,d", [(16, 64), (48, 192), (1024, 1024), (272, 3072), (96, 12288), (9216, 3072)])
def test_quantized_weights_match_oracle_bit_for_bit(m, d):
    import torch
    wb = synth.weights(m, d, seed=4000 + m)
    wb[min(3, m - 1), 64 * (d // 128):64 * (d // 128) + 64] = 0          # an all-zero group
    Wq, Sc = B.oq_adaln_quantize_weights(_dev(wb))
    q, s = B.oq_adaln_unpack(Wq, Sc, m, d)
    torch.cuda.synchronize()
    want_q, want_s = oad.rtn_int4(wb)
    assert np.array_equal(_bits(s), want_s)
    assert np.array_equal(q.cpu().numpy(), want_q)


@pytest.mark.parametrize("n", [1, 2, 5, 8, 11])
@pytest.mark.parametrize("m,d", [(48, 192), (1024, 1024), (272, 3072), (96, 12288), (18432, 3072)])
def test_linear_matches_oracle(m, d, n):
    import torch
    wb = synth.weights(m, d, seed=4100 + m)
    xb = _cond_tokens(n, d, seed=4200 + n)
    Wq, Sc = B.oq_adaln_quantize_weights(_dev(wb))
    X = _dev(xb)
    y32 = B.oq_adaln_linear(X, Wq, Sc, m, out_dtype=torch.float32)
    y16 = B.oq_adaln_linear(X, Wq, Sc, m)
    torch.cuda.synchronize()
    q, s = oad.rtn_int4(wb)
    rows = np.arange(m) if m <= 2048 else np.unique(np.concatenate([np.arange(64), np.arange(m - 64, m),
                                                                    np.random.default_rng(1).choice(m, 512, replace=False)]))
    ref = oad.adaln_linear(xb, q[rows], s[rows])
    got32 = y32.cpu().numpy().astype(np.float64)[:, rows]
    got16 = y16.float().cpu().numpy().astype(np.float64)[:, rows]
    assert np.linalg.norm(got32 - ref) <= F32_TOL * np.linalg.norm(ref)
    # element-wise: against the sum of absolute terms (cancellation-safe bound)
    xa = np.abs(obf.bf16_bits_to_f64(xb))
    wa = np.abs(oad.dequantize(q[rows], s[rows]))
    assert np.all(np.abs(got32 - ref) <= 4e-6 * (xa @ wa.T) + 1e-300)
    assert np.linalg.norm(got16 - ref) <= BF16_TOL * np.linalg.norm(ref)
    # the bf16 output is the rounding of the fp32 output
    assert torch.equal(y16, y32.to(torch.bfloat16))


def test_linear_is_deterministic_and_handles_strides():
    import torch
    m, d, n = 512, 3072, 3
    wb = synth.weights(m, d, seed=4300)
    Wq, Sc = B.oq_adaln_quantize_weights(_dev(wb))
    wide = torch.zeros((n, d + 64), dtype=torch.bfloat16, device="cuda")
    wide[:, :d] = _dev(_cond_tokens(n, d, 1))
    a = B.oq_adaln_linear(wide[:, :d], Wq, Sc, m, out_dtype=torch.float32)
    b = B.oq_adaln_linear(wide[:, :d].contiguous(), Wq, Sc, m, out_dtype=torch.float32)
    c = B.oq_adaln_linear(wide[:, :d], Wq, Sc, m, out_dtype=torch.float32)
    assert torch.equal(a, b) and torch.equal(a, c)
    # a token's result does not depend on which other tokens share the launch
    one = B.oq_adaln_linear(wide[1:2, :d], Wq, Sc, m, out_dtype=torch.float32)
    assert torch.equal(one[0], a[1])
    # output with a leading dimension
    out = torch.full((n, m + 8), 7.0, dtype=torch.float32, device="cuda")
    B.oq_adaln_linear(wide[:, :d], Wq, Sc, m, out=out[:, :m])
    assert torch.equal(out[:, :m], a) and torch.all(out[:, m:] == 7.0)


def test_empty_and_bad_arguments():
    import torch
    with pytest.raises(B.OqError) as e:
        B.oq_adaln_packed_bytes(24, 128)
    assert e.value.code == 2
    with pytest.raises(B.OqError) as e:
        B.oq_adaln_packed_bytes(32, 96)
    assert e.value.code == 2
    W = torch.zeros((32, 128), dtype=torch.bfloat16, device="cuda")
    Wq, Sc = B.oq_adaln_quantize_weights(W)
    X = torch.ones((0, 128), dtype=torch.bfloat16, device="cuda")
    assert B.oq_adaln_linear(X, Wq, Sc, 32).shape == (0, 32)
    X = torch.ones((2, 128), dtype=torch.bfloat16, device="cuda")
    y = B.oq_adaln_linear(X, Wq, Sc, 32, out_dtype=torch.float32)
    assert torch.all(y == 0)                 # all-zero weights: zero scales, zero output
    with pytest.raises(B.OqError) as e:
        B.oq_adaln_linear(X[:, 1:65], Wq, Sc, 32)       # misaligned rows
    assert e.value.code in (2, 3)
