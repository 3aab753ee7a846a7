"""The allocation-free layer entry point against the ordinary two-call path.

Callers that cannot allocate device memory when a layer has to run (a serving loop inside a fixed memory
budget, a thread that must not block on the allocator) use oq_linear_forward_noalloc, which keeps the
packed activations, their norms and the kernels' status word in a device array compiled into the library.
It launches the same kernels as oq_rotate_quantize_act + oq_qlinear, so the outputs must be identical.
This file sorts last on purpose: a run that stops at the first failure has then run every other test.
"""
import numpy as np
import pytest

from paper_2607_02461_b200 import binding as B
from paper_2607_02461_b200 import synth

pytestmark = pytest.mark.gpu


def _dev(bits_u16):
    import torch
    return torch.from_numpy(bits_u16.view(np.int16)).cuda().view(torch.bfloat16)


def test_noalloc_matches_ordinary_path_on_two_calls_in_a_row():
    import torch
    d, m, bits = 1024, 520, 4
    rot, cb = B.oq_make_rpbh(d, 128, 0), B.oq_build_codebook(d, bits)
    wq, wr = B.oq_quantize_weights(_dev(synth.weights(m, d, 2000)), rot, cb)     # also puts rot's tables on the device
    for call, (n, seed) in enumerate([(300, 11), (77, 12)]):                       # second call: smaller, other data
        X = _dev(synth.activations(n, d, seed))
        xq, xs = B.oq_rotate_quantize_act(X, rot, cb)
        want = B.oq_qlinear(xq, xs, cb, wq, wr, cb, d)
        want32 = B.oq_qlinear(xq, xs, cb, wq, wr, cb, d, out_dtype=torch.float32)
        got = torch.full((n, m), float("nan"), dtype=torch.bfloat16, device="cuda")
        got32 = torch.full((n, m), float("nan"), dtype=torch.float32, device="cuda")
        B.oq_linear_forward_noalloc(X, rot, cb, wq, wr, cb, got)
        B.oq_linear_forward_noalloc(X, rot, cb, wq, wr, cb, got32)
        torch.cuda.synchronize()
        assert B.oq_device_status() == 0
        # same kernels on the same data: identical, which is inside every tolerance the other tests use
        assert torch.equal(got, want), f"call {call}"
        rel = (got32.double() - want32.double()).norm() / want32.double().norm()
        assert rel.item() <= 1e-5 and torch.equal(got32, want32)


def test_noalloc_rejects_what_does_not_fit_and_unprepared_handles():
    import torch
    d = 1024
    cb = B.oq_build_codebook(d, 4)
    rot = B.oq_make_rpbh(d, 128, 0)
    wq, wr = B.oq_quantize_weights(_dev(synth.weights(64, d, 1)), rot, cb)
    big = torch.zeros((16385, d), dtype=torch.bfloat16, device="cuda")            # 16385 * 512 B > 8 MiB of indices
    out = torch.empty((16385, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.OqError) as e:
        B.oq_linear_forward_noalloc(big, rot, cb, wq, wr, cb, out)
    assert e.value.code == 6 and "8388608" in str(e.value)
    fresh = B.oq_make_rpbh(d, 128, 99)                                            # never used on the device
    with pytest.raises(B.OqError) as e:
        B.oq_linear_forward_noalloc(big[:8], fresh, cb, wq, wr, cb, out[:8])
    assert e.value.code == 1
