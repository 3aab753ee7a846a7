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


@pytest.mark.parametrize("d,bits", [(2048, 4), (3072, 3)])
def test_noalloc_back_to_back_on_the_tensor_core_path_without_allocating(d, bits):
    """The widths the benchmarks use run the tensor-core rotate+quantize kernel, launched with programmatic dependent
    launch: three calls in a row on one stream, no synchronisation in between, all sharing the one scratch array (every
    rotate+quantize overwrites what the GEMM before it reads).  Each must equal the two-call path bit for bit, and the
    device's free memory must not move while they run."""
    import torch
    m = 776
    rot, cb = B.oq_make_rpbh(d, 128, 0), B.oq_build_codebook(d, bits)
    assert B.oq_rq_plan(rot, cb)[0] == 3
    wq, wr = B.oq_quantize_weights(_dev(synth.weights(m, d, 2100 + bits)), rot, cb)
    Xs = [_dev(synth.activations(n, d, 30 + k)) for k, n in enumerate((513, 200, 1000))]
    wants = []
    for X in Xs:
        xq, xs = B.oq_rotate_quantize_act(X, rot, cb)
        wants.append(B.oq_qlinear(xq, xs, cb, wq, wr, cb, d))
    outs = [torch.full((X.shape[0], m), float("nan"), dtype=torch.bfloat16, device="cuda") for X in Xs]
    B.oq_linear_forward_noalloc(Xs[0], rot, cb, wq, wr, cb, outs[0])          # warm: first call on the device does the set-up
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for X, out in zip(Xs, outs):
        B.oq_linear_forward_noalloc(X, rot, cb, wq, wr, cb, out)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    assert B.oq_device_status() == 0
    for k, (got, want) in enumerate(zip(outs, wants)):
        assert torch.equal(got, want), f"call {k}"


def test_status_words_are_both_read_and_cleared():
    """A time-out recorded in the library's own status word must not hide (or leave behind) one in the scratch array's
    word, and the other way round: after one oq_device_status call both are clear and the next layer call is valid."""
    import torch
    d, m = 1024, 64
    rot, cb = B.oq_make_rpbh(d, 128, 0), B.oq_build_codebook(d, 4)
    wq, wr = B.oq_quantize_weights(_dev(synth.weights(m, d, 3)), rot, cb)
    X = _dev(synth.activations(40, d, 4))
    out = torch.empty((40, m), dtype=torch.bfloat16, device="cuda")
    B.oq_linear_forward_noalloc(X, rot, cb, wq, wr, cb, out)                   # the scratch word exists now
    torch.cuda.synchronize()
    assert B.oq_device_status() == 0
    B.oq_selftest_bounded_wait()                                              # a wait that simply runs out: code 9
    assert B.oq_device_status() == 9
    assert B.oq_device_status() == 0
    B.oq_linear_forward_noalloc(X, rot, cb, wq, wr, cb, out)
    xq, xs = B.oq_rotate_quantize_act(X, rot, cb)
    torch.cuda.synchronize()
    assert B.oq_device_status() == 0
    assert torch.equal(out, B.oq_qlinear(xq, xs, cb, wq, wr, cb, d))


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
