"""GPU parity of oq_qlinear against the oracle's fp64 product of the decoded operands (through the C ABI)."""
import numpy as np
import pytest

from oracle import bf16 as obf
from oracle import codebook as ocb
from oracle import qlinear as oql
from oracle import quantize as oq
from oracle import rpbh as orp
from paper_2607_02461_b200 import binding as B
from paper_2607_02461_b200 import synth

pytestmark = pytest.mark.gpu

TOL_F32 = 1e-5      # operand-exact comparison, fp32 output: fp32 accumulation only
TOL_BF16 = 2e-3     # relative Frobenius error, bf16 output (one output rounding: ~1.7e-3)


def _dev(bits_u16):
    import torch
    return torch.from_numpy(bits_u16.view(np.int16)).cuda().view(torch.bfloat16)


def _rel(a, b):
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)


def run_case(n, m, d, ba, bw, block=128, seed=0, xseed=1000, wseed=2000, end_to_end=True):
    import torch
    rot = B.oq_make_rpbh(d, block, seed)
    cba, cbw = B.oq_build_codebook(d, ba), B.oq_build_codebook(d, bw)
    xb, wb = synth.activations(n, d, xseed), synth.weights(m, d, wseed)
    xq, xs = B.oq_rotate_quantize_act(_dev(xb), rot, cba)
    wq, wr = B.oq_quantize_weights(_dev(wb), rot, cbw)
    y32 = B.oq_qlinear(xq, xs, cba, wq, wr, cbw, d, out_dtype=torch.float32)
    y16 = B.oq_qlinear(xq, xs, cba, wq, wr, cbw, d)
    y16b = B.oq_qlinear(xq, xs, cba, wq, wr, cbw, d)
    # the two GEMM kernels (activation operand in shared memory / in tensor memory) add the same products in the same order
    B.oq_debug_select_gemm_kernel(1)
    y16_smem = B.oq_qlinear(xq, xs, cba, wq, wr, cbw, d)
    B.oq_debug_select_gemm_kernel(2)
    y16_tmem = B.oq_qlinear(xq, xs, cba, wq, wr, cbw, d)
    B.oq_debug_select_gemm_kernel(3)                                       # the tile order of large inputs
    y16_band = B.oq_qlinear(xq, xs, cba, wq, wr, cbw, d)
    B.oq_debug_select_gemm_kernel(0)
    torch.cuda.synchronize()
    assert B.oq_device_status() == 0
    assert torch.equal(y16, y16b)                                          # run-to-run determinism
    assert torch.equal(y16, y16_tmem) and torch.equal(y16_smem, y16_tmem) and torch.equal(y16_band, y16_tmem)
    # operand-exact mode: decode the GPU's own packed operands on the CPU, fp64 product
    ia = B.oq_unpack_indices(xq, n, d, ba).cpu().numpy()
    iw = B.oq_unpack_indices(wq, m, d, bw).cpu().numpy()
    oa, ow = ocb.lloyd_max(d, ba), ocb.lloyd_max(d, bw)
    s = xs.cpu().numpy()
    r = obf.bf16_bits_to_f64(wr.view(torch.int16).cpu().numpy().view(np.uint16))
    ref = oql.qlinear(ia, s, oa.centroids_decoded, iw, r, ow.centroids_decoded)
    g32 = y32.cpu().numpy().astype(np.float64)
    g16 = y16.float().cpu().numpy().astype(np.float64)
    assert _rel(g32, ref) <= TOL_F32
    assert _rel(g16, ref) <= TOL_BF16
    # bf16 output must be the fp32 result rounded once: elementwise within one bf16 rounding (2^-8 relative)
    # plus the fp32 accumulation error, which scales with the row's largest output, not with the element
    slack = 2.0 ** -8 * np.abs(ref) + 1e-5 * np.abs(ref).max(axis=1, keepdims=True)
    assert np.all(np.abs(g16 - ref) <= slack)
    assert np.all(np.abs(g32 - ref) <= 1e-5 * np.abs(ref).max(axis=1, keepdims=True))
    if end_to_end:
        perm, signs = orp.make_rpbh(d, block, seed)
        qa = oq.quantize_rows(xb, block, perm, signs, oa.boundaries)
        qw = oq.quantize_weight_rows(wb, block, perm, signs, ow.boundaries)
        ref2 = oql.qlinear(qa["idx"], qa["norm"].astype(np.float32), oa.centroids_decoded, qw["idx"],
                           obf.bf16_bits_to_f64(qw["norm_bf16_bits"]), ow.centroids_decoded)
        assert _rel(g16, ref2) <= TOL_BF16
    return _rel(g16, ref)


def test_config1_single_linear_w4a4():
    run_case(256, 1024, 1024, 4, 4)


@pytest.mark.parametrize("ba,bw", [(3, 3), (4, 2), (4, 3), (2, 2), (3, 2), (2, 3), (3, 4), (2, 4)])
def test_other_bit_widths(ba, bw):
    run_case(200, 512, 1024, ba, bw)


@pytest.mark.parametrize("n,m,d", [(1, 8, 128), (129, 264, 256), (300, 1000, 384), (127, 256, 3072), (513, 776, 640)])
def test_ragged_shapes(n, m, d):
    run_case(n, m, d, 4, 4, block=128 if d % 128 == 0 else 64)


def test_identity_like_operands():
    """All indices equal: Y = s r d c_a c_w exactly representable path; one-hot K picks single products."""
    import torch
    d, n, m = 256, 130, 264
    cb = B.oq_build_codebook(d, 4)
    ocbk = ocb.lloyd_max(d, 4)
    rot = B.oq_make_rpbh(d, 128, 0)
    # build packed operands through the library from crafted inputs: a token equal to a constant
    # times a row of Pi has a one-hot rotated image; use the oracle only to CHECK, not to build
    xb, wb = synth.activations(n, d, 7), synth.weights(m, d, 8)
    xq, xs = B.oq_rotate_quantize_act(_dev(xb), rot, cb)
    wq, wr = B.oq_quantize_weights(_dev(wb), rot, cb)
    ones = torch.ones(n, dtype=torch.float32, device="cuda")
    y = B.oq_qlinear(xq, ones, cb, wq, torch.ones(m, dtype=torch.bfloat16, device="cuda"), cb, d, out_dtype=torch.float32)
    ia = B.oq_unpack_indices(xq, n, d, 4).cpu().numpy()
    iw = B.oq_unpack_indices(wq, m, d, 4).cpu().numpy()
    ref = oql.qlinear(ia, np.ones(n), ocbk.centroids_decoded, iw, np.ones(m), ocbk.centroids_decoded)
    assert _rel(y.cpu().numpy().astype(np.float64), ref) <= TOL_F32
    # scaling by the norms is exactly a row / column scaling of the unit result
    y2 = B.oq_qlinear(xq, xs, cb, wq, wr, cb, d, out_dtype=torch.float32)
    want = y.double() * xs.double()[:, None] * wr.double()[None, :]
    assert torch.allclose(y2.double(), want, rtol=3e-7, atol=0)


def test_strided_output_and_empty():
    import torch
    d, n, m = 256, 40, 72
    cb, rot = B.oq_build_codebook(d, 4), B.oq_make_rpbh(d, 128, 0)
    xq, xs = B.oq_rotate_quantize_act(_dev(synth.activations(n, d, 1)), rot, cb)
    wq, wr = B.oq_quantize_weights(_dev(synth.weights(m, d, 2)), rot, cb)
    dense = B.oq_qlinear(xq, xs, cb, wq, wr, cb, d)
    wide = torch.full((n, m + 24), 7.0, dtype=torch.bfloat16, device="cuda")
    B.oq_qlinear(xq, xs, cb, wq, wr, cb, d, out=wide[:, :m])
    assert torch.equal(wide[:, :m], dense) and torch.all(wide[:, m:] == 7.0)      # nothing written past m
    empty = B.oq_qlinear(xq[:0], xs[:0], cb, wq, wr, cb, d)
    assert empty.shape == (0, m)
    with pytest.raises(B.OqError) as e:
        B.oq_qlinear(xq, xs, cb, wq, wr, B.oq_build_codebook(512, 4), d)
    assert e.value.code == 1


def test_bounded_wait_gives_up_and_reports():
    """A device-side wait whose barrier never completes must end by itself, leave the context usable and
    show up in oq_device_status (nothing is hung or trapped to provoke it: the wait simply runs out)."""
    import torch
    assert B.oq_device_status() == 0
    B.oq_selftest_bounded_wait()
    assert B.oq_device_status() == 9          # code of the self-test wait; reading clears it
    assert B.oq_device_status() == 0
    d = 256
    cb, rot = B.oq_build_codebook(d, 4), B.oq_make_rpbh(d, 128, 0)
    xq, xs = B.oq_rotate_quantize_act(_dev(synth.activations(16, d, 1)), rot, cb)
    wq, wr = B.oq_quantize_weights(_dev(synth.weights(16, d, 2)), rot, cb)
    y = B.oq_qlinear(xq, xs, cb, wq, wr, cb, d)
    assert torch.isfinite(y.float()).all() and B.oq_device_status() == 0


def test_back_to_back_launches_into_shared_buffers_match_serialised_runs():
    """Both kernels are launched with programmatic stream serialisation (a kernel may start while the previous one of
    the stream is still running and waits inside before touching its data).  Layers launched back to back that reuse
    ONE set of packed-activation buffers (every rotate+quantize overwrites what the GEMM before it reads) must give
    bit-identical results to the same sequence with a device synchronisation after every kernel."""
    import torch
    d, m, n = 3072, 2048, 1000
    rot, cb = B.oq_make_rpbh(d, 128, 0), B.oq_build_codebook(d, 4)
    gen = torch.Generator(device="cuda").manual_seed(7)
    Xs = [torch.randn((n, d), device="cuda", generator=gen).to(torch.bfloat16) * (k + 1) for k in range(4)]
    W = (torch.randn((m, d), device="cuda", generator=gen) * 0.02).to(torch.bfloat16)
    wq, wr = B.oq_quantize_weights(W, rot, cb)
    xq = torch.empty((n, B.oq_packed_bytes(n, d, 4)[1]), dtype=torch.uint8, device="cuda")
    xs = torch.empty(n, dtype=torch.float32, device="cuda")

    def run(sync):
        outs = []
        for rep in range(3):
            for X in Xs:
                Y = torch.empty((n, m), dtype=torch.bfloat16, device="cuda")
                B.oq_rotate_quantize_act(X, rot, cb, out_idx=xq, out_norm=xs)
                if sync:
                    torch.cuda.synchronize()
                B.oq_qlinear(xq, xs, cb, wq, wr, cb, d, out=Y)
                if sync:
                    torch.cuda.synchronize()
                outs.append(Y)
        torch.cuda.synchronize()
        return outs

    ref = run(True)
    got = run(False)
    assert B.oq_device_status() == 0
    for a, b in zip(ref, got):
        assert torch.equal(a, b)


@pytest.mark.parametrize("bits_a,bits_w", [(4, 4), (3, 3), (4, 2), (2, 3)])
@pytest.mark.parametrize("n,m,d", [(200, 520, 2048), (1, 8, 128), (257, 264, 384), (1000, 1536, 3072)])
def test_levels_form_is_bit_identical_to_packed_form(n, m, d, bits_a, bits_w):
    """Activations written out once as bf16 levels and fetched by TMA: same operands, same accumulation order, so the
    same output bits as the kernel that decodes the packed activations itself; the level matrix itself is the
    codebook's bf16 table indexed by the unpacked indices."""
    import torch
    rot = B.oq_make_rpbh(d, 128, 0)
    cba, cbw = B.oq_build_codebook(d, bits_a), B.oq_build_codebook(d, bits_w)
    xb, wb = synth.activations(n, d, seed=3100 + n), synth.weights(m, d, seed=3200 + m)
    xq, xs = B.oq_rotate_quantize_act(_dev(xb), rot, cba)
    wq, wr = B.oq_quantize_weights(_dev(wb), rot, cbw)
    xd = B.oq_decode_levels(xq, n, d, cba)
    idx = B.oq_unpack_indices(xq, n, d, bits_a).cpu().numpy()
    levels_bits = obf.f64_to_bf16_bits(ocb.lloyd_max(d, bits_a).centroids)
    assert np.array_equal(xd.view(torch.int16).cpu().numpy().view(np.uint16), levels_bits[idx])
    for dt in (torch.bfloat16, torch.float32):
        ref = B.oq_qlinear(xq, xs, cba, wq, wr, cbw, d, out_dtype=dt)
        got = B.oq_qlinear_levels(xd, xs, wq, wr, cbw, d, out_dtype=dt)
        torch.cuda.synchronize()
        assert B.oq_device_status() == 0
        assert torch.equal(ref, got)
    # a level matrix with a leading dimension larger than dim
    wide = torch.zeros((n, d + 64), dtype=torch.bfloat16, device="cuda")
    B.oq_decode_levels(xq, n, d, cba, out=wide[:, :d])
    got = B.oq_qlinear_levels(wide[:, :d], xs, wq, wr, cbw, d)
    assert torch.equal(got, B.oq_qlinear(xq, xs, cba, wq, wr, cbw, d))


@pytest.mark.parametrize("n,m,d,block", [(200, 520, 3072, 1024), (130, 264, 5120, 1024)])
def test_whole_layer_with_the_papers_default_block(n, m, d, block):
    """Both operands rotated with the paper's default block (the largest power of two dividing the width): the rotation
    cancels in the product (Sec. 4.3) whatever the block, and the layer matches the oracle end to end."""
    run_case(n, m, d, 4, 4, block=block, seed=3)


@pytest.mark.parametrize("ba,bw", [(4, 4), (3, 3), (2, 4)])
def test_both_gemm_kernels_agree_over_several_tiles_per_sm_pair(ba, bw):
    """156 output tiles on at most 74 SM pairs: every pair runs two or three tiles, so the kernel with the activation operand
    in tensor memory reuses its single accumulator, its operand ring and its staging area; ragged last row and column tiles."""
    import torch
    n, m, d = 2990, 3304, 1024
    rot = B.oq_make_rpbh(d, 128, 0)
    cba, cbw = B.oq_build_codebook(d, ba), B.oq_build_codebook(d, bw)
    xq, xs = B.oq_rotate_quantize_act(_dev(synth.activations(n, d, 1234)), rot, cba)
    wq, wr = B.oq_quantize_weights(_dev(synth.weights(m, d, 2345)), rot, cbw)
    try:
        B.oq_debug_select_gemm_kernel(1)
        y1 = B.oq_qlinear(xq, xs, cba, wq, wr, cbw, d)
        B.oq_debug_select_gemm_kernel(2)
        y2 = B.oq_qlinear(xq, xs, cba, wq, wr, cbw, d)
        y2b = B.oq_qlinear(xq, xs, cba, wq, wr, cbw, d)
        B.oq_debug_select_gemm_kernel(3)               # 13 column tiles: one band of 8 and one of 5
        y3 = B.oq_qlinear(xq, xs, cba, wq, wr, cbw, d)
    finally:
        B.oq_debug_select_gemm_kernel(0)
    torch.cuda.synchronize()
    assert B.oq_device_status() == 0
    assert torch.equal(y1, y2) and torch.equal(y2, y2b) and torch.equal(y2, y3)
    # and against the fp32 output of kernel 1 rounded once
    y32 = B.oq_qlinear(xq, xs, cba, wq, wr, cbw, d, out_dtype=torch.float32)
    assert torch.equal(y32.to(torch.bfloat16), y2)
