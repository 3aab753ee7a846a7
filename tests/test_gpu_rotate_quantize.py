"""GPU parity of oq_rotate_quantize_act / oq_quantize_weights against the CPU oracle (through the C ABI)."""
import numpy as np
import pytest

from oracle import bf16 as obf
from oracle import codebook as ocb
from oracle import quantize as oq
from oracle import rpbh as orp
from paper_2607_02461_b200 import binding as B
from paper_2607_02461_b200 import synth

pytestmark = pytest.mark.gpu

ROT_TOL = 1e-5      # rotated activations: relative to the token's largest coordinate / Frobenius
BAND = 1e-5         # a level flip is allowed only within this (times the token's largest |t|) of a boundary


def _dev(bits_u16):
    import torch
    return torch.from_numpy(bits_u16.view(np.int16)).cuda().view(torch.bfloat16)


AUTO, GENERAL, REGISTERS, TENSOR, SLAB = 0, 1, 2, 3, 4    # oq_debug_select_rq_kernel


@pytest.fixture(autouse=True)
def _default_kernel_afterwards():
    yield
    B.oq_debug_select_rq_kernel(AUTO)


def check_rows(xb, block, seed, bits, weights=False, rows=None, kernel=AUTO):
    """Runs the GPU pass on xb (uint16 bf16 bits [N, d]) and compares with the oracle on `rows`."""
    import torch
    n, d = xb.shape
    rot, cb = B.oq_make_rpbh(d, block, seed), B.oq_build_codebook(d, bits)
    X = _dev(xb)
    dbg = torch.full((n, d), float("nan"), dtype=torch.float32, device="cuda")
    fn = B.oq_quantize_weights if weights else B.oq_rotate_quantize_act
    B.oq_debug_select_rq_kernel(kernel)
    idx_p, norm = fn(X, rot, cb, dbg_rotated=dbg)
    B.oq_debug_select_rq_kernel(AUTO)
    idx = B.oq_unpack_indices(idx_p, n, d, bits).cpu().numpy()
    torch.cuda.synchronize()
    assert B.oq_device_status() == 0
    sel = np.arange(n) if rows is None else np.asarray(rows)
    perm, signs = orp.make_rpbh(d, block, seed)
    ocbk = ocb.lloyd_max(d, bits)
    ref = (oq.quantize_weight_rows if weights else oq.quantize_rows)(xb[sel], block, perm, signs, ocbk.boundaries)
    z_gpu = dbg.cpu().numpy()[sel].astype(np.float64)
    z_ref = ref["rotated"]
    tok_max = np.abs(z_ref).max(axis=1)
    assert np.all(np.abs(z_gpu - z_ref).max(axis=1) <= ROT_TOL * tok_max + 1e-300)
    assert np.linalg.norm(z_gpu - z_ref) <= ROT_TOL * np.linalg.norm(z_ref) + 1e-300
    if weights:
        got = norm.view(torch.int16).cpu().numpy().view(np.uint16)[sel]
        want = ref["norm_bf16_bits"]
        off = got.astype(np.int32) - want.astype(np.int32)
        assert np.abs(off).max() <= 1                         # fp32 vs fp64 norm may straddle a bf16 rounding edge
        assert (off != 0).mean() <= 0.01
    else:
        got = norm.cpu().numpy()[sel].astype(np.float64)
        assert np.all(np.abs(got - ref["norm"]) <= 1e-6 * ref["norm"])
    # level indices: bit-exact except adjacent-bin flips inside the band around a boundary
    gi, ri = idx[sel].astype(np.int32), ref["idx"].astype(np.int32)
    flips = np.argwhere(gi != ri)
    tmax = np.abs(ref["unit"]).max(axis=1)
    ties = 0
    for r, k in flips:
        assert abs(gi[r, k] - ri[r, k]) == 1
        beta = ocbk.boundaries[min(gi[r, k], ri[r, k])]
        assert abs(ref["unit"][r, k] - beta) <= BAND * tmax[r]
        ties += ref["unit"][r, k] == beta          # exactly on a boundary: both neighbours are nearest (Eq. 3)
    return (len(flips) - ties) / gi.size


@pytest.mark.parametrize("bits", [4, 3, 2])
@pytest.mark.parametrize("d,block", [(1024, 128), (384, 64), (768, 256), (1024, 1024), (128, 8), (3072, 128),
                                     (5120, 256), (5120, 64), (13824, 128), (12288, 256), (1024, 256)])
def test_activation_rows_match_oracle(d, block, bits):
    xb = synth.activations(67 if d < 8000 else 21, d, seed=1000 + bits)   # ragged against any row tiling
    rate = check_rows(xb, block, 0, bits)
    assert rate <= 1e-4


@pytest.mark.parametrize("kernel", [GENERAL, REGISTERS, TENSOR, SLAB])
@pytest.mark.parametrize("bits", [4, 3, 2])
@pytest.mark.parametrize("d,n", [(128, 67), (256, 40), (1024, 67), (2048, 35), (3072, 67), (5120, 35), (12288, 21), (13824, 9)])
def test_every_kernel_matches_oracle_on_blocks_of_128(d, n, bits, kernel):
    """The four kernels compute the same function; blocks of 128 are the shape all of them support (the token-slab
    kernel from 1024 coordinates per row on; below that the selection falls back)."""
    xb = synth.activations(n, d, seed=1100 + bits)
    assert check_rows(xb, 128, 1, bits, kernel=kernel) <= 1e-4


@pytest.mark.parametrize("bits", [4, 3])
@pytest.mark.parametrize("block", [64, 256])
@pytest.mark.parametrize("d,n", [(256, 40), (1024, 67), (3072, 67), (5120, 35), (12288, 21), (13824, 9)])
@pytest.mark.parametrize("kernel", [TENSOR, SLAB])
def test_tensor_core_kernels_on_blocks_of_64_and_256(d, n, block, bits, kernel):
    """Blocks of 64 are two independent transforms per 128-coordinate tile row (block-diagonal operand); blocks of
    256 add one butterfly stage across the two tile rows of a block."""
    xb = synth.activations(n, d, seed=1300 + bits)
    assert check_rows(xb, block, 5, bits, kernel=kernel) <= 1e-4


@pytest.mark.parametrize("bits", [4, 3, 2])
@pytest.mark.parametrize("d,block,n", [(3072, 1024, 67), (3072, 512, 67), (5120, 1024, 35), (5120, 512, 35),
                                       (12288, 4096, 21), (12288, 2048, 21), (12288, 1024, 21), (13824, 512, 9),
                                       (1024, 1024, 40), (2048, 2048, 19), (4096, 4096, 9), (1024, 512, 67)])
def test_tensor_core_kernel_on_blocks_of_512_to_4096(d, block, n, bits):
    """The paper's default block is the largest power of two that divides the width (1024 for 3072 and 5120, 4096 for
    12288, 512 for 13824): H_{2^S} (x) H_128, i.e. S butterfly stages across the tile rows of a block after the
    tensor-core product.  The oracle applies the full-size Hadamard matrix."""
    xb = synth.activations(n, d, seed=1500 + bits)
    rot, cb = B.oq_make_rpbh(d, block, 6), B.oq_build_codebook(d, bits)
    B.oq_debug_select_rq_kernel(TENSOR)
    assert B.oq_rq_plan(rot, cb)[0] == TENSOR
    assert check_rows(xb, block, 6, bits, kernel=TENSOR) <= 1e-4


@pytest.mark.parametrize("n", [1, 3, 8, 9, 17])
@pytest.mark.parametrize("d,block", [(3072, 1024), (12288, 4096), (13824, 512)])
def test_large_blocks_with_few_rows_match_the_general_kernel(n, d, block):
    """Ragged groups with the multi-stage butterflies: rows that do not exist share warps with rows that do."""
    import torch
    xb = synth.activations(n, d, seed=1600 + n)
    rot, cb = B.oq_make_rpbh(d, block, 4), B.oq_build_codebook(d, 4)
    X = _dev(xb)
    B.oq_debug_select_rq_kernel(GENERAL)
    ref_idx, ref_norm = B.oq_rotate_quantize_act(X, rot, cb)
    B.oq_debug_select_rq_kernel(AUTO)
    assert B.oq_rq_plan(rot, cb)[0] == TENSOR
    idx, norm = B.oq_rotate_quantize_act(X, rot, cb)
    torch.cuda.synchronize()
    assert B.oq_device_status() == 0
    assert torch.allclose(norm, ref_norm, rtol=2e-6, atol=0)
    a = B.oq_unpack_indices(idx, n, d, 4).to(torch.int16)
    b = B.oq_unpack_indices(ref_idx, n, d, 4).to(torch.int16)
    diff = (a - b).abs()
    assert int(diff.max()) <= 1 and float((diff != 0).float().mean()) <= 2e-4


@pytest.mark.parametrize("kernel", [REGISTERS, TENSOR, SLAB])
def test_kernels_agree_with_each_other_on_many_groups(kernel):
    """More row groups than CTAs (several pipeline rounds per CTA), ragged last group: same packed words and
    norms (to rounding) as the general kernel."""
    import torch
    d, n = 1024, 148 * 16 * 3 + 5
    xb = synth.activations(n, d, seed=1200)
    rot, cb = B.oq_make_rpbh(d, 128, 2), B.oq_build_codebook(d, 4)
    X = _dev(xb)
    B.oq_debug_select_rq_kernel(GENERAL)
    ref_idx, ref_norm = B.oq_rotate_quantize_act(X, rot, cb)
    B.oq_debug_select_rq_kernel(kernel)
    idx, norm = B.oq_rotate_quantize_act(X, rot, cb)
    B.oq_debug_select_rq_kernel(AUTO)
    torch.cuda.synchronize()
    assert B.oq_device_status() == 0
    assert torch.allclose(norm, ref_norm, rtol=2e-6, atol=0)
    a = B.oq_unpack_indices(idx, n, d, 4).to(torch.int16)
    b = B.oq_unpack_indices(ref_idx, n, d, 4).to(torch.int16)
    diff = (a - b).abs()
    assert int(diff.max()) <= 1 and float((diff != 0).float().mean()) <= 1e-4


@pytest.mark.parametrize("kernel", [TENSOR, SLAB])
@pytest.mark.parametrize("n", [1, 2, 7, 8, 9, 15, 16, 17, 31, 33])
@pytest.mark.parametrize("d,block", [(3072, 128), (12288, 64), (5120, 256), (13824, 128), (1024, 128)])
def test_tensor_core_kernels_with_few_rows_and_padded_rows(n, d, block, kernel):
    """Fewer rows than one group, a ragged last group (also one whose second half is empty), and a leading dimension
    larger than dim: same indices as the general kernel (flips only between neighbours, rarely), same norms, and the
    all-zero row stays on the middle boundary."""
    import torch
    xb = synth.activations(n, d, seed=1400 + n)
    if n > 2:
        xb[n // 2, :] = 0
    rot, cb = B.oq_make_rpbh(d, block, 4), B.oq_build_codebook(d, 4)
    wide = torch.zeros((n, d + 64), dtype=torch.bfloat16, device="cuda")
    wide[:, :d] = _dev(xb)
    B.oq_debug_select_rq_kernel(GENERAL)
    ref_idx, ref_norm = B.oq_rotate_quantize_act(wide[:, :d], rot, cb)
    B.oq_debug_select_rq_kernel(kernel)
    assert B.oq_rq_plan(rot, cb)[0] == kernel
    idx, norm = B.oq_rotate_quantize_act(wide[:, :d], rot, cb)
    B.oq_debug_select_rq_kernel(AUTO)
    torch.cuda.synchronize()
    assert B.oq_device_status() == 0
    assert torch.allclose(norm, ref_norm, rtol=2e-6, atol=0)
    a = B.oq_unpack_indices(idx, n, d, 4).to(torch.int16)
    b = B.oq_unpack_indices(ref_idx, n, d, 4).to(torch.int16)
    diff = (a - b).abs()
    assert int(diff.max()) <= 1 and float((diff != 0).float().mean()) <= 1e-4
    if n > 2:
        assert norm[n // 2].item() == 0.0
        assert torch.all(a[n // 2] == 7)             # exact zero: the lower middle level (ties go down)


def test_config1_single_linear_activation_side():
    xb = synth.activations(256, 1024, seed=1000)
    assert check_rows(xb, 128, 0, 4) <= 1e-5


@pytest.mark.parametrize("bits", [4, 3, 2])
def test_weight_rows_match_oracle(bits):
    wb = synth.weights(200, 1024, seed=2000)
    wb[17, :] = 0
    assert check_rows(wb, 128, 0, bits, weights=True) <= 1e-4


def test_degenerate_tokens_and_strided_input():
    import torch
    d = 512
    x = np.zeros((5, d), np.float32)
    x[1, 100] = 30000.0
    x[2, :] = 1.5
    x[3, ::2] = -2.0 ** -120          # tiny values: squares underflow in fp32
    x[4, :] = np.random.default_rng(0).standard_normal(d) * 1e4
    xb = synth.to_bf16_bits(x)
    assert check_rows(xb, 128, 3, 4, rows=[0, 1, 2, 4]) <= 1e-4   # exact zeros sit on the middle boundary (ties)
    rot, cb = B.oq_make_rpbh(d, 128, 3), B.oq_build_codebook(d, 4)
    # leading dimension larger than dim
    wide = torch.zeros((5, d + 64), dtype=torch.bfloat16, device="cuda")
    wide[:, :d] = _dev(xb)
    a_idx, a_norm = B.oq_rotate_quantize_act(wide[:, :d], rot, cb)
    b_idx, b_norm = B.oq_rotate_quantize_act(_dev(xb), rot, cb)
    assert torch.equal(a_idx, b_idx) and torch.equal(a_norm, b_norm)
    assert a_norm[0].item() == 0.0
    z = B.oq_unpack_indices(a_idx, 5, d, 4)[0]
    assert torch.all(z == 7)           # t = 0 is equidistant from the two middle levels: ties go to the lower one


def test_empty_and_bad_arguments():
    import torch
    d = 256
    rot, cb = B.oq_make_rpbh(d, 128, 0), B.oq_build_codebook(d, 4)
    X = torch.zeros((0, d), dtype=torch.bfloat16, device="cuda")
    idx, nrm = B.oq_rotate_quantize_act(X, rot, cb)
    assert idx.shape[0] == 0 and nrm.numel() == 0
    with pytest.raises(B.OqError) as e:
        B.oq_rotate_quantize_act(torch.zeros((4, 384), dtype=torch.bfloat16, device="cuda"), rot, cb)
    assert e.value.code == 1
    X = torch.zeros((4, d + 8), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.OqError) as e:
        B.oq_rotate_quantize_act(X.view(-1)[1:1 + 4 * d].view(4, d), rot, cb)
    assert e.value.code == 3


@pytest.mark.parametrize("kernel", [AUTO, REGISTERS, TENSOR, SLAB])
def test_results_are_deterministic(kernel):
    import torch
    xb = synth.activations(300, 3072, seed=1001)
    rot, cb = B.oq_make_rpbh(3072, 128, 0), B.oq_build_codebook(3072, 4)
    X = _dev(xb)
    B.oq_debug_select_rq_kernel(kernel)
    a = B.oq_rotate_quantize_act(X, rot, cb)
    b = B.oq_rotate_quantize_act(X, rot, cb)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])


@pytest.mark.parametrize("d,block", [(3072, 1024), (12288, 4096), (13824, 512)])
def test_weight_rows_with_the_papers_default_blocks(d, block):
    """Offline weight quantization (Algorithm 1, "Offline") with the default block of each width: bf16 row norms."""
    wb = synth.weights(72, d, seed=2100 + block)
    wb[5, :] = 0
    assert check_rows(wb, block, 3, 4, weights=True) <= 1e-4
