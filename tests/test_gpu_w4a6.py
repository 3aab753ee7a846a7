"""GPU parity of the 6-bit activation path (W4A6, the video setting of Sec. 5.1): oq_rotate_quantize_act_levels and
oq_qlinear_levels against the CPU oracle.  The oracle's 64-level codebooks take minutes per width, so its centroids
are stored under tests/golden/ (written by tests/golden/make_codebook_b6.py from oracle.codebook alone)."""
import os

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

ROT_TOL = 1e-5
BAND = 1e-5
TOL_F32 = 1e-5
TOL_BF16 = 2e-3


def golden_centroids(d):
    path = os.path.join(os.path.dirname(__file__), "golden", f"lloyd_max_d{d}_b6.txt")
    return np.array([float(x) for x in open(path).read().split("\n") if x and not x.startswith("#")])


def _dev(bits_u16):
    import torch
    return torch.from_numpy(bits_u16.view(np.int16)).cuda().view(torch.bfloat16)


def _bits(t):
    import torch
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def quantize_and_check(xb, d, block, seed):
    """Runs the GPU pass and compares it with the oracle; returns (levels, norm, idx) of the GPU and the oracle's dict."""
    import torch
    n = xb.shape[0]
    cent = golden_centroids(d)
    bounds = 0.5 * (cent[:-1] + cent[1:])
    bounds[31] = 0.0
    rot, cb = B.oq_make_rpbh(d, block, seed), B.oq_build_codebook(d, 6)
    dbg = torch.full((n, d), float("nan"), dtype=torch.float32, device="cuda")
    lev, nrm, idx = B.oq_rotate_quantize_act_levels(_dev(xb), rot, cb, want_idx=True, dbg_rotated=dbg)
    torch.cuda.synchronize()
    assert B.oq_device_status() == 0
    perm, signs = orp.make_rpbh(d, block, seed)
    ref = oq.quantize_rows(xb, block, perm, signs, bounds)
    z_gpu, z_ref = dbg.cpu().numpy().astype(np.float64), ref["rotated"]
    assert np.all(np.abs(z_gpu - z_ref).max(axis=1) <= ROT_TOL * np.abs(z_ref).max(axis=1) + 1e-300)
    assert np.all(np.abs(nrm.cpu().numpy().astype(np.float64) - ref["norm"]) <= 1e-6 * ref["norm"])
    gi, ri = idx.cpu().numpy().astype(np.int32), ref["idx"].astype(np.int32)
    assert gi.min() >= 0 and gi.max() <= 63
    flips = np.argwhere(gi != ri)
    tmax = np.abs(ref["unit"]).max(axis=1)
    for r, k in flips:
        assert abs(gi[r, k] - ri[r, k]) == 1
        assert abs(ref["unit"][r, k] - bounds[min(gi[r, k], ri[r, k])]) <= BAND * tmax[r]
    assert len(flips) <= 2e-4 * gi.size
    # the level matrix is the bf16 table indexed by the GPU's own indices, bit for bit
    table = obf.f64_to_bf16_bits(cent)
    assert np.array_equal(_bits(lev), table[gi])
    return lev, nrm, gi, ref, cent


@pytest.mark.parametrize("d,block,n", [(3072, 128, 67), (3072, 1024, 35), (3072, 64, 33), (5120, 128, 35), (5120, 256, 19)])
def test_levels_indices_and_norms_match_oracle(d, block, n):
    xb = synth.activations(n, d, seed=5000 + n)
    if n > 4:
        xb[3, :] = 0                                   # an all-zero token: level 31 (ties go to the lower index), norm 0
    lev, nrm, gi, ref, cent = quantize_and_check(xb, d, block, 2)
    if n > 4:
        assert nrm[3].item() == 0.0 and np.all(gi[3] == 31)


@pytest.mark.parametrize("n,m,d", [(200, 520, 3072), (257, 264, 5120)])
def test_w4a6_linear_matches_oracle(n, m, d):
    import torch
    xb, wb = synth.activations(n, d, seed=5100 + n), synth.weights(m, d, seed=5200 + m)
    lev, nrm, gi, ref, cent = quantize_and_check(xb, d, 128, 0)
    rot, cbw = B.oq_make_rpbh(d, 128, 0), B.oq_build_codebook(d, 4)
    wq, wr = B.oq_quantize_weights(_dev(wb), rot, cbw)
    y32 = B.oq_qlinear_levels(lev, nrm, wq, wr, cbw, d, out_dtype=torch.float32)
    y16 = B.oq_qlinear_levels(lev, nrm, wq, wr, cbw, d)
    torch.cuda.synchronize()
    assert B.oq_device_status() == 0
    ow = ocb.lloyd_max(d, 4)
    levels_a = obf.bf16_bits_to_f64(obf.f64_to_bf16_bits(cent))
    iw = B.oq_unpack_indices(wq, m, d, 4).cpu().numpy()
    r = obf.bf16_bits_to_f64(_bits(wr))
    # operand-exact: the GPU's own indices and norms, fp64 product
    exact = oql.qlinear(gi, nrm.cpu().numpy(), levels_a, iw, r, ow.centroids_decoded)
    g32, g16 = y32.cpu().numpy().astype(np.float64), y16.float().cpu().numpy().astype(np.float64)
    assert np.linalg.norm(g32 - exact) <= TOL_F32 * np.linalg.norm(exact)
    assert np.linalg.norm(g16 - exact) <= TOL_BF16 * np.linalg.norm(exact)
    # end to end: the oracle quantizes the raw inputs itself
    perm, signs = orp.make_rpbh(d, 128, 0)
    qw = oq.quantize_weight_rows(wb, 128, perm, signs, ow.boundaries)
    e2e = oql.qlinear(ref["idx"], ref["norm"].astype(np.float32), levels_a, qw["idx"],
                      obf.bf16_bits_to_f64(qw["norm_bf16_bits"]), ow.centroids_decoded)
    assert np.linalg.norm(g16 - e2e) <= TOL_BF16 * np.linalg.norm(e2e)
    # six bits of activation are closer to the unquantized layer than four
    x = obf.bf16_bits_to_f64(xb)
    w = obf.bf16_bits_to_f64(wb)
    dense = x @ w.T
    cba4 = B.oq_build_codebook(d, 4)
    xq4, xs4 = B.oq_rotate_quantize_act(_dev(xb), rot, cba4)
    y4 = B.oq_qlinear(xq4, xs4, cba4, wq, wr, cbw, d, out_dtype=torch.float32).cpu().numpy().astype(np.float64)
    assert np.linalg.norm(g32 - dense) < np.linalg.norm(y4 - dense)


def test_full_flux_size_on_sampled_rows_and_outputs():
    """4608 tokens x 3072 -> 9216 (the FLUX qkv layer) in the launch configuration the block-step benchmark times:
    sampled token rows against the oracle's quantizer, sampled outputs against its fp64 product."""
    import torch
    n, d, m = 4608, 3072, 9216
    xb, wb = synth.activations(n, d, seed=5300), synth.weights(m, d, seed=5301)
    cent = golden_centroids(d)
    bounds = 0.5 * (cent[:-1] + cent[1:])
    bounds[31] = 0.0
    rot, cba, cbw = B.oq_make_rpbh(d, 128, 0), B.oq_build_codebook(d, 6), B.oq_build_codebook(d, 4)
    lev, nrm, idx = B.oq_rotate_quantize_act_levels(_dev(xb), rot, cba, want_idx=True)
    wq, wr = B.oq_quantize_weights(_dev(wb), rot, cbw)
    y = B.oq_qlinear_levels(lev, nrm, wq, wr, cbw, d, out_dtype=torch.float32)
    torch.cuda.synchronize()
    assert B.oq_device_status() == 0
    rng = np.random.default_rng(7)
    rows = np.unique(np.concatenate([[0, 1, 127, 128, 255, 256, n - 257, n - 256, n - 2, n - 1], rng.choice(n, 246, replace=False)]))
    perm, signs = orp.make_rpbh(d, 128, 0)
    ref = oq.quantize_rows(xb[rows], 128, perm, signs, bounds)
    gi = idx.cpu().numpy()[rows].astype(np.int32)
    ri = ref["idx"].astype(np.int32)
    diff = np.abs(gi - ri)
    assert diff.max() <= 1 and (diff != 0).mean() <= 2e-4
    assert np.all(np.abs(nrm.cpu().numpy()[rows].astype(np.float64) - ref["norm"]) <= 1e-6 * ref["norm"])
    assert np.array_equal(_bits(lev)[rows], obf.f64_to_bf16_bits(cent)[gi])
    cols = np.unique(np.concatenate([[0, 255, 256, m - 1], rng.choice(m, 252, replace=False)]))
    ow = ocb.lloyd_max(d, 4)
    iw = B.oq_unpack_indices(wq, m, d, 4).cpu().numpy()[cols]
    r = obf.bf16_bits_to_f64(_bits(wr))[cols]
    levels_a = obf.bf16_bits_to_f64(obf.f64_to_bf16_bits(cent))
    exact = oql.qlinear(gi, nrm.cpu().numpy()[rows], levels_a, iw, r, ow.centroids_decoded)
    got = y.cpu().numpy().astype(np.float64)[np.ix_(rows, cols)]
    assert np.linalg.norm(got - exact) <= TOL_F32 * np.linalg.norm(exact)


def test_host_buffer_layer_call_with_6bit_activations():
    """oq_linear_forward_host with a 64-level activation codebook: same bits as the two calls made by hand."""
    import torch
    n, m, d = 300, 520, 3072
    xb, wb = synth.activations(n, d, seed=5400), synth.weights(m, d, seed=5401)
    rot, cba, cbw = B.oq_make_rpbh(d, 128, 0), B.oq_build_codebook(d, 6), B.oq_build_codebook(d, 4)
    wq, wr = B.oq_quantize_weights(_dev(wb), rot, cbw)
    lev, nrm, _ = B.oq_rotate_quantize_act_levels(_dev(xb), rot, cba)
    want = B.oq_qlinear_levels(lev, nrm, wq, wr, cbw, d)
    Xh = torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16).pin_memory()
    Yh = torch.empty((n, m), dtype=torch.bfloat16).pin_memory()
    ws = torch.empty(B.oq_forward_workspace_bytes(n, d, m, 6), dtype=torch.uint8, device="cuda")
    B.oq_linear_forward_host(Xh, rot, cba, wq, wr, cbw, Yh, ws)
    torch.cuda.synchronize()
    assert B.oq_device_status() == 0
    assert torch.equal(Yh, want.cpu())
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.OqError) as e:
        B.oq_linear_forward_host(Xh, rot, cba, wq, wr, cbw, Yh, small)
    assert e.value.code == 6
