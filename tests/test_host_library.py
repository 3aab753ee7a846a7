"""CPU-only checks of liboq.so: it loads, exports every declared symbol, and its host-side offline
constructors agree with the independent oracle."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import codebook as ocb
from oracle import rpbh as orp
from paper_2607_02461_b200 import binding as B
from paper_2607_02461_b200 import build as oqbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    oqbuild.build()


def test_library_exports_every_declared_symbol():
    text = open(os.path.join(ROOT, "include", "oq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = set(re.findall(r"\b(oq_[a-z0-9_]+)\s*\(", text))
    assert {"oq_build_codebook", "oq_make_rpbh", "oq_quantize_weights", "oq_rotate_quantize_act", "oq_qlinear"} <= names
    L = ctypes.CDLL(os.path.join(ROOT, "paper_2607_02461_b200", "liboq.so"))
    for n in sorted(names):
        assert hasattr(L, n), f"{n} is declared in include/oq.h but not exported"
    assert B.oq_version().startswith("liboq")


@pytest.mark.parametrize("dim,bits", [(64, 1), (128, 2), (1024, 4), (3072, 3), (5120, 4), (12288, 2), (13824, 4)])
def test_codebook_matches_oracle(dim, bits):
    got, want = B.oq_build_codebook(dim, bits), ocb.lloyd_max(dim, bits)
    assert np.abs(got.centroids / want.centroids - 1).max() < 1e-11
    nz = want.boundaries != 0
    assert np.abs(got.boundaries[nz] / want.boundaries[nz] - 1).max() < 1e-11 if nz.any() else True
    assert got.boundaries[(1 << bits) // 2 - 1] == 0.0
    assert np.array_equal(got.boundaries_f32, want.boundaries_f32)          # bit-exact after rounding
    assert np.array_equal(got.centroids_bf16_bits, want.centroids_bf16_bits)


@pytest.mark.parametrize("dim,block,seed", [(8, 4, 0), (1024, 128, 0), (3072, 64, 7), (5120, 256, 1),
                                            (13824, 128, 0), (1920, 128, 2 ** 63 + 5)])
def test_rpbh_draw_is_bit_exact(dim, block, seed):
    got = B.oq_make_rpbh(dim, block, seed)
    perm, signs = orp.make_rpbh(dim, block, seed)
    assert np.array_equal(got.perm, perm) and np.array_equal(got.signs, signs)


def test_argument_errors():
    with pytest.raises(B.OqError) as e:
        B.oq_build_codebook(1024, 5)
    assert e.value.code == 2
    with pytest.raises(B.OqError) as e:
        B.oq_build_codebook(4, 2)
    assert e.value.code == 2
    with pytest.raises(B.OqError) as e:
        B.oq_make_rpbh(1000, 128, 0)
    assert e.value.code == 1
    with pytest.raises(B.OqError) as e:
        B.oq_make_rpbh(1024, 96, 0)
    assert e.value.code == 1
    with pytest.raises(B.OqError) as e:
        B.oq_make_rpbh(70000, 16, 0)
    assert e.value.code == 2
    with pytest.raises(B.OqError) as e:
        B.oq_packed_bytes(4, 1000, 4)
    assert e.value.code == 2
    assert B.lib().oq_build_codebook(1024, 4, None) == 1


def test_packed_sizes():
    assert B.oq_packed_bytes(256, 1024, 4) == (256 * 512, 512)
    assert B.oq_packed_bytes(3, 3072, 3) == (3 * 1152, 1152)
    assert B.oq_packed_bytes(0, 128, 2) == (0, 32)
    for d in (128, 1024, 13824):
        for b in (2, 3, 4):
            assert B.oq_packed_bytes(1, d, b)[1] % 16 == 0 and B.oq_packed_bytes(1, d, b)[1] * 8 == d * b


@pytest.mark.parametrize("dim,bits", [(64, 4), (1024, 4), (13824, 4), (3072, 3), (5120, 2), (128, 3)])
def test_level_search_polynomial_counts_boundaries(dim, bits):
    """The kernels find a level as floor(P(x)) with P evaluated in fp32 (fused multiply-adds, the last one
    adding 1.5 * 2^23 so that the integer part lands in the low mantissa bits).  Emulate exactly that and
    compare with the oracle's boundary count on a fine grid; mismatches may only sit within 1e-6 of a
    boundary (relative to the largest boundary)."""
    import ctypes as C
    cb = B.oq_build_codebook(dim, bits)
    coef = (C.c_float * 8)()
    clamp, centre, mid, deg = C.c_float(), C.c_float(), C.c_float(), C.c_int()
    L = B.lib()
    L.oq_codebook_level_poly.restype = C.c_int
    assert L.oq_codebook_level_poly(cb.handle, coef, C.byref(clamp), C.byref(centre), C.byref(mid), C.byref(deg)) == 0
    nb = (1 << bits) // 2 - 1
    assert deg.value == nb
    beta = ocb.lloyd_max(dim, bits).boundaries[nb + 1:]
    f32 = np.float32

    def fma(a, b, c):
        return (a.astype(np.float64) * np.asarray(b, np.float64) + np.float64(c)).astype(f32)

    t = np.concatenate([np.linspace(0, 1.3 * beta[-1], 1000001), np.linspace(1.3 * beta[-1], 1.0, 1001)])
    for s in (3.7, 1e-3, 4e4, 0.0):
        h = 128
        z = (t * np.sqrt(h) * (s + 1e-10)).astype(f32)
        kappa = f32(1.0) / f32(f32(np.sqrt(f32(h))) * f32(f32(s) + f32(1e-10)) * clamp.value)
        x = np.clip(fma(np.abs(z), kappa, 0.0), 0, 1)
        y = fma(x, f32(2), -centre.value)
        acc = np.full_like(y, coef[nb])
        for k in range(nb - 1, 0, -1):
            acc = fma(acc, y, coef[k])
        v = fma(acc, y, f32(mid.value + 12582912.0))
        mag = v.view(np.uint32).astype(np.int64) - 0x4B400000
        texact = z.astype(np.float64) / (np.sqrt(h) * (s + 1e-10))
        want = np.searchsorted(beta, texact, side="left")
        bad = mag != want
        assert mag.min() >= 0 and mag.max() <= nb
        if bad.any():
            dist = np.min(np.abs(texact[bad][:, None] - beta[None, :]), axis=1)
            assert dist.max() <= 1e-6 * beta[-1] and np.abs(mag - want)[bad].max() == 1


@pytest.mark.parametrize("dim,block,kernel,rows,tiles,slab", [
    (3072, 128, 3, 16, 3, 8),      # FLUX hidden size: 8 tokens per half group, 192 (token, block) pairs per half
    (12288, 128, 3, 4, 3, 2),      # FLUX MLP width
    (5120, 128, 3, 8, 3, 4),       # Wan hidden size: 160 pairs per half
    (13824, 128, 3, 2, 2, 2),      # Wan FFN width: 108 pairs per half, one tile per half
    (1024, 128, 2, 16, 0, 8),      # 64 pairs per half would fill half of the tiles: register kernel
    (3072, 64, 3, 16, 3, 8),       # blocks of 64 and 256 use the same 128-coordinate tile rows
    (3072, 256, 3, 16, 3, 8),
    (1024, 256, 2, 8, 0, 8),
    (3072, 1024, 3, 16, 3, 0),     # the paper's default blocks: same group shapes as blocks of 128
    (5120, 1024, 3, 8, 3, 0),
    (12288, 4096, 3, 4, 3, 0),
    (13824, 512, 3, 2, 2, 0),
    (1024, 1024, 1, 1, 0, 0),      # a quarter-full tile: general kernel
])
def test_rotate_quantize_plan(dim, block, kernel, rows, tiles, slab):
    """Host-side launch planning (no device needed): kernel choice and group shape for the benchmark widths; `slab` =
    tokens per slab of the token-slab kernel when it is selected (0: it does not take this block size)."""
    rot, cb = B.oq_make_rpbh(dim, block, 0), B.oq_build_codebook(dim, 4)
    k, r, t, smem = B.oq_rq_plan(rot, cb)
    assert (k, r, t) == (kernel, rows, tiles)
    assert smem <= 227 * 1024
    B.oq_debug_select_rq_kernel(1)
    try:
        assert B.oq_rq_plan(rot, cb)[0] == 1
        B.oq_debug_select_rq_kernel(4)
        k4, r4, t4, smem4 = B.oq_rq_plan(rot, cb)
        if slab:
            assert (k4, r4, t4) == (4, slab, 1) and smem4 <= 227 * 1024
        else:
            assert k4 != 4                 # falls back
    finally:
        B.oq_debug_select_rq_kernel(0)


def test_rotate_quantize_plan_rejects_mismatched_handles():
    rot = B.oq_make_rpbh(1024, 128, 0)
    with pytest.raises(B.OqError) as e:
        B.oq_rq_plan(rot, B.oq_build_codebook(2048, 4))
    assert e.value.code == 1
    with pytest.raises(B.OqError) as e:
        B.oq_debug_select_rq_kernel(7)
    assert e.value.code == 1
    with pytest.raises(B.OqError) as e:
        B.oq_debug_select_gemm_kernel(4)
    assert e.value.code == 1
    for k in (1, 2, 3, 0):
        B.oq_debug_select_gemm_kernel(k)
    # a width that is not a multiple of 128 has no fast path at all
    with pytest.raises(B.OqError) as e:
        B.oq_rq_plan(B.oq_make_rpbh(192, 64, 0), B.oq_build_codebook(192, 4))
    assert e.value.code == 2


def test_6bit_codebook_matches_the_stored_oracle_codebook():
    """64 levels (activations of the W4A6 setting): the library's Lloyd iteration against the oracle's centroids stored
    under tests/golden/, and the bf16 decode table."""
    import os
    from oracle import bf16 as obf
    for d in (3072, 5120):
        path = os.path.join(os.path.dirname(__file__), "golden", f"lloyd_max_d{d}_b6.txt")
        cent = np.array([float(x) for x in open(path).read().split("\n") if x and not x.startswith("#")])
        cb = B.oq_build_codebook(d, 6)
        assert np.allclose(cb.centroids, cent, rtol=1e-9, atol=0)
        assert np.array_equal(cb.centroids_bf16_bits, obf.f64_to_bf16_bits(cent))
        assert cb.boundaries[31] == 0.0 and np.all(np.diff(cb.boundaries) > 0)
    with pytest.raises(B.OqError) as e:
        B.oq_build_codebook(1024, 5)
    assert e.value.code == 2


def test_argument_checks_of_the_newer_entry_points_need_no_device():
    """Validation comes before any CUDA call: these return their error codes on a machine without a GPU."""
    L = B.lib()
    rot = B.oq_make_rpbh(3072, 128, 0)
    cb4, cb6 = B.oq_build_codebook(3072, 4), B.oq_build_codebook(3072, 6)
    null = ctypes.c_void_p(0)
    # 6-bit rotate+quantize wants a 6-bit codebook, and matching dims
    assert L.oq_rotate_quantize_act_levels(null, 4, 3072, 3072, rot.handle, cb4.handle, null, 3072, null, null, null, null) == 2
    assert L.oq_rotate_quantize_act_levels(null, 4, 1024, 1024, rot.handle, cb6.handle, null, 1024, null, null, null, null) == 1
    assert L.oq_rotate_quantize_act_levels(null, 0, 3072, 3072, rot.handle, cb6.handle, null, 3072, null, null, null, null) == 0
    assert L.oq_rotate_quantize_act_levels(null, 4, 3072, 3072, rot.handle, cb6.handle, null, 3072, null, null, null, null) == 1
    # the packed-index calls refuse a 6-bit codebook
    assert L.oq_rotate_quantize_act(null, 4, 3072, 3072, rot.handle, cb6.handle, null, null, null, null) == 2
    with pytest.raises(B.OqError) as e:
        B.oq_packed_bytes(4, 3072, 6)
    assert e.value.code == 2
    # level-matrix GEMM and decode
    assert L.oq_qlinear_levels(null, 3072, null, 4, null, null, 8, cb6.handle, 3072, null, 8, 0, null) == 2      # weight bits
    assert L.oq_qlinear_levels(null, 3072, null, 4, null, null, 8, cb4.handle, 3072, null, 8, 0, null) == 1      # NULL buffers
    assert L.oq_qlinear_levels(null, 3072, null, 0, null, null, 8, cb4.handle, 3072, null, 8, 0, null) == 0      # nothing to do
    assert L.oq_decode_levels(null, 4, 3072, cb6.handle, null, 3072, null) == 2
    assert L.oq_decode_levels(null, 4, 3072, None, null, 3072, null) == 1
    # AdaLN shapes
    assert L.oq_adaln_linear(null, 1, 128, null, null, 24, 128, null, 24, 0, null) == 2
    assert L.oq_adaln_linear(null, 1, 128, null, null, 32, 128, null, 32, 0, null) == 1
    assert L.oq_adaln_quantize_weights(null, 32, 96, 96, null, null, null) == 2
    assert B.oq_adaln_packed_bytes(32, 128) == (32 * 128 // 2, 2 * 32 * 128 // 64)
    assert B.oq_forward_workspace_bytes(10, 3072, 16, 6) > B.oq_forward_workspace_bytes(10, 3072, 16, 4)


def test_handles_and_errors_from_several_threads():
    """Handles may be built and used from several host threads at once; oq_last_error is per thread."""
    import threading
    results, errors = {}, []

    def work(k):
        try:
            cb = B.oq_build_codebook(1024 + 128 * k, 4)
            rot = B.oq_make_rpbh(1024 + 128 * k, 128, k)
            results[k] = (cb.centroids.copy(), rot.perm.copy(), B.oq_rq_plan(rot, cb)[0])
            try:
                B.oq_make_rpbh(100 + k, 64, 0)            # 64 does not divide 100 + k: an error on this thread only
            except B.OqError as e:
                results[("err", k)] = str(e)
        except Exception as e:      # pragma: no cover
            errors.append(repr(e))

    ts = [threading.Thread(target=work, args=(k,)) for k in range(6)]
    for t in ts:
        t.start()
    for t in ts:
        t.join()
    assert not errors
    for k in range(6):
        cb = B.oq_build_codebook(1024 + 128 * k, 4)
        rot = B.oq_make_rpbh(1024 + 128 * k, 128, k)
        assert np.array_equal(results[k][0], cb.centroids) and np.array_equal(results[k][1], rot.perm)
        assert ("err", k) in results and results[("err", k)]


def test_reference_arm_prints_the_contract_keys():
    """`bench.py --impl reference` (the CPU oracle timed on a bounded sample) prints one JSON line with the keys the
    benchmark contract asks for."""
    import json
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    res = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0",
                          "--workload", "single_w4a4"], capture_output=True, text=True, timeout=600, env=env)
    assert res.returncode == 0, res.stderr[-2000:]
    line = json.loads([l for l in res.stdout.splitlines() if l.startswith("{")][-1])
    for key in ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"):
        assert key in line, key
    assert line["impl"] == "reference" and line["value"] > 0 and line["config"]["workload"] == "single_w4a4"
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
