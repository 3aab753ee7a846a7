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
