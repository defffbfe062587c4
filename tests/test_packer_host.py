"""Host-side checks that need no GPU: the shared library loads and exports what the header
declares, and the C++ packer agrees bit-for-bit with the oracle's independent packer."""
import os
import re

import numpy as np
import pytest

from oracle import bcr_oracle as orc
from workloads import generators as gen

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2108_11033_b200.build import build_library
    build_library()
    from paper_2108_11033_b200 import binding
    return binding


def test_library_exports_every_declared_symbol(B):
    hdr = open(os.path.join(ROOT, "include", "grim.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(grim_[a-z0-9_]+)\s*\(", hdr))
    assert declared, "no declarations parsed"
    assert declared == set(B.EXPORTED)
    for name in declared:
        assert hasattr(B.lib, name), name
    assert "sm_100a" in B.grim_version()
    assert B.status_string(B.GRIM_ERR_NOT_BCR).startswith("mask")


CASES = [
    (256, 256, 16, 16, dict(dist="fixed", kr_fixed=8, kc_fixed=8)),
    (64, 27, 8, 32, dict(compression=8, dist="uniform")),
    (96, 153, 8, 32, dict(compression=10, dist="uniform")),
    (128, 256, 4, 16, dict(compression=16, dist="zipf")),
    (50, 200, 16, 64, dict(compression=4, dist="zipf", empty_frac=0.3)),
    (7, 5, 1, 1, dict(compression=2, dist="uniform")),
]


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("reorder", [False, True])
@pytest.mark.parametrize("case", CASES)
def test_pack_export_matches_oracle_bytes(B, case, reorder, dtype):
    M, K, bh, bw, kw = case
    W = gen.dense_weight(M, K, seed=50)
    mask = gen.bcr_mask(M, K, bh, bw, seed=51, **kw)
    flags = B.GRIM_PACK_HOST_ONLY | (B.GRIM_PACK_REORDER if reorder else 0)
    h = B.grim_bcr_pack(W, mask, bh, bw, dtype, flags)
    try:
        want = orc.pack_canonical(W, mask, bh, bw, dtype, reorder)
        got = B.grim_bcr_export(h)
        assert got == want
        info = B.grim_bcr_info(h)
        assert info.nnz == int(mask.sum()) and info.export_bytes == len(want)
        assert (info.M, info.K, info.bh, info.bw, info.on_device) == (M, K, bh, bw, 0)
        assert info.k_used == int((mask.sum(axis=0) > 0).sum())
        dense = B.grim_bcr_unpack_dense(h)
        assert np.array_equal(dense.astype(np.float64), orc.masked_weight(W, mask, dtype))
    finally:
        B.grim_bcr_destroy(h)


def test_pack_rejects_bad_input(B):
    W = gen.dense_weight(16, 32, seed=52)
    mask = gen.bcr_mask(16, 32, 8, 16, dist="fixed", kr_fixed=4, kc_fixed=8, seed=53)
    bad = mask.copy()
    r, c = np.argwhere(mask)[3]
    bad[r, c] = 0
    with pytest.raises(B.GrimError) as e:
        B.grim_bcr_pack(W, bad, 8, 16, 0, B.GRIM_PACK_HOST_ONLY)
    assert e.value.status == B.GRIM_ERR_NOT_BCR
    with pytest.raises(B.GrimError) as e:
        B.grim_bcr_pack(W, mask, 32, 16, 0, B.GRIM_PACK_HOST_ONLY)
    assert e.value.status == B.GRIM_ERR_UNSUPPORTED
    with pytest.raises(B.GrimError) as e:
        B.grim_bcr_pack(W, mask, 8, 16, 0, 64)
    assert e.value.status == B.GRIM_ERR_INVALID_ARG
    with pytest.raises(B.GrimError) as e:
        B.grim_bcr_pack(W, mask, 8, 16, 5, B.GRIM_PACK_HOST_ONLY)
    assert e.value.status == B.GRIM_ERR_DTYPE
    assert B.lib.grim_bcr_pack(None, 32, mask.ctypes.data, 32, 16, 32, 8, 16, 0, 2, None) == B.GRIM_ERR_INVALID_ARG
    # the mask is authoritative: a kept weight that is 0.0 stays stored
    W0 = W.copy()
    W0[r, c] = 0.0
    h = B.grim_bcr_pack(W0, mask, 8, 16, 0, B.GRIM_PACK_HOST_ONLY)
    assert B.grim_bcr_info(h).nnz == int(mask.sum())
    assert B.grim_bcr_export(h) == orc.pack_canonical(W0, mask, 8, 16, 0, False)
    B.grim_bcr_destroy(h)


def test_host_only_handle_refuses_compute(B):
    W = gen.dense_weight(16, 32, seed=54)
    mask = gen.bcr_mask(16, 32, 8, 16, dist="fixed", kr_fixed=4, kc_fixed=8, seed=55)
    h = B.grim_bcr_pack(W, mask, 8, 16, 0, B.GRIM_PACK_HOST_ONLY)
    mx = B.grim_mat_t(1, 32, 4, 4, 0)
    my = B.grim_mat_t(1, 16, 4, 4, 0)
    import ctypes as C
    assert B.lib.grim_bcr_spmm(h, C.byref(mx), C.byref(my), None) == B.GRIM_ERR_INVALID_ARG
    B.grim_bcr_destroy(h)


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("case", CASES)
def test_bcrc_export_matches_oracle(B, case, dtype):
    """The library's BCRC export (Section 4.3) against the oracle's, array by array."""
    M, K, bh, bw, kw = case
    W = gen.dense_weight(M, K, seed=56)
    mask = gen.bcr_mask(M, K, bh, bw, seed=57, **kw)
    h = B.grim_bcr_pack(W, mask, bh, bw, dtype, B.GRIM_PACK_HOST_ONLY)
    try:
        got = B.grim_bcr_export_bcrc(h)
        want = orc.bcrc_export(W, mask, dtype)
        for k in ("reorder", "row_offset", "occurrence", "column_stride", "compact_column"):
            assert np.array_equal(got[k], want[k]), k
        assert np.array_equal(got["weights"].view(np.uint32), want["weights"].view(np.uint32))
    finally:
        B.grim_bcr_destroy(h)


@pytest.mark.parametrize("case", [(24, 40, 4, 8, 0.6), (19, 45, 4, 16, 0.75), (32, 64, 8, 32, 0.875), (7, 5, 1, 1, 0.5),
                                  (16, 70, 16, 64, 0.5)])
def test_projection_matches_oracle(B, case):
    """The library's projection onto the BCR set (Section 5.2) takes the same decisions as the oracle's naive loop:
    masks equal bit for bit; and what it returns can be packed."""
    M, K, bh, bw, sparsity = case
    V = gen.normal_f32((M, K), 1.0, 58, 0)
    got = B.grim_bcr_project(V, bh, bw, sparsity)
    assert np.array_equal(got, orc.bcr_project(V, bh, bw, sparsity))
    h = B.grim_bcr_pack(V, got, bh, bw, 0, B.GRIM_PACK_HOST_ONLY)
    assert B.grim_bcr_info(h).nnz == int(got.sum()) <= np.floor((1 - sparsity) * M * K + 1e-9)
    B.grim_bcr_destroy(h)
