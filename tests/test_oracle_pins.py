"""Pins for the CPU oracle: checks against things the paper and the mathematics fix, none of
which re-use the oracle's own formula (brute-force loops, library routines on special
cases, printed counting examples, invariants)."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import bcr_oracle as orc
from workloads import generators as gen

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden_counts():
    out = {}
    with open(os.path.join(GOLDEN, "section3_counts.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split()
            out[k] = int(v)
    return out


def _brute_spmm(W, rowlists, collists, bh, bw, X):
    """Explicit loops over blocks, kept rows and kept columns (pure Python, exact fractions of fp64)."""
    M, K = W.shape
    N = X.shape[1]
    nbc = -(-K // bw)
    Y = [[0.0] * N for _ in range(M)]
    for b, (rows, cols) in enumerate(zip(rowlists, collists)):
        i, j = divmod(b, nbc)
        for a in rows:
            for c in cols:
                w = float(W[i * bh + a, j * bw + c])
                for n in range(N):
                    Y[i * bh + a][n] += w * float(X[j * bw + c, n])
    return np.array(Y)


def _mask_from_lists(M, K, bh, bw, rowlists, collists):
    nbc = -(-K // bw)
    m = np.zeros((M, K), np.uint8)
    for b, (rows, cols) in enumerate(zip(rowlists, collists)):
        i, j = divmod(b, nbc)
        for a in rows:
            for c in cols:
                m[i * bh + a, j * bw + c] = 1
    return m


# ---------------------------------------------------------------------------- multiply


def test_spmm_all_patterns_of_one_block_brute_force():
    """8x8 matrix, 4x4 blocks: block (0,1) runs through all 2^4 x 2^4 keep patterns."""
    g = np.random.default_rng(7)
    W = g.standard_normal((8, 8)).astype(np.float32)
    X = g.standard_normal((8, 3))
    fixed = [([0, 2], [1, 3]), None, ([1], [0, 1, 2]), ([0, 1, 2, 3], [2])]
    for rbits, cbits in itertools.product(range(16), range(16)):
        rows = [r for r in range(4) if rbits >> r & 1]
        cols = [c for c in range(4) if cbits >> c & 1]
        if (not rows) != (not cols):
            continue  # a mask cannot keep rows of a block without keeping columns
        lists = list(fixed)
        lists[1] = (rows, cols)
        rl = [l[0] for l in lists]
        cl = [l[1] for l in lists]
        mask = _mask_from_lists(8, 8, 4, 4, rl, cl)
        want = _brute_spmm(W, rl, cl, 4, 4, X)
        got = orc.spmm(W, mask, X)
        np.testing.assert_allclose(got, want, rtol=0, atol=1e-13)


def test_spmm_brute_force_ragged_grid():
    g = np.random.default_rng(8)
    M, K, bh, bw = 11, 13, 4, 5
    rk, ck = gen.bcr_keep_lists(M, K, bh, bw, compression=3, dist="uniform", seed=9)
    mask = gen.mask_from_keep(rk, ck, M, K)
    W = g.standard_normal((M, K)).astype(np.float32)
    X = g.standard_normal((K, 4))
    nbr, nbc = rk.shape[:2]
    rl = [list(np.flatnonzero(rk[i, j])) for i in range(nbr) for j in range(nbc)]
    cl = [list(np.flatnonzero(ck[i, j])) for i in range(nbr) for j in range(nbc)]
    np.testing.assert_allclose(orc.spmm(W, mask, X), _brute_spmm(W, rl, cl, bh, bw, X), rtol=0, atol=1e-13)


def test_spmm_all_kept_equals_library_matmul():
    g = np.random.default_rng(1)
    W = g.standard_normal((37, 29)).astype(np.float32)
    X = g.standard_normal((29, 5))
    want = (torch.from_numpy(W).double() @ torch.from_numpy(X)).numpy()
    np.testing.assert_allclose(orc.spmm(W, np.ones_like(W, np.uint8), X), want, rtol=1e-14, atol=1e-14)


def test_spmm_vector_input_is_gemv():
    g = np.random.default_rng(2)
    W = g.standard_normal((16, 16)).astype(np.float32)
    mask = gen.bcr_mask(16, 16, 4, 8, compression=2, seed=3)
    x = g.standard_normal(16)
    y = orc.spmm(W, mask, x)
    assert y.shape == (16, 1)
    for r in range(16):
        want = math.fsum(float(W[r, c]) * x[c] for c in range(16) if mask[r, c])
        assert abs(y[r, 0] - want) < 1e-13


def test_degenerate_block_sizes():
    """Section 3.2: 1x1 blocks are non-structured pruning; one block is whole row/column pruning."""
    g = np.random.default_rng(3)
    W = g.standard_normal((6, 7)).astype(np.float32)
    X = g.standard_normal((7, 2))
    # 1x1 blocks: any mask is valid
    mask = (g.random((6, 7)) < 0.4).astype(np.uint8)
    _, ok = orc.extract_blocks(mask, 1, 1)
    assert ok
    want = np.array([[math.fsum(float(W[r, c]) * X[c, n] for c in range(7) if mask[r, c]) for n in range(2)]
                     for r in range(6)])
    np.testing.assert_allclose(orc.spmm(W, mask, X), want, atol=1e-13)
    # one block: keep rows {0,2,5}, columns {1,2,6}
    rows, cols = [0, 2, 5], [1, 2, 6]
    mask = np.zeros((6, 7), np.uint8)
    mask[np.ix_(rows, cols)] = 1
    blocks, ok = orc.extract_blocks(mask, 6, 7)
    assert ok and list(blocks[0][0]) == rows and list(blocks[0][1]) == cols
    want = np.zeros((6, 2))
    want[rows] = W[np.ix_(rows, cols)].astype(np.float64) @ X[cols]
    np.testing.assert_allclose(orc.spmm(W, mask, X), want, atol=1e-13)


def test_pruned_rows_are_exactly_zero():
    g = np.random.default_rng(4)
    M, K, bh, bw = 32, 64, 8, 16
    rk, ck = gen.bcr_keep_lists(M, K, bh, bw, compression=4, seed=5)
    rk[:, :, 3] = False  # local row 3 kept in no block of any band
    mask = gen.mask_from_keep(rk, ck, M, K)
    W = g.standard_normal((M, K)).astype(np.float32)
    Y = orc.spmm(W, mask, g.standard_normal((K, 9)))
    dead = np.flatnonzero(mask.sum(axis=1) == 0)
    assert set(range(3, M, bh)) <= set(dead)
    assert np.all(Y[dead] == 0.0) and not np.any(np.signbit(Y[dead]))
    assert np.all(np.abs(Y[np.setdiff1d(np.arange(M), dead)]).sum(axis=1) > 0)


# ---------------------------------------------------------------------------- counting examples


def test_block_orientation_and_search_space_example():
    c = _golden_counts()
    M, K, bh, bw = c["layer_rows"], c["layer_cols"], c["block_rows"], c["block_cols"]
    assert M * K == c["total_weights"]
    nbr, nbc = M // bh, K // bw
    # a "column segment" is one column of one block: 4 rows x 16 cols blocks give 16 per block
    assert nbr * nbc * bw == c["column_segments"]
    # the other orientation would give a different count, so the example pins rows x cols
    assert (M // bw) * (K // bh) * bh != c["column_segments"]
    # column pruning only, half of the segments kept -> 2x pruning rate
    rk = np.ones((nbr, nbc, bh), bool)
    ck = np.zeros((nbr, nbc, bw), bool)
    flat = ck.reshape(-1)
    flat[np.random.default_rng(0).permutation(flat.size)[:c["kept_column_segments_at_2x"]]] = True
    mask = gen.mask_from_keep(rk, ck, M, K)
    blocks, ok = orc.extract_blocks(mask, bh, bw)
    assert ok and len(blocks) == nbr * nbc
    assert int(mask.sum()) == c["kept_weights_at_2x"]
    assert sum(len(r) * len(cc) for r, cc in blocks) == c["kept_weights_at_2x"]


def test_weights_per_block_example():
    c = _golden_counts()
    M, K = c["big_rows"], c["big_cols"]
    side = int(round(math.sqrt(M * K / c["big_blocks"])))
    assert (M // side) * (K // side) == c["big_blocks"]
    assert side * side / c["big_rate"] == c["big_weights_per_block"]
    mask = gen.bcr_mask(M, K, side, side, compression=c["big_rate"], dist="uniform", seed=11)
    blocks, ok = orc.extract_blocks(mask, side, side)
    assert ok
    per_block = np.array([len(r) * len(cc) for r, cc in blocks])
    assert per_block.sum() == mask.sum()
    assert abs(per_block.mean() / c["big_weights_per_block"] - 1.0) < 0.15


# ---------------------------------------------------------------------------- packing


@pytest.mark.parametrize("dtype", [orc.DTYPE_F32, orc.DTYPE_BF16])
@pytest.mark.parametrize("shape", [(32, 64, 8, 16), (19, 45, 4, 16), (64, 27, 8, 32)])
def test_pack_unpack_round_trip(shape, dtype):
    M, K, bh, bw = shape
    W = gen.dense_weight(M, K, seed=21)
    mask = gen.bcr_mask(M, K, bh, bw, compression=4, seed=22, empty_frac=0.2)
    buf = orc.pack_canonical(W, mask, bh, bw, dtype, reorder=True)
    u = orc.unpack_canonical(buf)
    assert np.array_equal(u["mask"], mask)
    if dtype == orc.DTYPE_F32:
        want = np.where(mask != 0, W, np.float32(0))
    else:
        want = np.where(mask != 0, torch.from_numpy(W).to(torch.bfloat16).float().numpy(), np.float32(0))
    assert np.array_equal(u["W"].view(np.uint32), want.view(np.uint32))
    assert u["nnz"] == int(mask.sum())
    assert np.array_equal(orc.masked_weight(W, mask, dtype), u["W"].astype(np.float64))


def _golden_canonical():
    out = {}
    for line in open(os.path.join(GOLDEN, "canonical_4x4_blocks2x2.txt")):
        line = line.strip()
        if line and not line.startswith("#"):
            name, hexs = line.split(":")
            out[name.strip()] = bytes.fromhex(hexs.replace(" ", ""))
    return out


def _golden_matrix():
    W = np.array([[1, 2, 3, 4], [5, 0, 0, 8], [-1, -2, 0.5, 0.25], [-3, -4, 1.5, -0.5]], dtype=np.float32)
    W.view(np.uint32)[1, 1] = 0x40C08000
    W.view(np.uint32)[1, 2] = 0x40E18000
    mask = np.array([[0, 1, 0, 0], [0, 1, 1, 1], [0, 0, 1, 1], [0, 0, 1, 1]], dtype=np.uint8)
    return W, mask


def test_pack_canonical_matches_hand_written_bytes():
    """The byte layout itself (field order, widths, value order, trailer) against a byte string typed out by hand
    from the layout in the public header - not produced by any packer."""
    g = _golden_canonical()
    W, mask = _golden_matrix()
    assert orc.pack_canonical(W, mask, 2, 2, orc.DTYPE_F32, reorder=True) == g["f32_reorder"]
    assert orc.pack_canonical(W, mask, 2, 2, orc.DTYPE_BF16, reorder=False) == g["bf16_plain"]
    u = orc.unpack_canonical(g["f32_reorder"])
    assert np.array_equal(u["mask"], mask) and list(u["row_perm"]) == [1, 2, 3, 0]
    assert np.array_equal(u["W"].view(np.uint32), np.where(mask != 0, W, np.float32(0)).view(np.uint32))


def test_pack_lists_sorted_and_nnz_accounting():
    M, K, bh, bw = 48, 96, 8, 32
    mask = gen.bcr_mask(M, K, bh, bw, compression=6, dist="zipf", seed=23)
    blocks, ok = orc.extract_blocks(mask, bh, bw)
    assert ok
    for i, (rows, cols) in enumerate(blocks):
        assert np.all(np.diff(rows) > 0) and np.all(np.diff(cols) > 0)
        bi, bj = divmod(i, K // bw)
        sub = mask[bi * bh:(bi + 1) * bh, bj * bw:(bj + 1) * bw]
        assert sub.sum() == len(rows) * len(cols)
    assert sum(len(r) * len(c) for r, c in blocks) == mask.sum()


def test_non_bcr_mask_is_detected():
    mask = gen.bcr_mask(16, 32, 8, 16, dist="fixed", kr_fixed=4, kc_fixed=8, seed=24)
    _, ok = orc.extract_blocks(mask, 8, 16)
    assert ok
    r, c = np.argwhere(mask)[5]
    bad = mask.copy()
    bad[r, c] = 0  # a hole inside a kept sub-matrix
    _, ok = orc.extract_blocks(bad, 8, 16)
    assert not ok
    with pytest.raises(ValueError):
        orc.pack_canonical(np.zeros((16, 32), np.float32), bad, 8, 16)


def test_row_permutation_groups_equal_work():
    """Section 4.2 / Section 6.4: after the reorder the per-row kept-weight counts are regular."""
    mask = gen.bcr_mask(64, 128, 8, 32, compression=5, dist="zipf", seed=25, empty_frac=0.1)
    mask[8:16] = 0
    perm = orc.row_permutation(mask)
    assert sorted(perm.tolist()) == list(range(64))
    nnz = mask.sum(axis=1).astype(np.int64)[perm]
    assert np.all(np.diff(nnz) <= 0)
    assert np.all(nnz[-8:] == 0)
    for a, b in zip(perm[:-1], perm[1:]):
        if mask[a].sum() == mask[b].sum():
            assert a < b


def test_bf16_rounding_against_library_and_ties():
    g = np.random.default_rng(5)
    a = np.concatenate([g.standard_normal(4096).astype(np.float32) * s for s in (1e-3, 1.0, 1e4)])
    want = torch.from_numpy(a).to(torch.bfloat16).float().numpy()
    assert np.array_equal(orc.round_to_bf16(a).view(np.uint32), want.view(np.uint32))
    # ties go to the even bf16 neighbour: bf16 has 8 significand bits, spacing 2^-7 at 1.0
    assert orc.round_to_bf16(np.float32(1.0 + 2.0 ** -8)) == np.float32(1.0)
    assert orc.round_to_bf16(np.float32(1.0 + 3 * 2.0 ** -8)) == np.float32(1.0 + 2.0 ** -6)
    assert orc.round_to_bf16(np.float32(1.0 + 2.0 ** -8 + 2.0 ** -20)) == np.float32(1.0 + 2.0 ** -7)
    assert orc.round_to_bf16(np.float32(-0.0)).view(np.uint32) == 0x80000000


# ---------------------------------------------------------------------------- convolution


def _brute_conv(W4, x, bias, stride, pad):
    Nb, C, H, Wd = x.shape
    Co, _, KH, KW = W4.shape
    OH = (H + 2 * pad - KH) // stride + 1
    OW = (Wd + 2 * pad - KW) // stride + 1
    out = np.zeros((Nb, Co, OH, OW))
    for n in range(Nb):
        for o in range(Co):
            for oh in range(OH):
                for ow in range(OW):
                    acc = float(bias[o])
                    for c in range(C):
                        for kh in range(KH):
                            for kw in range(KW):
                                ih = oh * stride + kh - pad
                                iw = ow * stride + kw - pad
                                if 0 <= ih < H and 0 <= iw < Wd:
                                    acc += float(W4[o, c, kh, kw]) * float(x[n, c, ih, iw])
                    out[n, o, oh, ow] = acc
    return out


@pytest.mark.parametrize("stride,pad,ks", [(1, 1, 3), (2, 1, 3), (1, 0, 1), (1, 2, 5)])
def test_conv_brute_force_with_mask(stride, pad, ks):
    g = np.random.default_rng(6)
    C, Co, H = 5, 8, 6
    K = C * ks * ks
    W = g.standard_normal((Co, K)).astype(np.float32)
    mask = gen.bcr_mask(Co, K, 4, 8, compression=2, seed=31)
    x = g.standard_normal((2, C, H, H + 1))
    bias = g.standard_normal(Co)
    W4 = np.where(mask != 0, W, 0).astype(np.float64).reshape(Co, C, ks, ks)
    want = _brute_conv(W4, x, bias, stride, pad)
    got = orc.conv2d(W, mask, x, bias, ksize=ks, stride=stride, pad=pad)
    np.testing.assert_allclose(got, want, atol=1e-12)
    got_relu = orc.conv2d(W, mask, x, bias, ksize=ks, stride=stride, pad=pad, relu=True)
    np.testing.assert_allclose(got_relu, np.maximum(want, 0), atol=1e-12)


def test_conv_all_kept_equals_library_conv():
    g = np.random.default_rng(7)
    C, Co, H = 6, 10, 9
    W = g.standard_normal((Co, C * 9)).astype(np.float32)
    x = g.standard_normal((3, C, H, H))
    bias = g.standard_normal(Co)
    want = torch.nn.functional.conv2d(torch.from_numpy(x), torch.from_numpy(W).double().reshape(Co, C, 3, 3),
                                      torch.from_numpy(bias), stride=1, padding=1).numpy()
    got = orc.conv2d(W, np.ones_like(W, np.uint8), x, bias, ksize=3, stride=1, pad=1)
    np.testing.assert_allclose(got, want, atol=1e-12)


def test_conv_1x1_is_spmm_on_reshaped_input():
    g = np.random.default_rng(8)
    C, Co, H = 16, 12, 5
    W = g.standard_normal((Co, C)).astype(np.float32)
    mask = gen.bcr_mask(Co, C, 4, 8, compression=2, seed=33)
    x = g.standard_normal((1, C, H, H))
    got = orc.conv2d(W, mask, x, None, ksize=1)
    want = _brute_spmm(W, *zip(*[(list(r), list(c)) for r, c in orc.extract_blocks(mask, 4, 8)[0]]), 4, 8,
                       x.reshape(C, H * H))
    np.testing.assert_allclose(got.reshape(Co, H * H), want, atol=1e-12)


def test_maxpool():
    x = np.arange(2 * 3 * 4 * 6, dtype=np.float64).reshape(2, 3, 4, 6)
    x[0, 0, 0, 0] = 1e3
    want = torch.nn.functional.max_pool2d(torch.from_numpy(x), 2, 2).numpy()
    assert np.array_equal(orc.maxpool2x2(x), want)


# ---------------------------------------------------------------------------- GRU


def _gru_layers(in_f, H, L, seed, all_kept):
    m = gen.gru_model(in_f, H, L, T=1, bh=4, bw=8, compression=2, seed=seed)
    if all_kept:
        for lay in m["layers"]:
            lay["mask_ih"][:] = 1
            lay["mask_hh"][:] = 1
    return m["layers"]


def test_gru_all_kept_equals_library_gru():
    in_f, H, L, T = 7, 12, 2, 9
    layers = _gru_layers(in_f, H, L, seed=41, all_kept=True)
    x = np.random.default_rng(9).standard_normal((T, in_f))
    ref = torch.nn.GRU(in_f, H, L).double()
    with torch.no_grad():
        for l, lay in enumerate(layers):
            getattr(ref, f"weight_ih_l{l}").copy_(torch.from_numpy(lay["W_ih"]).double())
            getattr(ref, f"weight_hh_l{l}").copy_(torch.from_numpy(lay["W_hh"]).double())
            getattr(ref, f"bias_ih_l{l}").copy_(torch.from_numpy(lay["b_ih"]).double())
            getattr(ref, f"bias_hh_l{l}").copy_(torch.from_numpy(lay["b_hh"]).double())
        h0 = torch.from_numpy(np.random.default_rng(10).standard_normal((L, 1, H)))
        y, hT = ref(torch.from_numpy(x)[:, None, :], h0)
    got_y, got_h = orc.gru_seq(layers, x, h0=h0[:, 0].numpy())
    np.testing.assert_allclose(got_y, y[:, 0].numpy(), atol=1e-12)
    np.testing.assert_allclose(got_h, hT[:, 0].numpy(), atol=1e-12)


def test_gru_single_step_closed_form_with_mask():
    """T = 1 and h0 = 0: q = b_hh, so h = (1 - z) * n with scalar formulas evaluated entry by entry."""
    in_f, H = 9, 8
    lay = _gru_layers(in_f, H, 1, seed=42, all_kept=False)[0]
    x = np.random.default_rng(11).standard_normal(in_f)
    y, hT = orc.gru_seq([lay], x[None, :])
    for u in range(H):
        def pre(row):
            return math.fsum(float(lay["W_ih"][row, c]) * x[c] for c in range(in_f) if lay["mask_ih"][row, c]) \
                + float(lay["b_ih"][row])
        r = 1 / (1 + math.exp(-(pre(u) + float(lay["b_hh"][u]))))
        z = 1 / (1 + math.exp(-(pre(H + u) + float(lay["b_hh"][H + u]))))
        n = math.tanh(pre(2 * H + u) + r * float(lay["b_hh"][2 * H + u]))
        assert abs(y[0, u] - (1 - z) * n) < 1e-13
    assert np.array_equal(y[0], hT[0])


def test_gru_two_steps_by_hand_uses_previous_state_and_mask():
    """Second step by scalar loops: catches a dropped z*h term, a swapped gate or an ignored hidden mask."""
    in_f, H = 5, 4
    lay = _gru_layers(in_f, H, 1, seed=43, all_kept=False)[0]
    x = np.random.default_rng(12).standard_normal((2, in_f))
    y, _ = orc.gru_seq([lay], x)
    h = [0.0] * H
    for t in range(2):
        def dot(Wn, mn, row, v):
            return math.fsum(float(lay[Wn][row, c]) * v[c] for c in range(len(v)) if lay[mn][row, c])
        new = []
        for u in range(H):
            gi = [dot("W_ih", "mask_ih", g * H + u, x[t]) + float(lay["b_ih"][g * H + u]) for g in range(3)]
            gh = [dot("W_hh", "mask_hh", g * H + u, h) + float(lay["b_hh"][g * H + u]) for g in range(3)]
            r = 1 / (1 + math.exp(-(gi[0] + gh[0])))
            z = 1 / (1 + math.exp(-(gi[1] + gh[1])))
            n = math.tanh(gi[2] + r * gh[2])
            new.append((1 - z) * n + z * h[u])
        h = new
        np.testing.assert_allclose(y[t], h, atol=1e-13)


# ---------------------------------------------------------------------------- BCRC (Section 4.3)


def test_bcrc_reproduces_the_fragments_quoted_in_the_text():
    """Section 4.3 quotes the first entries of the arrays of its (unavailable) figure: reorder 0, 3; row offset 0, 3;
    column stride 0, 3; the first column list 0, 3, 6; occurrence 0, 2 (rows 0 and 1 of the reordered matrix share
    that list).  A matrix with that property: original rows 0 and 3 keep columns 0, 3, 6; the other rows keep fewer."""
    mask = np.zeros((4, 8), np.uint8)
    mask[0, [0, 3, 6]] = 1
    mask[3, [0, 3, 6]] = 1
    mask[1, [1, 4]] = 1
    mask[2, [2]] = 1
    W = np.arange(1, 33, dtype=np.float32).reshape(4, 8)
    b = orc.bcrc_export(W, mask)
    assert list(b["reorder"][:2]) == [0, 3]
    assert list(b["row_offset"][:2]) == [0, 3]
    assert list(b["column_stride"][:2]) == [0, 3]
    assert list(b["compact_column"][:3]) == [0, 3, 6]
    assert list(b["occurrence"][:2]) == [0, 2]
    # the shared list is stored once: 3 + 2 + 1 column ids for 3 + 3 + 2 + 1 weights
    assert len(b["compact_column"]) == 6 and len(b["weights"]) == 9
    assert list(b["weights"][:6]) == [1, 4, 7, 25, 28, 31]


@pytest.mark.parametrize("shape", [(32, 64, 8, 16, 4.0), (19, 45, 4, 16, 3.0), (48, 96, 16, 32, 6.0)])
def test_bcrc_invariants(shape):
    M, K, bh, bw, c = shape
    W = gen.dense_weight(M, K, seed=24)
    mask = gen.bcr_mask(M, K, bh, bw, compression=c, seed=25, empty_frac=0.2)
    b = orc.bcrc_export(W, mask)
    want = np.where(mask != 0, W, np.float32(0))
    assert np.array_equal(orc.bcrc_to_dense(b, M, K).view(np.uint32), want.view(np.uint32))   # rebuilds the masked weight
    assert sorted(b["reorder"]) == list(range(M))                                               # a permutation
    nnz_sorted = np.diff(b["row_offset"])
    assert np.all(nnz_sorted[:-1] >= nnz_sorted[1:]) and b["row_offset"][-1] == int(mask.sum())
    for g in range(len(b["occurrence"]) - 1):                                                   # groups are maximal runs
        cols = b["compact_column"][b["column_stride"][g]:b["column_stride"][g + 1]]
        assert np.all(np.diff(cols) > 0)
        for p in range(b["occurrence"][g], b["occurrence"][g + 1]):
            assert np.array_equal(np.flatnonzero(mask[b["reorder"][p]]), cols)
        if g > 0:
            prev = b["compact_column"][b["column_stride"][g - 1]:b["column_stride"][g]]
            assert not np.array_equal(prev, cols)
    assert orc.index_bytes_bcrc(b) <= orc.index_bytes_csr(mask) + 4 * (2 * M + 3)   # never worse than CSR + its fixed arrays


def test_bcrc_reduces_to_csr_when_no_two_rows_share_a_list():
    """With all column lists distinct every row is its own group, and (compact_column, column_stride) are the column ids
    and row pointers of CSR for the reordered matrix (library routine: scipy.sparse.csr_matrix)."""
    import scipy.sparse as sp
    rng = np.random.default_rng(26)
    M, K = 12, 40
    mask = np.zeros((M, K), np.uint8)
    for r in range(M):
        mask[r, rng.choice(K, size=3 + r, replace=False)] = 1   # different lengths: all lists differ
    W = gen.dense_weight(M, K, seed=27)
    b = orc.bcrc_export(W, mask)
    assert len(b["occurrence"]) == M + 1
    csr = sp.csr_matrix(np.where(mask != 0, W, 0)[b["reorder"]])
    csr.sort_indices()
    assert np.array_equal(csr.indices, b["compact_column"]) and np.array_equal(csr.indptr, b["column_stride"])
    assert np.array_equal(csr.data.astype(np.float32), b["weights"])


def test_bcrc_saves_column_ids_when_rows_share_lists():
    """One block per row band (block = whole row width): every kept row of a band shares the band's column list, so BCRC
    stores one list per band where CSR stores one per row (Section 4.3's argument for the format)."""
    M, K, bh = 64, 128, 8
    mask = gen.bcr_mask(M, K, bh, 64, compression=4, seed=28)   # two blocks per band
    b = orc.bcrc_export(gen.dense_weight(M, K, seed=29), mask)
    assert len(b["compact_column"]) < int(mask.sum())
    assert orc.index_bytes_bcrc(b) < orc.index_bytes_csr(mask)


# ---------------------------------------------------------------------------- projection onto the BCR set (Section 5.2)


def test_projection_with_unit_blocks_is_magnitude_pruning():
    """1 x 1 blocks: the BCR set is plain sparsity and the Euclidean projection is textbook - keep the largest
    magnitudes.  The greedy steps must give exactly that."""
    V = gen.normal_f32((12, 17), 1.0, 30, 0)
    for sparsity in (0.0, 0.5, 0.9, 1.0):
        mask = orc.bcr_project(V, 1, 1, sparsity)
        k = int(np.floor((1 - sparsity) * V.size + 1e-9))
        order = np.argsort(-np.abs(V).ravel(), kind="stable")
        want = np.zeros(V.size, np.uint8)
        want[order[:k]] = 1
        assert int(mask.sum()) == k and np.array_equal(mask.ravel(), want)


@pytest.mark.parametrize("seed", [31, 32, 33, 34])
def test_projection_is_feasible_and_never_beats_the_exact_one(seed):
    """Tiny blocks, exhaustive search: the greedy result lies in the set (BCR structure, enough zeros), so its distance
    can only be >= the exact projection's; and the exact search itself is checked on the case where it is obvious."""
    V = gen.normal_f32((4, 6), 1.0, seed, 0)
    for sparsity in (0.3, 0.5, 0.75):
        mask = orc.bcr_project(V, 2, 3, sparsity)
        _, ok = orc.extract_blocks(mask, 2, 3)
        assert ok and mask.sum() <= np.floor((1 - sparsity) * V.size + 1e-9)
        exact_mask, exact_loss = orc.bcr_project_exact(V, 2, 3, sparsity)
        _, ok2 = orc.extract_blocks(exact_mask, 2, 3)
        assert ok2 and exact_mask.sum() <= np.floor((1 - sparsity) * V.size + 1e-9)
        loss = float((V.astype(np.float64)[mask == 0] ** 2).sum())
        assert abs(float((V.astype(np.float64)[exact_mask == 0] ** 2).sum()) - exact_loss) < 1e-9
        assert loss >= exact_loss - 1e-12
        assert loss <= 2.5 * exact_loss + 1e-12      # and it is not far off on these inputs


def test_exact_projection_on_an_obvious_case():
    """One 2 x 2 block, half the entries must go: a dominant column is what stays."""
    V = np.array([[5.0, 0.1], [4.0, 0.2]], np.float32)
    mask, loss = orc.bcr_project_exact(V, 2, 2, 0.5)
    assert np.array_equal(mask, [[1, 0], [1, 0]]) and abs(loss - (0.01 + 0.04)) < 1e-6
    assert np.array_equal(orc.bcr_project(V, 2, 2, 0.5), mask)
