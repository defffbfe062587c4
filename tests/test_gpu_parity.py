"""GPU parity: every CUDA entry point against the fp64 CPU oracle, element by element, through the C ABI.

Tolerances (fixed requirements of this library): fp32 results  ||Y - Y*||_F / ||Y*||_F <= 1e-5;
bf16 inputs with fp32 accumulation  max |err| <= 2e-2 * ||W row||_2 * ||X col||_2 (plus |bias| where
a bias is added); packing is bit-exact (tests/test_packer_host.py).  Rows kept by no block must be
exactly +0.
"""
import numpy as np
import pytest
import torch

from oracle import bcr_oracle as orc
from parity_util import F32_TOL, assert_close, rel_fro
from workloads import generators as gen

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2108_11033_b200.build import build_library
    build_library()
    from paper_2108_11033_b200 import binding
    return binding


def to_dev(a, bf16=False):
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()
    return t.to(torch.bfloat16) if bf16 else t


def check_spmm(B, W, mask, X, bh, bw, *, bf16=False, flags=0, tile_n=0, y_bf16=False, path=0):
    M, K = W.shape
    X = gen.bf16_representable(X) if bf16 else np.asarray(X, np.float32)
    N = X.shape[1]
    dt = B.GRIM_BF16 if bf16 else B.GRIM_F32
    h = B.grim_bcr_pack(W, mask, bh, bw, dt, flags)
    try:
        if bf16:
            B.grim_bcr_reserve(h, N)  # workspace of the split tensor-core multiply, where the library chooses it
        Xd = to_dev(X, bf16)
        Yd = torch.full((M, N), float("nan"), device="cuda", dtype=torch.bfloat16 if y_bf16 else torch.float32)
        if tile_n or path:
            B.grim_bcr_spmm_ex(h, Xd, Yd, tile_n=tile_n, path=path)
        else:
            B.grim_bcr_spmm(h, Xd, Yd)
        torch.cuda.synchronize()
        assert B.grim_bcr_status(h) == B.GRIM_OK
        got = Yd.float().cpu().numpy().astype(np.float64)
        want = orc.spmm(W, mask, X, dt)
        dead = np.flatnonzero(mask.sum(axis=1) == 0)
        assert np.all(got[dead] == 0.0) and not np.any(np.signbit(got[dead])), "pruned rows must be exactly +0"
        Wm = orc.masked_weight(W, mask, dt)
        scale = np.linalg.norm(Wm, axis=1)[:, None] * np.linalg.norm(X.astype(np.float64), axis=0)[None, :]
        assert_close(got, want, scale, bf16_in=bf16, out_bf16=y_bf16, what=f"spmm {M}x{K}x{N}")
    finally:
        B.grim_bcr_destroy(h)


# ---------------------------------------------------------------------------------------- SpMM / GEMV


def test_config1_spmm_fp32(B):
    c = gen.config1_spmm()
    check_spmm(B, c["W"], c["mask"], c["X"], c["bh"], c["bw"])


SHAPES = [
    # M, K, bh, bw, generator kwargs
    (256, 256, 16, 16, dict(dist="fixed", kr_fixed=8, kc_fixed=8)),
    (200, 333, 8, 32, dict(compression=6, dist="uniform")),
    (96, 153, 8, 32, dict(compression=10, dist="uniform")),
    (130, 260, 4, 16, dict(compression=8, dist="zipf")),
    (150, 500, 16, 64, dict(compression=4, dist="zipf", empty_frac=0.25)),
    (64, 27, 8, 32, dict(compression=3, dist="uniform")),
    (33, 40, 3, 5, dict(compression=2, dist="uniform")),
    (24, 48, 1, 1, dict(compression=3, dist="uniform")),
    (16, 64, 16, 64, dict(compression=4, dist="uniform")),
]


@pytest.mark.parametrize("N", [1, 3, 16, 37, 64, 130, 260])
@pytest.mark.parametrize("shape", SHAPES)
def test_spmm_fp32_small(B, shape, N):
    M, K, bh, bw, kw = shape
    W = gen.dense_weight(M, K, seed=60)
    mask = gen.bcr_mask(M, K, bh, bw, seed=61, **kw)
    X = gen.normal_f32((K, N), 1.0, 62, 0)
    check_spmm(B, W, mask, X, bh, bw)


@pytest.mark.parametrize("N", [1, 5, 64, 200])
@pytest.mark.parametrize("shape", SHAPES[1:6])
def test_spmm_bf16_small(B, shape, N):
    M, K, bh, bw, kw = shape
    W = gen.dense_weight(M, K, seed=63)
    mask = gen.bcr_mask(M, K, bh, bw, seed=64, **kw)
    X = gen.normal_f32((K, N), 1.0, 65, 0)
    check_spmm(B, W, mask, X, bh, bw, bf16=True)
    check_spmm(B, W, mask, X, bh, bw, bf16=True, y_bf16=True)


@pytest.mark.parametrize("tile_n", [16, 32, 64, 128])
@pytest.mark.parametrize("reorder", [0, 1])
def test_spmm_tiles_and_reorder(B, tile_n, reorder):
    M, K, bh, bw = 512, 768, 8, 32
    W = gen.dense_weight(M, K, seed=66)
    mask = gen.bcr_mask(M, K, bh, bw, compression=8, dist="zipf", seed=67, empty_frac=0.1)
    mask[40:56] = 0  # two fully pruned bands
    X = gen.normal_f32((K, 150), 1.0, 68, 0)
    check_spmm(B, W, mask, X, bh, bw, flags=reorder, tile_n=tile_n)


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("case", [(512, 768, 8, 32, 1), (512, 768, 8, 32, 2), (300, 520, 4, 16, 4), (300, 520, 4, 16, 1),
                                  (260, 700, 16, 64, 1), (96, 153, 8, 32, 2), (64, 27, 8, 32, 1), (33, 40, 3, 5, 1)])
def test_register_tiled_kernel_explicit(B, case, bf16):
    """The N > 16 register-tiled kernel asked for by name (path 1), with each number of band groups per
    thread block, on a ragged column count (TMA loader: aligned X; gather loader: covered by the strided test)."""
    M, K, bh, bw, groups = case
    W = gen.dense_weight(M, K, seed=73)
    mask = gen.bcr_mask(M, K, bh, bw, compression=6, dist="zipf", seed=74, empty_frac=0.1)
    mask[: 2 * bh] = 0
    X = gen.normal_f32((K, 328), 1.0, 75, 0)
    check_spmm(B, W, mask, X, bh, bw, bf16=bf16, tile_n=groups, path=1, flags=1)


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("case", [(512, 768, 8, 32, 8, 328), (512, 768, 8, 32, 8, 600), (300, 520, 4, 16, 8, 328),
                                  (300, 520, 4, 16, 9, 515), (96, 153, 8, 32, 8, 257), (64, 27, 8, 32, 8, 1024)])
def test_register_tiled_kernel_two_pieces_per_lane(B, case, bf16):
    """The same kernel with 256-column tiles (a lane owns two 4-column pieces; tile_n 8 and 9), on column counts that
    leave the second piece partly or wholly empty in the last tile."""
    M, K, bh, bw, tile_n, N = case
    W = gen.dense_weight(M, K, seed=173)
    mask = gen.bcr_mask(M, K, bh, bw, compression=6, dist="zipf", seed=174, empty_frac=0.1)
    mask[: 2 * bh] = 0
    X = gen.normal_f32((K, N), 1.0, 175, 0)
    check_spmm(B, W, mask, X, bh, bw, bf16=bf16, tile_n=tile_n, path=1, flags=1)


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("case", [(512, 768, 8, 32, 17, 16), (512, 768, 8, 32, 18, 12), (512, 768, 8, 32, 20, 9),
                                  (300, 520, 4, 16, 20, 16), (260, 700, 16, 64, 17, 16), (96, 153, 8, 32, 17, 5),
                                  (64, 27, 8, 32, 17, 1), (2048, 1024, 8, 32, 17 + 256 * 3, 16)])
def test_register_tiled_kernel_narrow_tile(B, case, bf16):
    """The 16-column tile for N <= 16 (a lane owns one column, the halves of a warp split each chunk's kept columns;
    tile_n 17, 18, 20 = 1, 2, 4 band groups per thread block), unsplit and split over the block columns."""
    M, K, bh, bw, tile_n, N = case
    W = gen.dense_weight(M, K, seed=183)
    mask = gen.bcr_mask(M, K, bh, bw, compression=6, dist="zipf", seed=184, empty_frac=0.1)
    mask[: 2 * bh] = 0
    X = gen.normal_f32((K, N), 1.0, 185, 0)
    check_spmm(B, W, mask, X, bh, bw, bf16=bf16, tile_n=tile_n, path=1, flags=1)


@pytest.mark.parametrize("row_tiles", [1, 2])
def test_tensor_core_row_tiles_per_block(B, row_tiles):
    """One or two 128-row tiles per thread block (two share every X tile), on a row count that leaves the last
    thread block with a single, partly filled tile."""
    M, K, bh, bw, N = 328, 700, 8, 32, 520
    W = gen.dense_weight(M, K, seed=97)
    mask = gen.bcr_mask(M, K, bh, bw, compression=5, dist="uniform", seed=98, empty_frac=0.1)
    X = gen.normal_f32((K, N), 1.0, 99, 0)
    check_spmm(B, W, mask, X, bh, bw, bf16=True, path=2, tile_n=row_tiles, flags=1)


@pytest.mark.parametrize("y_bf16", [False, True])
@pytest.mark.parametrize("case", [(256, 512, 8, 32, 256), (200, 333, 8, 32, 328), (300, 520, 4, 16, 520), (260, 700, 16, 64, 264),
                                  (96, 153, 8, 32, 1024), (512, 2048, 16, 64, 776)])
def test_tensor_core_kernel_explicit(B, case, y_bf16):
    """The tcgen05 path asked for by name (path 2): bf16 operands, fp32 accumulation in tensor memory; ragged M, K
    and N, empty blocks, pruned bands, every supported block shape."""
    M, K, bh, bw, N = case
    W = gen.dense_weight(M, K, seed=87)
    mask = gen.bcr_mask(M, K, bh, bw, compression=6, dist="zipf", seed=88, empty_frac=0.1)
    mask[: 2 * bh] = 0
    X = gen.normal_f32((K, N), 1.0, 89, 0)
    check_spmm(B, W, mask, X, bh, bw, bf16=True, path=2, flags=1, y_bf16=y_bf16)


@pytest.mark.parametrize("y_bf16", [False, True])
@pytest.mark.parametrize("case", [(256, 512, 8, 32, 512), (328, 700, 8, 32, 520), (300, 520, 4, 16, 1032), (260, 700, 16, 64, 264),
                                  (96, 153, 8, 32, 1024), (512, 2048, 16, 64, 776), (640, 320, 4, 32, 600), (400, 256, 8, 16, 520),
                                  (384, 448, 16, 16, 512), (384, 448, 16, 32, 136), (200, 333, 4, 64, 328), (1100, 900, 8, 64, 1544)])
def test_paired_tensor_core_kernel_explicit(B, case, y_bf16):
    """The paired tcgen05 kernel asked for by name (path 5): two thread blocks multiply 256 rows x 512 columns
    together.  Ragged M, K and N, an odd number of 128-row tiles (the last pair has one empty partner), a single
    tile, empty blocks, pruned bands, every supported block shape."""
    M, K, bh, bw, N = case
    W = gen.dense_weight(M, K, seed=187)
    mask = gen.bcr_mask(M, K, bh, bw, compression=6, dist="zipf", seed=188, empty_frac=0.1)
    mask[: 2 * bh] = 0
    X = gen.normal_f32((K, N), 1.0, 189, 0)
    check_spmm(B, W, mask, X, bh, bw, bf16=True, path=5, flags=1, y_bf16=y_bf16)


@pytest.mark.parametrize("split", [2, 5, 8])
def test_split_multiply(B, split):
    """Few output tiles: several thread blocks share a tile's block columns and add their partial sums into a
    zeroed Y (pruned rows must stay exactly +0)."""
    M, K, bh, bw = 160, 2100, 8, 32
    W = gen.dense_weight(M, K, seed=83)
    mask = gen.bcr_mask(M, K, bh, bw, compression=8, dist="uniform", seed=84, empty_frac=0.2)
    mask[16:24] = 0
    X = gen.normal_f32((K, 200), 1.0, 85, 0)
    check_spmm(B, W, mask, X, bh, bw, path=1, tile_n=1 + 256 * split)


def test_conv_split_with_bias_and_relu(B):
    """A layer with few output pixels and many input channels takes the split path (separate bias / ReLU pass)."""
    L = gen.conv_layer(1, 96, 48, 9, ksize=3, bh=8, bw=32, compression=4, seed=86)
    check_conv(B, L, L["x"], ksize=3, stride=1, pad=1, bf16=False)
    check_conv(B, L, L["x"], ksize=3, stride=1, pad=1, bf16=False, relu=False)


@pytest.mark.parametrize("N", [2, 7, 12, 16])
def test_lane_per_column_kernel_explicit(B, N):
    M, K, bh, bw = 200, 333, 16, 64
    W = gen.dense_weight(M, K, seed=76)
    mask = gen.bcr_mask(M, K, bh, bw, compression=5, dist="uniform", seed=77)
    X = gen.normal_f32((K, N), 1.0, 78, 0)
    for variant in (0, 1, 2):  # default choice, values staged in registers, values streamed through shared memory
        check_spmm(B, W, mask, X, bh, bw, path=3, tile_n=variant)
        check_spmm(B, W, mask, X, bh, bw, bf16=True, path=3, tile_n=variant)


STREAM_CASES = [
    # M, K, bh, bw, generator kwargs: more bands than SMs, several bands per thread block, ragged edges
    (3000, 1500, 8, 32, dict(compression=4, dist="uniform")),
    (2500, 700, 16, 64, dict(compression=6, dist="zipf", empty_frac=0.1)),
    (20001, 96, 4, 16, dict(compression=3, dist="uniform")),   # > 32 bands per thread block: several batches
    (1190, 20000, 8, 32, dict(compression=16, dist="zipf")),   # vector too long for shared memory: gathered
]


@pytest.mark.parametrize("bf16", [False, True])
def test_small_n_edge_cases(B, bf16):
    """Default routing for N <= 16 on degenerate shapes: nothing kept at all, a single band shorter than a block, a
    matrix narrower than a block, one kept element, and the widest K the 16-bit column words can address."""
    for M, K, bh, bw, kw in [
        (40, 64, 8, 32, dict(compression=4, dist="uniform", empty_frac=1.0)),   # every block empty
        (5, 300, 8, 32, dict(compression=2, dist="uniform")),                   # one ragged band
        (100, 7, 4, 16, dict(compression=2, dist="uniform")),                   # K smaller than a block
        (64, 65536, 16, 64, dict(compression=64, dist="zipf")),                 # widest K of the chunk layout
    ]:
        W = gen.dense_weight(M, K, seed=180)
        mask = gen.bcr_mask(M, K, bh, bw, seed=181, **kw)
        for N in (1, 3, 16):
            X = gen.normal_f32((K, N), 1.0, 182, N)
            check_spmm(B, W, mask, X, bh, bw, bf16=bf16)
    W = gen.dense_weight(24, 96, seed=183)
    mask = np.zeros((24, 96), np.uint8)
    mask[9, 70] = 1  # a single kept element
    check_spmm(B, W, mask, gen.normal_f32((96, 1), 1.0, 184, 0), 8, 32, bf16=bf16)


@pytest.mark.parametrize("N", [1, 4, 9, 16])
@pytest.mark.parametrize("case", STREAM_CASES)
def test_streaming_kernel_explicit(B, case, N):
    M, K, bh, bw, kw = case
    W = gen.dense_weight(M, K, seed=170)
    mask = gen.bcr_mask(M, K, bh, bw, seed=171, **kw)
    mask[bh * 3:bh * 5] = 0  # two fully pruned bands
    X = gen.normal_f32((K, N), 1.0, 172, 0)
    check_spmm(B, W, mask, X, bh, bw, path=3, tile_n=2)
    check_spmm(B, W, mask, X, bh, bw, bf16=True, path=3, tile_n=2, y_bf16=(N == 4))


def test_spmm_strided_operands_and_errors(B):
    M, K, bh, bw, N = 64, 96, 8, 32, 20
    W = gen.dense_weight(M, K, seed=69)
    mask = gen.bcr_mask(M, K, bh, bw, compression=4, seed=70)
    h = B.grim_bcr_pack(W, mask, bh, bw, B.GRIM_F32, 0)
    Xfull = torch.randn(K, N + 7, device="cuda")
    Yfull = torch.zeros(M, N + 3, device="cuda")
    X, Y = Xfull[:, 2:2 + N], Yfull[:, 1:1 + N]  # ld > cols, unaligned start
    B.grim_bcr_spmm(h, X, Y)
    torch.cuda.synchronize()
    want = orc.spmm(W, mask, X.cpu().numpy())
    assert rel_fro(Y.cpu().numpy(), want) <= F32_TOL
    assert float(Yfull[:, 0].abs().max()) == 0.0 and float(Yfull[:, 1 + N:].abs().max()) == 0.0
    with pytest.raises(B.GrimError) as e:
        B.grim_bcr_spmm(h, torch.zeros(K + 1, N, device="cuda"), torch.zeros(M, N, device="cuda"))
    assert e.value.status == B.GRIM_ERR_SHAPE
    with pytest.raises(B.GrimError) as e:
        B.grim_bcr_spmm(h, torch.zeros(K, N, device="cuda", dtype=torch.bfloat16), torch.zeros(M, N, device="cuda"))
    assert e.value.status == B.GRIM_ERR_DTYPE
    with pytest.raises(B.GrimError) as e:
        B.grim_bcr_spmm(h, torch.zeros(K, N, device="cuda"), torch.zeros(M, N, device="cuda", dtype=torch.bfloat16))
    assert e.value.status == B.GRIM_ERR_DTYPE
    B.grim_bcr_destroy(h)


@pytest.mark.parametrize("case", [(4096, 1, 8.0, 8, 32, "uniform", False), (4096, 16, 16.0, 4, 16, "zipf", False),
                                  (2048, 128, 4.0, 16, 64, "zipf", True), (4096, 1, 4.0, 16, 64, "zipf", True),
                                  (1024, 1024, 8.0, 8, 32, "uniform", False)])
def test_sweep_points(B, case):
    M, N, c, bh, bw, dist, bf16 = case
    s = gen.sweep_case(M, N, c, bh, bw, dist, bf16=bf16)
    check_spmm(B, s["W"], s["mask"], s["X"], bh, bw, bf16=bf16, flags=1)


@pytest.mark.parametrize("N", [1, 4])
def test_streaming_kernel_chained_launches(B, N):
    """The streaming kernel is launched with programmatic stream serialization: a launch may begin (tables, barriers,
    first weight copies) while the launch before it still runs, and waits for it before it reads X or writes Y.  A chain
    of dependent products through two ping-pong buffers, queued without any host synchronisation, must therefore give
    what the oracle gives step by step - both the read-after-write (X of a step is Y of the step before) and the
    write-after-read (Y of a step is X of the step before) orders are exercised."""
    M = 2048
    s = gen.sweep_case(M, N, 4.0, 8, 32, "uniform")
    W = (s["W"] * 8.0).astype(np.float32)  # keeps the iterates at the same scale from step to step
    h = B.grim_bcr_pack(W, s["mask"], 8, 32, B.GRIM_F32, 1)
    try:
        bufs = [to_dev(s["X"]), torch.empty(M, N, device="cuda")]
        steps = 6
        for i in range(steps):
            B.grim_bcr_spmm_ex(h, bufs[i & 1], bufs[(i + 1) & 1], path=3, tile_n=2)
        torch.cuda.synchronize()
        assert B.grim_bcr_status(h) == B.GRIM_OK
        want = s["X"].astype(np.float64)
        for i in range(steps):
            want = orc.spmm(W, s["mask"], want.astype(np.float32)).astype(np.float64)
        got = bufs[steps & 1].cpu().numpy()
        assert rel_fro(got, want) <= 10 * F32_TOL, rel_fro(got, want)
    finally:
        B.grim_bcr_destroy(h)


@pytest.mark.parametrize("reps", [3, -3])
def test_tune_returns_a_valid_choice(B, reps):
    """reps > 0 times back-to-back launches, reps < 0 launches after an L2 flush each (cold operands)."""
    s = gen.sweep_case(1024, 96, 8.0, 8, 32, "uniform")
    h = B.grim_bcr_pack(s["W"], s["mask"], 8, 32, B.GRIM_F32, 0)
    X = to_dev(s["X"])
    Y = torch.empty(1024, 96, device="cuda")
    best = B.grim_bcr_tune(h, X, Y, reps=reps)
    assert best["path"] in (1, 2, 3, 4) and best["ms"] > 0
    B.grim_bcr_spmm_ex(h, X, Y, tile_n=best["tile_n"], path=best["path"])
    torch.cuda.synchronize()
    assert rel_fro(Y.cpu().numpy(), orc.spmm(s["W"], s["mask"], s["X"])) <= F32_TOL
    # the answer is kept in the handle: the plain call now launches exactly what the explicit call launches
    Y.fill_(float("nan"))
    n0 = B.grim_launch_count()
    B.grim_bcr_spmm_ex(h, X, Y, tile_n=best["tile_n"], path=best["path"])
    n_explicit = B.grim_launch_count() - n0
    Y2 = torch.full_like(Y, float("nan"))
    B.grim_bcr_spmm(h, X, Y2)
    assert B.grim_launch_count() - n0 - n_explicit == n_explicit
    torch.cuda.synchronize()
    assert torch.equal(Y, Y2) or rel_fro(Y2.cpu().numpy(), Y.cpu().numpy()) <= 1e-6  # (a split multiply adds in any order)
    B.grim_bcr_destroy(h)


def test_regime_flags_keep_one_set_of_layouts(B):
    """A handle packed for narrow right-hand sides only multiplies N <= 16, one packed for wide ones N > 16; the other
    regime is refused before any launch, and each holds less device memory than a handle with every layout."""
    s = gen.sweep_case(1024, 64, 8.0, 8, 32, "uniform")
    X64, X4 = to_dev(s["X"]), to_dev(s["X"][:, :4])
    want = orc.spmm(s["W"], s["mask"], s["X"])
    free0 = torch.cuda.mem_get_info()[0]
    h_all = B.grim_bcr_pack(s["W"], s["mask"], 8, 32, B.GRIM_F32, 0)
    used_all = free0 - torch.cuda.mem_get_info()[0]
    B.grim_bcr_destroy(h_all)
    for flag, ok_x, bad_x in ((B.GRIM_PACK_NARROW_ONLY, X4, X64), (B.GRIM_PACK_WIDE_ONLY, X64, X4)):
        free1 = torch.cuda.mem_get_info()[0]
        h = B.grim_bcr_pack(s["W"], s["mask"], 8, 32, B.GRIM_F32, flag)
        assert free1 - torch.cuda.mem_get_info()[0] <= used_all
        Y = torch.full((1024, ok_x.shape[1]), float("nan"), device="cuda")
        B.grim_bcr_spmm(h, ok_x, Y)
        torch.cuda.synchronize()
        assert rel_fro(Y.cpu().numpy(), want[:, :ok_x.shape[1]]) <= F32_TOL
        with pytest.raises(B.GrimError) as e:
            B.grim_bcr_spmm(h, bad_x, torch.empty(1024, bad_x.shape[1], device="cuda"))
        assert e.value.status == B.GRIM_ERR_UNSUPPORTED
        B.grim_bcr_destroy(h)


# ---------------------------------------------------------------------------------------- convolution


def conv_col_norms(x, ksize, stride, pad):
    """||im2col column||_2 per output pixel: sqrt of the box-sum of x^2 over the receptive field."""
    xx = torch.from_numpy(np.asarray(x, np.float64) ** 2)
    ones = torch.ones(1, xx.shape[1], ksize, ksize, dtype=torch.float64)
    return torch.sqrt(torch.nn.functional.conv2d(xx, ones, stride=stride, padding=pad)).numpy()  # N,1,OH,OW


def check_conv(B, L, batch_x, *, ksize, stride, pad, bf16, relu=True, out_bf16=False, kernel_flags=0):
    W, mask, bias = L["W"], L["mask"], L["bias"]
    dt = B.GRIM_BF16 if bf16 else B.GRIM_F32
    x = gen.bf16_representable(batch_x) if bf16 else batch_x
    h = B.grim_bcr_pack(W, mask, L["bh"], L["bw"], dt, 0)
    try:
        xd = to_dev(x, bf16)
        Nb, C, H, Wd = x.shape
        OH = (H + 2 * pad - ksize) // stride + 1
        OW = (Wd + 2 * pad - ksize) // stride + 1
        out = torch.full((Nb, W.shape[0], OH, OW), float("nan"), device="cuda",
                         dtype=torch.bfloat16 if out_bf16 else torch.float32)
        if bf16:
            B.grim_bcr_reserve(h, Nb * OH * OW)
        B.grim_bcr_conv2d(h, xd, out, ksize, stride, pad, bias=to_dev(bias), relu=relu, kernel_flags=kernel_flags)
        torch.cuda.synchronize()
        assert B.grim_bcr_status(h) == B.GRIM_OK
        got = out.float().cpu().numpy().astype(np.float64)
        want = orc.conv2d(W, mask, x, bias, ksize=ksize, stride=stride, pad=pad, relu=relu, dtype=dt)
        Wm = orc.masked_weight(W, mask, dt)
        scale = np.linalg.norm(Wm, axis=1)[None, :, None, None] * conv_col_norms(x, ksize, stride, pad)
        assert_close(got, want, scale, bf16_in=bf16, out_bf16=out_bf16,
                     bias_abs=np.abs(bias.astype(np.float64))[None, :, None, None], what="conv")
    finally:
        B.grim_bcr_destroy(h)


@pytest.mark.parametrize("geom", [(3, 1, 1), (3, 2, 1), (1, 1, 0), (5, 1, 2), (3, 1, 0)])
@pytest.mark.parametrize("bf16", [False, True])
def test_conv_small(B, geom, bf16):
    ks, stride, pad = geom
    L = gen.conv_layer(2, 12, 40, 13, ksize=ks, bh=8, bw=32, compression=4, seed=71)
    x = np.maximum(gen.normal_f32((3, 12, 13, 11), 1.0, 72, 0), 0)
    check_conv(B, L, x, ksize=ks, stride=stride, pad=pad, bf16=bf16)
    check_conv(B, L, x, ksize=ks, stride=stride, pad=pad, bf16=bf16, relu=False, out_bf16=bf16)


@pytest.mark.parametrize("bf16", [False, True])
def test_conv_11x11_and_1x1(B, bf16):
    """The large kernels of the paper's 3 x 3 against 11 x 11 comparison (Section 6.3), at stride 1 and at the stride 4
    of the classic first layer that uses them, and 1 x 1 kernels, which run as plain products per image (wide enough
    pixel counts to reach the tensor-core kernels with bf16)."""
    L = gen.conv_layer(2, 6, 48, 23, ksize=11, bh=8, bw=32, compression=5, seed=110)
    check_conv(B, L, L["x"], ksize=11, stride=1, pad=5, bf16=bf16)
    check_conv(B, L, L["x"], ksize=11, stride=4, pad=2, bf16=bf16, relu=False, out_bf16=bf16)
    L1 = gen.conv_layer(3, 96, 264, 24, ksize=1, bh=8, bw=32, compression=4, seed=111)
    check_conv(B, L1, L1["x"], ksize=1, stride=1, pad=0, bf16=bf16)
    check_conv(B, L1, L1["x"], ksize=1, stride=1, pad=0, bf16=bf16, relu=False, out_bf16=bf16)
    L2 = gen.conv_layer(2, 40, 72, 7, ksize=1, bh=4, bw=16, compression=3, seed=112)   # odd pixel count: unaligned rows
    check_conv(B, L2, L2["x"], ksize=1, stride=1, pad=0, bf16=bf16)


@pytest.mark.parametrize("bf16", [False, True])
def test_config3_conv_batch1(B, bf16):
    L = gen.conv_layer(1, 512, 512, 28, bf16=bf16)
    check_conv(B, L, L["x"], ksize=3, stride=1, pad=1, bf16=bf16)


def test_config3_conv_batch32_sampled(B):
    """Full-size launch (batch 32, the shape the benchmark times); the oracle checks 4 of the 32 images."""
    L = gen.conv_layer(32, 512, 512, 28)
    h = B.grim_bcr_pack(L["W"], L["mask"], 16, 64, B.GRIM_F32, 0)
    xd = to_dev(L["x"])
    out = torch.empty(32, 512, 28, 28, device="cuda")
    B.grim_bcr_conv2d(h, xd, out, 3, 1, 1, bias=to_dev(L["bias"]), relu=True)
    torch.cuda.synchronize()
    pick = [0, 7, 19, 31]
    want = orc.conv2d(L["W"], L["mask"], L["x"][pick], L["bias"], ksize=3, stride=1, pad=1, relu=True)
    assert rel_fro(out[pick].cpu().numpy(), want) <= F32_TOL
    B.grim_bcr_destroy(h)


def test_maxpool(B):
    x = torch.randn(2, 5, 8, 12, device="cuda")
    out = torch.empty(2, 5, 4, 6, device="cuda")
    B.grim_maxpool2x2(x, out)
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy().astype(np.float64), orc.maxpool2x2(x.cpu().numpy().astype(np.float64)))
    xb = x.to(torch.bfloat16)
    ob = torch.empty(2, 5, 4, 6, device="cuda", dtype=torch.bfloat16)
    B.grim_maxpool2x2(xb, ob)
    torch.cuda.synchronize()
    assert np.array_equal(ob.float().cpu().numpy().astype(np.float64),
                          orc.maxpool2x2(xb.float().cpu().numpy().astype(np.float64)))


def test_vgg_stack_small_image_per_layer(B):
    """Config-4 layer shapes at a 32x32 image: each layer is checked with the oracle fed the GPU's own
    previous-layer output (bf16 in, fp32 accumulate, bf16 out)."""
    net = gen.vgg16_stack(2, image=32)
    cur = to_dev(net["x"], True)
    for L in net["layers"]:
        h = B.grim_bcr_pack(L["W"], L["mask"], net["bh"], net["bw"], B.GRIM_BF16, 0)
        Nb, C, H, Wd = cur.shape
        out = torch.empty(Nb, L["cout"], H, Wd, device="cuda", dtype=torch.bfloat16)
        B.grim_bcr_conv2d(h, cur, out, 3, 1, 1, bias=to_dev(L["bias"]), relu=True)
        torch.cuda.synchronize()
        x_np = cur.float().cpu().numpy()
        want = orc.conv2d(L["W"], L["mask"], x_np, L["bias"], ksize=3, stride=1, pad=1, relu=True, dtype=orc.DTYPE_BF16)
        Wm = orc.masked_weight(L["W"], L["mask"], orc.DTYPE_BF16)
        scale = np.linalg.norm(Wm, axis=1)[None, :, None, None] * conv_col_norms(x_np, 3, 1, 1)
        assert_close(out.float().cpu().numpy(), want, scale, bf16_in=True, out_bf16=True,
                     bias_abs=np.abs(L["bias"].astype(np.float64))[None, :, None, None], what=f"vgg layer {L['cout']}")
        B.grim_bcr_destroy(h)
        if L["pool"]:
            pooled = torch.empty(Nb, L["cout"], H // 2, Wd // 2, device="cuda", dtype=torch.bfloat16)
            B.grim_maxpool2x2(out, pooled)
            cur = pooled
        else:
            cur = out


@pytest.mark.parametrize("layer", [0, 1, 4, 8, 12])
def test_vgg_full_size_layers(B, layer):
    """Config-4 layers at their real 224x224 sizes (batch 1, the launch shapes the benchmark times): first layer
    (K = 27, ragged), the widest pixel count, and one layer per resolution down to 14x14."""
    net = gen.vgg16_stack(1)
    L = net["layers"][layer]
    x = gen.bf16_representable(np.maximum(gen.normal_f32((1, L["cin"], L["hw"], L["hw"]), 1.0, 93, layer), 0))
    LL = dict(W=L["W"], mask=L["mask"], bias=L["bias"], bh=net["bh"], bw=net["bw"])
    check_conv(B, LL, x, ksize=3, stride=1, pad=1, bf16=True, out_bf16=True)


def test_conv_bf16_batch_crossing_images(B):
    """Tensor-core convolution with an image size that is not a multiple of the 8-pixel pieces or of the 256-column
    tile, several images, fp32 and bf16 outputs."""
    L = gen.conv_layer(5, 24, 72, 15, ksize=3, bh=8, bw=32, compression=5, seed=94)
    check_conv(B, L, L["x"], ksize=3, stride=1, pad=1, bf16=True)
    check_conv(B, L, L["x"], ksize=3, stride=1, pad=1, bf16=True, relu=False, out_bf16=True)


@pytest.mark.parametrize("shape", [(12, 12, 7), (8, 16, 9), (16, 10, 5), (24, 16, 3), (10, 14, 5), (14, 14, 3)])
@pytest.mark.parametrize("bh", [4, 8, 16])
def test_conv_bf16_staged_planes(B, shape, bh):
    """Tensor-core convolution on planes whose size is a multiple of 8 pixels, or of 4 (the variants that stage the
    input planes in shared memory by bulk copies / by 8-byte copies): 256-pixel tiles that meet two or three images, a
    ragged last tile, several K tiles, all block heights."""
    H, Wd, batch = shape
    C, Cout, bw = 20, 136, 32
    rng_seed = 300 + H + Wd + bh
    W = gen.dense_weight(Cout, C * 9, seed=rng_seed)
    mask = gen.bcr_mask(Cout, C * 9, bh, bw, compression=4, dist="uniform", seed=rng_seed + 1)
    bias = gen.normal_f32((Cout,), 0.1, rng_seed + 2, 0)
    x = np.maximum(gen.normal_f32((batch, C, H, Wd), 1.0, rng_seed + 3, 0), 0)
    L = dict(W=W, mask=mask, bias=bias, bh=bh, bw=bw)
    check_conv(B, L, x, ksize=3, stride=1, pad=1, bf16=True)
    check_conv(B, L, x, ksize=3, stride=1, pad=1, bf16=True, relu=False, out_bf16=True)


@pytest.mark.parametrize("shape", [(12, 12, 7), (8, 16, 9), (16, 10, 5), (24, 16, 3), (10, 14, 5), (14, 14, 3), (7, 9, 4), (15, 15, 5)])
@pytest.mark.parametrize("bh,cout", [(4, 136), (8, 300), (16, 520)])
def test_conv_bf16_paired_kernel(B, shape, bh, cout):
    """The paired tensor-core convolution asked for by name: planes staged by bulk copies (multiples of 8 pixels), by
    8-byte copies (multiples of 4) and read from global memory (others); tiles that meet two or three images, pixel
    counts that leave the odd block of a pair with a partial or an empty tile, one to five row tiles (odd counts give
    the last pair an empty partner), fp32 and bf16 outputs."""
    H, Wd, batch = shape
    C, bw = 20, 32
    rng_seed = 400 + H + Wd + bh
    W = gen.dense_weight(cout, C * 9, seed=rng_seed)
    mask = gen.bcr_mask(cout, C * 9, bh, bw, compression=4, dist="uniform", seed=rng_seed + 1)
    bias = gen.normal_f32((cout,), 0.1, rng_seed + 2, 0)
    x = np.maximum(gen.normal_f32((batch, C, H, Wd), 1.0, rng_seed + 3, 0), 0)
    L = dict(W=W, mask=mask, bias=bias, bh=bh, bw=bw)
    check_conv(B, L, x, ksize=3, stride=1, pad=1, bf16=True, kernel_flags=B.GRIM_CONV_PAIRED)
    check_conv(B, L, x, ksize=3, stride=1, pad=1, bf16=True, relu=False, out_bf16=True, kernel_flags=B.GRIM_CONV_PAIRED)


@pytest.mark.parametrize("y_bf16", [False, True])
def test_tensor_core_split_over_k(B, y_bf16):
    """Few output tiles and a long K: the tensor-core multiply is split over K (partial sums through the fp32
    scratch, second pass for the output), matrix and convolution forms, with pruned bands and a ragged last K tile."""
    M, K, bh, bw = 300, 3100, 8, 32
    W = gen.dense_weight(M, K, seed=310)
    mask = gen.bcr_mask(M, K, bh, bw, compression=6, dist="zipf", seed=311)
    mask[16:32] = 0
    X = gen.normal_f32((K, 304), 1.0, 312, 0)  # row stride a multiple of 16 bytes (TMA)
    check_spmm(B, W, mask, X, bh, bw, bf16=True, path=2, y_bf16=y_bf16)
    C, Cout = 176, 200
    Wc = gen.dense_weight(Cout, C * 9, seed=313)
    maskc = gen.bcr_mask(Cout, C * 9, 16, 64, compression=5, dist="uniform", seed=314)
    L = dict(W=Wc, mask=maskc, bias=gen.normal_f32((Cout,), 0.1, 315, 0), bh=16, bw=64)
    for H, Wd, batch in ((12, 12, 3), (7, 9, 2)):  # staged planes / planes read from global memory
        x = np.maximum(gen.normal_f32((batch, C, H, Wd), 1.0, 316, H), 0)
        check_conv(B, L, x, ksize=3, stride=1, pad=1, bf16=True, out_bf16=y_bf16)


# ---------------------------------------------------------------------------------------- GRU


def build_gru(B, m, max_T):
    hi, hh = [], []
    for lay in m["layers"]:
        hi.append(B.grim_bcr_pack(lay["W_ih"], lay["mask_ih"], m["bh"], m["bw"], B.GRIM_F32, 0))
        hh.append(B.grim_bcr_pack(lay["W_hh"], lay["mask_hh"], m["bh"], m["bw"], B.GRIM_F32, 0))
    g = B.grim_gru_create(hi, hh, [l["b_ih"] for l in m["layers"]], [l["b_hh"] for l in m["layers"]], max_T)
    return g, hi + hh


def check_gru(B, m, h0=None, grid_kernel=False):
    T, H, L = m["T"], m["hidden"], len(m["layers"])
    g, handles = build_gru(B, m, T)
    try:
        if grid_kernel:  # a poll limit selects the cooperative-grid kernel instead of the cluster kernel
            B.grim_gru_debug_barrier(g, -1, 1 << 22)
        x = to_dev(m["x"])
        y = torch.full((T, H), float("nan"), device="cuda")
        hT = torch.full((L, H), float("nan"), device="cuda")
        for _ in range(2):  # the handle is reusable
            B.grim_gru_seq(g, x, y, h0=to_dev(h0) if h0 is not None else None, hT=hT)
            assert B.grim_gru_status(g) == B.GRIM_OK
        want_y, want_h = orc.gru_seq(m["layers"], m["x"], h0=h0)
        assert rel_fro(y.cpu().numpy(), want_y) <= F32_TOL, rel_fro(y.cpu().numpy(), want_y)
        assert rel_fro(hT.cpu().numpy(), want_h) <= F32_TOL
    finally:
        B.grim_gru_destroy(g)
        for h in handles:
            B.grim_bcr_destroy(h)


@pytest.mark.parametrize("cfg", [(20, 64, 1, 7, 8, 32), (37, 128, 2, 13, 8, 32), (16, 96, 3, 5, 4, 16),
                                 (50, 256, 2, 9, 16, 64)])
def test_gru_small(B, cfg):
    in_f, H, L, T, bh, bw = cfg
    m = gen.gru_model(in_f, H, L, T, bh=bh, bw=bw, compression=4, seed=80)
    check_gru(B, m)
    h0 = gen.normal_f32((L, H), 0.5, 81, 0)
    check_gru(B, m, h0=h0)
    check_gru(B, m, h0=h0, grid_kernel=True)


def test_gru_four_layers_and_odd_hidden_size(B):
    """Four layers (run one after the other: the wavefront schedule is kept to three) against the oracle, and a
    hidden size that is a multiple of the block height but not of 4 is refused at creation."""
    check_gru(B, gen.gru_model(24, 128, 4, 70, bh=8, bw=32, compression=4, seed=97))
    m = gen.gru_model(12, 30, 1, 3, bh=6, bw=16, compression=2, seed=98)
    with pytest.raises(B.GrimError) as e:
        build_gru(B, m, 3)
    assert e.value.status == B.GRIM_ERR_UNSUPPORTED


@pytest.mark.parametrize("grid_kernel", [False, True])
def test_config2_gru_full(B, grid_kernel):
    check_gru(B, gen.gru_model(), grid_kernel=grid_kernel)


@pytest.mark.parametrize("chunks", [1, 2, 5, 8])
def test_gru_layer_pipelining_gives_the_same_result(B, chunks):
    """Three layers cut into `chunks` pieces in time and run as a wavefront on internal streams: same outputs and
    final states as the oracle, with and without an initial state, on a sequence length that does not divide."""
    m = gen.gru_model(30, 128, 3, 53, bh=8, bw=32, compression=4, seed=95)
    T, H, L = m["T"], m["hidden"], 3
    g, handles = build_gru(B, m, T)
    try:
        B.grim_gru_set_pipeline(g, chunks)
        h0 = gen.normal_f32((L, H), 0.5, 96, 0)
        for init in (None, h0):
            y = torch.full((T, H), float("nan"), device="cuda")
            hT = torch.full((L, H), float("nan"), device="cuda")
            B.grim_gru_seq(g, to_dev(m["x"]), y, h0=to_dev(init) if init is not None else None, hT=hT)
            assert B.grim_gru_status(g) == B.GRIM_OK
            want_y, want_h = orc.gru_seq(m["layers"], m["x"], h0=init)
            assert rel_fro(y.cpu().numpy(), want_y) <= F32_TOL
            assert rel_fro(hT.cpu().numpy(), want_h) <= F32_TOL
    finally:
        B.grim_gru_destroy(g)
        for h in handles:
            B.grim_bcr_destroy(h)


@pytest.mark.parametrize("cfg", [(153, 1024, 2, 32), (37, 128, 3, 5), (20, 64, 1, 1)])
def test_gru_batched_step(B, cfg):
    """One time step for a batch of sequences (the paper's timed GRU shape is sequence length 1, batch 32), two steps in a
    row so that the carried state is used: against the oracle run per batch element."""
    in_f, H, L, batch = cfg
    m = gen.gru_model(in_f, H, L, 2, compression=10 if H == 1024 else 4, seed=99)
    g, handles = build_gru(B, m, 2 * batch + 2)
    try:
        xs = [gen.normal_f32((batch, in_f), 1.0, 100, t) for t in range(2)]
        h = to_dev(gen.normal_f32((L, batch, H), 0.5, 101, 0))
        h_np = h.cpu().numpy().astype(np.float64)
        y = torch.full((batch, H), float("nan"), device="cuda")
        for t in range(2):
            B.grim_gru_step(g, to_dev(xs[t]), h, y)
            torch.cuda.synchronize()
            want_y = np.empty((batch, H))
            for b in range(batch):
                yb, hb = orc.gru_seq(m["layers"], xs[t][b:b + 1], h0=h_np[:, b])
                want_y[b], h_np[:, b] = yb[0], hb
            assert rel_fro(y.cpu().numpy(), want_y) <= F32_TOL
            assert rel_fro(h.cpu().numpy(), h_np) <= F32_TOL
        with pytest.raises(B.GrimError) as e:
            B.grim_gru_step(g, torch.zeros(2 * batch + 2, in_f, device="cuda"), torch.zeros(L, 2 * batch + 2, H, device="cuda"))
        assert e.value.status == B.GRIM_ERR_SHAPE
    finally:
        B.grim_gru_destroy(g)
        for hd in handles:
            B.grim_bcr_destroy(hd)


def test_gru_bounded_wait_reports_timeout(B):
    """One thread block stays away from the step barrier: every wait runs out after a small bound, the
    kernel returns by itself and the status word says so; afterwards the handle works normally."""
    m = gen.gru_model(20, 256, 1, 6, bh=8, bw=32, compression=4, seed=82)
    g, handles = build_gru(B, m, 6)
    x = to_dev(m["x"])
    y = torch.zeros(6, 256, device="cuda")
    B.grim_gru_debug_barrier(g, 1, 20000)
    B.grim_gru_seq(g, x, y)
    assert B.grim_gru_status(g) == B.GRIM_ERR_TIMEOUT
    B.grim_gru_debug_barrier(g, -1, 0)
    B.grim_gru_seq(g, x, y)
    assert B.grim_gru_status(g) == B.GRIM_OK
    want_y, _ = orc.gru_seq(m["layers"], m["x"])
    assert rel_fro(y.cpu().numpy(), want_y) <= F32_TOL
    B.grim_gru_destroy(g)
    for h in handles:
        B.grim_bcr_destroy(h)
