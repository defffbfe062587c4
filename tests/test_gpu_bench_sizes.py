"""GPU parity at the sizes and launch configurations the benchmark times (default routing, reorder as in the
bench).  The full fp64 product is too slow at these sizes, so the oracle computes sampled output rows (every
output row is an independent product) or sampled images, element by element; rows kept by no block are checked
over the whole output."""
import numpy as np
import pytest
import torch

from oracle import bcr_oracle as orc
from parity_util import assert_close
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


def sampled_spmm_check(B, s, bh, bw, *, bf16, reorder, rows=192, seed=0):
    W, mask = s["W"], s["mask"]
    X = gen.bf16_representable(s["X"]) if bf16 else np.asarray(s["X"], np.float32)
    M, N = W.shape[0], X.shape[1]
    dt = B.GRIM_BF16 if bf16 else B.GRIM_F32
    h = B.grim_bcr_pack(W, mask, bh, bw, dt, B.GRIM_PACK_REORDER if reorder else 0)
    try:
        Y = torch.full((M, N), float("nan"), device="cuda")
        B.grim_bcr_spmm(h, to_dev(X, bf16), Y)
        torch.cuda.synchronize()
        assert B.grim_bcr_status(h) == B.GRIM_OK
        got = Y.cpu().numpy()
        assert np.all(np.isfinite(got))
        dead = np.flatnonzero(mask.sum(axis=1) == 0)
        assert np.all(got[dead] == 0.0) and not np.any(np.signbit(got[dead]))
        pick = np.sort(gen.rng(900 + seed, 0).choice(M, size=min(rows, M), replace=False))
        want = orc.spmm(W[pick], mask[pick], X, dt)
        Wm = orc.masked_weight(W[pick], mask[pick], dt)
        scale = np.linalg.norm(Wm, axis=1)[:, None] * np.linalg.norm(X.astype(np.float64), axis=0)[None, :]
        assert_close(got[pick], want, scale, bf16_in=bf16, out_bf16=False, what=f"spmm {M}^2 N={N}")
    finally:
        B.grim_bcr_destroy(h)


@pytest.mark.parametrize("reorder", [1, 0])
@pytest.mark.parametrize("case", [(1, 4.0, False), (1, 4.0, True), (16, 4.0, False), (16, 4.0, True),
                                  (128, 8.0, False), (128, 8.0, True), (1024, 8.0, False), (1024, 8.0, True)])
def test_sweep_8192_points(B, case, reorder):
    """The 8192 x 8192 corner of the sweep: the matrix-vector product (c = 4), N = 16, N = 128 and N = 1024 in fp32
    and bf16, 8 x 32 blocks, with and without the reorder."""
    N, c, bf16 = case
    s = gen.sweep_case(8192, N, c, 8, 32, "uniform", bf16=bf16)
    sampled_spmm_check(B, s, 8, 32, bf16=bf16, reorder=reorder, seed=N)


@pytest.mark.parametrize("case", [(4096, 1, 4.0, 16, 64, "zipf", False), (4096, 1024, 16.0, 4, 16, "zipf", True),
                                  (4096, 1024, 8.0, 16, 64, "uniform", False)])
def test_sweep_4096_points(B, case):
    M, N, c, bh, bw, dist, bf16 = case
    s = gen.sweep_case(M, N, c, bh, bw, dist, bf16=bf16)
    sampled_spmm_check(B, s, bh, bw, bf16=bf16, reorder=1, seed=M + N)


def conv_col_norms(x, ksize, stride, pad):
    xx = torch.from_numpy(np.asarray(x, np.float64) ** 2)
    ones = torch.ones(1, xx.shape[1], ksize, ksize, dtype=torch.float64)
    return torch.sqrt(torch.nn.functional.conv2d(xx, ones, stride=stride, padding=pad)).numpy()


def conv_images_check(L, x_np, got, pick, *, bf16, out_bf16, what):
    """got: the GPU's output for images `pick` of x_np (already a NumPy array)."""
    dt = orc.DTYPE_BF16 if bf16 else orc.DTYPE_F32
    xs = x_np[pick]
    want = orc.conv2d(L["W"], L["mask"], xs, L["bias"], ksize=3, stride=1, pad=1, relu=True, dtype=dt)
    Wm = orc.masked_weight(L["W"], L["mask"], dt)
    scale = np.linalg.norm(Wm, axis=1)[None, :, None, None] * conv_col_norms(xs, 3, 1, 1)
    assert_close(got, want, scale, bf16_in=bf16, out_bf16=out_bf16,
                 bias_abs=np.abs(L["bias"].astype(np.float64))[None, :, None, None], what=what)


@pytest.mark.parametrize("bf16", [False, True])
def test_config3_conv_batch32(B, bf16):
    """512 -> 512, 28 x 28, batch 32 as the benchmark launches it (bf16: the staged tensor-core launch with bf16
    output); the oracle checks four images, among them the first and the last."""
    L = gen.conv_layer(32, 512, 512, 28, bf16=bf16)
    x = gen.bf16_representable(L["x"]) if bf16 else L["x"]
    h = B.grim_bcr_pack(L["W"], L["mask"], 16, 64, B.GRIM_BF16 if bf16 else B.GRIM_F32, B.GRIM_PACK_REORDER)
    try:
        out = torch.full((32, 512, 28, 28), float("nan"), device="cuda", dtype=torch.bfloat16 if bf16 else torch.float32)
        if bf16:
            B.grim_bcr_reserve(h, 32 * 28 * 28)
        B.grim_bcr_conv2d(h, to_dev(x, bf16), out, 3, 1, 1, bias=to_dev(L["bias"]), relu=True)
        torch.cuda.synchronize()
        assert B.grim_bcr_status(h) == B.GRIM_OK
        assert bool(torch.isfinite(out.float()).all())
        pick = [0, 9, 22, 31]
        conv_images_check(L, x, out[pick].float().cpu().numpy(), pick, bf16=bf16, out_bf16=bf16, what="config 3 batch 32")
    finally:
        B.grim_bcr_destroy(h)


@pytest.mark.parametrize("batch", [1, 16])
def test_config4_vgg_stack_full_size(B, batch):
    """All 13 layers at 224 x 224, batch 1 and 16, run as the benchmark runs them (bf16 in and out, ReLU fused,
    max-pools between); every layer is checked on two images with the oracle fed the GPU's own input of that layer."""
    net = gen.vgg16_stack(batch)
    cur = to_dev(net["x"], True)
    pick = [0] if batch == 1 else [0, batch - 1]
    for li, L in enumerate(net["layers"]):
        h = B.grim_bcr_pack(L["W"], L["mask"], net["bh"], net["bw"], B.GRIM_BF16, B.GRIM_PACK_REORDER)
        Nb, C, H, Wd = cur.shape
        out = torch.full((Nb, L["cout"], H, Wd), float("nan"), device="cuda", dtype=torch.bfloat16)
        B.grim_bcr_reserve(h, Nb * H * Wd)  # as the benchmark does at set-up
        B.grim_bcr_conv2d(h, cur, out, 3, 1, 1, bias=to_dev(L["bias"]), relu=True)
        torch.cuda.synchronize()
        assert B.grim_bcr_status(h) == B.GRIM_OK
        assert bool(torch.isfinite(out.float()).all()), f"layer {li + 1}"
        x_np = cur[pick].float().cpu().numpy()
        conv_images_check(L, x_np, out[pick].float().cpu().numpy(), list(range(len(pick))), bf16=True, out_bf16=True,
                          what=f"vgg layer {li + 1} batch {batch}")
        B.grim_bcr_destroy(h)
        if L["pool"]:
            pooled = torch.empty(Nb, L["cout"], H // 2, Wd // 2, device="cuda", dtype=torch.bfloat16)
            B.grim_maxpool2x2(out, pooled)
            cur = pooled
        else:
            cur = out
