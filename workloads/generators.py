"""Seeded synthetic inputs shaped like the paper's workloads.

This module is shared by the CPU oracle's tests and by the CUDA path's tests and
benchmark.  It holds no arithmetic of the method itself: it only draws dense
weights, BCR keep-masks and activations from a counter-based generator (Philox
keyed by (seed, stream)), so that both sides see identical inputs.

The BCR pattern follows Section 3.2 of the paper: the weight matrix is tiled into
equal blocks of bh rows by bw columns (the "4x16" of the search-space example in
Section 3.2 is 4 rows by 16 columns), and inside each block whole rows and whole
columns are dropped independently; what survives in a block is a full sub-matrix.
The pruning rate c is total weights / kept weights.

The trained VGG-16 / GRU weights and the ImageNet / TIMIT data of Section 6 are not
needed for the multiply itself; these inputs stand in for them.
"""
from __future__ import annotations

import numpy as np
import torch

# ----------------------------------------------------------------------------------------------
# generator plumbing
# ----------------------------------------------------------------------------------------------


def rng(seed: int, stream: int = 0) -> np.random.Generator:
    """Counter-based generator: one independent stream per (seed, stream) pair."""
    return np.random.Generator(np.random.Philox(key=[int(seed) & (2**64 - 1), int(stream) & (2**64 - 1)]))


def normal_f32(shape, std: float, seed: int, stream: int) -> np.ndarray:
    return (rng(seed, stream).standard_normal(shape) * std).astype(np.float32)


def bf16_representable(a: np.ndarray) -> np.ndarray:
    """Round an fp32 array to the nearest bf16 value (library conversion), returned as fp32.

    Used only to make *inputs* that a bf16 run can hold exactly; the oracle and the CUDA
    packer each have their own rounding for the weights.
    """
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32))
    return t.to(torch.bfloat16).to(torch.float32).numpy()


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """fp32 array holding bf16-representable values -> uint16 bit patterns."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> 16).astype(np.uint16)


# ----------------------------------------------------------------------------------------------
# BCR keep-masks
# ----------------------------------------------------------------------------------------------


def _kr_pmf(h: int, dist: str, zipf_s: float) -> np.ndarray:
    k = np.arange(1, h + 1, dtype=np.float64)
    if dist == "uniform":
        p = np.ones(h)
    elif dist == "zipf":
        p = k ** (-zipf_s)
    else:
        raise ValueError(dist)
    return p / p.sum()


def bcr_keep_lists(M: int, K: int, bh: int, bw: int, *, compression: float | None = None,
                   dist: str = "uniform", seed: int = 0, stream: int = 100,
                   kr_fixed: int | None = None, kc_fixed: int | None = None,
                   zipf_s: float = 1.2, empty_frac: float = 0.0, band_zipf: float = 0.0):
    """Draw per-block keep flags.

    Returns (rowkeep, colkeep): bool arrays of shape (nbr, nbc, bh) and (nbr, nbc, bw).
    Edge blocks of a ragged grid only ever keep rows / columns that exist.

    dist = "fixed": exactly kr_fixed rows and kc_fixed columns per block.
    dist = "uniform": kept-row count uniform on 1..bh.  dist = "zipf": P(kr = k) ~ k^-s.
    In the last two the kept-column count is chosen per block so that the expected tile
    size is bh*bw/compression: kc = floor(t) + [u < frac(t)], t = clamp(s / E[kr], 1, bw).
    band_zipf > 0 makes whole block rows (bands) heavy or light: band i gets the share rank_i^-band_zipf of the
    kept columns (ranks are a random permutation of the bands, shares scaled to mean 1), so that the work per band
    is skewed the way the kept-row counts are skewed per block - the case a band schedule has something to balance.
    """
    g = rng(seed, stream)
    nbr = -(-M // bh)
    nbc = -(-K // bw)
    hb = np.minimum(bh, M - np.arange(nbr) * bh)  # rows that exist in block-row i
    wb = np.minimum(bw, K - np.arange(nbc) * bw)
    HB = np.broadcast_to(hb[:, None], (nbr, nbc))
    WB = np.broadcast_to(wb[None, :], (nbr, nbc))

    if dist == "fixed":
        kr = np.minimum(int(kr_fixed), HB).astype(np.int64)
        kc = np.minimum(int(kc_fixed), WB).astype(np.int64)
    else:
        kr = np.empty((nbr, nbc), dtype=np.int64)
        ekr = np.empty((nbr, nbc), dtype=np.float64)
        u_kr = g.random((nbr, nbc))
        for h in np.unique(hb):
            pmf = _kr_pmf(int(h), dist, zipf_s)
            cdf = np.cumsum(pmf)
            sel = HB == h
            kr[sel] = 1 + np.searchsorted(cdf, u_kr[sel], side="right").clip(0, h - 1)
            ekr[sel] = float((pmf * np.arange(1, h + 1)).sum())
        s = HB * WB / float(compression)
        if band_zipf > 0.0:
            share = (1.0 + g.permutation(nbr)) ** (-float(band_zipf))
            s = s * (share / share.mean())[:, None]
        t = np.clip(s / ekr, 1.0, WB)
        u_kc = g.random((nbr, nbc))
        kc = (np.floor(t) + (u_kc < (t - np.floor(t)))).astype(np.int64)
        kc = np.minimum(kc, WB)
    if empty_frac > 0.0:
        dead = g.random((nbr, nbc)) < empty_frac
        kr = np.where(dead, 0, kr)
        kc = np.where(dead, 0, kc)

    def subset(count, extent, width):
        keys = g.random((nbr, nbc, width))
        keys = np.where(np.arange(width)[None, None, :] < extent[:, :, None], keys, 2.0)
        srt = np.sort(keys, axis=-1)
        idx = np.clip(count - 1, 0, width - 1)
        thr = np.take_along_axis(srt, idx[:, :, None], axis=-1)
        keep = keys <= thr
        keep &= (count > 0)[:, :, None]
        keep &= keys < 1.5
        return keep

    rowkeep = subset(kr, HB, bh)
    colkeep = subset(kc, WB, bw)
    return rowkeep, colkeep


def mask_from_keep(rowkeep: np.ndarray, colkeep: np.ndarray, M: int, K: int) -> np.ndarray:
    """Expand per-block keep flags to an M x K uint8 mask (1 = kept)."""
    nbr, nbc, bh = rowkeep.shape
    bw = colkeep.shape[2]
    m = rowkeep[:, :, :, None] & colkeep[:, :, None, :]
    m = m.transpose(0, 2, 1, 3).reshape(nbr * bh, nbc * bw)
    return np.ascontiguousarray(m[:M, :K]).astype(np.uint8)


def bcr_mask(M, K, bh, bw, **kw) -> np.ndarray:
    rk, ck = bcr_keep_lists(M, K, bh, bw, **kw)
    return mask_from_keep(rk, ck, M, K)


def dense_weight(M: int, K: int, seed: int, stream: int = 1, std: float = 0.05) -> np.ndarray:
    """Dense fp32 weight N(0, std); pruned positions also hold values - the mask decides."""
    return normal_f32((M, K), std, seed, stream)


# ----------------------------------------------------------------------------------------------
# the five benchmark configurations
# ----------------------------------------------------------------------------------------------


def config1_spmm(seed: int = 1):
    """Single fp32 SpMM: W 256x256, 16x16 blocks keeping 8 of 16 rows and columns, X 256x64."""
    M = K = 256
    W = dense_weight(M, K, seed)
    mask = bcr_mask(M, K, 16, 16, dist="fixed", kr_fixed=8, kc_fixed=8, seed=seed)
    X = normal_f32((K, 64), 1.0, seed, 2)
    return dict(W=W, mask=mask, X=X, bh=16, bw=16)


def gru_model(in_features: int = 153, hidden: int = 1024, layers: int = 2, T: int = 200,
              bh: int = 8, bw: int = 32, compression: float = 10.0, seed: int = 2,
              dist: str = "uniform"):
    """GRU inference inputs: per layer W_ih (3H x in), W_hh (3H x H) with gate order r, z, n,
    two bias vectors, BCR masks at the given compression, x of shape (T, in)."""
    out = dict(T=T, hidden=hidden, layers=[], bh=bh, bw=bw)
    for l in range(layers):
        kin = in_features if l == 0 else hidden
        st = 10 * l
        lay = dict(
            W_ih=dense_weight(3 * hidden, kin, seed, 11 + st),
            W_hh=dense_weight(3 * hidden, hidden, seed, 12 + st),
            b_ih=normal_f32((3 * hidden,), 0.05, seed, 13 + st),
            b_hh=normal_f32((3 * hidden,), 0.05, seed, 14 + st),
            mask_ih=bcr_mask(3 * hidden, kin, bh, bw, compression=compression, dist=dist, seed=seed, stream=15 + st),
            mask_hh=bcr_mask(3 * hidden, hidden, bh, bw, compression=compression, dist=dist, seed=seed, stream=16 + st),
        )
        out["layers"].append(lay)
    out["x"] = normal_f32((T, in_features), 1.0, seed, 3)
    return out


def conv_layer(batch: int, cin: int, cout: int, hw: int, *, ksize: int = 3, bh: int = 16, bw: int = 64,
               compression: float = 8.0, seed: int = 3, bf16: bool = False, stream0: int = 0,
               dist: str = "uniform"):
    """One conv layer: weight (cout, cin, k, k) viewed as cout x (cin*k*k) in OIHW order,
    BCR mask on that matrix, bias N(0, 0.05), input ReLU(N(0,1)) in NCHW."""
    K = cin * ksize * ksize
    W = dense_weight(cout, K, seed, stream0 + 21)
    mask = bcr_mask(cout, K, bh, bw, compression=compression, dist=dist, seed=seed, stream=stream0 + 22)
    bias = normal_f32((cout,), 0.05, seed, stream0 + 23)
    x = np.maximum(normal_f32((batch, cin, hw, hw), 1.0, seed, stream0 + 24), 0.0)
    if bf16:
        x = bf16_representable(x)
    return dict(W=W, mask=mask, bias=bias, x=x, cin=cin, cout=cout, hw=hw, ksize=ksize, bh=bh, bw=bw)


VGG16_CHANNELS = [64, 64, 128, 128, 256, 256, 256, 512, 512, 512, 512, 512, 512]
VGG16_POOL_AFTER = {1, 3, 6, 9, 12}  # zero-based conv index followed by a 2x2/2 max-pool


def vgg16_stack(batch: int, *, image: int = 224, bh: int = 8, bw: int = 32, compression: float = 8.0,
                seed: int = 4, bf16: bool = True):
    """The 13 conv layers of VGG-16 with synthetic BCR-pruned weights and an N(0,1) image."""
    layers = []
    cin = 3
    hw = image
    for i, cout in enumerate(VGG16_CHANNELS):
        K = cin * 9
        layers.append(dict(
            W=dense_weight(cout, K, seed, 100 + 10 * i),
            mask=bcr_mask(cout, K, bh, bw, compression=compression, dist="uniform", seed=seed, stream=101 + 10 * i),
            bias=normal_f32((cout,), 0.05, seed, 102 + 10 * i),
            cin=cin, cout=cout, hw=hw, pool=(i in VGG16_POOL_AFTER)))
        cin = cout
        if i in VGG16_POOL_AFTER:
            hw //= 2
    x = normal_f32((batch, 3, image, image), 1.0, seed, 5)
    if bf16:
        x = bf16_representable(x)
    return dict(layers=layers, x=x, bh=bh, bw=bw)


def sweep_case(M: int, N: int, compression: float, bh: int, bw: int, dist: str, seed: int = 5, bf16: bool = False):
    """One point of the SpMM sweep: square W (M = K), X K x N."""
    W = dense_weight(M, M, seed, 31)
    mask = bcr_mask(M, M, bh, bw, compression=compression, dist=dist, seed=seed, stream=32)
    X = normal_f32((M, N), 1.0, seed, 33)
    if bf16:
        X = bf16_representable(X)
    return dict(W=W, mask=mask, X=X, bh=bh, bw=bw)
