"""Block-size selection (Section 5.1 of the paper, "Block Size Optimization").

Smaller blocks prune more freely (better accuracy), larger blocks run faster; the paper picks, per layer and pruning
rate, the smallest block size whose speed is still acceptable, by timing SYNTHESISED layers: random weights with a
random BCR mask of the wanted rate and block size, because the rate, not the position of the kept weights, is what
decides the time.  The candidates are walked from small to large and the walk stops at the first size that no
longer improves the time by the factor `threshold` (the paper leaves its value open; 1.05 here).

Only argument handling and the loop live here; the timed step is the library's multiply.
"""
from __future__ import annotations

import statistics


def synthesize(M: int, K: int, rate: float, size, seed: int = 9, dist: str = "uniform"):
    """A stand-in for a layer: weight shape as the original, random values, a random BCR mask at `rate` x compression
    with blocks of `size` = (rows, cols)."""
    from workloads import generators as gen
    bh, bw = size
    return dict(W=gen.dense_weight(M, K, seed, 41), mask=gen.bcr_mask(M, K, bh, bw, compression=rate, dist=dist, seed=seed, stream=42),
                bh=bh, bw=bw)


def run_layer(layer, N: int, bf16: bool = False, reps: int = 20) -> float:
    """Median time in milliseconds of Y = W X for the synthesised layer on the current CUDA device (L2 flushed before
    every launch)."""
    import numpy as np
    import torch
    from . import binding as B
    from workloads import generators as gen
    dt = B.GRIM_BF16 if bf16 else B.GRIM_F32
    h = B.grim_bcr_pack(layer["W"], layer["mask"], layer["bh"], layer["bw"], dt, B.GRIM_PACK_REORDER)
    try:
        K = layer["W"].shape[1]
        X = torch.from_numpy(gen.normal_f32((K, N), 1.0, 9, 43)).cuda()
        if bf16:
            X = X.to(torch.bfloat16)
        Y = torch.empty(layer["W"].shape[0], N, device="cuda")
        flush = torch.empty(1 << 28, dtype=torch.uint8, device="cuda")
        for _ in range(3):
            B.grim_bcr_spmm(h, X, Y)
        ms = []
        for _ in range(reps):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            B.grim_bcr_spmm(h, X, Y)
            e1.record()
            e1.synchronize()
            ms.append(e0.elapsed_time(e1))
        assert B.grim_bcr_status(h) == B.GRIM_OK
        return float(statistics.median(ms))
    finally:
        B.grim_bcr_destroy(h)


def find_opt_blk(shape, rate: float, block_sizes, N: int = 64, threshold: float = 1.05, time_layer=None, **kw):
    """The smallest block size of `block_sizes` (ordered small to large) beyond which growing the block no longer pays.

    Each candidate is synthesised at `rate` and timed (`time_layer(layer)` -> milliseconds; by default the library's
    multiply with N right-hand-side columns).  A candidate is accepted while it beats the best time so far by at least
    the factor `threshold`; the first one that does not ends the walk.  Returns (size, ms, trace) with trace the list
    of (size, ms) that were timed; size is None when block_sizes is empty.
    """
    M, K = shape
    timer = time_layer or (lambda layer: run_layer(layer, N, **kw))
    best_size, best_ms, trace = None, float("inf"), []
    for size in block_sizes:
        ms = timer(synthesize(M, K, rate, size))
        trace.append((tuple(size), ms))
        if best_ms / ms < threshold:
            break
        best_size, best_ms = tuple(size), ms
    return best_size, (best_ms if best_size is not None else None), trace
