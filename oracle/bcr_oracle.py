"""CPU oracle for the BCR sparse multiply (test infrastructure - never on the product path).

Plain, slow, obviously-correct fp64 NumPy code that states WHAT the hot path computes:
a weight matrix pruned with the Block-based Column-Row scheme of Section 3.2 (tile the
matrix into equal blocks; in each block drop whole rows and whole columns; survivors of a
block form a full sub-matrix) multiplied by dense activations.  Because the method only
skips structural zeros, its result has a plain definition, and the oracle is that
definition written out: expand to a dense matrix with zeros and multiply.

  * matrix x matrix / matrix x vector: the unified GEMM/GEMV view of Section 3.1;
  * convolution: the direct definition (Section 3.1 maps CONV to GEMM; the oracle does
    NOT go through im2col, so the index map of the fast path is checked independently);
  * GRU: Section 6.1 only names a 2-layer GRU; the recurrence used is the common
    library variant with gate order r, z, n, two bias vectors and the reset gate applied
    to the hidden-side pre-activation of the candidate;
  * canonical packed form + row reorder: Sections 4.2-4.3 store only kept weights plus
    shared per-block index lists after a row reorder that groups similar rows.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this module.
It shares no code with the CUDA library or its Python binding.

Pins (tests/test_oracle_pins.py): brute force over explicit block/row/column loops on tiny
matrices, all-kept masks against dense library matmul / conv2d / GRU, 1x1-block and
one-block degenerate cases of Section 3.2, the counting examples of Section 3.2
(64x64 layer with 4x16 blocks -> 1024 column segments; 1024x1024 in 64 blocks at 8x ->
2048 weights per block), pack -> unpack round trip, exact-zero pruned rows, closed-form
single-step GRU.  The BCRC array fragments of Section 4.3 refer to a figure that is not
available, so nothing here reproduces that format: BCRC export is "parity unpinned" and
not implemented in this file.
"""
from __future__ import annotations

import struct

import numpy as np

MAGIC = int.from_bytes(b"GRIMBCR1", "little")
DTYPE_F32 = 0
DTYPE_BF16 = 1


# ----------------------------------------------------------------------------------------------
# value handling
# ----------------------------------------------------------------------------------------------


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round fp32 to the nearest bf16 (ties to even); result returned as fp32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    r = ((u + 0x7FFF + lsb) >> 16) << 16
    return (r & 0xFFFFFFFF).astype(np.uint32).view(np.float32).reshape(a.shape)


def masked_weight(W: np.ndarray, mask: np.ndarray, dtype: int = DTYPE_F32) -> np.ndarray:
    """Dense M x K fp64 matrix: kept weights (rounded to bf16 first for the bf16 path), zeros elsewhere.

    The mask is authoritative (Section 3.2): a kept weight whose value is 0.0 is still kept.
    """
    Wv = np.asarray(W, dtype=np.float32)
    if dtype == DTYPE_BF16:
        Wv = round_to_bf16(Wv)
    return np.where(np.asarray(mask) != 0, Wv.astype(np.float64), 0.0)


# ----------------------------------------------------------------------------------------------
# the multiply (Section 3.1)
# ----------------------------------------------------------------------------------------------


def spmm(W, mask, X, dtype: int = DTYPE_F32) -> np.ndarray:
    """Y = (W .* mask) @ X in fp64.  X is K x N (N = 1 gives the matrix-vector case)."""
    Wm = masked_weight(W, mask, dtype)
    X = np.asarray(X, dtype=np.float64)
    if X.ndim == 1:
        X = X[:, None]
    return Wm @ X


def conv2d(W, mask, x, bias=None, *, ksize: int, stride: int = 1, pad: int = 0, relu: bool = False,
           dtype: int = DTYPE_F32) -> np.ndarray:
    """Direct convolution, NCHW, fp64.

    W / mask are Cout x (Cin*KH*KW) with the K axis flattened as k = (c*KH + kh)*KW + kw.
    out[n,o,oh,ow] = bias[o] + sum_{c,kh,kw} Wm[o,c,kh,kw] * in[n,c,oh*stride+kh-pad,ow*stride+kw-pad]
    with zeros outside the image.
    """
    x = np.asarray(x, dtype=np.float64)
    Nb, C, H, Wd = x.shape
    KH = KW = int(ksize)
    Wm = masked_weight(W, mask, dtype)
    Cout = Wm.shape[0]
    assert Wm.shape[1] == C * KH * KW
    W4 = Wm.reshape(Cout, C, KH, KW)
    OH = (H + 2 * pad - KH) // stride + 1
    OW = (Wd + 2 * pad - KW) // stride + 1
    xp = np.zeros((Nb, C, H + 2 * pad, Wd + 2 * pad), dtype=np.float64)
    xp[:, :, pad:pad + H, pad:pad + Wd] = x
    out = np.zeros((Nb, Cout, OH, OW), dtype=np.float64)
    for kh in range(KH):
        for kw in range(KW):
            win = xp[:, :, kh:kh + stride * (OH - 1) + 1:stride, kw:kw + stride * (OW - 1) + 1:stride]
            # sum over input channels c: out[n,o,:,:] += W4[o,c,kh,kw] * win[n,c,:,:]
            out += np.einsum("oc,nchw->nohw", W4[:, :, kh, kw], win, optimize=True)
    if bias is not None:
        out += np.asarray(bias, dtype=np.float64)[None, :, None, None]
    if relu:
        out = np.maximum(out, 0.0)
    return out


def maxpool2x2(x: np.ndarray) -> np.ndarray:
    """2x2 max-pool, stride 2, NCHW (even H and W)."""
    Nb, C, H, Wd = x.shape
    return x.reshape(Nb, C, H // 2, 2, Wd // 2, 2).max(axis=(3, 5))


def _sigmoid(v):
    return 1.0 / (1.0 + np.exp(-v))


def gru_seq(layers, x, h0=None, dtype: int = DTYPE_F32):
    """Multi-layer GRU over a sequence, batch 1, fp64.

    layers: list of dicts with W_ih (3H x in), mask_ih, W_hh (3H x H), mask_hh, b_ih, b_hh; rows in
    gate order r, z, n.  x: T x in.  Per step and layer, with g = W_ih x_t + b_ih, q = W_hh h + b_hh:
        r = sigmoid(g_r + q_r); z = sigmoid(g_z + q_z); n = tanh(g_n + r * q_n); h' = (1 - z) * n + z * h.
    Layer l > 0 takes layer l-1's h_t as x_t.  Returns (y: T x H of the last layer, hT: L x H).
    """
    seq = np.asarray(x, dtype=np.float64)
    T = seq.shape[0]
    hT = []
    for li, lay in enumerate(layers):
        Wi = masked_weight(lay["W_ih"], lay["mask_ih"], dtype)
        Wh = masked_weight(lay["W_hh"], lay["mask_hh"], dtype)
        bi = np.asarray(lay["b_ih"], dtype=np.float64)
        bh_ = np.asarray(lay["b_hh"], dtype=np.float64)
        H = Wh.shape[1]
        h = np.zeros(H) if h0 is None else np.asarray(h0[li], dtype=np.float64).copy()
        out = np.empty((T, H))
        for t in range(T):
            g = Wi @ seq[t] + bi
            q = Wh @ h + bh_
            r = _sigmoid(g[:H] + q[:H])
            z = _sigmoid(g[H:2 * H] + q[H:2 * H])
            n = np.tanh(g[2 * H:] + r * q[2 * H:])
            h = (1.0 - z) * n + z * h
            out[t] = h
        seq = out
        hT.append(h)
    return seq, np.stack(hT)


# ----------------------------------------------------------------------------------------------
# block structure, canonical packed form, row reorder (Sections 3.2, 4.2, 4.3)
# ----------------------------------------------------------------------------------------------


def extract_blocks(mask: np.ndarray, bh: int, bw: int):
    """Per block (row-major over the block grid): kept-row and kept-column lists, block-local, ascending.

    A row (column) of a block is kept when any of its entries is kept.  Returns (blocks, ok)
    where ok is False when some block's mask is not the outer product of its two keep
    vectors, i.e. the matrix is not BCR-pruned on this grid.  Edge blocks of a ragged grid
    are smaller; their indices stay block-local.
    """
    mask = np.asarray(mask) != 0
    M, K = mask.shape
    nbr = -(-M // bh)
    nbc = -(-K // bw)
    blocks = []
    ok = True
    for i in range(nbr):
        for j in range(nbc):
            sub = mask[i * bh:(i + 1) * bh, j * bw:(j + 1) * bw]
            rk = sub.any(axis=1)
            ck = sub.any(axis=0)
            if not np.array_equal(sub, np.outer(rk, ck)):
                ok = False
            blocks.append((np.flatnonzero(rk), np.flatnonzero(ck)))
    return blocks, ok


def row_permutation(mask: np.ndarray) -> np.ndarray:
    """Row reorder of Section 4.2 in a fully specified form: rows sorted by kept-weight count,
    largest first, ties by original index (so rows with equal work sit together and empty
    rows come last).  perm[p] = original row placed at position p."""
    nnz = (np.asarray(mask) != 0).sum(axis=1)
    return np.argsort(-nnz, kind="stable").astype(np.int32)


def pack_canonical(W, mask, bh: int, bw: int, dtype: int = DTYPE_F32, reorder: bool = False) -> bytes:
    """Canonical packed form as a little-endian byte string.

    header: 8 x int64 (magic, M, K, bh, bw, nbr, nbc, dtype)
    per block in row-major grid order: u16 kr, u16 kc, u16 rows[kr], u16 cols[kc],
        values[kr*kc] row-major over (rows, cols): fp32, or bf16 bit patterns (u16)
    trailer: int32 row_perm[M] (identity unless reorder)
    """
    W = np.asarray(W, dtype=np.float32)
    mask = np.asarray(mask)
    M, K = W.shape
    blocks, ok = extract_blocks(mask, bh, bw)
    if not ok:
        raise ValueError("mask is not block-wise column-row structured")
    nbr = -(-M // bh)
    nbc = -(-K // bw)
    out = [struct.pack("<8q", MAGIC, M, K, bh, bw, nbr, nbc, dtype)]
    Wv = round_to_bf16(W) if dtype == DTYPE_BF16 else W
    for b, (rows, cols) in enumerate(blocks):
        i, j = divmod(b, nbc)
        out.append(struct.pack("<2H", len(rows), len(cols)))
        out.append(rows.astype("<u2").tobytes())
        out.append(cols.astype("<u2").tobytes())
        tile = Wv[np.ix_(i * bh + rows, j * bw + cols)] if len(rows) and len(cols) else np.zeros((0, 0), np.float32)
        tile = np.ascontiguousarray(tile, dtype=np.float32)
        if dtype == DTYPE_BF16:
            out.append((tile.view(np.uint32) >> 16).astype("<u2").tobytes())
        else:
            out.append(tile.astype("<f4").tobytes())
    perm = row_permutation(mask) if reorder else np.arange(M, dtype=np.int32)
    out.append(perm.astype("<i4").tobytes())
    return b"".join(out)


def unpack_canonical(buf: bytes):
    """Inverse of pack_canonical: returns dict(W fp32 dense with zeros, mask u8, row_perm, header fields)."""
    magic, M, K, bh, bw, nbr, nbc, dtype = struct.unpack_from("<8q", buf, 0)
    if magic != MAGIC:
        raise ValueError("bad magic")
    off = 64
    W = np.zeros((M, K), dtype=np.float32)
    mask = np.zeros((M, K), dtype=np.uint8)
    nnz = 0
    for i in range(nbr):
        for j in range(nbc):
            kr, kc = struct.unpack_from("<2H", buf, off)
            off += 4
            rows = np.frombuffer(buf, "<u2", kr, off).astype(np.int64)
            off += 2 * kr
            cols = np.frombuffer(buf, "<u2", kc, off).astype(np.int64)
            off += 2 * kc
            n = kr * kc
            if dtype == DTYPE_BF16:
                bits = np.frombuffer(buf, "<u2", n, off).astype(np.uint32) << 16
                vals = bits.view(np.float32)
                off += 2 * n
            else:
                vals = np.frombuffer(buf, "<f4", n, off)
                off += 4 * n
            if n:
                W[np.ix_(i * bh + rows, j * bw + cols)] = vals.reshape(kr, kc)
                mask[np.ix_(i * bh + rows, j * bw + cols)] = 1
            nnz += n
    perm = np.frombuffer(buf, "<i4", M, off).copy()
    off += 4 * M
    if off != len(buf):
        raise ValueError("trailing bytes")
    return dict(W=W, mask=mask, row_perm=perm, M=M, K=K, bh=bh, bw=bw, nbr=nbr, nbc=nbc, dtype=dtype, nnz=nnz)


# ----------------------------------------------------------------------------------------------
# BCRC, the paper's storage format (Section 4.3).  parity unpinned against the paper's own worked example: the
# figure that carries it is not in the available text.  The fragments the text quotes (reorder 0, 3; row offset 0, 3;
# column stride 0, 3; first column list 0, 3, 6; occurrence 0, 2) are reproduced by a test on a matrix built to have
# them, and the arrays are pinned by what they must satisfy: they rebuild the masked weight exactly, every group's
# rows have exactly the stored list, and with no two equal lists the column arrays reduce to CSR of the reordered
# matrix.
# ----------------------------------------------------------------------------------------------


def bcrc_export(W, mask, dtype: int = DTYPE_F32):
    """The six arrays of Section 4.3 for the masked weight.

    Rows are reordered by kept-weight count (largest first), then by column list (lexicographic), then by row id: rows
    with equal lists become neighbours and form a group whose list is stored once.  reorder[p] = original row at
    position p; row_offset[p] = first weight of reordered row p; occurrence[g] = first reordered row of group g;
    column_stride[g] = first entry of group g's list in compact_column; weights = kept weights row by row.
    """
    Wm = masked_weight(W, mask, dtype)
    keep = np.asarray(mask) != 0
    M = keep.shape[0]
    lists = [tuple(int(c) for c in np.flatnonzero(keep[r])) for r in range(M)]
    order = sorted(range(M), key=lambda r: (-len(lists[r]), lists[r], r))
    reorder, row_offset, occurrence, column_stride, compact, weights = [], [0], [], [], [], []
    for p, r in enumerate(order):
        reorder.append(r)
        if p == 0 or lists[r] != lists[order[p - 1]]:
            occurrence.append(p)
            column_stride.append(len(compact))
            compact.extend(lists[r])
        weights.extend(float(Wm[r, c]) for c in lists[r])
        row_offset.append(len(weights))
    occurrence.append(M)
    column_stride.append(len(compact))
    return dict(reorder=np.array(reorder, np.int32), row_offset=np.array(row_offset, np.int64),
                occurrence=np.array(occurrence, np.int32), column_stride=np.array(column_stride, np.int64),
                compact_column=np.array(compact, np.int32), weights=np.array(weights, np.float32))


def bcrc_to_dense(b, M: int, K: int) -> np.ndarray:
    """Rebuilds the dense fp32 matrix from the six arrays (what a kernel that walks BCRC would read)."""
    out = np.zeros((M, K), np.float32)
    for g in range(len(b["occurrence"]) - 1):
        cols = b["compact_column"][b["column_stride"][g]:b["column_stride"][g + 1]]
        for p in range(b["occurrence"][g], b["occurrence"][g + 1]):
            w = b["weights"][b["row_offset"][p]:b["row_offset"][p + 1]]
            assert len(w) == len(cols)
            out[b["reorder"][p], cols] = w
    return out


def index_bytes_bcrc(b) -> int:
    """Bytes of everything in BCRC that is not a weight (32-bit entries, as CSR is counted below)."""
    return 4 * (len(b["reorder"]) + len(b["row_offset"]) + len(b["occurrence"]) + len(b["column_stride"]) + len(b["compact_column"]))


def index_bytes_csr(mask) -> int:
    """Bytes of CSR's row pointers and column ids for the same matrix (32-bit entries)."""
    keep = np.asarray(mask) != 0
    return 4 * (keep.shape[0] + 1 + int(keep.sum()))


# ----------------------------------------------------------------------------------------------
# Projection onto the BCR-sparse set (Section 5.2, Eq. (4)).  The paper names the Euclidean projection but gives no
# algorithm for it.  Two functions: the exact projection by exhaustive search (tiny inputs only; this is the
# definition), and the greedy line-removal steps the library takes, written out naively (every cost recomputed from
# scratch at every step).
# ----------------------------------------------------------------------------------------------


def bcr_project_exact(V, bh: int, bw: int, sparsity: float):
    """The nearest BCR-sparse matrix by brute force: every choice of kept rows and kept columns per block, subject to
    kept entries <= (1 - sparsity) * M * K, minimising the sum of squares of the removed entries.  Returns (mask, loss).
    Exponential: a few blocks of at most 3 x 3."""
    V = np.asarray(V, dtype=np.float64)
    M, K = V.shape
    nbr, nbc = -(-M // bh), -(-K // bw)
    budget = int(np.floor((1.0 - sparsity) * M * K + 1e-9))
    total = float((V ** 2).sum())
    per_block = []
    for i in range(nbr):
        for j in range(nbc):
            sub = V[i * bh:(i + 1) * bh, j * bw:(j + 1) * bw]
            r, c = sub.shape
            opts = {}
            for rm in range(1 << r):
                for cm in range(1 << c):
                    rk = np.array([(rm >> t) & 1 for t in range(r)], bool)
                    ck = np.array([(cm >> t) & 1 for t in range(c)], bool)
                    n = int(rk.sum() * ck.sum())
                    e = float((sub[np.ix_(rk, ck)] ** 2).sum())
                    if n not in opts or e > opts[n][0]:      # per block only the best energy for each count matters
                        opts[n] = (e, np.outer(rk, ck))
            per_block.append(opts)
    best = {0: (0.0, [])}                                       # kept count -> (kept energy, chosen masks)
    for opts in per_block:
        nxt = {}
        for n0, (e0, ch) in best.items():
            for n1, (e1, m1) in opts.items():
                if n0 + n1 <= budget and (n0 + n1 not in nxt or e0 + e1 > nxt[n0 + n1][0]):
                    nxt[n0 + n1] = (e0 + e1, ch + [m1])
        best = nxt
    e, ch = max(best.values(), key=lambda t: t[0])
    mask = np.zeros((M, K), np.uint8)
    for b, m in enumerate(ch):
        i, j = divmod(b, nbc)
        mask[i * bh:i * bh + m.shape[0], j * bw:j * bw + m.shape[1]] = m
    return mask, total - e


def bcr_project(V, bh: int, bw: int, sparsity: float) -> np.ndarray:
    """Greedy projection: all rows and columns of all blocks start kept; a line is one row or one column of one block
    and costs the mean square of its entries still kept (summed in index order, in double precision); the cheapest
    line (ties: smallest id = block * (bh + bw) + row, or + bh + column) is removed until at most
    (1 - sparsity) * M * K entries are kept.  Returns the keep mask."""
    V = np.asarray(V, dtype=np.float32)
    M, K = V.shape
    nbr, nbc = -(-M // bh), -(-K // bw)
    budget = int(np.floor((1.0 - sparsity) * M * K + 1e-9))
    rowkeep = [[[True] * min(bh, M - i * bh) for j in range(nbc)] for i in range(nbr)]
    colkeep = [[[True] * min(bw, K - j * bw) for j in range(nbc)] for i in range(nbr)]
    kept = M * K

    def cost(i, j, l):
        rk, ck = rowkeep[i][j], colkeep[i][j]
        if l < bh:
            if l >= len(rk) or not rk[l]:
                return None
            vals = [float(V[i * bh + l, j * bw + c]) for c in range(len(ck)) if ck[c]]
        else:
            c = l - bh
            if c >= len(ck) or not ck[c]:
                return None
            vals = [float(V[i * bh + r, j * bw + c]) for r in range(len(rk)) if rk[r]]
        if not vals:
            return None
        s = 0.0
        for v in vals:
            s += v * v
        return s / len(vals)

    while kept > budget:
        best = None
        for i in range(nbr):
            for j in range(nbc):
                for l in range(bh + bw):
                    c = cost(i, j, l)
                    if c is not None and (best is None or c < best[0]):     # strict: the first (smallest id) wins ties
                        best = (c, i, j, l)
        if best is None:
            break
        _, i, j, l = best
        if l < bh:
            kept -= sum(colkeep[i][j])
            rowkeep[i][j][l] = False
        else:
            kept -= sum(rowkeep[i][j])
            colkeep[i][j][l - bh] = False
    mask = np.zeros((M, K), np.uint8)
    for i in range(nbr):
        for j in range(nbc):
            m = np.outer(rowkeep[i][j], colkeep[i][j])
            mask[i * bh:i * bh + m.shape[0], j * bw:j * bw + m.shape[1]] = m
    return mask
