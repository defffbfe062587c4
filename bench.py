#!/usr/bin/env python
"""Benchmark of the BCR sparse multiply on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload gru|gemv|spmm|conv] [--impl ours|reference]

One "step" is one pass of the whole hot path over one batch of seeded synthetic input.  The default
workload is the GRU configuration (2 layers, hidden 1024, 153 input features, T = 200, 8x32 blocks, 10x
compression): two hoisted sparse projections plus two persistent recurrent kernels.  The metric is
effective GFLOP/s = 2 * nnz * N / time (N = number of right-hand-side columns / time steps).

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead (a deliberately plain
dense fp64 program; its ratio to the GPU number says nothing about kernel quality).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "BCR SpMM/GEMV effective GFLOP/s (2*nnz*N)"

UNIT = "GFLOP/s"
CSRC = os.path.join(ROOT, "paper_2108_11033_b200", "csrc")


def profile_traffic(workload_name):
    """DRAM traffic per launch of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum of one ncu
    capture), read from the summary under profiles/ whose `workload:` line names this workload.  A summary records
    the SHA-1 of the kernel's source file at capture time (`source_sha1: <file> <hash>`); when the file has changed
    since, the counters no longer describe the kernel and None is returned."""
    import hashlib
    pdir = os.path.join(ROOT, "profiles")
    if not os.path.isdir(pdir):
        return None
    for fn in sorted(os.listdir(pdir)):
        try:
            fields = {}
            for line in open(os.path.join(pdir, fn)):
                if ":" in line and line.split(":", 1)[0].strip() in ("workload", "traffic_bytes_per_launch", "source_sha1"):
                    k, v = line.split(":", 1)
                    fields[k.strip()] = v.strip()
            if fields.get("workload") != workload_name or "traffic_bytes_per_launch" not in fields:
                continue
            src, sha = fields.get("source_sha1", " ").split()
            with open(os.path.join(CSRC, src), "rb") as f:
                if hashlib.sha1(f.read()).hexdigest() != sha:
                    return None
            return float(fields["traffic_bytes_per_launch"])
        except Exception:
            continue
    return None


_SWEEP_CACHE = {}


def sweep_inputs(M, N, c, bh, bw, dist, bf16):
    """Same inputs as workloads.generators.sweep_case (seed 5); the weight and the mask of a (size, compression, block,
    distribution) are generated once and shared by the records that use them."""
    from workloads import generators as gen
    key = (M, c, bh, bw, dist)
    if key not in _SWEEP_CACHE:
        if len(_SWEEP_CACHE) >= 2:
            _SWEEP_CACHE.pop(next(iter(_SWEEP_CACHE)))
        _SWEEP_CACHE[key] = (gen.dense_weight(M, M, 5, 31), gen.bcr_mask(M, M, bh, bw, compression=c, dist=dist, seed=5, stream=32))
    W, mask = _SWEEP_CACHE[key]
    X = gen.normal_f32((M, N), 1.0, 5, 33)
    if bf16:
        X = gen.bf16_representable(X)
    return dict(W=W, mask=mask, X=X, bh=bh, bw=bw)


def parity_rows(W, mask, X, got_rows, pick, bf16, out_bf16=False):
    """Sampled output rows against the CPU oracle (outside every timed region), element by element."""
    from oracle import bcr_oracle as orc
    from workloads.tolerances import assert_close
    dt = orc.DTYPE_BF16 if bf16 else orc.DTYPE_F32
    want = orc.spmm(W[pick], mask[pick], X, dt)
    Wm = orc.masked_weight(W[pick], mask[pick], dt)
    scale = np.linalg.norm(Wm, axis=1)[:, None] * np.linalg.norm(X.astype(np.float64), axis=0)[None, :]
    assert_close(got_rows, want, scale, bf16_in=bf16, out_bf16=out_bf16, what="sampled rows")


def parity_conv(L, x_np, got, bf16, out_bf16, rows):
    """Output channels `rows` of a 3x3 / stride 1 / pad 1 convolution with bias and ReLU against the CPU oracle;
    x_np: the images (NCHW, the values the GPU read), got: the GPU's output [images, len(rows), H, W]."""
    import torch
    from oracle import bcr_oracle as orc
    from workloads.tolerances import assert_close
    dt = orc.DTYPE_BF16 if bf16 else orc.DTYPE_F32
    W, mask, bias = L["W"][rows], L["mask"][rows], L["bias"][rows]
    want = orc.conv2d(W, mask, x_np, bias, ksize=3, stride=1, pad=1, relu=True, dtype=dt)
    Wm = orc.masked_weight(W, mask, dt)
    xx = torch.from_numpy(np.asarray(x_np, np.float64) ** 2)
    ones = torch.ones(1, xx.shape[1], 3, 3, dtype=torch.float64)
    col = torch.sqrt(torch.nn.functional.conv2d(xx, ones, padding=1)).numpy()  # norm of each im2col column
    scale = np.linalg.norm(Wm, axis=1)[None, :, None, None] * col
    assert_close(got, want, scale, bf16_in=bf16, out_bf16=out_bf16, bias_abs=np.abs(bias.astype(np.float64))[None, :, None, None],
                 what="sampled channels")


def min_index_bytes(info):
    """The smallest index a BCR matrix needs: one row bitmask and one column bitmask per non-empty block."""
    return info.nonempty_blocks * (info.bh + info.bw) / 8.0


L2_BYTES = 126e6
MAX_ROTATION = 12


def rotation_sets(working_set_bytes):
    """Number of operand sets a workload rotates through so that a set has left L2 (126 MB) before it is used again:
    the sets touched in between must add up to well over the L2 size.  1 = too many would be needed (small working
    set): such a workload is timed one launch at a time with an L2 flush before each."""
    need = int(math.ceil(1.3 * L2_BYTES / max(working_set_bytes, 1.0))) + 1
    return need if need <= MAX_ROTATION else 1


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                    bf16_tflops_burst=float(d["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1400.0, bf16_tflops_burst=1590.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.gpu)], stdout=fd, stderr=subprocess.DEVNULL)
            os.close(fd)
        except Exception:
            self.proc = None

    def stop(self):
        out = dict(sm_mhz=None, sm_max_mhz=None, reasons=[], samples=0)
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        try:
            rows = [l.strip().split(", ") for l in open(self.path) if l.strip()]
            os.unlink(self.path)
            sm = [float(r[1]) for r in rows]
            names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
            reasons = sorted({n for r in rows for n, v in zip(names, r[5:9]) if v.strip().lower() == "active"})
            out = dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=float(rows[0][2]) if rows else None,
                       reasons=reasons, samples=len(rows))
        except Exception:
            pass
        return out


# ------------------------------------------------------------------------------------------------ workloads


class GruWorkload:
    name = "gru_2x1024_in153_T200_bcr8x32_c10_fp32"
    dtype = "f32"

    def __init__(self, sample_T=200):
        from workloads import generators as gen
        self.m = gen.gru_model()
        self.T, self.H = self.m["T"], self.m["hidden"]
        self.nnz = sum(int(l["mask_ih"].sum()) + int(l["mask_hh"].sum()) for l in self.m["layers"])
        self.flops = 2.0 * self.nnz * self.T
        self.sample_T = sample_T

    def setup(self, B, torch):
        m = self.m
        self.B, self.torch = B, torch
        self.hi = [B.grim_bcr_pack(l["W_ih"], l["mask_ih"], m["bh"], m["bw"], B.GRIM_F32, B.GRIM_PACK_REORDER) for l in m["layers"]]
        self.hh = [B.grim_bcr_pack(l["W_hh"], l["mask_hh"], m["bh"], m["bw"], B.GRIM_F32, B.GRIM_PACK_REORDER) for l in m["layers"]]
        self.g = B.grim_gru_create(self.hi, self.hh, [l["b_ih"] for l in m["layers"]], [l["b_hh"] for l in m["layers"]], self.T)
        self.x_host = torch.from_numpy(m["x"]).pin_memory()
        self.y_host = torch.empty(self.T, self.H).pin_memory()
        self.x = self.x_host.cuda()
        self.y = torch.empty(self.T, self.H, device="cuda")
        B.grim_gru_profile(self.g, True)
        # Bytes the pass has to move once: every layer's packed W_ih and W_hh (values + index words), the input, the
        # hoisted pre-activations written and read back, the inter-layer and output sequences.  (W_hh stays on chip
        # for the whole sequence, so it is NOT counted once per time step; the figure that does count it per step is
        # reported beside this one as notional.)
        self.kernel_bytes, self.min_bytes, self.notional_bytes = 0.0, 0.0, 0.0
        for hi, hh in zip(self.hi, self.hh):
            ii, ih = B.grim_bcr_info(hi), B.grim_bcr_info(hh)
            acts = ii.K * self.T * 4 + 2 * self.T * 3 * self.H * 4 + self.T * self.H * 4
            self.kernel_bytes += ii.value_bytes + ii.index_bytes_spmm + ih.value_bytes + ih.index_bytes_gemv + acts
            self.min_bytes += ii.value_bytes + min_index_bytes(ii) + ih.value_bytes + min_index_bytes(ih) + acts
            self.notional_bytes += self.T * (ih.value_bytes + ih.index_bytes_gemv + 3 * self.H * 4 + 2 * self.H * 4)
        self.h2d = self.x_host.numel() * 4
        self.d2h = self.y_host.numel() * 4
        self.kernel = "gru_cluster_reg_kernel"
        self.peak_kind = "alu"
        self.force_bound = "hbm"  # far from any throughput roof: a chain of T dependent steps (latency-bound)

    def step(self):
        self.B.grim_gru_seq(self.g, self.x, self.y)

    def step_e2e(self):
        xd = self.x_host.cuda(non_blocking=True)
        self.B.grim_gru_seq(self.g, xd, self.y)
        self.y_host.copy_(self.y, non_blocking=True)

    def kernel_ms(self):
        return self.B.grim_gru_profile_read(self.g)[1]

    def check(self):
        """Status word, then the whole output sequence of the last pass against the oracle."""
        from oracle import bcr_oracle as orc
        from workloads.tolerances import F32_TOL, rel_fro
        self.torch.cuda.synchronize()
        assert self.B.grim_gru_status(self.g) == self.B.GRIM_OK, "a bounded device wait gave up"
        want, _ = orc.gru_seq(self.m["layers"], self.m["x"])
        got = self.y.cpu().numpy()
        assert np.all(np.isfinite(got)) and rel_fro(got, want) <= F32_TOL, rel_fro(got, want)

    def close(self):
        self.B.grim_gru_destroy(self.g)
        for h in self.hi + self.hh:
            self.B.grim_bcr_destroy(h)

    def oracle_sample(self):
        from oracle import bcr_oracle as orc
        Ts = self.sample_T
        t0 = time.perf_counter()
        orc.gru_seq(self.m["layers"], self.m["x"][:Ts])
        dt = time.perf_counter() - t0
        return 2.0 * self.nnz * Ts / dt / 1e9, f"first {Ts} of {self.T} time steps, both layers, dense fp64 NumPy mat-vec"


class SpmmWorkload:
    """One point of the SpMM sweep (square W).  N = 1 runs the matrix-vector kernel."""

    def __init__(self, M=8192, N=1, c=8.0, bh=8, bw=32, dist="uniform", bf16=False, inputs=None, name=None):
        self.M, self.N, self.bf16 = M, N, bf16
        self.s = inputs if inputs is not None else sweep_inputs(M, N, c, bh, bw, dist, bf16)
        self.bh, self.bw = bh, bw
        self.name = name or f"spmm_M{M}_K{M}_N{N}_c{c:g}_{bh}x{bw}_{dist}_{'bf16' if bf16 else 'fp32'}"
        self.dtype = "bf16" if bf16 else "f32"
        self.nnz = int(self.s["mask"].sum())
        self.flops = 2.0 * self.nnz * N
        self.dense_elems = int(self.s["mask"].size)

    def setup(self, B, torch):
        self.B, self.torch = B, torch
        s = self.s
        dt = B.GRIM_BF16 if self.bf16 else B.GRIM_F32
        # one regime's device layouts where only that regime's kernels can take the request; 8 <= N <= 16 is served by
        # kernels of both regimes (the tile search decides), so those handles keep every layout
        self.pack_flags = B.GRIM_PACK_REORDER | (B.GRIM_PACK_NARROW_ONLY if self.N < 8 else
                                                 (B.GRIM_PACK_WIDE_ONLY if self.N > 16 else 0))
        self.h = B.grim_bcr_pack(s["W"], s["mask"], self.bh, self.bw, dt, self.pack_flags)
        tdt = torch.bfloat16 if self.bf16 else torch.float32
        self.x_host = torch.from_numpy(s["X"]).to(tdt).pin_memory()
        self.x = self.x_host.cuda()
        self.y = torch.empty(self.M, self.N, device="cuda")
        self.y_host = torch.empty(self.M, self.N).pin_memory()
        i = B.grim_bcr_info(self.h)
        esz = 2 if self.bf16 else 4
        idx = i.index_bytes_gemv if self.N <= 16 else i.index_bytes_spmm
        self.kernel_bytes = float(i.value_bytes + idx + i.k_used * self.N * esz + self.M * self.N * 4)
        self.min_bytes = float(i.value_bytes + min_index_bytes(i) + i.k_used * self.N * esz + self.M * self.N * 4)
        self.h2d = self.x_host.numel() * esz
        self.d2h = self.y_host.numel() * 4
        tc = self.bf16 and self.N >= 128 and self.bh in (4, 8, 16) and self.bw in (16, 32, 64)
        self.kernel = "bcr_stream_kernel" if self.N <= 16 else ("bcr_tc_kernel" if tc else "bcr_ffma_kernel")
        self.peak_kind = "tensor" if tc else "alu"
        if tc:
            self.kernel_bytes = float(i.value_bytes + i.index_bytes_tc + i.k_used * self.N * esz + self.M * self.N * 4)
        self._ev = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
        # operand sets the timed steps rotate through (own copy of the packed matrix, of X and of Y each)
        self.sets = [(self.h, self.x, self.y)]
        for _ in range(rotation_sets(self.kernel_bytes) - 1):
            h = B.grim_bcr_pack(s["W"], s["mask"], self.bh, self.bw, dt, self.pack_flags)
            self.sets.append((h, self.x.clone(), torch.empty_like(self.y)))
        self.rotating = len(self.sets) > 1
        self.per_step_events = True
        self._i = 0
        # tile-shape search (Section 4.5): every handle times the candidate kernels / tiles for this request once and
        # keeps the answer; the plain multiply below then uses it
        self.tuned = None
        for h, x, y in self.sets:
            if self.bf16 and self.N >= 8:
                B.grim_bcr_reserve(h, self.N)  # workspace of the split tensor-core multiply (used when the grid is small)
            # operands that are streamed from HBM every step (the rotating sets) are tuned with a cold L2 as well
            self.tuned = B.grim_bcr_tune(h, x, y, reps=-5 if self.rotating else 5)
        torch.cuda.synchronize()
        names = {1: "bcr_ffma_kernel", 2: "bcr_tc_kernel", 4: "bcr_spmm_kernel", 5: "bcr_tc2_kernel",
                 3: "bcr_skinny_kernel" if self.tuned["tile_n"] == 1 else "bcr_stream_kernel"}
        self.kernel = names.get(self.tuned["path"], self.kernel)
        self.peak_kind = "tensor" if self.tuned["path"] in (2, 5) else "alu"
        if self.peak_kind == "tensor":
            self.kernel_bytes = float(i.value_bytes + i.index_bytes_tc + i.k_used * self.N * esz + self.M * self.N * 4)

    def step(self):
        h, x, y = self.sets[self._i % len(self.sets)]
        self._i += 1
        if self.per_step_events:
            self._ev[0].record()
        self.B.grim_bcr_spmm(h, x, y)
        if self.per_step_events:
            self._ev[1].record()

    def step_e2e(self):
        xd = self.x_host.cuda(non_blocking=True)
        self.B.grim_bcr_spmm(self.h, xd, self.y)
        self.y_host.copy_(self.y, non_blocking=True)

    def e2e_pipelined(self, steps):
        """End to end as a serving loop would run it: every step copies its X from pinned host memory, multiplies and
        copies its Y back to pinned host memory, on three streams (copy in, multiply, copy out) over three sets of
        device buffers, so that the copies of neighbouring steps overlap the multiply.  Returns the device time of all
        steps in ms (one event pair around the whole loop on the current stream, which the three streams fork from
        and join)."""
        torch, B = self.torch, self.B
        nb = 3
        cur = torch.cuda.current_stream()
        s_in, s_k, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
        xd = [torch.empty_like(self.x) for _ in range(nb)]
        yd = [torch.empty_like(self.y) for _ in range(nb)]
        yh = [torch.empty(self.M, self.N).pin_memory() for _ in range(nb)]
        ev = lambda: torch.cuda.Event()
        in_done, k_done, out_done = [ev() for _ in range(nb)], [ev() for _ in range(nb)], [ev() for _ in range(nb)]
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        t0.record(cur)
        for st in (s_in, s_k, s_out):
            st.wait_event(t0)
        for k in range(steps):
            b = k % nb
            with torch.cuda.stream(s_in):
                if k >= nb:
                    s_in.wait_event(k_done[b])      # the multiply that read this X buffer is done
                xd[b].copy_(self.x_host, non_blocking=True)
                in_done[b].record(s_in)
            with torch.cuda.stream(s_k):
                s_k.wait_event(in_done[b])
                if k >= nb:
                    s_k.wait_event(out_done[b])     # the copy that read this Y buffer is done
                B.grim_bcr_spmm(self.h, xd[b], yd[b], stream=s_k)
                k_done[b].record(s_k)
            with torch.cuda.stream(s_out):
                s_out.wait_event(k_done[b])
                yh[b].copy_(yd[b], non_blocking=True)
                out_done[b].record(s_out)
        for st in (s_in, s_k, s_out):
            cur.wait_stream(st)
        t1.record(cur)
        t1.synchronize()
        self.y_host.copy_(yh[(steps - 1) % nb])
        # what came back to the host is the product (outside the timed region): every buffer's sampled rows
        pick = np.sort(np.random.default_rng(3).choice(self.M, size=min(16, self.M), replace=False))
        for b in range(min(nb, steps)):
            got = yh[b].numpy()
            assert np.all(np.isfinite(got))
            parity_rows(self.s["W"], self.s["mask"], self.s["X"], got[pick], pick, self.bf16)
        return t0.elapsed_time(t1)

    def kernel_ms(self):
        self._ev[1].synchronize()
        return self._ev[0].elapsed_time(self._ev[1])

    def check(self):
        """Status words of every handle used, then sampled output rows of the last launch against the oracle."""
        torch = self.torch
        torch.cuda.synchronize()
        for h, _, _ in self.sets:
            assert self.B.grim_bcr_status(h) == self.B.GRIM_OK, "a bounded device wait gave up"
        _, x, y = self.sets[(self._i - 1) % len(self.sets)] if self._i else self.sets[0]
        pick = np.sort(np.random.default_rng(1).choice(self.M, size=min(64, self.M), replace=False))
        got = y.cpu().numpy()
        assert np.all(np.isfinite(got))
        parity_rows(self.s["W"], self.s["mask"], self.s["X"], got[pick], pick, self.bf16)

    def close(self):
        for h, _, _ in self.sets:
            self.B.grim_bcr_destroy(h)
        self.sets = []

    def oracle_sample(self, rows=None, cols=256):
        """Times the oracle on the first `rows` rows of W (all by default) and the first `cols` columns of X."""
        from oracle import bcr_oracle as orc
        n = min(self.N, cols)
        r = self.M if rows is None else min(self.M, rows)
        W, mask = self.s["W"][:r], self.s["mask"][:r]
        t0 = time.perf_counter()
        orc.spmm(W, mask, self.s["X"][:, :n], 1 if self.bf16 else 0)
        dt = time.perf_counter() - t0
        return 2.0 * float(mask.sum()) * n / dt / 1e9, \
            f"first {r} of {self.M} rows of W, first {n} of {self.N} columns of X, masked dense fp64 NumPy matmul"


class ConvWorkload:
    def __init__(self, batch=32, bf16=False):
        from workloads import generators as gen
        self.L = gen.conv_layer(batch, 512, 512, 28, bf16=bf16)
        self.batch, self.bf16 = batch, bf16
        self.name = f"conv3x3_512to512_28x28_b{batch}_bcr16x64_c8_{'bf16' if bf16 else 'fp32'}"
        self.dtype = "bf16" if bf16 else "f32"
        self.nnz = int(self.L["mask"].sum())
        self.flops = 2.0 * self.nnz * batch * 28 * 28
        self.dense_elems = int(self.L["mask"].size)

    def setup(self, B, torch):
        self.B, self.torch = B, torch
        L = self.L
        dt = B.GRIM_BF16 if self.bf16 else B.GRIM_F32
        tdt = torch.bfloat16 if self.bf16 else torch.float32
        self.h = B.grim_bcr_pack(L["W"], L["mask"], 16, 64, dt, B.GRIM_PACK_REORDER | B.GRIM_PACK_WIDE_ONLY)
        if self.bf16:
            B.grim_bcr_reserve(self.h, self.batch * 28 * 28)
        self.x_host = torch.from_numpy(L["x"]).to(tdt).pin_memory()
        self.x = self.x_host.cuda()
        self.bias = torch.from_numpy(L["bias"]).cuda()
        self.y = torch.empty(self.batch, 512, 28, 28, device="cuda", dtype=tdt)
        self.y_host = torch.empty(self.batch, 512, 28, 28, dtype=tdt).pin_memory()
        i = B.grim_bcr_info(self.h)
        esz = 2 if self.bf16 else 4
        idx = i.index_bytes_tc if self.bf16 else i.index_bytes_spmm
        self.kernel_bytes = float(i.value_bytes + idx + self.x.numel() * esz + self.y.numel() * esz)
        self.min_bytes = float(i.value_bytes + min_index_bytes(i) + self.x.numel() * esz + self.y.numel() * esz)
        self.h2d = self.x_host.numel() * esz
        self.d2h = self.y_host.numel() * esz
        self.kernel = "bcr_tc_kernel (implicit im2col)" if self.bf16 else "bcr_ffma_kernel (implicit im2col)"
        self.peak_kind = "tensor" if self.bf16 else "alu"
        self._ev = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
        self.sets = [(self.h, self.x, self.y)]
        for _ in range(rotation_sets(self.kernel_bytes) - 1):
            h = B.grim_bcr_pack(L["W"], L["mask"], 16, 64, dt, B.GRIM_PACK_REORDER | B.GRIM_PACK_WIDE_ONLY)
            if self.bf16:
                B.grim_bcr_reserve(h, self.batch * 28 * 28)
            self.sets.append((h, self.x.clone(), torch.empty_like(self.y)))
        self.rotating = len(self.sets) > 1
        self.per_step_events = True
        self._i = 0

    def step(self):
        h, x, y = self.sets[self._i % len(self.sets)]
        self._i += 1
        if self.per_step_events:
            self._ev[0].record()
        self.B.grim_bcr_conv2d(h, x, y, 3, 1, 1, bias=self.bias, relu=True)
        if self.per_step_events:
            self._ev[1].record()

    def step_e2e(self):
        xd = self.x_host.cuda(non_blocking=True)
        self.B.grim_bcr_conv2d(self.h, xd, self.y, 3, 1, 1, bias=self.bias, relu=True)
        self.y_host.copy_(self.y, non_blocking=True)

    def kernel_ms(self):
        self._ev[1].synchronize()
        return self._ev[0].elapsed_time(self._ev[1])

    def check(self):
        """Status words, then the first and the last image of the last launch on 64 sampled output channels."""
        self.torch.cuda.synchronize()
        for h, _, _ in self.sets:
            assert self.B.grim_bcr_status(h) == self.B.GRIM_OK, "a bounded device wait gave up"
        _, x, y = self.sets[(self._i - 1) % len(self.sets)] if self._i else self.sets[0]
        assert bool(self.torch.isfinite(y.float()).all())
        imgs = sorted({0, self.batch - 1})
        rows = np.sort(np.random.default_rng(2).choice(512, size=64, replace=False))
        got = y[imgs].float().cpu().numpy()[:, rows]
        parity_conv(self.L, x[imgs].float().cpu().numpy(), got, self.bf16, self.bf16, rows)

    def close(self):
        for h, _, _ in self.sets:
            self.B.grim_bcr_destroy(h)
        self.sets = []

    def oracle_sample(self):
        from oracle import bcr_oracle as orc
        L = self.L
        t0 = time.perf_counter()
        orc.conv2d(L["W"], L["mask"], L["x"][:1], L["bias"], ksize=3, stride=1, pad=1, relu=True, dtype=1 if self.bf16 else 0)
        dt = time.perf_counter() - t0
        return 2.0 * self.nnz * 28 * 28 / dt / 1e9, f"1 of {self.batch} images, direct fp64 NumPy convolution with the masked dense weight"

class VggWorkload:
    """The 13 convolution layers of VGG-16 (3x3, stride 1, pad 1, ReLU; 2x2 max-pool after layers 2, 4, 7, 10, 13),
    every layer BCR-pruned 8x with 8x32 blocks, bf16 activations and weights, fp32 accumulation."""

    def __init__(self, batch=1, image=224):
        from workloads import generators as gen
        self.net = gen.vgg16_stack(batch, image=image)
        self.batch, self.image = batch, image
        self.name = f"vgg16_convstack_{image}x{image}_b{batch}_bcr8x32_c8_bf16"
        self.dtype = "bf16"
        self.nnz = sum(int(L["mask"].sum()) for L in self.net["layers"])
        self.flops = sum(2.0 * int(L["mask"].sum()) * batch * L["hw"] * L["hw"] for L in self.net["layers"])
        self.peak_kind = "tensor"
        self.dense_elems = sum(int(L["mask"].size) for L in self.net["layers"])
        self.kernel = "bcr_tc_kernel (implicit im2col, per layer)"

    def setup(self, B, torch):
        self.B, self.torch = B, torch
        net = self.net
        self.h, self.bias, self.bufs, self.info = [], [], [], []
        self.x_host = torch.from_numpy(net["x"]).to(torch.bfloat16).pin_memory()
        self.x = self.x_host.cuda()
        cur_hw = self.image
        for L in net["layers"]:
            self.h.append(B.grim_bcr_pack(L["W"], L["mask"], net["bh"], net["bw"], B.GRIM_BF16,
                                          B.GRIM_PACK_REORDER | B.GRIM_PACK_WIDE_ONLY))
            B.grim_bcr_reserve(self.h[-1], self.batch * cur_hw * cur_hw)
            self.bias.append(torch.from_numpy(L["bias"]).cuda())
            out = torch.empty(self.batch, L["cout"], cur_hw, cur_hw, device="cuda", dtype=torch.bfloat16)
            pooled = None
            if L["pool"]:
                cur_hw //= 2
                pooled = torch.empty(self.batch, L["cout"], cur_hw, cur_hw, device="cuda", dtype=torch.bfloat16)
            self.bufs.append((out, pooled))
            self.info.append(B.grim_bcr_info(self.h[-1]))
        self.y_host = torch.empty_like(self.bufs[-1][1], device="cpu").pin_memory()
        self.ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in net["layers"]]
        self.layer_bytes, self.layer_flops = [], []
        for L, i in zip(net["layers"], self.info):
            npx = self.batch * L["hw"] * L["hw"]
            self.layer_bytes.append(float(i.value_bytes + i.index_bytes_tc + 2 * L["cin"] * npx + 2 * L["cout"] * npx))
            self.layer_flops.append(2.0 * i.nnz * npx)
        self.kernel_bytes = sum(self.layer_bytes)
        self.min_bytes = sum(float(i.value_bytes + min_index_bytes(i)) + 2.0 * (L["cin"] + L["cout"]) * self.batch * L["hw"] ** 2
                             for L, i in zip(net["layers"], self.info))
        self.h2d = self.x_host.numel() * 2
        self.d2h = self.y_host.numel() * 2
        self.layer_ms = [[] for _ in net["layers"]]

    def _run(self, x):
        B = self.B
        cur = x
        for li, L in enumerate(self.net["layers"]):
            out, pooled = self.bufs[li]
            self.ev[li][0].record()
            B.grim_bcr_conv2d(self.h[li], cur, out, 3, 1, 1, bias=self.bias[li], relu=True)
            self.ev[li][1].record()
            if pooled is not None:
                B.grim_maxpool2x2(out, pooled)
                cur = pooled
            else:
                cur = out
        return cur

    def step(self):
        self._run(self.x)

    def step_e2e(self):
        xd = self.x_host.cuda(non_blocking=True)
        self.y_host.copy_(self._run(xd), non_blocking=True)

    def kernel_ms(self):
        self.ev[-1][1].synchronize()
        ms = [a.elapsed_time(b) for a, b in self.ev]
        for li, m in enumerate(ms):
            self.layer_ms[li].append(m)
        return sum(ms)

    def check(self):
        """Every layer of the last pass, on the last image and 32 sampled output channels, with the oracle fed the
        values the GPU read as that layer's input."""
        self.torch.cuda.synchronize()
        for h in self.h:
            assert self.B.grim_bcr_status(h) == self.B.GRIM_OK, "a bounded device wait gave up"
        cur = self.x
        img = [self.batch - 1]
        for li, L in enumerate(self.net["layers"]):
            out, pooled = self.bufs[li]
            rows = np.sort(np.random.default_rng(3 + li).choice(L["cout"], size=min(32, L["cout"]), replace=False))
            assert bool(self.torch.isfinite(out[img].float()).all()), f"layer {li + 1}"
            parity_conv(L, cur[img].float().cpu().numpy(), out[img].float().cpu().numpy()[:, rows], True, True, rows)
            cur = pooled if pooled is not None else out

    def close(self):
        for h in self.h:
            self.B.grim_bcr_destroy(h)
        self.h = []

    def extra(self, peaks):
        """Per-layer time and fraction of the binding roofline (HBM bytes vs the measured dense bf16 tensor rate)."""
        import statistics
        alu_peak = peaks["bf16_tflops_burst"] * 1e12
        rows = []
        for li, L in enumerate(self.net["layers"]):
            ms = statistics.mean(self.layer_ms[li]) if self.layer_ms[li] else None
            t_hbm = self.layer_bytes[li] / (peaks["hbm_gbs"] * 1e9)
            t_alu = self.layer_flops[li] / alu_peak
            rows.append(dict(layer=li + 1, cout=L["cout"], cin=L["cin"], hw=L["hw"], ms=ms,
                             bound="hbm" if t_hbm >= t_alu else "tensor",
                             frac=(max(t_hbm, t_alu) / (ms * 1e-3)) if ms else None))
        return dict(layers=rows)

    def oracle_sample(self):
        from oracle import bcr_oracle as orc
        L = self.net["layers"][7]  # conv 8 (256 -> 512 at 1/8 resolution): a mid-sized layer
        hw = L["hw"]
        x = np.maximum(np.random.default_rng(0).standard_normal((1, L["cin"], hw, hw)).astype(np.float32), 0)
        t0 = time.perf_counter()
        orc.conv2d(L["W"], L["mask"], x, L["bias"], ksize=3, stride=1, pad=1, relu=True, dtype=1)
        dt = time.perf_counter() - t0
        return 2.0 * int(L["mask"].sum()) * hw * hw / dt / 1e9, \
            f"layer 8 of 13 on one image ({L['cin']}->{L['cout']} at {hw}x{hw}), direct fp64 NumPy convolution with the masked dense weight"


def make_workload(args):
    w = args.workload
    if w == "suite":  # the headline point of the sweep; the other configurations follow as records
        return SpmmWorkload(M=8192, N=1024, c=8.0, bh=8, bw=32, dist="uniform", bf16=False)
    if w == "gru":
        return GruWorkload()
    if w == "gemv":
        return SpmmWorkload(M=args.size, N=1, c=args.compression, bh=args.bh, bw=args.bw, dist=args.dist, bf16=args.bf16)
    if w == "spmm":
        return SpmmWorkload(M=args.size, N=args.ncols, c=args.compression, bh=args.bh, bw=args.bw, dist=args.dist, bf16=args.bf16)
    if w == "conv":
        return ConvWorkload(batch=args.batch, bf16=args.bf16)
    if w == "vgg":
        return VggWorkload(batch=args.batch if args.batch != 32 else 1, image=args.image)
    raise SystemExit(f"unknown workload {w}")


# ------------------------------------------------------------------------------------------------ arms


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = make_workload(args)
    if isinstance(wl, GruWorkload):
        wl.sample_T = 50
    kw = {}
    if isinstance(wl, SpmmWorkload):
        # size the per-step sample so that the whole run takes about two minutes: start small, time it once, grow the
        # number of rows (then of columns) in proportion
        budget = 120.0 / max(1, args.steps + args.warmup)
        kw = dict(rows=min(wl.M, 256), cols=min(wl.N, 64))
        t0 = time.perf_counter()
        wl.oracle_sample(**kw)
        scale = budget / max(time.perf_counter() - t0, 1e-3)
        rows = int(min(wl.M, max(64, kw["rows"] * scale)))
        cols = int(min(wl.N, max(kw["cols"], kw["cols"] * scale * kw["rows"] / rows)))
        kw = dict(rows=rows, cols=cols)
    for _ in range(args.warmup):
        wl.oracle_sample(**kw)
    vals, t0 = [], time.perf_counter()
    for _ in range(args.steps):
        v, what = wl.oracle_sample(**kw)
        vals.append(v)
    total = time.perf_counter() - t0
    # harmonic mean over steps = total work / total time
    value = len(vals) / sum(1.0 / v for v in vals)
    cores = len(os.sched_getaffinity(0))
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps, warmup=args.warmup,
                ms_per_step=1e3 * total / args.steps, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="f64", data="synthetic", impl="reference",
                config=dict(workload=wl.name, note="CPU oracle; each step is a bounded sample of the workload"),
                cpu_baseline=dict(value=value, unit=UNIT, cores=cores, kind="oracle", sample=what),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0), gpu_launches=0)
    print(json.dumps(line))


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks of the default process group (identity when there
    is none): a multi-GPU number is the slowest rank's."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def aggregate_value(flops_per_rank_step, steps, total_ms, world):
    """Whole-job throughput in GFLOP/s: every rank (replica) does the same work; time is the slowest rank's."""
    return world * flops_per_rank_step * steps / (total_ms * 1e-3) / 1e9


def run_ours(args):
    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    from paper_2108_11033_b200.build import build_library
    build_library()
    from paper_2108_11033_b200 import binding as B

    bench = Bench(B, torch)
    suite = args.workload == "suite"
    wl = make_workload(args)
    wl.setup(B, torch)
    warmup = max(args.warmup, 3)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(warmup):
        wl.step()
    barrier()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    B.grim_launch_count_reset()
    barrier()
    total_ms, k_ms = bench.time_steps(wl, args.steps)
    barrier()
    launches = B.grim_launch_count()
    try:
        wl.check()
        parity = "ok"
    except AssertionError as e:
        parity = ("FAIL: " + str(e))[:300]

    # end to end: host buffers, copies inside the timed region
    for _ in range(2):
        wl.step_e2e()
    barrier()
    e2e_pipelined = hasattr(wl, "e2e_pipelined")
    if e2e_pipelined:
        # copies of neighbouring steps overlap the multiply (three streams); every step's X comes from the host and
        # every step's Y goes back to it, so nothing is served from L2 and no flush is needed between steps
        e2e_ms = wl.e2e_pipelined(args.steps)
        barrier()
    else:
        ev2 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        for k in range(args.steps):
            bench.flush_l2()
            ev2[k][0].record()
            wl.step_e2e()
            ev2[k][1].record()
        barrier()
        e2e_ms = sum(a.elapsed_time(b) for a, b in ev2)

    # the other target configurations, one record each (rank 0 at N = 1 only: they are single-GPU measurements)
    configs = None
    if suite and rank == 0 and world == 1:
        configs = [record_of(bench, wl, "config 5: SpMM 8192^2, N = 1024, c = 8, fp32 (headline)", k_ms, parity)]
        only = set(args.only.split(",")) if args.only else None
        for i, (label, make) in enumerate(suite_workloads()):
            if only is not None and str(i) not in only:
                continue
            try:
                configs.append(measure_config(bench, label, make))
            except Exception as e:  # a record that cannot be measured is reported, not dropped
                configs.append(dict(config=label, parity="FAIL: " + repr(e)[:300]))
    clocks = sampler.stop() if rank == 0 else None

    total_ms, e2e_ms = max_over_ranks([total_ms, e2e_ms], device="cuda")

    if rank == 0:
        value = aggregate_value(wl.flops, args.steps, total_ms, world)
        e2e_value = aggregate_value(wl.flops, args.steps, e2e_ms, world)
        roof = bench.roofline(wl, k_ms)
        roof["parity"] = parity
        cpu_v, cpu_what = wl.oracle_sample()
        rotating = bool(getattr(wl, "rotating", False))
        line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=warmup,
                    ms_per_step=total_ms / args.steps, higher_is_better=True, scaling="weak", vs_baseline=None,
                    dtype=wl.dtype, data="synthetic",
                    config=dict(workload=wl.name, nnz=wl.nnz,
                                l2=(f"inputs larger than L2: the steps rotate through {len(wl.sets)} operand sets of "
                                    f"{wl.kernel_bytes / 1e6:.0f} MB, launches queued back to back" if rotating else
                                    "flushed between timed iterations (1 GiB write, then a 512 MiB read that leaves no dirty lines)"),
                                parallelism="replicas only" if world > 1 else "1 GPU"),
                    clocks=clocks,
                    e2e=dict(value=e2e_value, unit=UNIT, h2d_bytes_per_step=wl.h2d, d2h_bytes_per_step=wl.d2h,
                             ms_per_step=e2e_ms / args.steps,
                             how=("steps pipelined over three streams: host-to-device copy of X, multiply, device-to-host "
                                  "copy of Y, every step from and to pinned host buffers" if e2e_pipelined else
                                  "one step at a time: copy in, compute, copy out")),
                    gpu_launches=int(launches), roofline=roof,
                    cpu_baseline=dict(value=cpu_v, unit=UNIT, cores=len(os.sched_getaffinity(0)), kind="oracle",
                                      sample=cpu_what))
        if configs is not None:
            line["configs"] = configs
            line["ffma_peak_tflops_measured"] = bench.ffma_tflops
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


class Bench:
    """What every measurement needs: the binding, torch, the L2 flush, the peaks."""

    def __init__(self, B, torch):
        self.B, self.torch = B, torch
        # written before timed iterations: evicts the working set from L2 (126 MB) and keeps the GPU busy long enough for
        # the host to queue the step behind it, so that no host latency sits between the events
        self.flush = torch.empty(1 << 30, dtype=torch.uint8, device="cuda")
        self.peaks = measured_peaks()
        # fp32 FMA ceiling: measured with a register-only micro-kernel at run time (it follows the clock the GPU
        # sustains); the figure derived from unit counts and the maximum clock is kept beside it for context
        self.ffma_tflops = B.grim_measure_ffma_peak()
        self.ffma_derived = 148 * 128 * 2 * 1.965e9 / 1e12

    def flush_l2(self):
        # the write evicts the working set; the read of half the buffer behind it pushes the write's dirty lines out
        # to HBM, so that the timed step does not pay for writing them back when its own reads evict them
        self.flush.zero_()
        self.flush[: 1 << 29].view(self.torch.int64).sum()

    def time_steps(self, wl, steps):
        """Times exactly `steps` steps of a workload; returns (total ms over the steps, mean ms of the dominant kernel).
        Workloads whose operands exceed L2 rotate through operand sets and are queued back to back behind a few
        flushes (the time between the two events is that of the launches alone); the others are timed one step at a
        time with an L2 flush before each."""
        torch = self.torch
        if bool(getattr(wl, "rotating", False)):
            wl.per_step_events = False
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            for _ in range(2 + min(steps, 400) // 8):
                self.flush_l2()
            e0.record()
            for _ in range(steps):
                wl.step()
            e1.record()
            e1.synchronize()
            wl.per_step_events = True
            total = e0.elapsed_time(e1)
            return total, total / steps
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        kernel_ms = []
        for k in range(steps):
            self.flush_l2()
            ev[k][0].record()
            wl.step()
            ev[k][1].record()
            kernel_ms.append(wl.kernel_ms())
        torch.cuda.synchronize()
        return sum(a.elapsed_time(b) for a, b in ev), statistics.mean(kernel_ms)

    def roofline(self, wl, k_ms):
        """Binding bound of the dominant kernel: the slower of (algorithmic bytes at the measured HBM bandwidth) and
        (effective flops 2*nnz*N at the peak of the unit that does the arithmetic: the measured fp32 FMA rate, or the
        measured dense bf16 tensor rate for the tcgen05 kernel)."""
        peaks = self.peaks
        flop_peak = peaks["bf16_tflops_burst"] if wl.peak_kind == "tensor" else self.ffma_tflops
        t_hbm = wl.kernel_bytes / (peaks["hbm_gbs"] * 1e9)
        t_min = getattr(wl, "min_bytes", wl.kernel_bytes) / (peaks["hbm_gbs"] * 1e9)
        t_flop = wl.flops / (flop_peak * 1e12)
        bound = getattr(wl, "force_bound", None) or ("hbm" if t_hbm >= t_flop else wl.peak_kind)
        t = k_ms * 1e-3
        if bound == "hbm":
            achieved = wl.kernel_bytes / t / 1e9
            roof = dict(bound="hbm", achieved=achieved, peak=peaks["hbm_gbs"], unit="GB/s", frac=achieved / peaks["hbm_gbs"],
                        frac_min_index=t_min / t, traffic=None, kernel=wl.kernel, kernel_ms=k_ms,
                        algorithmic_bytes=wl.kernel_bytes, min_index_bytes_total=getattr(wl, "min_bytes", None),
                        peak_source=peaks["source"] + " HBM copy bandwidth")
        else:
            achieved = wl.flops / t / 1e12
            roof = dict(bound=bound, achieved=achieved, peak=flop_peak, unit="TFLOP/s", frac=achieved / flop_peak, traffic=None,
                        kernel=wl.kernel, kernel_ms=k_ms,
                        peak_source=("measured dense bf16 (burst)" if bound == "tensor" else
                                     f"measured fp32 FMA micro-kernel at run time (derived from unit counts at the maximum "
                                     f"clock: {self.ffma_derived:.1f})"))
        roof["traffic"] = profile_traffic(wl.name)
        roof["t_hbm_us"] = t_hbm * 1e6
        roof["t_flop_us"] = t_flop * 1e6
        if hasattr(wl, "extra"):
            roof.update(wl.extra(peaks))
        return roof


def suite_workloads():
    """The five target configurations as (label, constructor) pairs, in an order that lets consecutive records share
    generated weights.  The headline point (8192^2, N = 1024, c = 8, fp32) is measured by the main timed region."""
    from workloads import generators as gen

    def config1():
        c = gen.config1_spmm()
        return SpmmWorkload(M=256, N=64, c=4.0, bh=16, bw=16, inputs=c, name="config1_spmm_M256_K256_N64_16x16_keep8x8_fp32")

    S = SpmmWorkload
    return [
        ("config 1: SpMM 256^2, N = 64, fp32", config1),
        ("config 2: GRU 2 x 1024, T = 200, fp32", GruWorkload),
        ("config 3: conv 512->512 28^2, batch 1, fp32", lambda: ConvWorkload(1, False)),
        ("config 3: conv 512->512 28^2, batch 1, bf16", lambda: ConvWorkload(1, True)),
        ("config 3: conv 512->512 28^2, batch 32, fp32", lambda: ConvWorkload(32, False)),
        ("config 3: conv 512->512 28^2, batch 32, bf16", lambda: ConvWorkload(32, True)),
        ("config 4: VGG-16 conv stack, batch 1, bf16", lambda: VggWorkload(1)),
        ("config 4: VGG-16 conv stack, batch 16, bf16", lambda: VggWorkload(16)),
        ("config 5: GEMV 4096^2, c = 4, fp32", lambda: S(4096, 1, 4.0)),
        ("config 5: GEMV 8192^2, c = 4, fp32", lambda: S(8192, 1, 4.0)),
        ("config 5: GEMV 8192^2, c = 4, bf16", lambda: S(8192, 1, 4.0, bf16=True)),
        ("config 5: SpMM 8192^2, N = 16, c = 4, fp32", lambda: S(8192, 16, 4.0)),
        ("config 5: SpMM 8192^2, N = 16, c = 4, bf16", lambda: S(8192, 16, 4.0, bf16=True)),
        ("config 5: SpMM 8192^2, N = 128, c = 8, fp32", lambda: S(8192, 128, 8.0)),
        ("config 5: SpMM 8192^2, N = 128, c = 8, bf16", lambda: S(8192, 128, 8.0, bf16=True)),
        ("config 5: SpMM 8192^2, N = 1024, c = 8, bf16", lambda: S(8192, 1024, 8.0, bf16=True)),
    ]


def record_of(bench, wl, label, ms, parity):
    """One entry of the `configs` array."""
    roof = bench.roofline(wl, ms)
    rec = dict(config=label, workload=wl.name, dtype=wl.dtype, nnz=wl.nnz, ms=ms, gflops=wl.flops / (ms * 1e-3) / 1e9,
               bound=roof["bound"], frac=roof["frac"], frac_min_index=roof.get("frac_min_index"), kernel=wl.kernel,
               t_hbm_us=roof["t_hbm_us"], t_flop_us=roof["t_flop_us"], parity=parity)
    if "layers" in roof:
        rec["layers"] = roof["layers"]
    if getattr(wl, "tuned", None):
        rec["tuned"] = dict(path=wl.tuned["path"], tile_n=wl.tuned["tile_n"])
    if isinstance(wl, GruWorkload):
        rec["bound"] = "latency (hbm figure: bytes moved once)"
        rec["us_per_time_step"] = ms * 1e3 / wl.T
        rec["notional_frac_if_W_hh_were_streamed_every_step"] = wl.notional_bytes / (bench.peaks["hbm_gbs"] * 1e9) / (ms * 1e-3)
    if wl.peak_kind == "tensor":
        # the tensor-core kernel multiplies zero-filled tiles: at best the dense rate divided by the compression
        rec["structural_ceiling_gflops"] = bench.peaks["bf16_tflops_burst"] * 1e3 * wl.nnz / getattr(wl, "dense_elems", wl.nnz)
    return rec


def measure_config(bench, label, make, min_s=0.5):
    """Sets a workload up, times it for at least `min_s` seconds (so that the clock sampler sees it), checks the last
    output against the oracle and the handles' status words, and releases it."""
    torch = bench.torch
    wl = make()
    wl.setup(bench.B, torch)
    for _ in range(3):
        wl.step()
    torch.cuda.synchronize()
    if bool(getattr(wl, "rotating", False)):
        _, est = bench.time_steps(wl, 20)
        n = int(min(20000, max(20, math.ceil(min_s * 1e3 / max(est, 1e-4)))))
        _, ms = bench.time_steps(wl, n)
    else:
        # one launch at a time behind an L2 flush; the flushes count towards the duration (the GPU is busy throughout)
        samples, t0 = [], time.perf_counter()
        while len(samples) < 20 or (time.perf_counter() - t0 < min_s and len(samples) < 2000):
            bench.flush_l2()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            wl.step()
            e1.record()
            e1.synchronize()
            # the stack and the GRU report the whole pass (their latency is the figure of merit); single kernels too
            samples.append(e0.elapsed_time(e1))
            if hasattr(wl, "layer_ms"):
                wl.kernel_ms()
        ms = statistics.median(samples)
    try:
        wl.check()
        parity = "ok"
    except AssertionError as e:
        parity = ("FAIL: " + str(e))[:300]
    rec = record_of(bench, wl, label, ms, parity)
    wl.close()
    del wl
    torch.cuda.empty_cache()
    return rec


def run_sweep(args):
    """The SpMM sweep: square W with M = K in {1024, 4096, 8192}, N in {1, 16, 128, 1024}, compression in {4, 8, 16},
    blocks in {4x16, 8x32, 16x64}, fp32 and bf16, kept-row counts uniform or Zipf(1.2), with and without reorder.
    Writes one JSON line per run to --out and prints a one-line summary.  (--sweep-sizes etc. restrict the grid.)"""
    import itertools
    import torch
    torch.cuda.set_device(0)
    from paper_2108_11033_b200.build import build_library
    build_library()
    from paper_2108_11033_b200 import binding as B
    from workloads import generators as gen

    peaks = measured_peaks()
    alu_peak = 148 * 128 * 2 * 1.965e9
    flush = torch.empty(1 << 30, dtype=torch.uint8, device="cuda")
    sizes = [int(v) for v in args.sweep_sizes.split(",")]
    ncols = [int(v) for v in args.sweep_ncols.split(",")]
    comps = [float(v) for v in args.sweep_compressions.split(",")]
    blocks = [tuple(int(t) for t in v.split("x")) for v in args.sweep_blocks.split(",")]
    out = open(args.out, "w")
    fracs, n_runs = [], 0
    t_start = time.perf_counter()
    for M, c, (bh, bw), dist_name in itertools.product(sizes, comps, blocks, ["uniform", "zipf"]):
        W = gen.dense_weight(M, M, 5, 31)
        mask = gen.bcr_mask(M, M, bh, bw, compression=c, dist=dist_name, seed=5, stream=32)
        nnz = int(mask.sum())
        Xf = gen.normal_f32((M, max(ncols)), 1.0, 5, 33)
        for bf16, reorder in itertools.product([False, True], [1, 0]):
            h = B.grim_bcr_pack(W, mask, bh, bw, B.GRIM_BF16 if bf16 else B.GRIM_F32, reorder)
            if bf16:
                B.grim_bcr_reserve(h, min(max(ncols), 256))  # workspace of the split tensor-core multiply (small grids)
            info = B.grim_bcr_info(h)
            esz = 2 if bf16 else 4
            for N in ncols:
                X = torch.from_numpy(np.ascontiguousarray(Xf[:, :N])).cuda()
                if bf16:
                    X = X.to(torch.bfloat16)
                Y = torch.empty(M, N, device="cuda")
                # the library's default routing: bf16 handles take the tensor-core tiles from N = 8, fp32 handles with
                # blocks of 8 rows or more the CUDA-core kernel from N = 8, everything narrower the lane-per-column kernel
                tc = bf16 and N >= 8
                cuda_core = not tc and (N > 16 or (N >= 8 and bh >= 8 and not bf16))
                idx = info.index_bytes_tc if tc else (info.index_bytes_spmm if cuda_core else info.index_bytes_gemv)
                nbytes = float(info.value_bytes + idx + info.k_used * N * esz + M * N * 4)
                flops = 2.0 * nnz * N
                for _ in range(3):
                    B.grim_bcr_spmm(h, X, Y)
                ms = []
                for _ in range(args.steps):
                    flush.zero_()
                    flush[: 1 << 29].view(torch.int64).sum()  # leaves no dirty lines for the timed launch to write back
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    B.grim_bcr_spmm(h, X, Y)
                    e1.record()
                    e1.synchronize()
                    ms.append(e0.elapsed_time(e1))
                status = B.grim_bcr_status(h)  # a bounded device-side wait that gave up leaves Y invalid: flag the record
                t = statistics.median(ms) * 1e-3
                t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9)
                t_flop = flops / (peaks["bf16_tflops_burst"] * 1e12 if tc else alu_peak)
                rec = dict(M=M, N=N, c=c, block=f"{bh}x{bw}", dist=dist_name, dtype="bf16" if bf16 else "f32", reorder=reorder,
                           nnz=nnz, ms=t * 1e3, gflops=flops / t / 1e9, bound="hbm" if t_hbm >= t_flop else ("tensor" if tc else "alu"),
                           frac=max(t_hbm, t_flop) / t, kernel="tc" if tc else ("ffma" if cuda_core else "stream"), status=int(status))
                out.write(json.dumps(rec) + "\n")
                fracs.append(rec["frac"])
                n_runs += 1
            B.grim_bcr_destroy(h)
        out.flush()
    out.close()
    print(json.dumps(dict(metric="SpMM sweep: fraction of the binding roofline", runs=n_runs, median_frac=statistics.median(fracs),
                          min_frac=min(fracs), max_frac=max(fracs), wall_s=time.perf_counter() - t_start, out=args.out)))


def run_bcrc_study(args):
    """Extra (non-weight) data of BCRC against CSR (Section 6.4 of the paper reports 30.1 % - 97.1 % less for its
    models) on seeded BCR masks: the library's BCRC export of a host-only handle, 32-bit entries on both sides.  Host
    only; prints one JSON line per matrix.  BCRC wins where rows share column lists, i.e. with few block columns per
    band (the paper prunes in 8 - 256 large blocks per matrix); with hundreds of small blocks per band no two rows
    keep the same columns and BCRC carries its fixed arrays on top of what CSR stores."""
    from paper_2108_11033_b200.build import build_library
    build_library()
    from paper_2108_11033_b200 import binding as B
    from workloads import generators as gen
    cases = [(1024, 64, 16, 64, 8.0), (1024, 128, 16, 64, 8.0), (1024, 256, 16, 64, 8.0), (1024, 512, 16, 64, 8.0),
             (1024, 128, 16, 64, 4.0), (1024, 128, 8, 32, 8.0), (1024, 1024, 16, 64, 8.0), (1024, 1024, 8, 32, 8.0),
             (1024, 1024, 4, 16, 8.0), (512, 4608, 16, 64, 8.0), (3072, 1024, 8, 32, 10.0)]
    for M, K, bh, bw, c in cases:
        mask = gen.bcr_mask(M, K, bh, bw, compression=c, dist="uniform", seed=5, stream=32)
        h = B.grim_bcr_pack(np.zeros((M, K), np.float32), mask, bh, bw, B.GRIM_F32, B.GRIM_PACK_HOST_ONLY)
        b = B.grim_bcr_export_bcrc(h)
        B.grim_bcr_destroy(h)
        nnz = int(mask.sum())
        bcrc = 4 * (len(b["reorder"]) + len(b["row_offset"]) + len(b["occurrence"]) + len(b["column_stride"]) + len(b["compact_column"]))
        csr = 4 * (M + 1 + nnz)
        print(json.dumps(dict(M=M, K=K, block=f"{bh}x{bw}", blocks_per_band=-(-K // bw), compression=c, nnz=nnz,
                              groups=len(b["occurrence"]) - 1, column_ids_bcrc=len(b["compact_column"]), column_ids_csr=nnz,
                              index_bytes_bcrc=bcrc, index_bytes_csr=csr, saving=1.0 - bcrc / csr,
                              total_saving=1.0 - (bcrc + 4 * nnz) / (csr + 4 * nnz))))


def run_reorder_study(args):
    """What the band schedule (Section 4.2, GRIM_PACK_REORDER) buys when the work per band is skewed: matrices whose
    bands get Zipf-distributed shares of the kept columns (generators.bcr_keep_lists, band_zipf), timed with the
    schedule off and on through the library's default routing.  One JSON line per point."""
    import torch
    torch.cuda.set_device(0)
    from paper_2108_11033_b200.build import build_library
    build_library()
    from paper_2108_11033_b200 import binding as B
    from workloads import generators as gen
    flush = torch.empty(1 << 30, dtype=torch.uint8, device="cuda")
    for M, skew, bf16 in [(4096, 1.0, False), (8192, 1.0, False), (8192, 0.5, False), (8192, 1.0, True)]:
        W = gen.dense_weight(M, M, 7, 41)
        mask = gen.bcr_mask(M, M, 8, 32, compression=8.0, dist="uniform", seed=7, stream=42, band_zipf=skew)
        band = mask.reshape(M // 8, 8, M).sum(axis=(1, 2))
        Xf = gen.normal_f32((M, 1024), 1.0, 7, 43)
        times = {}
        for reorder in (0, 1):
            h = B.grim_bcr_pack(W, mask, 8, 32, B.GRIM_BF16 if bf16 else B.GRIM_F32, reorder)
            if bf16:
                B.grim_bcr_reserve(h, 256)
            for N in (1, 16, 128, 1024):
                X = torch.from_numpy(np.ascontiguousarray(Xf[:, :N])).cuda()
                X = X.to(torch.bfloat16) if bf16 else X
                Y = torch.empty(M, N, device="cuda")
                for _ in range(3):
                    B.grim_bcr_spmm(h, X, Y)
                ms = []
                for _ in range(args.steps if args.steps < 50 else 7):
                    flush.zero_()
                    flush[: 1 << 29].view(torch.int64).sum()
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    B.grim_bcr_spmm(h, X, Y)
                    e1.record()
                    e1.synchronize()
                    ms.append(e0.elapsed_time(e1))
                assert B.grim_bcr_status(h) == 0
                times[(reorder, N)] = statistics.median(ms)
            B.grim_bcr_destroy(h)
        for N in (1, 16, 128, 1024):
            print(json.dumps(dict(M=M, N=N, dtype="bf16" if bf16 else "f32", band_zipf=skew, nnz=int(mask.sum()),
                                  heaviest_band_over_mean=float(band.max() / band.mean()),
                                  ms_schedule_off=times[(0, N)], ms_schedule_on=times[(1, N)],
                                  off_over_on=times[(0, N)] / times[(1, N)])), flush=True)


def run_block_sweep(args):
    """Time against number of blocks for one 1024 x 1024 matrix at 10x (the experiment of Section 5.1, left panel of its
    figure) with the block shapes the packer takes, and the block size the search of that section then picks."""
    import torch
    torch.cuda.set_device(0)
    from paper_2108_11033_b200.build import build_library
    build_library()
    from paper_2108_11033_b200 import blocksize as bs
    sizes = [(1, 1), (1, 4), (2, 8), (4, 16), (8, 32), (16, 64)]
    for N in (1, 64, 1024):
        rows = []
        for size in sizes:
            layer = bs.synthesize(1024, 1024, 10.0, size)
            rows.append(dict(block=f"{size[0]}x{size[1]}", blocks=(1024 // size[0]) * (1024 // size[1]),
                             nnz=int(layer["mask"].sum()), ms=bs.run_layer(layer, N)))
        pick, ms, trace = bs.find_opt_blk((1024, 1024), 10.0, sizes[1:], N=N, threshold=1.05)
        print(json.dumps(dict(experiment="time vs number of blocks, 1024 x 1024, 10x, fp32", N=N, points=rows,
                              find_opt_blk=dict(threshold=1.05, picked=pick, ms=ms, timed=[[list(t[0]), t[1]] for t in trace]))))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="suite", choices=["suite", "gru", "gemv", "spmm", "conv", "vgg"])
    ap.add_argument("--only", default="", help="suite: comma-separated indices of the extra records to measure (default: all)")
    ap.add_argument("--image", type=int, default=224)
    ap.add_argument("--size", type=int, default=8192)
    ap.add_argument("--ncols", type=int, default=128)
    ap.add_argument("--compression", type=float, default=8.0)
    ap.add_argument("--bh", type=int, default=8)
    ap.add_argument("--bw", type=int, default=32)
    ap.add_argument("--dist", default="uniform", choices=["uniform", "zipf"])
    ap.add_argument("--bf16", action="store_true")
    ap.add_argument("--batch", type=int, default=32)
    ap.add_argument("--sweep", action="store_true", help="run the SpMM sweep instead of one workload")
    ap.add_argument("--sweep-sizes", default="1024,4096,8192")
    ap.add_argument("--sweep-ncols", default="1,16,128,1024")
    ap.add_argument("--sweep-compressions", default="4,8,16")
    ap.add_argument("--sweep-blocks", default="4x16,8x32,16x64")
    ap.add_argument("--out", default="sweep.jsonl")
    ap.add_argument("--bcrc-study", action="store_true", help="host only: index bytes of the BCRC export against CSR")
    ap.add_argument("--block-sweep", action="store_true", help="time vs number of blocks at 1024 x 1024, 10x, and the block-size search")
    ap.add_argument("--reorder-study", action="store_true", help="band schedule off / on for matrices with skewed work per band")
    args = ap.parse_args()
    if args.reorder_study:
        run_reorder_study(args)
        return
    if args.block_sweep:
        run_block_sweep(args)
        return
    if args.bcrc_study:
        run_bcrc_study(args)
        return
    if args.sweep:
        run_sweep(args)
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
