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

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum, bytes) of the dominant kernel per step, from one ncu
# capture of the same command (summaries under profiles/); None where the kernel has changed since or was not captured.
TRAFFIC = {
    "gru_2x1024_in153_T200_bcr8x32_c10_fp32": 6 * 3.519e6,  # six launches (2 layers x 3 chunks) of 3.5 MB each
    "spmm_M4096_K4096_N1024_c8_8x32_uniform_fp32": 27.68e6,
    "spmm_M8192_K8192_N1_c4_8x32_uniform_fp32": 85.27e6,
    "spmm_M8192_K8192_N1024_c8_8x32_uniform_bf16": 47.60e6,
}
UNIT = "GFLOP/s"


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
        # algorithmic bytes of the recurrent kernel (dominant): per step the kept values and their index
        # words of W_hh, the three pre-activation rows, h read and h written; summed over the layers
        self.kernel_bytes = 0.0
        for hh in self.hh:
            i = B.grim_bcr_info(hh)
            self.kernel_bytes += self.T * (i.value_bytes + i.index_bytes_gemv + 3 * self.H * 4 + 2 * self.H * 4)
        self.h2d = self.x_host.numel() * 4
        self.d2h = self.y_host.numel() * 4
        self.kernel = "gru_cluster_reg_kernel"
        self.peak_kind = "alu"
        self.force_bound = "hbm"  # a chain of dependent steps: reported against the streamed-bytes figure

    def step(self):
        self.B.grim_gru_seq(self.g, self.x, self.y)

    def step_e2e(self):
        xd = self.x_host.cuda(non_blocking=True)
        self.B.grim_gru_seq(self.g, xd, self.y)
        self.y_host.copy_(self.y, non_blocking=True)

    def kernel_ms(self):
        return self.B.grim_gru_profile_read(self.g)[1]

    def check(self):
        assert self.B.grim_gru_status(self.g) == self.B.GRIM_OK

    def oracle_sample(self):
        from oracle import bcr_oracle as orc
        Ts = self.sample_T
        t0 = time.perf_counter()
        orc.gru_seq(self.m["layers"], self.m["x"][:Ts])
        dt = time.perf_counter() - t0
        return 2.0 * self.nnz * Ts / dt / 1e9, f"first {Ts} of {self.T} time steps, both layers, dense fp64 NumPy mat-vec"


class SpmmWorkload:
    """One point of the SpMM sweep (square W).  N = 1 runs the matrix-vector kernel."""

    def __init__(self, M=8192, N=1, c=8.0, bh=8, bw=32, dist="uniform", bf16=False, conv=False):
        from workloads import generators as gen
        self.M, self.N, self.bf16 = M, N, bf16
        self.s = gen.sweep_case(M, N, c, bh, bw, dist, bf16=bf16)
        self.bh, self.bw = bh, bw
        self.name = f"spmm_M{M}_K{M}_N{N}_c{c:g}_{bh}x{bw}_{dist}_{'bf16' if bf16 else 'fp32'}"
        self.dtype = "bf16" if bf16 else "f32"
        self.nnz = int(self.s["mask"].sum())
        self.flops = 2.0 * self.nnz * N
        self.copies = 1

    def setup(self, B, torch):
        self.B, self.torch = B, torch
        s = self.s
        dt = B.GRIM_BF16 if self.bf16 else B.GRIM_F32
        self.h = B.grim_bcr_pack(s["W"], s["mask"], self.bh, self.bw, dt, B.GRIM_PACK_REORDER)
        tdt = torch.bfloat16 if self.bf16 else torch.float32
        self.x_host = torch.from_numpy(s["X"]).to(tdt).pin_memory()
        self.x = self.x_host.cuda()
        self.y = torch.empty(self.M, self.N, device="cuda")
        self.y_host = torch.empty(self.M, self.N).pin_memory()
        i = B.grim_bcr_info(self.h)
        esz = 2 if self.bf16 else 4
        idx = i.index_bytes_gemv if self.N <= 16 else i.index_bytes_spmm
        self.kernel_bytes = float(i.value_bytes + idx + i.k_used * self.N * esz + self.M * self.N * 4)
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
            h = B.grim_bcr_pack(s["W"], s["mask"], self.bh, self.bw, dt, B.GRIM_PACK_REORDER)
            self.sets.append((h, self.x.clone(), torch.empty_like(self.y)))
        self.rotating = len(self.sets) > 1
        self.per_step_events = True
        self._i = 0

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

    def kernel_ms(self):
        self._ev[1].synchronize()
        return self._ev[0].elapsed_time(self._ev[1])

    def check(self):
        pass

    def oracle_sample(self):
        from oracle import bcr_oracle as orc
        n = min(self.N, 64)
        t0 = time.perf_counter()
        orc.spmm(self.s["W"], self.s["mask"], self.s["X"][:, :n], 1 if self.bf16 else 0)
        dt = time.perf_counter() - t0
        return 2.0 * self.nnz * n / dt / 1e9, f"first {n} of {self.N} columns, masked dense fp64 NumPy matmul"


class ConvWorkload:
    def __init__(self, batch=32, bf16=False):
        from workloads import generators as gen
        self.L = gen.conv_layer(batch, 512, 512, 28, bf16=bf16)
        self.batch, self.bf16 = batch, bf16
        self.name = f"conv3x3_512to512_28x28_b{batch}_bcr16x64_c8_{'bf16' if bf16 else 'fp32'}"
        self.dtype = "bf16" if bf16 else "f32"
        self.nnz = int(self.L["mask"].sum())
        self.flops = 2.0 * self.nnz * batch * 28 * 28

    def setup(self, B, torch):
        self.B, self.torch = B, torch
        L = self.L
        dt = B.GRIM_BF16 if self.bf16 else B.GRIM_F32
        tdt = torch.bfloat16 if self.bf16 else torch.float32
        self.h = B.grim_bcr_pack(L["W"], L["mask"], 16, 64, dt, B.GRIM_PACK_REORDER)
        self.x_host = torch.from_numpy(L["x"]).to(tdt).pin_memory()
        self.x = self.x_host.cuda()
        self.bias = torch.from_numpy(L["bias"]).cuda()
        self.y = torch.empty(self.batch, 512, 28, 28, device="cuda", dtype=tdt)
        self.y_host = torch.empty(self.batch, 512, 28, 28, dtype=tdt).pin_memory()
        i = B.grim_bcr_info(self.h)
        esz = 2 if self.bf16 else 4
        idx = i.index_bytes_tc if self.bf16 else i.index_bytes_spmm
        self.kernel_bytes = float(i.value_bytes + idx + self.x.numel() * esz + self.y.numel() * esz)
        self.h2d = self.x_host.numel() * esz
        self.d2h = self.y_host.numel() * esz
        self.kernel = "bcr_tc_kernel (implicit im2col)" if self.bf16 else "bcr_ffma_kernel (implicit im2col)"
        self.peak_kind = "tensor" if self.bf16 else "alu"
        self._ev = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
        self.sets = [(self.h, self.x, self.y)]
        for _ in range(rotation_sets(self.kernel_bytes) - 1):
            h = B.grim_bcr_pack(L["W"], L["mask"], 16, 64, dt, B.GRIM_PACK_REORDER)
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
        pass

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
        self.kernel = "bcr_tc_kernel (implicit im2col, per layer)"

    def setup(self, B, torch):
        self.B, self.torch = B, torch
        net = self.net
        self.h, self.bias, self.bufs, self.info = [], [], [], []
        self.x_host = torch.from_numpy(net["x"]).to(torch.bfloat16).pin_memory()
        self.x = self.x_host.cuda()
        cur_hw = self.image
        for L in net["layers"]:
            self.h.append(B.grim_bcr_pack(L["W"], L["mask"], net["bh"], net["bw"], B.GRIM_BF16, B.GRIM_PACK_REORDER))
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
        pass

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
    for _ in range(args.warmup):
        wl.oracle_sample()
    vals, t0 = [], time.perf_counter()
    for _ in range(args.steps):
        v, what = wl.oracle_sample()
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

    wl = make_workload(args)
    wl.setup(B, torch)
    # written before every timed iteration: evicts the working set from L2 (126 MB) and keeps the GPU busy
    # long enough for the host to queue the step behind it, so that no host latency sits between the events
    flush = torch.empty(1 << 30, dtype=torch.uint8, device="cuda")

    def flush_l2():
        # the write evicts the working set; the read of half the buffer behind it pushes the write's dirty lines out
        # to HBM, so that the timed step does not pay for writing them back when its own reads evict them
        flush.zero_()
        flush[: 1 << 29].view(torch.int64).sum()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        wl.step()
    wl.check()
    barrier()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    B.grim_launch_count_reset()
    kernel_ms = []
    rotating = bool(getattr(wl, "rotating", False))
    barrier()
    if rotating:
        wl.per_step_events = False
        # Inputs larger than L2: the steps rotate through operand sets, so every launch reads from HBM, and they are
        # queued back to back behind a few flushes (which keep the GPU busy while the host queues all steps): the
        # time between the two events is that of the launches alone, without per-launch host or event latency.
        for _ in range(2 + args.steps // 8):
            flush_l2()
        ev[0][0].record()
        for k in range(args.steps):
            wl.step()
        ev[0][1].record()
        barrier()
        total_ms = ev[0][0].elapsed_time(ev[0][1])
        kernel_ms = [total_ms / args.steps]
    else:
        for k in range(args.steps):
            flush_l2()  # evict the working set from L2 between timed iterations (not timed)
            ev[k][0].record()
            wl.step()
            ev[k][1].record()
            kernel_ms.append(wl.kernel_ms())
        barrier()
        total_ms = sum(a.elapsed_time(b) for a, b in ev)
    launches = B.grim_launch_count()
    wl.check()

    # end to end: host buffers, copies inside the timed region
    for _ in range(2):
        wl.step_e2e()
    barrier()
    ev2 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for k in range(args.steps):
        flush_l2()
        ev2[k][0].record()
        wl.step_e2e()
        ev2[k][1].record()
    barrier()
    e2e_ms = sum(a.elapsed_time(b) for a, b in ev2)
    clocks = sampler.stop() if rank == 0 else None

    total_ms, e2e_ms = max_over_ranks([total_ms, e2e_ms], device="cuda")

    if rank == 0:
        peaks = measured_peaks()
        value = aggregate_value(wl.flops, args.steps, total_ms, world)
        e2e_value = aggregate_value(wl.flops, args.steps, e2e_ms, world)
        k_ms = statistics.mean(kernel_ms)
        # binding roofline of the dominant kernel: the slower of (algorithmic bytes at the measured HBM bandwidth) and
        # (effective flops 2*nnz*N at the peak of the unit that does the arithmetic: plain fp32 FMA pipes, derived as
        # 148 SMs x 128 lanes x 2 flop x 1.965 GHz, or the measured dense bf16 tensor rate for the tcgen05 kernel)
        alu_peak = 148 * 128 * 2 * 1.965e9 / 1e12
        flop_peak = peaks["bf16_tflops_burst"] if wl.peak_kind == "tensor" else alu_peak
        t_hbm = wl.kernel_bytes / (peaks["hbm_gbs"] * 1e9)
        t_flop = wl.flops / (flop_peak * 1e12)
        bound = getattr(wl, "force_bound", None) or ("hbm" if t_hbm >= t_flop else wl.peak_kind)
        if bound == "hbm":
            achieved = wl.kernel_bytes / (k_ms * 1e-3) / 1e9
            roof = dict(bound="hbm", achieved=achieved, peak=peaks["hbm_gbs"], unit="GB/s", frac=achieved / peaks["hbm_gbs"],
                        traffic=None, kernel=wl.kernel, kernel_ms=k_ms, algorithmic_bytes=wl.kernel_bytes,
                        peak_source=peaks["source"])
        else:
            achieved = wl.flops / (k_ms * 1e-3) / 1e12
            roof = dict(bound=bound, achieved=achieved, peak=flop_peak, unit="TFLOP/s", frac=achieved / flop_peak, traffic=None,
                        kernel=wl.kernel, kernel_ms=k_ms,
                        peak_source=("measured dense bf16 (burst)" if bound == "tensor"
                                     else "derived: 148 SM x 128 FMA lanes x 2 x 1.965 GHz"))
        roof["traffic"] = TRAFFIC.get(wl.name)
        roof["t_hbm_us"] = t_hbm * 1e6
        roof["t_flop_us"] = t_flop * 1e6
        if hasattr(wl, "extra"):
            roof.update(wl.extra(peaks))
        cpu_v, cpu_what = wl.oracle_sample()
        line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=max(args.warmup, 3),
                    ms_per_step=total_ms / args.steps, higher_is_better=True, scaling="weak", vs_baseline=None,
                    dtype=wl.dtype, data="synthetic",
                    config=dict(workload=wl.name, nnz=wl.nnz,
                                l2=(f"inputs larger than L2: the steps rotate through {len(wl.sets)} operand sets of "
                                    f"{wl.kernel_bytes / 1e6:.0f} MB, launches queued back to back" if rotating else
                                    "flushed between timed iterations (1 GiB write, then a 512 MiB read that leaves no dirty lines)"),
                                parallelism="replicas only" if world > 1 else "1 GPU"),
                    clocks=clocks,
                    e2e=dict(value=e2e_value, unit=UNIT, h2d_bytes_per_step=wl.h2d, d2h_bytes_per_step=wl.d2h,
                             ms_per_step=e2e_ms / args.steps),
                    gpu_launches=int(launches), roofline=roof,
                    cpu_baseline=dict(value=cpu_v, unit=UNIT, cores=len(os.sched_getaffinity(0)), kind="oracle",
                                      sample=cpu_what))
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()

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
            info = B.grim_bcr_info(h)
            esz = 2 if bf16 else 4
            for N in ncols:
                X = torch.from_numpy(np.ascontiguousarray(Xf[:, :N])).cuda()
                if bf16:
                    X = X.to(torch.bfloat16)
                Y = torch.empty(M, N, device="cuda")
                tc = bf16 and N >= 128
                idx = info.index_bytes_gemv if N <= 16 else (info.index_bytes_tc if tc else info.index_bytes_spmm)
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
                t = statistics.median(ms) * 1e-3
                t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9)
                t_flop = flops / (peaks["bf16_tflops_burst"] * 1e12 if tc else alu_peak)
                rec = dict(M=M, N=N, c=c, block=f"{bh}x{bw}", dist=dist_name, dtype="bf16" if bf16 else "f32", reorder=reorder,
                           nnz=nnz, ms=t * 1e3, gflops=flops / t / 1e9, bound="hbm" if t_hbm >= t_flop else ("tensor" if tc else "alu"),
                           frac=max(t_hbm, t_flop) / t, kernel="skinny" if N <= 16 else ("tc" if tc else "ffma"))
                out.write(json.dumps(rec) + "\n")
                fracs.append(rec["frac"])
                n_runs += 1
            B.grim_bcr_destroy(h)
        out.flush()
    out.close()
    print(json.dumps(dict(metric="SpMM sweep: fraction of the binding roofline", runs=n_runs, median_frac=statistics.median(fracs),
                          min_frac=min(fracs), max_frac=max(fracs), wall_s=time.perf_counter() - t_start, out=args.out)))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="gru", choices=["gru", "gemv", "spmm", "conv", "vgg"])
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
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
