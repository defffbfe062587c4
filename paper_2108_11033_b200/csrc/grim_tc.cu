// Tensor-core (tcgen05) kernel for Y = W * X with bf16 operands and fp32 accumulation, large N
// (Section 3.1: every layer is a GEMM; Sections 4.3 - 4.4: compact storage, expanded only on chip).
//
// The packed weights never exist in dense form in HBM.  A thread block owns 128 rows of W (in schedule
// order) and 256 output columns and walks K in tiles of 64.  Per K tile
//   - one thread asks TMA for the 64 x 256 tile of X (128-byte swizzle, the layout the tensor core reads
//     directly as the N-major operand) and for the packed records of the thread block's bands,
//   - twelve warps in three groups expand those records into a 128 x 64 bf16 tile in shared memory (the K-major
//     128-byte-swizzled layout of the other operand): clear it, then one 2-byte store per kept value at the
//     offset the packer stored beside it,
//   - one thread issues four tcgen05.mma (128 x 256 x 16) that accumulate in tensor memory.
// A ring of stages with full / ready / empty mbarriers overlaps the three.  After the last K tile the eight
// warps read the accumulators back (tcgen05.ld), add bias, apply the activation and store Y.
//
// The multiply therefore runs at the tensor core's dense rate on a tile whose density is that of the
// pruned matrix; it is chosen for bf16 handles when N is large, where even so it is several times faster
// than the CUDA-core kernels.  Every wait is bounded; tensor memory is released on every exit path.
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <cstring>

#include "grim_device.cuh"
#include "grim_im2col.cuh"
#include "grim_internal.h"

namespace grim {
namespace {

constexpr int kTcWorkers = 12;     // warps that expand the packed weights; the first eight also run the epilogue
constexpr int kTcGroups = 3;       // the workers form groups that take K tiles in turn, so that expansions overlap
constexpr int kTcGroupWarps = kTcWorkers / kTcGroups;
constexpr int kTcGroupThreads = 32 * kTcGroupWarps;
constexpr int kTcThreads = 64 + 32 * kTcWorkers;  // warp 0: copies, warp 1: tensor core, then the workers
constexpr int kTcBuilders = 12;    // convolution only: warps that build the X tile from the NCHW input
constexpr int kTcBuildGroups = 3;  // they form groups that take K tiles in turn, like the expansion warps
constexpr int kTcBuildGroupWarps = kTcBuilders / kTcBuildGroups;
constexpr int kTcConvThreads = kTcThreads + 32 * kTcBuilders;
constexpr int kTM = 128;          // rows of W per thread block
constexpr int kTQ = 256;          // output columns per thread block
constexpr int kTK = 64;           // K per stage
constexpr int kTcStages = 4;        // ring slots at most; fewer when the packed records are large
constexpr int kATileBytes = kTM * kTK * 2;   // 16 KiB
constexpr int kBTileBytes = kTQ * kTK * 2;   // 32 KiB
constexpr int kTcHdrBytes = 1024;
constexpr int kTcRecSlots = 8;      // ring of packed records (small), deeper than the ring of tiles so that records
                                    // are on chip well before the weight tile they expand into becomes free
constexpr unsigned kTmemCols = 256;

struct TcParams {
  const RcStage* stage;
  const uint8_t* blob;
  const uint32_t* band_order;
  unsigned* status;
  int nbr, M, K, bh, nkt;
  int bh_shift, slots_per_tile, nstages, nrec;
  int mt, mtiles;  // row tiles (128 rows each) per thread block: 1 or 2 (they share every X tile); tiles in the matrix
  uint32_t stage_bytes, rec_stride;
  unsigned spin_limit;
  int64_t in_elems;  // convolution: elements of the input tensor
  int seg_off, seg_len;  // staged convolution: elements in front of the tile's first pixel / per channel segment
  int nseg;              // staged convolution: slots of the ring of staged planes
  int ksplit, kt_per;    // > 1: blockIdx.z takes kt_per K tiles and adds its partial sums into the fp32 scratch `acc`
  float* acc;            // [M][ncols] when ksplit > 1
  uint32_t seg_bytes;    // bytes of one such slot
  SpmmArgs a;
};

using namespace ptx;

// Shared-memory matrix descriptor of the tensor core: start address, leading / stride byte offsets
// (all without their 4 low bits), descriptor version 1, 128-byte swizzle.
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: fp32 accumulate, bf16 x bf16, A K-major, B N-major, M = 128, N = 256.
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) | ((kTQ >> 3) << 17) | ((kTM >> 4) << 24);

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(kIdesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// CONV: 0 = X is a matrix (TMA tiles); 1 = implicit im2col, the builders read the NCHW input from global memory;
// 2 = implicit im2col, the input planes the tile needs are first staged in shared memory by bulk copies; 3 = the same
// with 8-byte asynchronous copies per lane, for planes whose size is a multiple of 4 but not of 8 pixels (their starts
// are not all 16-byte aligned).
template <int BH, int CONV>
__global__ void __launch_bounds__(CONV ? kTcConvThreads : kTcThreads, 1) bcr_tc_kernel(const __grid_constant__ CUtensorMap tmX, const TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  // tiles must start on a 1 KiB boundary (the swizzle pattern repeats every 8 rows of 128 bytes)
  // the launch that follows in the stream may start as SMs free up: it waits (griddepcontrol.wait) before it reads or
  // writes anything this launch touches
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full = reinterpret_cast<uint64_t*>(smem);        // the X tile of a stage has landed
  uint64_t* ready = full + kTcStages;                        // the expanded weight tile of a stage is written
  uint64_t* empty = ready + kTcStages;                         // the tensor core is done with a stage
  uint64_t* built = empty + kTcStages;                         // convolution: the X tile of a stage is written
  uint64_t* acc_done = built + kTcStages;                      // all multiplies of the tile are complete
  uint64_t* rec_full = acc_done + 1;                           // a packed record has landed
  unsigned* s_done = reinterpret_cast<unsigned*>(smem + 640);    // [record slot] warps that have finished expanding it
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + 384);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + 388);
  uint64_t* seg_free = reinterpret_cast<uint64_t*>(smem + 704);  // staged convolution: the builders are done with a slot of planes
  uint32_t* s_meta = reinterpret_cast<uint32_t*>(smem + 512);  // [record slot] bytes of the packed record (0: none)
  uint8_t* stages = smem + kTcHdrBytes;
  const uint32_t stage_bytes = p.stage_bytes;
  uint8_t* recs = stages + (size_t)p.nstages * stage_bytes;
  uint8_t* segs = recs + (size_t)p.nrec * p.mt * p.rec_stride;  // staged convolution: ring of input planes

  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
  const SpmmArgs& a = p.a;
  const int64_t q0 = (int64_t)blockIdx.x * kTQ;
  const int pos0 = blockIdx.y * p.mt * p.slots_per_tile;  // first band (schedule position) of this thread block's rows
  const uint32_t b_off = (uint32_t)p.mt * kATileBytes;     // the X tile follows the weight tiles in a stage
  const uint32_t tmem_cols = kTmemCols * (uint32_t)p.mt;
  // K tiles of this thread block: all of them, or its share of a split multiply; kt below counts them from 0
  const int kbase = p.ksplit > 1 ? (int)blockIdx.z * p.kt_per : 0;
  const int nkt = p.ksplit > 1 ? (p.nkt - kbase < p.kt_per ? p.nkt - kbase : p.kt_per) : p.nkt;
  const int ns = p.nstages, nr = p.nrec;
  Im2colCtx im;
  if (CONV) {
    im.a = &p.a; im.K = p.K; im.in_elems = (int)p.in_elems; im.seg_off = p.seg_off; im.seg_len = p.seg_len; im.nseg = p.nseg;
    im.seg_bytes = p.seg_bytes; im.q0 = q0; im.nkt = nkt; im.kbase = kbase; im.ns = ns; im.stages = stages;
    im.stage_bytes = stage_bytes; im.b_off = b_off; im.segs = segs; im.empty = empty; im.seg_full = full;
    im.seg_free = seg_free; im.built = built; im.built_rank = -1; im.cluster_waits = false; im.spin_limit = p.spin_limit;
    im.s_abort = s_abort;
  }

  if (tid == 0) {
    for (int s = 0; s < kTcStages; ++s) {
      mbar_init(full + s, CONV == 3 ? 32u : 1u);  // completed by TMA byte counts, or by the copy warp's 32 lanes
      mbar_init(ready + s, kTcGroupWarps);
      mbar_init(empty + s, 1);
      mbar_init(built + s, kTcBuildGroupWarps);
      mbar_init(seg_free + s, kTcBuildGroupWarps);
    }
    for (int s = 0; s < kTcRecSlots; ++s) {
      mbar_init(rec_full + s, 1);
      s_done[s] = 0;
    }
    mbar_init(acc_done, 1);
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *s_tmem;
  // (programmatic dependent launch) whatever earlier launches in the stream wrote - X, a cleared scratch or Y - is
  // complete and visible from here on; up to here only the packed matrix and this block's own shared memory were touched
  asm volatile("griddepcontrol.wait;" ::: "memory");

  // Requests the packed records of K tile k (one per row tile) into record slot rs; one thread.
  auto request_records = [&](int k, int rs) {
    uint32_t bytes[2] = {0u, 0u}, off[2] = {0u, 0u}, total = 0;
    for (int m = 0; m < p.mt; ++m) {
      const int t = (int)blockIdx.y * p.mt + m;
      if (t < p.mtiles) {
        const RcStage se = p.stage[(int64_t)t * p.nkt + kbase + k];
        bytes[m] = se.bytes; off[m] = se.off16;
      }
      s_meta[rs * 2 + m] = bytes[m];
      total += bytes[m];
    }
    mbar_arrive_expect_tx(rec_full + rs, total);
    for (int m = 0; m < p.mt; ++m)
      if (bytes[m]) bulk_load(recs + (size_t)(rs * p.mt + m) * p.rec_stride, p.blob + (size_t)off[m] * 16, bytes[m], rec_full + rs);
  };

  bool failed = false;
  int fail_site = 0;
  if (warp == 0) {
    // ------------------------------------------------------------------ copies
    if (lane == 0) {
      // the first records (the ring of records is deeper than the ring of tiles); later ones are requested by the
      // expansion warps as they free a record slot
      for (int rk = 0; rk < nr && rk < nkt; ++rk) request_records(rk, rk);
      for (int kt = 0; kt < nkt && !CONV; ++kt) {  // the convolution builds its X tiles itself
        const int slot = kt % ns;
        if (kt >= ns && !mbar_wait(empty + slot, (unsigned)((kt / ns - 1) & 1), p.spin_limit, s_abort)) { failed = true, fail_site = 1; break; }
        uint8_t* st = stages + (size_t)slot * stage_bytes;
        // 64-column boxes that lie wholly past the last column are not requested (their part of the tile keeps
        // whatever it held; the accumulator columns computed from it are never stored)
        const int nbox = (int)((a.ncols - q0 + 63) / 64) < kTQ / 64 ? (int)((a.ncols - q0 + 63) / 64) : kTQ / 64;
        mbar_arrive_expect_tx(full + slot, (unsigned)(nbox * 64 * kTK * 2));
#pragma unroll
        for (int i = 0; i < kTQ / 64; ++i)
          if (i < nbox) tma_load_2d(st + b_off + i * (64 * kTK * 2), &tmX, (int)q0 + 64 * i, (kbase + kt) * kTK, full + slot);
      }
    }
    if (CONV >= 2) {
      // staged implicit im2col: the input planes of every K tile are copied into a ring of shared-memory segments
      if (!conv_copy_planes<CONV>(im, lane)) failed = true, fail_site = 1;
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ tensor core
    if (lane == 0) {
      for (int kt = 0; kt < nkt; ++kt) {
        const int slot = kt % ns;
        const unsigned par = (unsigned)((kt / ns) & 1);
        if ((!CONV && !mbar_wait(full + slot, par, p.spin_limit, s_abort)) || !mbar_wait(ready + slot, par, p.spin_limit, s_abort) ||
            (CONV && !mbar_wait(built + slot, par, p.spin_limit, s_abort))) { failed = true, fail_site = 2; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t a_addr = smem_u32(stages + (size_t)slot * stage_bytes);
        const uint32_t b_addr = a_addr + b_off;
        for (int m = 0; m < p.mt; ++m) {
#pragma unroll
          for (int s = 0; s < kTK / 16; ++s) {
            // A: K-major, rows 128 bytes apart, 8-row groups 1 KiB apart; 16 K-elements = 32 bytes further on
            const uint64_t ad = smem_desc(a_addr + m * kATileBytes + s * 32, 16, 1024);
            // B: N-major, 64-column groups 8 KiB apart, 8-row K groups 1 KiB apart; 16 K-rows = 2 KiB further on
            const uint64_t bd = smem_desc(b_addr + s * 2048, 64 * kTK * 2, 1024);
            umma_bf16(tmem_base + (uint32_t)m * kTmemCols, ad, bd, (kt > 0 || s > 0) ? 1u : 0u);
          }
        }
        umma_commit(empty + slot);  // arrives when the multiplies above have read their operands
      }
      if (!failed) umma_commit(acc_done);
    }
  } else if (CONV && warp >= 2 + kTcWorkers) {
    // ------------------------------------------------------------------ implicit im2col (3x3, stride 1, pad 1)
    const int bgrp = (warp - 2 - kTcWorkers) / kTcBuildGroupWarps;
    const int bt = tid - kTcThreads - bgrp * (32 * kTcBuildGroupWarps);  // 0 .. 127 inside the group
    if (!conv_build_tiles<CONV>(im, bgrp, kTcBuildGroups, bt, lane, fail_site)) failed = true;
  } else {
    // ------------------------------------------------------------------ expansion of the packed weights
    const int grp = (warp - 2) / kTcGroupWarps;               // this warp's group
    const int wt = tid - 64 - grp * kTcGroupThreads;           // 0 .. kTcGroupThreads - 1 inside the group
    for (int kt = grp; kt < nkt; kt += kTcGroups) {
      const int slot = kt % ns, rs = kt % nr;
      // the weight tile of the slot is free once the multiplies of its previous use are done; the record is
      // normally long there
      if (kt >= ns && !__all_sync(0xffffffffu, mbar_wait(empty + slot, (unsigned)((kt / ns - 1) & 1), p.spin_limit, s_abort))) { failed = true, fail_site = 4; break; }
      if (!__all_sync(0xffffffffu, mbar_wait(rec_full + rs, (unsigned)((kt / nr) & 1), p.spin_limit, s_abort))) { failed = true, fail_site = 5; break; }
      uint8_t* st = stages + (size_t)slot * stage_bytes;
      // clear the tile, meet, then one 2-byte store per kept value at the offset stored beside it
      for (int m = 0; m < p.mt; ++m)
        ptx::expand_scatter<kTcGroupThreads>(smem_u32(recs + (size_t)(rs * p.mt + m) * p.rec_stride), s_meta[rs * 2 + m],
                                             smem_u32(st + m * kATileBytes), wt, 1 + grp);
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> visible to the tensor core
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(ready + slot);
        // the last warp of the group to finish with the record frees its slot: it requests the record that uses
        // the slot next (every read of the old record precedes that warp's count)
        if (atomicAdd(s_done + rs, 1u) == (unsigned)kTcGroupWarps - 1u) {
          s_done[rs] = 0;
          if (kt + nr < nkt) request_records(kt + nr, rs);
        }
      }
      if (__any_sync(0xffffffffu, failed)) { failed = true; break; }
    }
    // ------------------------------------------------------------------ epilogue
    const bool epilogue_warp = warp - 2 < 8;  // two warps per quarter of the tensor-memory lanes
    if (epilogue_warp && !__any_sync(0xffffffffu, failed)) {
      if (!__all_sync(0xffffffffu, mbar_wait(acc_done, 0, p.spin_limit, s_abort))) failed = true, fail_site = 8;
    }
    if (epilogue_warp && !__any_sync(0xffffffffu, failed)) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int quarter = warp & 3;                 // the tensor-memory lanes this warp may read
      const int trow = quarter * 32 + lane;         // row of the tile held by this thread's lane
      const int r = trow & (BH - 1);
      const int cb0 = ((warp - 2) >> 2) * (kTQ / 64), cb1 = cb0 + kTQ / 64;  // warps 2-5: columns 0-127, warps 6-9: 128-255
      for (int m = 0; m < p.mt; ++m) {
      const int pos = pos0 + m * p.slots_per_tile + (trow >> p.bh_shift);
      int64_t row = -1;
      if (pos < p.nbr && (int)blockIdx.y * p.mt + m < p.mtiles) row = (int64_t)p.band_order[pos] * p.bh + r;
      const bool row_ok = row >= 0 && row < p.M;
      const float bias = (row_ok && a.bias) ? __ldg(a.bias + row) : 0.f;
      for (int cb = cb0; cb < cb1; ++cb) {
        uint32_t v[32];
        tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(m * (int)kTmemCols + cb * 32), v);
        const int64_t q = q0 + cb * 32;
        if (!row_ok || q >= a.ncols) continue;
        if (p.ksplit > 1) {
          // split multiply: partial sums go to the zeroed fp32 scratch; bias, activation and the output layout are
          // applied by a pass over the scratch when all parts are in
          float* dst = p.acc + row * a.ncols + q;
          if (q + 31 < a.ncols && (reinterpret_cast<uintptr_t>(dst) & 15) == 0) {
            // eight 16-byte reductions instead of thirty-two 4-byte ones
#pragma unroll
            for (int i = 0; i < 8; ++i)
              asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst + 4 * i), "f"(__uint_as_float(v[4 * i])),
                           "f"(__uint_as_float(v[4 * i + 1])), "f"(__uint_as_float(v[4 * i + 2])), "f"(__uint_as_float(v[4 * i + 3]))
                           : "memory");
          } else {
            for (int i = 0; i < 32 && q + i < a.ncols; ++i) atomicAdd(dst + i, __uint_as_float(v[i]));
          }
          continue;
        }
        float t[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          t[i] = __uint_as_float(v[i]) + bias;
          if (a.relu) t[i] = fmaxf(t[i], 0.f);
        }
        int64_t off0 = row * a.y_sr + q;
        bool full_chunk = q + 31 < a.ncols;
        if (CONV) {
          // NCHW output: 32 consecutive pixels of one channel are contiguous while they stay inside one image
          const int64_t ohw = (int64_t)a.OH * a.OW;
          const int64_t img = q / ohw, pix = q - img * ohw;
          off0 = (img * p.M + row) * ohw + pix;
          if (pix + 31 >= ohw || !full_chunk) {
            for (int i = 0; i < 32 && q + i < a.ncols; ++i) {
              const int64_t im = (q + i) / ohw, px = (q + i) - im * ohw;
              const int64_t o = (im * p.M + row) * ohw + px;
              if (a.y_dtype == GRIM_F32) static_cast<float*>(a.Y)[o] = t[i];
              else static_cast<__nv_bfloat16*>(a.Y)[o] = __float2bfloat16_rn(t[i]);
            }
            continue;
          }
        }
        if (a.y_dtype == GRIM_F32) {
          float* y = static_cast<float*>(a.Y) + off0;
          if (full_chunk && ((reinterpret_cast<uintptr_t>(y) & 15) == 0)) {
#pragma unroll
            for (int i = 0; i < 8; ++i) reinterpret_cast<float4*>(y)[i] = make_float4(t[4 * i], t[4 * i + 1], t[4 * i + 2], t[4 * i + 3]);
          } else {
            for (int i = 0; i < 32 && q + i < a.ncols; ++i) y[i] = t[i];
          }
        } else {
          __nv_bfloat16* y = static_cast<__nv_bfloat16*>(a.Y) + off0;
          if (full_chunk && ((reinterpret_cast<uintptr_t>(y) & 15) == 0)) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              uint4 u;
              __nv_bfloat162 b0 = __floats2bfloat162_rn(t[8 * i], t[8 * i + 1]), b1 = __floats2bfloat162_rn(t[8 * i + 2], t[8 * i + 3]);
              __nv_bfloat162 b2 = __floats2bfloat162_rn(t[8 * i + 4], t[8 * i + 5]), b3 = __floats2bfloat162_rn(t[8 * i + 6], t[8 * i + 7]);
              u.x = *reinterpret_cast<unsigned*>(&b0); u.y = *reinterpret_cast<unsigned*>(&b1);
              u.z = *reinterpret_cast<unsigned*>(&b2); u.w = *reinterpret_cast<unsigned*>(&b3);
              reinterpret_cast<uint4*>(y)[i] = u;
            }
          } else {
            for (int i = 0; i < 32 && q + i < a.ncols; ++i) y[i] = __float2bfloat16_rn(t[i]);
          }
        }
      }
      }  // row tiles
    }
  }

  if (__any_sync(0xffffffffu, failed)) {
    *s_abort = 1;
    if (fail_site) atomicOr(p.status, (unsigned)GRIM_ERR_TIMEOUT | (1u << (8 + fail_site)));
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
}

// Second pass of a split multiply: scratch + bias -> activation -> Y in its layout and type.
__global__ void tc_finalize_kernel(const float* __restrict__ acc, int64_t ncols, int M, const float* __restrict__ bias, int relu,
                                   void* Y, int y_dtype, int64_t y_sr, int conv, int64_t ohw) {
  const int64_t total = (int64_t)M * ncols;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t row = i / ncols, q = i - row * ncols;
    float v = acc[i] + (bias ? __ldg(bias + row) : 0.f);
    if (relu) v = fmaxf(v, 0.f);
    int64_t off = row * y_sr + q;
    if (conv) {
      const int64_t img = q / ohw, pix = q - img * ohw;
      off = (img * M + row) * ohw + pix;
    }
    if (y_dtype == GRIM_F32) static_cast<float*>(Y)[off] = v;
    else static_cast<__nv_bfloat16*>(Y)[off] = __float2bfloat16_rn(v);
  }
}

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess) {
      cudaGetLastError();
      p = nullptr;
    }
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

size_t tc_stage_bytes(int mt) { return (size_t)mt * kATileBytes + kBTileBytes; }
size_t tc_rec_stride(const grim_bcr* h) { return ((size_t)h->td_max_rec + 127) & ~size_t(127); }
// extra: bytes besides the operand tiles and the records (the ring of staged input planes of the convolution)
size_t tc_smem_need(const grim_bcr* h, int mt, int stages, int nrec, size_t extra = 0) {
  return 1024 + kTcHdrBytes + (size_t)stages * tc_stage_bytes(mt) + (size_t)nrec * mt * tc_rec_stride(h) + extra;
}
// Ring sizes that fit: as many tile slots as possible first (they carry the bulk of the bytes in flight), then as
// many record slots as are left, at least as many as tile slots.
// At least as many tile slots as expansion groups: a group then never waits on a barrier that is more than one
// phase behind it (parity waits cannot tell phases two apart).
bool tc_rings(const grim_bcr* h, int mt, int* stages, int* nrec, size_t extra = 0) {
  for (int s = kTcStages; s >= kTcGroups; --s)
    for (int r = kTcRecSlots; r >= s; --r)
      if (tc_smem_need(h, mt, s, r, extra) <= 226 * 1024) { *stages = s; *nrec = r; return true; }
  return false;
}
// Row tiles per thread block: two share every X tile (half the L2 traffic per flop, which is what bounds the
// kernel) when that still leaves enough thread blocks for the GPU and three tile slots fit.
int tc_row_tiles(const grim_bcr* h, int64_t qtiles, size_t extra = 0) {
  int s = 0, r = 0;
  if (h->tc_mtiles >= 2 && qtiles * ((h->tc_mtiles + 1) / 2) >= 96 && tc_rings(h, 2, &s, &r, extra) && s >= 3) return 2;
  return 1;
}
}  // namespace

bool tc_path_supported(const grim_bcr* h, const SpmmArgs& a) {
  if (h->device < 0 || h->dtype != GRIM_BF16 || !h->d_td_stage || !h->d_status) return false;
  if (a.x_dtype != GRIM_BF16 || reinterpret_cast<uintptr_t>(a.X) % 16 != 0) return false;
  if (a.conv) {
    // the tile builder covers the common same-size 3x3 convolution; other geometries use the CUDA-core kernel
    if (a.KH != 3 || a.KW != 3 || a.stride != 1 || a.pad != 1 || a.OH != a.H || a.OW != a.W) return false;
    if (a.ncols / ((int64_t)a.OH * a.OW) * a.C * a.H * a.W >= (int64_t(1) << 31) - 64) return false;
  } else if (a.x_sq != 1 || a.y_sq != 1 || (a.x_sk * 2) % 16 != 0) {
    return false;
  }
  if (a.ncols <= 0 || a.ncols > (int64_t(1) << 31) - kTQ || h->td_max_rec == 0) return false;
  int st_ = 0, nr_ = 0;
  if (!tc_rings(h, 1, &st_, &nr_)) return false;
  if (h->tc_mtiles > 65535) return false;
  return encode_tiled_fn() != nullptr;
}

grim_status_t launch_spmm_tc(const grim_bcr* h, const SpmmArgs& a, cudaStream_t s) {
  if (!tc_path_supported(h, a)) return GRIM_ERR_UNSUPPORTED;
  TcParams p;
  p.stage = h->d_td_stage; p.blob = h->d_td_blob; p.band_order = h->d_band_order; p.status = h->d_status;
  p.nbr = (int)h->nbr; p.M = (int)h->M; p.K = (int)h->K; p.bh = h->bh; p.nkt = (int)h->tc_ktiles;
  p.bh_shift = h->bh == 4 ? 2 : (h->bh == 8 ? 3 : 4);
  p.slots_per_tile = kTM / h->bh;
  const int64_t qtiles_ = (a.ncols + kTQ - 1) / kTQ;
  size_t extra = 0, seg_bytes = 0;
  p.seg_off = p.seg_len = 0;
  p.nseg = kImSegSlots;
  bool staged = conv_staging(a, &p.seg_off, &p.seg_len, &seg_bytes);
  const int want_mt = (a.tile_n == 1 || a.tile_n == 2) ? a.tile_n : tc_row_tiles(h, qtiles_, 0);
  if (staged) {
    // the ring of planes is as deep as shared memory allows without giving up the second row tile (which halves the
    // tile-building work per output); without room for even two slots the planes are read from global memory
    staged = false;
    for (int n = kImSegSlots; n >= 2 && !staged; --n) {
      int s_ = 0, r_ = 0;
      if (tc_rings(h, want_mt, &s_, &r_, n * seg_bytes) && (want_mt == 1 || s_ >= 3)) { p.nseg = n; staged = true; }
    }
  }
  extra = staged ? p.nseg * seg_bytes : 0;
  p.seg_bytes = (uint32_t)seg_bytes;
  p.mt = want_mt;
  p.mtiles = (int)h->tc_mtiles;
  if (!tc_rings(h, p.mt, &p.nstages, &p.nrec, extra)) { p.mt = 1; tc_rings(h, 1, &p.nstages, &p.nrec, extra); }
  p.stage_bytes = (uint32_t)tc_stage_bytes(p.mt);
  p.rec_stride = (uint32_t)tc_rec_stride(h);
  p.spin_limit = 1u << 20;
  p.a = a;

  p.in_elems = a.conv ? a.ncols / ((int64_t)a.OH * a.OW) * a.C * a.H * a.W : 0;
  // Split over K when the grid would leave most of the GPU idle (small pixel or column counts): several thread
  // blocks share an output tile, each takes a run of K tiles and adds its partial sums into an fp32 scratch that the
  // handle owns (grown on first use), and a second pass applies bias, activation and the output layout.
  p.ksplit = 1; p.kt_per = p.nkt; p.acc = nullptr;
  {
    const int64_t blocks = qtiles_ * ((h->tc_mtiles + p.mt - 1) / p.mt);
    const int sms = sm_count(h->device);
    // (measured on the VGG-16 layers: worth it from about 16 K tiles per block; with fewer, clearing the scratch,
    // the reductions into it and the second pass cost more than the shorter K loop saves)
    int want = (int)std::min<int64_t>(16, sms / std::max<int64_t>(blocks, 1));
    want = std::min(want, p.nkt / 4);  // at least four K tiles per part
    const size_t need = (size_t)h->M * (size_t)a.ncols * 4;
    if (want >= 2 && p.nkt >= 16 && blocks * 2 <= sms && need <= ((size_t)1 << 30)) {
      // the scratch is reserved ahead of time (grim_bcr_reserve); without it, or when it is too small, the multiply runs unsplit
      if (h->d_tc_acc && h->tc_acc_bytes >= need) {
        p.kt_per = (p.nkt + want - 1) / want;
        p.ksplit = (p.nkt + p.kt_per - 1) / p.kt_per;
        p.acc = h->d_tc_acc;
        if (p.ksplit < 2) { p.ksplit = 1; p.kt_per = p.nkt; p.acc = nullptr; }
        else if (cudaMemsetAsync(p.acc, 0, need, s) != cudaSuccess) return GRIM_ERR_CUDA;
      }
    }
  }
  auto finalize = [&]() -> grim_status_t {
    if (p.ksplit <= 1) return GRIM_OK;
    const int64_t total = (int64_t)h->M * a.ncols;
    const int blocks = (int)std::min<int64_t>((total + 255) / 256, (int64_t)sm_count(h->device) * 8);
    tc_finalize_kernel<<<blocks, 256, 0, s>>>(p.acc, a.ncols, (int)h->M, a.bias, a.relu, a.Y, a.y_dtype, a.y_sr, a.conv,
                                              (int64_t)a.OH * a.OW);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? GRIM_OK : GRIM_ERR_CUDA;
  };
  CUtensorMap tm;
  memset(&tm, 0, sizeof(tm));
  if (a.conv) {
    const bool bulk = ((int64_t)a.OH * a.OW) % 8 == 0;
    auto kern = staged ? (bulk ? (h->bh == 4 ? bcr_tc_kernel<4, 2> : (h->bh == 8 ? bcr_tc_kernel<8, 2> : bcr_tc_kernel<16, 2>))
                               : (h->bh == 4 ? bcr_tc_kernel<4, 3> : (h->bh == 8 ? bcr_tc_kernel<8, 3> : bcr_tc_kernel<16, 3>)))
                       : (h->bh == 4 ? bcr_tc_kernel<4, 1> : (h->bh == 8 ? bcr_tc_kernel<8, 1> : bcr_tc_kernel<16, 1>));
    const size_t smem = tc_smem_need(h, p.mt, p.nstages, p.nrec, extra);
    if (ensure_dynamic_smem(reinterpret_cast<const void*>(kern), smem) != cudaSuccess) return GRIM_ERR_CUDA;
    dim3 grid((unsigned)((a.ncols + kTQ - 1) / kTQ), (unsigned)((h->tc_mtiles + p.mt - 1) / p.mt), (unsigned)p.ksplit);
    const cudaError_t le = launch_pdl(kern, grid, dim3(kTcConvThreads), smem, s, tm, p);
    count_launch();
    if (le != cudaSuccess) { cudaGetLastError(); return GRIM_ERR_CUDA; }
    return finalize();
  }
  const cuuint64_t dims[2] = {(cuuint64_t)a.ncols, (cuuint64_t)h->K};
  const cuuint64_t strides[1] = {(cuuint64_t)(a.x_sk * 2)};
  const cuuint32_t box[2] = {64, (cuuint32_t)kTK};
  const cuuint32_t estr[2] = {1, 1};
  if (encode_tiled_fn()(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(a.X), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return GRIM_ERR_CUDA;
  const size_t smem = tc_smem_need(h, p.mt, p.nstages, p.nrec);
  auto kern = h->bh == 4 ? bcr_tc_kernel<4, 0> : (h->bh == 8 ? bcr_tc_kernel<8, 0> : bcr_tc_kernel<16, 0>);
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), smem);
  if (e != cudaSuccess) return GRIM_ERR_CUDA;
  const int64_t qtiles = (a.ncols + kTQ - 1) / kTQ;
  const int64_t mtiles = (h->tc_mtiles + p.mt - 1) / p.mt;
  dim3 grid((unsigned)qtiles, (unsigned)mtiles, (unsigned)p.ksplit);
  const cudaError_t le = launch_pdl(kern, grid, dim3(kTcThreads), smem, s, tm, p);
  count_launch();
  if (le != cudaSuccess) { cudaGetLastError(); return GRIM_ERR_CUDA; }
  return finalize();
}

}  // namespace grim
