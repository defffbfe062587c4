// Paired tensor-core kernel (tcgen05, cta_group::2) for Y = W * X with bf16 operands, fp32 accumulation, large N
// (Section 3.1: every layer is a GEMM; Sections 4.3 - 4.4: compact storage that is expanded only on chip, every
// needed piece of data loaded once and reused).
//
// Two thread blocks on neighbouring SMs (a cluster of two) own 256 rows of W (schedule order) and 512 output
// columns.  Each block expands ITS 128 rows of a 64-wide K tile from the packed record into shared memory once,
// and that one expansion feeds 512 output columns: the pair issues tcgen05.mma with M = 256, N = 256 twice per
// 16-wide K step (two accumulators of 256 columns fill the 512 columns of tensor memory), each block supplying
// its half of W's rows and its half (128 columns) of every X operand.  Against a single block multiplying
// 128 x 256 per expansion, a block here reads half the X bytes per flop from shared memory and expands a quarter
// of the weight tiles per flop.
//
// Roles per block: warp 0 requests X tiles (TMA, 128-byte swizzle) and packed records (bulk copies); warp 1 and
// the last warp of the even block issue the multiplies, one accumulator each; twelve warps in three groups expand
// records (clear the tile, then one 2-byte store per kept value at the offset stored beside it: a few instructions
// per value, no index arithmetic); eight of them read the accumulators back at the end.  Everything the odd block
// produces is reported straight to the even block's barriers (its TMA loads count their bytes there, its warps
// arrive across the cluster).  All waits are bounded; tensor memory is released on every path.
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <cstring>

#include "grim_device.cuh"
#include "grim_im2col.cuh"
#include "grim_internal.h"

namespace grim {
namespace {

using namespace ptx;

constexpr int kWorkers = 12, kGroups = 3, kGroupWarps = kWorkers / kGroups, kGroupThreads = 32 * kGroupWarps;
constexpr int kIssueWarp2 = 2 + kWorkers;  // second issuing warp (the last warp of the block)
constexpr int kThreads = 64 + 32 * kWorkers + 32;
constexpr int kBuilders = 12, kBuildGroups = 3;  // convolution only: warps that build the X tile from the NCHW input
constexpr int kConvThreads = kThreads + 32 * kBuilders;
constexpr int kRows = 128;              // rows of W per block
constexpr int kColsPerBlock = 256;      // X columns staged per block per K tile
constexpr int kPairCols = 512;          // output columns per pair
constexpr int kK = 64;                  // K per stage
constexpr int kMaxStages = 4, kRecSlots = 8;
constexpr int kABytes = kRows * kK * 2;            // 16 KiB
constexpr int kBBytes = kColsPerBlock * kK * 2;    // 32 KiB
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kHdrBytes = 1024;
constexpr unsigned kTmemCols = 512;

struct Tc2Params {
  const RcStage* stage;
  const uint8_t* blob;
  const uint32_t* band_order;
  unsigned* status;
  int nbr, M, K, bh, bw, nkt, mtiles;
  int bh_shift, slots_per_tile, nstages, nrec;
  uint32_t rec_stride;
  unsigned spin_limit;
  int flags;
  int in_elems, seg_off, seg_len, nseg;  // convolution (see grim_im2col.cuh)
  uint32_t seg_bytes;
  SpmmArgs a;
};

// Shared-memory matrix descriptor: start address, leading / stride byte offsets (all without their 4 low bits),
// descriptor version 1, 128-byte swizzle.
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: fp32 accumulate, bf16 x bf16, A K-major, B N-major, M = 256 (both blocks), N = 256.
constexpr uint32_t kIdesc2 = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) | ((256u >> 3) << 17) | ((256u >> 4) << 24);

__device__ __forceinline__ void umma2_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(kIdesc2), "r"(accumulate)
      : "memory");
}
// Arrives on the barrier at this CTA-local address in both blocks of the pair once the multiplies issued so far
// have completed.
__device__ __forceinline__ void umma2_commit_both(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(smem_u32(bar)), "h"((unsigned short)3) : "memory");
}
// TMA tile load issued by either block of a pair whose bytes are counted on a barrier given as a shared::cluster
// address (here: the even block's).  No multicast: every block loads its own tile.
__device__ __forceinline__ void tma_load_2d_pair(void* dst, const void* tensor_map, int x, int y, uint32_t bar_cluster_addr) {
  asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(smem_u32(dst)), "l"(tensor_map), "r"(x), "r"(y), "r"(bar_cluster_addr) : "memory");
}
// Asks TMA to bring a tile into L2 only (no shared-memory destination, nothing to wait for).
__device__ __forceinline__ void tma_prefetch_2d(const void* tensor_map, int x, int y) {
  asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global [%0, {%1, %2}];" ::"l"(tensor_map), "r"(x), "r"(y) : "memory");
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

// CONV: 0 = X is a matrix (TMA tiles); 1, 2, 3 = implicit im2col, the X tiles are built on chip (grim_im2col.cuh).
template <int CONV>
__global__ void __launch_bounds__(CONV ? kConvThreads : kThreads, 1) bcr_tc2_kernel(const __grid_constant__ CUtensorMap tmX, const Tc2Params p) {
  extern __shared__ uint8_t smem_raw[];
  // tiles start on a 1 KiB boundary (the swizzle pattern repeats every 8 rows of 128 bytes); the offset from the
  // the launch that follows in the stream may start as SMs free up: it waits (griddepcontrol.wait) before it reads or
  // writes anything this launch touches
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // start of the block's shared memory is the same in both blocks, which the paired multiply relies on
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  // One barrier per stage IN THE EVEN BLOCK collects everything the multiplies of that stage need from both blocks:
  // the X tiles (one arrival of the even block's copy thread that announces the bytes of both blocks; the odd
  // block's TMA loads complete their bytes on this barrier too) and the expanded weight tiles (one arrival per
  // expansion warp of either block, the odd block's across the cluster).  The issuing threads wait once per stage
  // (under load every dependent shared-memory access costs a few hundred cycles) and nothing is relayed.
  uint64_t* ready = reinterpret_cast<uint64_t*>(smem);
  uint64_t* empty = ready + kMaxStages;                   // the pair's multiplies on a stage are done (set in both blocks)
  uint64_t* acc_done = empty + kMaxStages;                // all multiplies are complete (set in both blocks)
  uint64_t* rec_full = acc_done + 1;                      // a packed record has landed
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + 384);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + 388);
  uint32_t* s_meta = reinterpret_cast<uint32_t*>(smem + 512);  // [record slot] bytes of the record (0: the tile is empty)
  unsigned* s_done = reinterpret_cast<unsigned*>(smem + 640);  // [record slot] warps that have finished with it
  uint64_t* seg_full = reinterpret_cast<uint64_t*>(smem + 704);  // staged convolution: the planes of a K tile have landed
  uint64_t* seg_free = reinterpret_cast<uint64_t*>(smem + 768);  // ... and the builders are done with them
  uint8_t* stages = smem + kHdrBytes;
  uint8_t* recs = stages + (size_t)p.nstages * kStageBytes;
  uint8_t* segs = recs + (size_t)p.nrec * p.rec_stride;

  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
  const SpmmArgs& a = p.a;
  const uint32_t rank = cluster_ctarank();  // 0: issues the multiplies; 1: its partner
  const int tile = (int)blockIdx.x;          // 128-row tile of W (blockIdx.x = 2 * pair + rank)
  const bool has_tile = tile < p.mtiles;
  const int64_t q0 = (int64_t)blockIdx.y * kPairCols;   // first output column of the pair
  const int64_t qb = q0 + (int64_t)rank * kColsPerBlock;  // first X column this block stages
  const int ns = p.nstages, nr = p.nrec, nkt = p.nkt;

  if (tid == 0) {
    for (int s = 0; s < kMaxStages; ++s) {
      // matrix: the copy thread + the expansion warps of both blocks; convolution: expansion and builder warps
      mbar_init(ready + s, CONV ? 2 * kGroupWarps + 2 * kImBuildWarps : 1 + 2 * kGroupWarps);
      mbar_init(empty + s, 2);  // one arrival per issuing thread
      mbar_init(seg_full + s, CONV == 3 ? 32u : 1u);  // completed by byte counts, or by the copy warp's 32 lanes
      mbar_init(seg_free + s, kImBuildWarps);
    }
    for (int s = 0; s < kRecSlots; ++s) {
      mbar_init(rec_full + s, 1);
      s_done[s] = 0;
    }
    mbar_init(acc_done, 2);
    *s_abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync_all();  // both blocks' barriers exist before either signals the other
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *s_tmem;
  // (programmatic dependent launch) whatever earlier launches in the stream wrote - X, a cleared scratch or Y - is
  // complete and visible from here on; up to here only the packed matrix and this block's own shared memory were touched
  asm volatile("griddepcontrol.wait;" ::: "memory");

  // Requests the packed record of K tile k into record slot rs; one thread.
  auto request_record = [&](int k, int rs) {
    uint32_t bytes = 0, off = 0;
    if (has_tile) {
      const RcStage se = p.stage[(int64_t)tile * p.nkt + k];
      bytes = se.bytes; off = se.off16;
    }
    s_meta[rs] = bytes;
    mbar_arrive_expect_tx(rec_full + rs, bytes);
    if (bytes) bulk_load(recs + (size_t)rs * p.rec_stride, p.blob + (size_t)off * 16, bytes, rec_full + rs);
  };

  bool failed = false;
  int fail_site = 0;
  Im2colCtx im;
  if (CONV) {
    im.a = &p.a; im.K = p.K; im.in_elems = p.in_elems; im.seg_off = p.seg_off; im.seg_len = p.seg_len; im.nseg = p.nseg;
    im.seg_bytes = p.seg_bytes; im.q0 = qb; im.nkt = nkt; im.kbase = 0; im.ns = ns; im.stages = stages;
    im.stage_bytes = kStageBytes; im.b_off = kABytes; im.segs = segs; im.empty = empty; im.seg_full = seg_full;
    im.seg_free = seg_free; im.built = ready; im.built_rank = rank == 0 ? -1 : 0; im.cluster_waits = true;
    im.spin_limit = p.spin_limit; im.s_abort = s_abort;
  }
  if (warp == 0) {
    // ------------------------------------------------------------------ copies
    if (CONV) {
      if (lane == 0)
        for (int rk = 0; rk < nr && rk < nkt; ++rk) request_record(rk, rk);
      __syncwarp();
      if (CONV >= 2 && !conv_copy_planes<CONV>(im, lane)) failed = true, fail_site = 1;
    } else if (lane == 0) {
      for (int rk = 0; rk < nr && rk < nkt; ++rk) request_record(rk, rk);
      // 64-column boxes wholly past the last column are not requested (their part of the tile keeps whatever it
      // held; the accumulator columns computed from it are never stored)
      auto boxes_from = [&](int64_t first) {
        const int64_t n = (a.ncols - first + 63) / 64;
        return (int)(n < 0 ? 0 : (n > kColsPerBlock / 64 ? kColsPerBlock / 64 : n));
      };
      const int nbox = boxes_from(qb);
      const unsigned pair_bytes = (unsigned)((boxes_from(q0) + boxes_from(q0 + kColsPerBlock)) * 64 * kK * 2);
      // the even block's barrier, as seen from this block
      uint32_t ready0;
      asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ready0) : "r"(smem_u32(ready)), "r"(0));
      // X tiles are asked into L2 kPrefetch K tiles ahead of their load into shared memory: all row pairs walk K in
      // step, so without it every load of the ring would wait for HBM, and the ring is only a few tiles deep
      constexpr int kPrefetch = 8;
      for (int kt = 0; kt < kPrefetch && kt < nkt; ++kt)
        for (int i = 0; i < nbox; ++i) tma_prefetch_2d(&tmX, (int)qb + 64 * i, kt * kK);
      for (int kt = 0; kt < nkt; ++kt) {
        const int slot = kt % ns;
        if (kt + kPrefetch < nkt)
          for (int i = 0; i < nbox; ++i) tma_prefetch_2d(&tmX, (int)qb + 64 * i, (kt + kPrefetch) * kK);
        if (kt >= ns && !mbar_wait<true>(empty + slot, (unsigned)((kt / ns - 1) & 1), p.spin_limit, s_abort, 20)) { failed = true, fail_site = 1; break; }
        uint8_t* bt = stages + (size_t)slot * kStageBytes + kABytes;
        if (rank == 0) mbar_arrive_expect_tx(ready + slot, pair_bytes);
#pragma unroll
        for (int i = 0; i < kColsPerBlock / 64; ++i)
          if (i < nbox) tma_load_2d_pair(bt + i * (64 * kK * 2), &tmX, (int)qb + 64 * i, kt * kK, ready0 + (uint32_t)slot * 8u);
      }
    }
  } else if (warp == 1 || warp == kIssueWarp2) {
    if (lane == 0 && rank == 0 && !((p.flags & 1) && warp != 1)) {
      // ------------------------------------------------------------------ tensor core (even block)
      // Two issuing threads, one per accumulator.  Issuing is asynchronous but the queue is short, so a thread is
      // held while its multiplies wait their turn; its poll of the next stage's barrier (a few hundred cycles
      // while the tensor core reads shared memory flat out) then overlaps the other thread's multiplies.
      // The barrier of the NEXT stage is tested (without blocking) before this stage's multiplies are issued and the
      // answer is read after them, so that in the steady state, where operands are in place well ahead, no
      // shared-memory round trip sits between the multiplies of consecutive stages.
      const int acc = warp == 1 ? 0 : 1;
      bool have = false;
      for (int kt = 0; kt < nkt; ++kt) {
        const int slot = kt % ns;
        const unsigned par = (unsigned)((kt / ns) & 1);
        if (!have && !mbar_wait<true>(ready + slot, par, p.spin_limit << 3, s_abort, 0)) { failed = true, fail_site = 2; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        have = kt + 1 < nkt && mbar_test_wait_cluster(ready + (kt + 1) % ns, (unsigned)(((kt + 1) / ns) & 1));
        const uint32_t a_addr = smem_u32(stages + (size_t)slot * kStageBytes);
        const uint32_t b_addr = a_addr + kABytes;
        for (int ac = (p.flags & 1) ? 0 : acc; ac <= ((p.flags & 1) ? 1 : acc); ++ac) {
#pragma unroll
          for (int s = 0; s < kK / 16; ++s) {
            // A: K-major, rows 128 bytes apart, 8-row groups 1 KiB apart; 16 K-elements = 32 bytes further on
            const uint64_t ad = smem_desc(a_addr + s * 32, 16, 1024);
            // B: N-major, 64-column panels 8 KiB apart, 8-row K groups 1 KiB apart; 16 K-rows = 2 KiB further on;
            // accumulator `ac` takes panels 2 * ac and 2 * ac + 1 of each block
            const uint64_t bd = smem_desc(b_addr + ac * (2 * 64 * kK * 2) + s * 2048, 64 * kK * 2, 1024);
            umma2_bf16(tmem_base + (uint32_t)ac * 256u, ad, bd, (kt > 0 || s > 0) ? 1u : 0u);
          }
        }
        umma2_commit_both(empty + slot);  // arrives in both blocks when this thread's multiplies have read their operands
        if (p.flags & 1) umma2_commit_both(empty + slot);
      }
      if (!failed) umma2_commit_both(acc_done);
      if (!failed && (p.flags & 1)) umma2_commit_both(acc_done);
    }
  } else if (CONV && warp > kIssueWarp2) {
    // ------------------------------------------------------------------ implicit im2col: this block's 256 pixels
    const int bgrp = (warp - kIssueWarp2 - 1) / kImBuildWarps;
    const int bt = tid - kThreads - bgrp * (32 * kImBuildWarps);
    if (!conv_build_tiles<CONV>(im, bgrp, kBuildGroups, bt, lane, fail_site)) failed = true;
  } else {
    // ------------------------------------------------------------------ expansion of the packed weights
    const int grp = (warp - 2) / kGroupWarps;
    const int wt = tid - 64 - grp * kGroupThreads;
    for (int kt = grp; kt < nkt; kt += kGroups) {
      const int slot = kt % ns, rs = kt % nr;
      if (kt >= ns && !__all_sync(0xffffffffu, mbar_wait<true>(empty + slot, (unsigned)((kt / ns - 1) & 1), p.spin_limit, s_abort, 32))) { failed = true, fail_site = 4; break; }
      if (!__all_sync(0xffffffffu, mbar_wait(rec_full + rs, (unsigned)((kt / nr) & 1), p.spin_limit, s_abort))) { failed = true, fail_site = 5; break; }
      expand_scatter<kGroupThreads>(smem_u32(recs + (size_t)rs * p.rec_stride), s_meta[rs],
                                    smem_u32(stages + (size_t)slot * kStageBytes), wt, 1 + grp);
      fence_proxy_async();  // generic-proxy writes -> visible to the tensor core
      __syncwarp();
      if (lane == 0) {
        if (rank == 0) mbar_arrive(ready + slot);
        else mbar_arrive_remote(ready + slot, 0);
        // the last warp of the group to finish with the record frees its slot: it requests the record that uses
        // the slot next (every read of the old record precedes that warp's count)
        if (atomicAdd(s_done + rs, 1u) == (unsigned)kGroupWarps - 1u) {
          s_done[rs] = 0;
          if (kt + nr < nkt) request_record(kt + nr, rs);
        }
      }
    }
    // ------------------------------------------------------------------ epilogue
    const bool epilogue_warp = warp - 2 < 8;  // two warps per quarter of the tensor-memory lanes, one per accumulator
    if (epilogue_warp && !__any_sync(0xffffffffu, failed)) {
      if (!__all_sync(0xffffffffu, mbar_wait<true>(acc_done, 0, p.spin_limit, s_abort))) failed = true, fail_site = 6;
    }
    if (epilogue_warp && !__any_sync(0xffffffffu, failed)) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int quarter = warp & 3;
      const int trow = quarter * 32 + lane;
      const int acc = (warp - 2) >> 2;
      const int pos = tile * p.slots_per_tile + (trow >> p.bh_shift);
      int64_t row = -1;
      if (has_tile && pos < p.nbr) row = (int64_t)p.band_order[pos] * p.bh + (trow & (p.bh - 1));
      const bool row_ok = row >= 0 && row < p.M;
      const float bias = (row_ok && a.bias) ? __ldg(a.bias + row) : 0.f;
      const int row_i = row_ok ? (int)row : -1;
      for (int cb = 0; cb < 8; ++cb) {
        uint32_t v[32];
        tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * 256 + cb * 32), v);
        // accumulator column c came from X column 256 * (c / 128) + 128 * acc + c % 128 of the pair's 512
        const int c = cb * 32;
        const int64_t q = q0 + 256 * (c >> 7) + 128 * acc + (c & 127);
        if (q >= a.ncols) continue;  // (uniform over the warp)
        float t[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          t[i] = __uint_as_float(v[i]) + bias;
          if (a.relu) t[i] = fmaxf(t[i], 0.f);
        }
        // Through shared memory, so that a warp instruction writes one row's 32 consecutive columns (a whole
        // 128-byte line) instead of 16 bytes of 32 different rows: stage[lane][i] with a row pitch of 33 words is free
        // of bank conflicts both ways.  (The stage buffers are free: all multiplies have completed.)
        float* stg = reinterpret_cast<float*>(stages) + (warp - 2) * (33 * 32);
#pragma unroll
        for (int i = 0; i < 32; ++i) stg[lane * 33 + i] = t[i];
        __syncwarp();
        // element (row r, column qq) of the output: matrix Y[r * y_sr + qq]; convolution (NCHW, qq = image * OH*OW +
        // pixel): out[(image * M + r) * OH*OW + pixel] - per column a base offset, per row a stride
        const int64_t ohw = CONV ? (int64_t)a.OH * a.OW : 1;
        const int64_t rstride = CONV ? ohw : a.y_sr;
        auto col_base = [&](int64_t qq) -> int64_t {
          if (!CONV) return qq;
          const int64_t img = qq / ohw;
          return img * p.M * ohw + (qq - img * ohw);
        };
        if (a.y_dtype == GRIM_F32) {
          float* Y = static_cast<float*>(a.Y);
          const bool col_ok = q + lane < a.ncols;
          const int64_t base = col_base(q + lane);
#pragma unroll 8
          for (int r = 0; r < 32; ++r) {
            const int rr = __shfl_sync(0xffffffffu, row_i, r);
            const float val = stg[r * 33 + lane];
            if (rr >= 0 && col_ok) Y[(int64_t)rr * rstride + base] = val;
          }
        } else {
          // bf16: a lane takes two neighbouring columns, a warp instruction two rows of 64 bytes each
          __nv_bfloat16* Y = static_cast<__nv_bfloat16*>(a.Y);
          const int c2 = (lane & 15) * 2;
          const int64_t base0 = col_base(q + c2), base1 = col_base(q + c2 + 1);
          const bool ok0 = q + c2 < a.ncols, ok1 = q + c2 + 1 < a.ncols;
#pragma unroll 8
          for (int r2 = 0; r2 < 32; r2 += 2) {
            const int r = r2 + (lane >> 4);
            const int rr = __shfl_sync(0xffffffffu, row_i, r);
            const float v0 = stg[r * 33 + c2], v1 = stg[r * 33 + c2 + 1];
            if (rr < 0 || !ok0) continue;
            __nv_bfloat16* y = Y + (int64_t)rr * rstride + base0;
            if (ok1 && base1 == base0 + 1 && (reinterpret_cast<uintptr_t>(y) & 3) == 0) {
              *reinterpret_cast<__nv_bfloat162*>(y) = __floats2bfloat162_rn(v0, v1);
            } else {
              y[0] = __float2bfloat16_rn(v0);
              if (ok1) Y[(int64_t)rr * rstride + base1] = __float2bfloat16_rn(v1);
            }
          }
        }
        __syncwarp();
      }
    }
  }

  if (__any_sync(0xffffffffu, failed)) {
    *s_abort = 1;
    if (fail_site) atomicOr(p.status, (unsigned)GRIM_ERR_TIMEOUT | (1u << (8 + fail_site)));
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync_all();  // neither block leaves (or frees tensor memory) while the other may still use its memory
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
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

size_t rec_stride_of(const grim_bcr* h) { return ((size_t)h->td_max_rec + 127) & ~size_t(127); }
// extra: bytes besides the operand tiles and the records (the ring of staged input planes of the convolution)
size_t smem_need(const grim_bcr* h, int stages, int nrec, size_t extra = 0) {
  return 1024 + kHdrBytes + (size_t)stages * kStageBytes + (size_t)nrec * rec_stride_of(h) + extra;
}
// As many tile slots as fit (at least as many as expansion groups, so that no wait is ever more than one barrier
// phase behind), then as many record slots as are left, at least as many as tile slots.
bool rings(const grim_bcr* h, int* stages, int* nrec, size_t extra = 0) {
  for (int s = kMaxStages; s >= kGroups; --s)
    for (int r = kRecSlots; r >= s; --r)
      if (smem_need(h, s, r, extra) <= 227 * 1024) { *stages = s; *nrec = r; return true; }
  return false;
}

}  // namespace

bool tc2_path_supported(const grim_bcr* h, const SpmmArgs& a) {
  if (h->device < 0 || h->dtype != GRIM_BF16 || !h->d_td_stage || !h->d_status || h->td_max_rec == 0) return false;
  if (a.x_dtype != GRIM_BF16 || reinterpret_cast<uintptr_t>(a.X) % 16 != 0) return false;
  if (a.conv) {
    if (!conv_tiles_supported(a)) return false;
  } else if (a.x_sq != 1 || a.y_sq != 1 || (a.x_sk * 2) % 16 != 0) {
    return false;
  }
  if (a.ncols <= 0 || a.ncols > (int64_t(1) << 31) - kPairCols) return false;
  if ((a.ncols + kPairCols - 1) / kPairCols > 65535) return false;
  int s = 0, r = 0;
  if (!rings(h, &s, &r)) return false;
  return encode_tiled_fn() != nullptr;
}

grim_status_t launch_spmm_tc2(const grim_bcr* h, const SpmmArgs& a, cudaStream_t s) {
  if (!tc2_path_supported(h, a)) return GRIM_ERR_UNSUPPORTED;
  Tc2Params p;
  p.stage = h->d_td_stage; p.blob = h->d_td_blob; p.band_order = h->d_band_order; p.status = h->d_status;
  p.nbr = (int)h->nbr; p.M = (int)h->M; p.K = (int)h->K; p.bh = h->bh; p.bw = h->bw; p.nkt = (int)h->tc_ktiles;
  p.mtiles = (int)h->tc_mtiles;
  p.bh_shift = h->bh == 4 ? 2 : (h->bh == 8 ? 3 : 4);
  p.slots_per_tile = kRows / h->bh;
  p.rec_stride = (uint32_t)rec_stride_of(h);
  p.spin_limit = 1u << 20;
  p.flags = a.conv ? 0 : a.tile_n;
  p.a = a;
  // convolution: stage the input planes in shared memory when their size allows and a ring of at least two
  // segments fits beside three tile slots; otherwise the builders read them from global memory
  size_t seg_bytes = 0, extra = 0;
  int mode = 0;
  p.in_elems = 0; p.seg_off = p.seg_len = 0; p.nseg = kImSegSlots; p.seg_bytes = 0;
  if (a.conv) {
    mode = 1;
    p.in_elems = (int)(a.ncols / ((int64_t)a.OH * a.OW) * a.C * a.H * a.W);
    if (conv_staging(a, &p.seg_off, &p.seg_len, &seg_bytes)) {
      for (int n = kImSegSlots; n >= 2 && mode == 1; --n) {
        int s_ = 0, r_ = 0;
        if (rings(h, &s_, &r_, n * seg_bytes)) { p.nseg = n; mode = ((int64_t)a.OH * a.OW) % 8 == 0 ? 2 : 3; }
      }
    }
    if (mode > 1) { extra = p.nseg * seg_bytes; p.seg_bytes = (uint32_t)seg_bytes; }
  }
  if (!rings(h, &p.nstages, &p.nrec, extra)) return GRIM_ERR_UNSUPPORTED;
  CUtensorMap tm;
  memset(&tm, 0, sizeof(tm));
  if (!a.conv) {
    const cuuint64_t dims[2] = {(cuuint64_t)a.ncols, (cuuint64_t)h->K};
    const cuuint64_t strides[1] = {(cuuint64_t)(a.x_sk * 2)};
    const cuuint32_t box[2] = {64, (cuuint32_t)kK};
    const cuuint32_t estr[2] = {1, 1};
    if (encode_tiled_fn()(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(a.X), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return GRIM_ERR_CUDA;
  }
  const size_t smem = smem_need(h, p.nstages, p.nrec, extra);
  using Kern = void (*)(const CUtensorMap, const Tc2Params);
  const Kern kerns[4] = {bcr_tc2_kernel<0>, bcr_tc2_kernel<1>, bcr_tc2_kernel<2>, bcr_tc2_kernel<3>};
  Kern kern = kerns[mode];
  if (ensure_dynamic_smem(reinterpret_cast<const void*>(kern), smem) != cudaSuccess) return GRIM_ERR_CUDA;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(2 * ((h->tc_mtiles + 1) / 2)), (unsigned)((a.ncols + kPairCols - 1) / kPairCols), 1);
  cfg.blockDim = dim3(a.conv ? kConvThreads : kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // may begin while the launch before it still runs
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tm, p);
  count_launch();
  return e == cudaSuccess ? GRIM_OK : GRIM_ERR_CUDA;
}

}  // namespace grim
