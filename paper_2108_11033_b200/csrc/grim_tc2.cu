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
// Roles per block: warp 0 requests X tiles (TMA, 128-byte swizzle) and packed records (bulk copies); warp 1 of
// the even block issues the multiplies, warp 1 of the odd block tells the even block when its operands are in
// place; twelve warps in three groups expand records, a thread building 16-byte pieces of the tile in registers
// from one block descriptor and a run of consecutive values (no clearing pass, no scattered 2-byte stores); eight
// of them read the accumulators back at the end.  All waits are bounded; tensor memory is released on every path.
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <cstring>

#include "grim_device.cuh"
#include "grim_internal.h"

namespace grim {
namespace {

using namespace ptx;

constexpr int kWorkers = 12, kGroups = 3, kGroupWarps = kWorkers / kGroups, kGroupThreads = 32 * kGroupWarps;
constexpr int kThreads = 64 + 32 * kWorkers;
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

// One band's share of a thread's piece: block-local row `lr` of a band with descriptor (colmask of the thread's
// segment, rowmask, first value), `kc` kept columns in the whole block, `prefix` kept columns of the block in front of
// the piece, `sub` the piece's 8 column bits.  Returns the 8 bf16 values (zeros where nothing is kept) as 4 words.
__device__ __forceinline__ void piece_of_row(uint32_t vals_s, uint32_t rowmask, uint32_t lr, uint32_t val_off, uint32_t kc,
                                             uint32_t prefix, uint32_t sub, const uint32_t (&off2)[8], uint32_t (&w)[4]) {
  const bool kept = (rowmask >> lr) & 1u;
  const uint32_t a = __popc(rowmask & ((1u << lr) - 1u));
  const uint32_t base = vals_s + 2u * (val_off + a * kc + prefix);
  uint32_t v[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    unsigned short h = 0;
    // not volatile: the loads of all eight rows may be issued together; their address depends on the descriptor
    // loads, which are ordered after the wait for the record
    if (kept && ((sub >> e) & 1u)) asm("ld.shared.u16 %0, [%1];" : "=h"(h) : "r"(base + off2[e]));
    v[e] = h;
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) w[i] = v[2 * i] | (v[2 * i + 1] << 16);
}

// Expands one packed record into the 128 x 64 bf16 weight tile at shared address a_s (K-major rows of 128 bytes,
// 16-byte pieces XOR-ed with the row's low three bits: the tensor core's 128-byte swizzle).  Called by the
// kGroupThreads threads of one group; thread wt owns piece j = wt & 7 (columns 8j .. 8j + 7) of rows 8 * (wt >> 3) ..
// + 7.  rec_s = shared address of the record, or 0 when the tile keeps nothing (zeros are written).
template <int BH, int BW>
__device__ __forceinline__ void expand_tile(uint32_t rec_s, uint32_t a_s, int wt) {
  constexpr int SEG = BW < kTdSeg ? BW : kTdSeg;  // columns per descriptor
  constexpr int NSEG = kK / SEG;                  // descriptors per band
  constexpr int BANDS = kRows / BH;
  const uint32_t j = (uint32_t)wt & 7u, rg = (uint32_t)wt >> 3;
  const uint32_t seg = (8u * j) / SEG, shift = (8u * j) % SEG;
  const uint32_t vals_s = rec_s + (uint32_t)(BANDS * NSEG * sizeof(TdDesc));
  constexpr int NB = BH == 4 ? 2 : 1;  // bands met by the thread's 8 rows
  uint32_t colmask[NB], rowmask[NB], val_off[NB], kc[NB], prefix[NB], sub[NB];
  uint32_t off2[NB][8];
#pragma unroll
  for (int b = 0; b < NB; ++b) {
    const uint32_t band = BH == 4 ? 2u * rg + b : (BH == 8 ? rg : rg >> 1);
    colmask[b] = rowmask[b] = val_off[b] = kc[b] = prefix[b] = 0u;
    if (rec_s) {
      const uint32_t d_s = rec_s + (band * NSEG + seg) * (uint32_t)sizeof(TdDesc);
      uint32_t c0, m0;
      asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(c0), "=r"(m0) : "r"(d_s));
      colmask[b] = c0; rowmask[b] = m0 & 0xFFFFu; val_off[b] = m0 >> 16;
      kc[b] = __popc(c0);
      if (BW == 64) {  // the other half of the block: its kept columns count towards the row length (and, for the
                       // upper half, towards the columns in front of the piece)
        uint32_t c1;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(c1) : "r"(d_s ^ (uint32_t)sizeof(TdDesc)));
        kc[b] += __popc(c1);
        if (seg & 1u) prefix[b] = __popc(c1);
      }
      prefix[b] += __popc(c0 & ((1u << shift) - 1u));
    }
    sub[b] = (colmask[b] >> shift) & 0xFFu;
#pragma unroll
    for (int e = 0; e < 8; ++e) off2[b][e] = 2u * __popc(sub[b] & ((1u << e) - 1u));
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int b = BH == 4 ? (i >> 2) : 0;
    const uint32_t lr = BH == 4 ? (uint32_t)(i & 3) : (BH == 8 ? (uint32_t)i : 8u * (rg & 1u) + (uint32_t)i);
    uint32_t w[4];
    piece_of_row(vals_s, rowmask[b], lr, val_off[b], kc[b], prefix[b], sub[b], off2[b], w);
    const uint32_t row = 8u * rg + (uint32_t)i;
    sts128(a_s + row * 128u + ((j ^ (uint32_t)i) << 4), w[0], w[1], w[2], w[3]);
  }
}

template <int BH, int BW>
__global__ void __launch_bounds__(kThreads, 1) bcr_tc2_kernel(const __grid_constant__ CUtensorMap tmX, const Tc2Params p) {
  extern __shared__ uint8_t smem_raw[];
  // tiles start on a 1 KiB boundary (the swizzle pattern repeats every 8 rows of 128 bytes); the offset from the
  // start of the block's shared memory is the same in both blocks, which the paired multiply relies on
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full = reinterpret_cast<uint64_t*>(smem);   // this block's X tile of a stage has landed
  uint64_t* ready = full + kMaxStages;                    // this block's expanded weight tile of a stage is written
  uint64_t* empty = ready + kMaxStages;                   // the pair's multiplies on a stage are done (set in both blocks)
  uint64_t* peer_ok = empty + kMaxStages;                 // even block only: the odd block's operands of a stage are in place
  uint64_t* acc_done = peer_ok + kMaxStages;              // all multiplies are complete (set in both blocks)
  uint64_t* rec_full = acc_done + 1;                      // a packed record has landed
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(smem + 384);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + 388);
  uint32_t* s_meta = reinterpret_cast<uint32_t*>(smem + 512);  // [record slot] bytes of the record (0: the tile is empty)
  unsigned* s_done = reinterpret_cast<unsigned*>(smem + 640);  // [record slot] warps that have finished with it
  uint8_t* stages = smem + kHdrBytes;
  uint8_t* recs = stages + (size_t)p.nstages * kStageBytes;

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
      mbar_init(full + s, 1);
      mbar_init(ready + s, kGroupWarps);
      mbar_init(empty + s, 1);
      mbar_init(peer_ok + s, 1);
    }
    for (int s = 0; s < kRecSlots; ++s) {
      mbar_init(rec_full + s, 1);
      s_done[s] = 0;
    }
    mbar_init(acc_done, 1);
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
  if (warp == 0) {
    // ------------------------------------------------------------------ copies
    if (lane == 0) {
      for (int rk = 0; rk < nr && rk < nkt; ++rk) request_record(rk, rk);
      // 64-column boxes wholly past the last column are not requested (their part of the tile keeps whatever it
      // held; the accumulator columns computed from it are never stored)
      int nbox = (int)((a.ncols - qb + 63) / 64);
      nbox = nbox < 0 ? 0 : (nbox > kColsPerBlock / 64 ? kColsPerBlock / 64 : nbox);
      for (int kt = 0; kt < nkt; ++kt) {
        const int slot = kt % ns;
        if (kt >= ns && !mbar_wait<true>(empty + slot, (unsigned)((kt / ns - 1) & 1), p.spin_limit, s_abort)) { failed = true, fail_site = 1; break; }
        uint8_t* bt = stages + (size_t)slot * kStageBytes + kABytes;
        mbar_arrive_expect_tx(full + slot, (unsigned)(nbox * 64 * kK * 2));
#pragma unroll
        for (int i = 0; i < kColsPerBlock / 64; ++i)
          if (i < nbox) tma_load_2d(bt + i * (64 * kK * 2), &tmX, (int)qb + 64 * i, kt * kK, full + slot);
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      // ------------------------------------------------------------------ tensor core (even block)
      for (int kt = 0; kt < nkt; ++kt) {
        const int slot = kt % ns;
        const unsigned par = (unsigned)((kt / ns) & 1);
        if (!mbar_wait(full + slot, par, p.spin_limit, s_abort) || !mbar_wait(ready + slot, par, p.spin_limit, s_abort) ||
            !mbar_wait<true>(peer_ok + slot, par, p.spin_limit, s_abort)) { failed = true, fail_site = 2; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t a_addr = smem_u32(stages + (size_t)slot * kStageBytes);
        const uint32_t b_addr = a_addr + kABytes;
#pragma unroll
        for (int acc = 0; acc < 2; ++acc) {
#pragma unroll
          for (int s = 0; s < kK / 16; ++s) {
            // A: K-major, rows 128 bytes apart, 8-row groups 1 KiB apart; 16 K-elements = 32 bytes further on
            const uint64_t ad = smem_desc(a_addr + s * 32, 16, 1024);
            // B: N-major, 64-column panels 8 KiB apart, 8-row K groups 1 KiB apart; 16 K-rows = 2 KiB further on;
            // accumulator `acc` takes panels 2 * acc and 2 * acc + 1 of each block
            const uint64_t bd = smem_desc(b_addr + acc * (2 * 64 * kK * 2) + s * 2048, 64 * kK * 2, 1024);
            umma2_bf16(tmem_base + (uint32_t)acc * 256u, ad, bd, (kt > 0 || s > 0) ? 1u : 0u);
          }
        }
        umma2_commit_both(empty + slot);  // arrives in both blocks when the multiplies above have read their operands
      }
      if (!failed) umma2_commit_both(acc_done);
    } else if (lane == 0) {
      // ------------------------------------------------------------------ odd block: report operands in place
      for (int kt = 0; kt < nkt; ++kt) {
        const int slot = kt % ns;
        const unsigned par = (unsigned)((kt / ns) & 1);
        if (!mbar_wait(full + slot, par, p.spin_limit, s_abort) || !mbar_wait(ready + slot, par, p.spin_limit, s_abort)) { failed = true, fail_site = 3; break; }
        mbar_arrive_remote(peer_ok + slot, 0);
      }
    }
  } else {
    // ------------------------------------------------------------------ expansion of the packed weights
    const int grp = (warp - 2) / kGroupWarps;
    const int wt = tid - 64 - grp * kGroupThreads;
    for (int kt = grp; kt < nkt; kt += kGroups) {
      const int slot = kt % ns, rs = kt % nr;
      if (kt >= ns && !__all_sync(0xffffffffu, mbar_wait<true>(empty + slot, (unsigned)((kt / ns - 1) & 1), p.spin_limit, s_abort))) { failed = true, fail_site = 4; break; }
      if (!__all_sync(0xffffffffu, mbar_wait(rec_full + rs, (unsigned)((kt / nr) & 1), p.spin_limit, s_abort))) { failed = true, fail_site = 5; break; }
      const uint32_t rec_s = s_meta[rs] ? smem_u32(recs + (size_t)rs * p.rec_stride) : 0u;
      expand_tile<BH, BW>(rec_s, smem_u32(stages + (size_t)slot * kStageBytes), wt);
      fence_proxy_async();  // generic-proxy writes -> visible to the tensor core
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(ready + slot);
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
      if (has_tile && pos < p.nbr) row = (int64_t)p.band_order[pos] * p.bh + (trow & (BH - 1));
      const bool row_ok = row >= 0 && row < p.M;
      const float bias = (row_ok && a.bias) ? __ldg(a.bias + row) : 0.f;
      for (int cb = 0; cb < 8; ++cb) {
        uint32_t v[32];
        tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * 256 + cb * 32), v);
        // accumulator column c came from X column 256 * (c / 128) + 128 * acc + c % 128 of the pair's 512
        const int c = cb * 32;
        const int64_t q = q0 + 256 * (c >> 7) + 128 * acc + (c & 127);
        if (!row_ok || q >= a.ncols) continue;
        float t[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          t[i] = __uint_as_float(v[i]) + bias;
          if (a.relu) t[i] = fmaxf(t[i], 0.f);
        }
        const bool full_chunk = q + 31 < a.ncols;
        const int64_t off0 = row * a.y_sr + q;
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
size_t smem_need(const grim_bcr* h, int stages, int nrec) {
  return 1024 + kHdrBytes + (size_t)stages * kStageBytes + (size_t)nrec * rec_stride_of(h);
}
// As many tile slots as fit (at least as many as expansion groups, so that no wait is ever more than one barrier
// phase behind), then as many record slots as are left, at least as many as tile slots.
bool rings(const grim_bcr* h, int* stages, int* nrec) {
  for (int s = kMaxStages; s >= kGroups; --s)
    for (int r = kRecSlots; r >= s; --r)
      if (smem_need(h, s, r) <= 227 * 1024) { *stages = s; *nrec = r; return true; }
  return false;
}

using Tc2Kernel = void (*)(const CUtensorMap, const Tc2Params);
Tc2Kernel kernel_for(int bh, int bw) {
  if (bh == 4) return bw == 16 ? bcr_tc2_kernel<4, 16> : (bw == 32 ? bcr_tc2_kernel<4, 32> : bcr_tc2_kernel<4, 64>);
  if (bh == 8) return bw == 16 ? bcr_tc2_kernel<8, 16> : (bw == 32 ? bcr_tc2_kernel<8, 32> : bcr_tc2_kernel<8, 64>);
  return bw == 16 ? bcr_tc2_kernel<16, 16> : (bw == 32 ? bcr_tc2_kernel<16, 32> : bcr_tc2_kernel<16, 64>);
}

}  // namespace

bool tc2_path_supported(const grim_bcr* h, const SpmmArgs& a) {
  if (h->device < 0 || h->dtype != GRIM_BF16 || !h->d_td_stage || !h->d_status || h->td_max_rec == 0) return false;
  if (a.conv || a.x_dtype != GRIM_BF16 || reinterpret_cast<uintptr_t>(a.X) % 16 != 0) return false;
  if (a.x_sq != 1 || a.y_sq != 1 || (a.x_sk * 2) % 16 != 0) return false;
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
  rings(h, &p.nstages, &p.nrec);
  p.rec_stride = (uint32_t)rec_stride_of(h);
  p.spin_limit = 1u << 20;
  p.a = a;
  CUtensorMap tm;
  memset(&tm, 0, sizeof(tm));
  const cuuint64_t dims[2] = {(cuuint64_t)a.ncols, (cuuint64_t)h->K};
  const cuuint64_t strides[1] = {(cuuint64_t)(a.x_sk * 2)};
  const cuuint32_t box[2] = {64, (cuuint32_t)kK};
  const cuuint32_t estr[2] = {1, 1};
  if (encode_tiled_fn()(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(a.X), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return GRIM_ERR_CUDA;
  const size_t smem = smem_need(h, p.nstages, p.nrec);
  Tc2Kernel kern = kernel_for(h->bh, h->bw);
  // the attribute is kept by the kernel: set once per (kernel, size) and again only when a larger size is needed
  static size_t attr_set[3][3] = {};
  size_t& have = attr_set[p.bh_shift - 2][h->bw == 16 ? 0 : (h->bw == 32 ? 1 : 2)];
  if (have < smem) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return GRIM_ERR_CUDA;
    have = smem;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(2 * ((h->tc_mtiles + 1) / 2)), (unsigned)((a.ncols + kPairCols - 1) / kPairCols), 1);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tm, p);
  count_launch();
  return e == cudaSuccess ? GRIM_OK : GRIM_ERR_CUDA;
}

}  // namespace grim
