// Register-tiled CUDA-core kernel for Y = W * X (Sections 3.1, 4.2 - 4.5): N > 16 and, with its narrow tile, N <= 16.
//
// One thread block (16 warps) owns BPW groups of 16 row bands and a tile of 128 or 256 output columns and walks
// the block columns.  Per block column a slab of X (bw rows x the tile's columns) is brought into shared memory
// once - by TMA when X is a plain row-major matrix, otherwise by 4-byte cp.async gathers (strided X, or the
// implicit im2col of Section 4.5 taken directly from the NCHW input) - together with the packed records of
// the thread block's bands for that block column.  A ring of stages with full / empty mbarriers lets warps
// run up to a stage apart, which absorbs the uneven work of bands (Section 4.2's load imbalance).
//
// A warp owns one band per group, a lane four output columns of each of one or two 128-column pieces.  Per block
// the lane loads the slab rows of the kept columns into registers once (each needed input row is read once and
// reused by every kept row - the load-redundancy idea of Section 4.4) and then, per kept row, reads the row's
// weights with broadcast 128-bit loads and multiplies: packed two-column FMAs (fma.rn.f32x2), so that a lane issues
// half as many instructions for the same flops - the kernel is short of issue slots and of shared-memory bandwidth,
// not of FMA units.  With two pieces per lane the slab addresses, the weight loads and the row tests of a block are
// shared by twice the FMAs (measured 17 % faster than one piece; two bands per warp buy nothing).  Accumulator
// registers are indexed statically: the rows of the band are walked in order with one warp-uniform test of the
// block's row mask each.  Grids that would leave most SMs idle are split over block columns (partial sums added
// into a zeroed Y).
//
// Narrow tile (N <= 16): a lane owns one output column and the two halves of a warp split the kept columns of a
// chunk; the stages are small, so the ring is deeper (8 slots, 6 in flight) and two thread blocks share an SM.
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <cstring>

#include "grim_device.cuh"
#include "grim_internal.h"

namespace grim {
namespace {

constexpr int kFThreads = 512;
constexpr int kFWarps = 16;
constexpr int kTN = 128;          // output columns per thread block and piece
constexpr int kNarrowTN = 16;     // ... of the narrow variant
constexpr int kStages = 4;        // ring slots
constexpr int kAhead = 2;         // stages requested ahead of the one being multiplied
// The narrow variant's stages are small (a 2 KiB slab and a few KiB of records): with two in flight a thread block
// moves about 7 KiB per memory latency, far below its share of the bandwidth; its ring is deeper.
constexpr int kNarrowStages = 8;
constexpr int kNarrowAhead = 6;
constexpr int kMaxRing = 8;
constexpr int kJlistCap = 2048;   // block columns per matrix the stage list can hold
constexpr int kHdrBytes = (192 + kMaxRing * 16 + kJlistCap * 2 + 127) / 128 * 128;  // barriers, flags, per-slot blob sizes, stage list

enum { kModeTma = 0, kModeGather = 1 };

struct FParams {
  const RcStage* stage;
  const uint8_t* blob;
  const uint32_t* band_order;
  unsigned* status;
  int nbr, nbc, M, K, bh, bw, ngroups;
  uint32_t blob_stride, slab_bytes;
  unsigned spin_limit;
  int slab_ld;  // floats between slab rows: kTN, or kTN + 4 when the gather writes down the columns (X stored q-major)
  int ksplit;  // > 1: blockIdx.z takes a share of the block columns and adds its partial sums into a zeroed Y
  SpmmArgs a;
};

// (mbarrier, bulk-copy and TMA wrappers: grim_device.cuh)
using namespace ptx;

__device__ __forceinline__ void cp_async4_zfill(void* dst, const void* src, bool valid) {
  const unsigned n = valid ? 4u : 0u;
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(smem_u32(dst)), "l"(src), "r"(n) : "memory");
}
// One slab element: fp32 activations go through cp.async; bf16 activations are widened on the way (a 2-byte
// cp.async does not exist), so the slab always holds fp32.
__device__ __forceinline__ void gather_elem(float* dst, const void* X, int64_t off, bool valid, bool x_bf16) {
  if (!x_bf16) {
    cp_async4_zfill(dst, static_cast<const float*>(X) + (valid ? off : 0), valid);
  } else {
    unsigned short u = 0;
    if (valid) u = __ldg(static_cast<const unsigned short*>(X) + off);
    *dst = __uint_as_float((unsigned)u << 16);
  }
}
__device__ __forceinline__ void cp_async16_cg(void* dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}

// Four neighbouring slab elements of one row as two packed pairs (fp32 bit patterns, low word = lower column).
__device__ __forceinline__ ulonglong2 ld_x4(const float* slab, unsigned col, int lane4, int sld) {
  return *reinterpret_cast<const ulonglong2*>(slab + col * sld + lane4);
}
__device__ __forceinline__ ulonglong2 ld_x4(const __nv_bfloat16* slab, unsigned col, int lane4, int sld) {
  const uint2 u = *reinterpret_cast<const uint2*>(slab + col * sld + lane4);
  ulonglong2 r;
  r.x = ((unsigned long long)(u.x & 0xFFFF0000u) << 32) | (unsigned long long)(u.x << 16);
  r.y = ((unsigned long long)(u.y & 0xFFFF0000u) << 32) | (unsigned long long)(u.y << 16);
  return r;
}
// Packed fp32 multiply-add on two neighbouring output columns: one instruction, two FMAs per lane.  The FMA pipe
// does the same flops either way; what the packed form saves is issue slots, which this kernel is short of (loads,
// address arithmetic and row tests share them with the FMAs).
__device__ __forceinline__ void ffma2(unsigned long long& acc, unsigned long long w2, unsigned long long x2) {
  asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc) : "l"(w2), "l"(x2));
}
// (w, w): the weight operand of a packed FMA.  Built in registers: storing the weights twice so that a load delivers
// the pair was measured 16 % slower - the shared-memory pipe is the scarcer resource here, not the ALU.
__device__ __forceinline__ unsigned long long dup2(float w) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %1};" : "=l"(r) : "f"(w));
  return r;
}
__device__ __forceinline__ float2 unpack2(unsigned long long v) {
  float2 f;
  asm("mov.b64 {%0, %1}, %2;" : "=f"(f.x), "=f"(f.y) : "l"(v));
  return f;
}

// One slab element (narrow tiles).
__device__ __forceinline__ float ld_x1(const float* slab, unsigned col, int q, int sld) { return slab[col * sld + q]; }
__device__ __forceinline__ float ld_x1(const __nv_bfloat16* slab, unsigned col, int q, int sld) {
  return __uint_as_float((unsigned)reinterpret_cast<const unsigned short*>(slab)[col * sld + q] << 16);
}

// CW: 128-column pieces of the output tile per lane (a lane owns four columns of each piece).
// CW = 0 is the narrow tile for right-hand sides of at most 16 columns: a lane owns ONE output column, and the two
// halves of a warp split the kept columns of a chunk between them (lanes 0-15 the first four, lanes 16-31 the
// other four; their sums meet in one shuffle at the end).  The kept values then stream through shared memory once
// and each costs a quarter of a broadcast load and one FMA per lane - no per-lane gathers from global memory.
template <int BH, int BPW, int CW, typename XT, int MODE>
__global__ void __launch_bounds__(kFThreads, CW == 0 ? 2 : 1) bcr_ffma_kernel(const __grid_constant__ CUtensorMap tmX, const FParams p) {
  constexpr bool NARROW = CW == 0;
  constexpr int NS = NARROW ? kNarrowStages : kStages, AH = NARROW ? kNarrowAhead : kAhead;  // ring slots, stages in flight
  constexpr int TN = NARROW ? kNarrowTN : kTN * CW;  // output columns per thread block
  extern __shared__ __align__(128) uint8_t smem[];
  uint64_t* full = reinterpret_cast<uint64_t*>(smem);
  uint64_t* empty = full + kMaxRing;
  // the launch that follows in the stream may start as SMs free up: it waits (griddepcontrol.wait) before it reads or
  // writes anything this launch touches
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + 128);
  int* s_nst = reinterpret_cast<int*>(smem + 132);
  uint32_t* s_meta = reinterpret_cast<uint32_t*>(smem + 192);               // [ring slot][4] blob bytes per band group
  const uint16_t* jlist = reinterpret_cast<const uint16_t*>(smem + 192 + kMaxRing * 16);  // non-empty block columns, ascending
  uint8_t* slots = smem + kHdrBytes;
  const uint32_t slot_bytes = p.slab_bytes + BPW * p.blob_stride;
  const int sld = MODE == kModeTma ? TN : p.slab_ld;

  const int tid = threadIdx.x, lane = tid & 31;
  // broadcast from lane 0 so that the compiler knows the warp index (and all that derives from it) is the same
  // in every lane: branches on the band's header and row mask then need no divergence handling
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
  const SpmmArgs& a = p.a;
  const int64_t q0 = (int64_t)blockIdx.x * TN;
  const int g0 = blockIdx.y * BPW;

  if (warp == 0) {
    int n = 0;
    for (int j0 = 0; j0 < p.nbc; j0 += 32) {
      const int j = j0 + lane;
      bool f = false;
      if (j < p.nbc)
        for (int b = 0; b < BPW; ++b)
          if (g0 + b < p.ngroups) f = f || p.stage[(int64_t)(g0 + b) * p.nbc + j].bytes != 0;
      const unsigned m = __ballot_sync(0xffffffffu, f);
      if (f) const_cast<uint16_t*>(jlist)[n + __popc(m & ((1u << lane) - 1u))] = (uint16_t)j;
      n += __popc(m);
    }
    if (lane == 0) {
      *s_nst = n;
      *s_abort = 0;
      for (int s = 0; s < NS; ++s) {
        mbar_init(full + s, MODE == kModeTma ? 1u : (unsigned)kFThreads);
        mbar_init(empty + s, kFWarps);
      }
      fence_mbar_init();
    }
  }
  __syncthreads();
  // (programmatic dependent launch) whatever earlier launches in the stream wrote - X, a cleared scratch or Y - is
  // complete and visible from here on; up to here only the packed matrix and this block's own shared memory were touched
  asm volatile("griddepcontrol.wait;" ::: "memory");
  // with a split over block columns this thread block multiplies only its share of the stage list
  const int nst_all = *s_nst;
  const int n_lo = (int)((int64_t)blockIdx.z * nst_all / p.ksplit), n_hi = (int)((int64_t)(blockIdx.z + 1) * nst_all / p.ksplit);
  const int nst = n_hi - n_lo;
  jlist += n_lo;

  // per-thread constants of the gather loader: this thread always fills column qq of the slab
  const int qq = tid & (TN - 1);
  constexpr int kRowStep = kFThreads / TN;  // slab rows between two elements of a thread
  const int kk0 = tid / TN;  // first slab row
  int ih0 = 0, iw0 = 0;
  int64_t qoff = 0;
  bool q_ok = false;
  if (MODE == kModeGather) {
    const int64_t q = q0 + qq;
    q_ok = q < a.ncols;
    if (a.conv) {
      const int64_t ohw = (int64_t)a.OH * a.OW;
      const int64_t img = q_ok ? q / ohw : 0;
      const int pix = q_ok ? (int)(q - img * ohw) : 0;
      const int oh = pix / a.OW, ow = pix - oh * a.OW;
      ih0 = oh * a.stride - a.pad;
      iw0 = ow * a.stride - a.pad;
      qoff = img * a.C * a.H * a.W + (int64_t)ih0 * a.W + iw0;
    } else {
      qoff = q * a.x_sq;
    }
  }

  // Requests stage n (the n-th non-empty block column) into its ring slot.
  auto request = [&](int n) {
    const int slot = n % NS;
    const int j = jlist[n];
    uint8_t* base = slots + (size_t)slot * slot_bytes;
    if (MODE == kModeTma) {
      // one thread: sizes first (read by the consumers after the barrier completes), then the copies
      uint32_t bytes[BPW], off[BPW], total = p.slab_bytes;
#pragma unroll
      for (int b = 0; b < BPW; ++b) {
        bytes[b] = 0; off[b] = 0;
        if (g0 + b < p.ngroups) {
          const RcStage se = p.stage[(int64_t)(g0 + b) * p.nbc + j];
          bytes[b] = se.bytes; off[b] = se.off16;
        }
        s_meta[slot * 4 + b] = bytes[b];
        total += bytes[b];
      }
      mbar_arrive_expect_tx(full + slot, total);
      tma_load_2d(base, &tmX, (int)q0, j * p.bw, full + slot);
#pragma unroll
      for (int b = 0; b < BPW; ++b)
        if (bytes[b]) bulk_load(base + p.slab_bytes + b * p.blob_stride, p.blob + (size_t)off[b] * 16, bytes[b], full + slot);
    } else {
      float* slab = reinterpret_cast<float*>(base);
      const void* X = a.X;
      const bool xb = a.x_dtype == GRIM_BF16;
      int64_t k = (int64_t)j * p.bw + kk0;
      if (a.conv) {
        const int khw = a.KH * a.KW;
        int c = (int)(k / khw);
        int rem = (int)(k - (int64_t)c * khw);
        int kh = rem / a.KW, kw = rem - kh * a.KW;
        for (int kk = kk0; kk < p.bw; kk += kRowStep, k += kRowStep) {
          const int ih = ih0 + kh, iw = iw0 + kw;
          const bool ok = q_ok && k < p.K && ih >= 0 && ih < a.H && iw >= 0 && iw < a.W;
          gather_elem(slab + kk * sld + qq, X, qoff + ((int64_t)c * a.H + kh) * a.W + kw, ok, xb);
          kw += kRowStep;
          while (kw >= a.KW) { kw -= a.KW; ++kh; }
          while (kh >= a.KH) { kh -= a.KH; ++c; }
        }
      } else if (a.x_sq == 1) {
        for (int kk = kk0; kk < p.bw; kk += kRowStep, k += kRowStep) {
          const bool ok = q_ok && k < p.K;
          gather_elem(slab + kk * sld + qq, X, k * a.x_sk + qoff, ok, xb);
        }
      } else {
        // X stored q-major: consecutive threads take consecutive k so that the reads coalesce; the padded row
        // stride keeps the column-wise shared-memory writes to a few bank conflicts
        for (int e = tid; e < p.bw * TN; e += kFThreads) {
          const int kk = e % p.bw, qe = e / p.bw;
          const int64_t ke = (int64_t)j * p.bw + kk, q = q0 + qe;
          const bool ok = q < a.ncols && ke < p.K;
          gather_elem(slab + kk * sld + qe, X, ke * a.x_sk + q * a.x_sq, ok, xb);
        }
      }
#pragma unroll
      for (int b = 0; b < BPW; ++b) {
        uint32_t bytes = 0, off = 0;
        if (g0 + b < p.ngroups) {
          const RcStage se = p.stage[(int64_t)(g0 + b) * p.nbc + j];
          bytes = se.bytes; off = se.off16;
        }
        if (tid == 0) s_meta[slot * 4 + b] = bytes;
        uint8_t* dst = base + p.slab_bytes + b * p.blob_stride;
        const uint8_t* src = p.blob + (size_t)off * 16;
        for (uint32_t i = tid * 16; i < bytes; i += kFThreads * 16) cp_async16_cg(dst + i, src + i);
      }
      if (xb) __threadfence_block();  // the widened elements were written with ordinary stores
      cp_async_arrive_noinc(full + slot);
    }
  };

  // accumulators as packed pairs of neighbouring columns: [band][row][pair]; pairs 2c, 2c + 1 belong to piece c
  unsigned long long acc[BPW][BH][NARROW ? 1 : 2 * CW];
  float nacc[BPW][NARROW ? BH : 1];  // narrow tiles: one column per lane
#pragma unroll
  for (int b = 0; b < BPW; ++b)
#pragma unroll
    for (int r = 0; r < BH; ++r) {
#pragma unroll
      for (int c = 0; c < (NARROW ? 1 : 2 * CW); ++c) acc[b][r][c] = 0ull;
      if (NARROW) nacc[b][NARROW ? r : 0] = 0.f;
    }
  const int lane4 = lane * 4;
  const int nhalf = lane >> 4, nq = lane & 15;  // narrow tiles: which four columns of a chunk, which output column

  // prologue: the first AH stages go into fresh slots
  for (int n = 0; n < AH && n < nst; ++n)
    if (MODE != kModeTma || tid == 0) request(n);

  bool failed = false;
  for (int n = 0; n < nst; ++n) {
    // ---- producer duty: request stage n + AH; its slot was last used by stage n + AH - NS
    const int m = n + AH;
    if (m < nst) {
      const bool mine = MODE != kModeTma || (warp == (n % kFWarps) && lane == 0);
      if (mine) {
        bool ok = true;
        if (m >= NS) ok = mbar_wait(empty + m % NS, (unsigned)((m / NS - 1) & 1), p.spin_limit, s_abort, 0);
        if (ok) request(m);
        else failed = true;
      }
    }
    if (__any_sync(0xffffffffu, failed)) { failed = true; break; }
    // ---- wait for stage n
    const int slot = n % NS;
    if (!mbar_wait(full + slot, (unsigned)((n / NS) & 1), p.spin_limit, s_abort, 0)) failed = true;
    if (__any_sync(0xffffffffu, failed)) { failed = true; break; }
    const uint8_t* base = slots + (size_t)slot * slot_bytes;
    const XT* slab = reinterpret_cast<const XT*>(base);
#pragma unroll
    for (int b = 0; b < BPW; ++b) {
      if (s_meta[slot * 4 + b] == 0) continue;
      const uint8_t* blob = base + p.slab_bytes + b * p.blob_stride;
      const uint32_t hdr = __shfl_sync(0xffffffffu, reinterpret_cast<const uint32_t*>(blob)[warp], 0);
      const int kr = (hdr >> 16) & 0xFF, nch = hdr >> 24;
      if (kr == 0) continue;
      const uint8_t* rec = blob + (hdr & 0xFFFFu) * 16;
      const unsigned rm = __shfl_sync(0xffffffffu, *reinterpret_cast<const unsigned*>(rec), 0);  // kept rows of this block
      const uint8_t* cols = rec + 8;
      const float4* wp = reinterpret_cast<const float4*>(rec + ((8 + nch * kRcChunk + 15) & ~15));
      // The slab rows of KS kept columns are held in registers at a time: all eight of a chunk for one piece per
      // lane, four when a lane owns two pieces (the registers go to the accumulators instead).
      if constexpr (NARROW) {
        const float4* wq0 = wp + nhalf;
        for (int ch = 0; ch < nch; ++ch) {
          const uint2 cc = *reinterpret_cast<const uint2*>(cols + ch * kRcChunk);
          const unsigned c4 = nhalf ? cc.y : cc.x;
          float x[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) x[e] = ld_x1(slab, (c4 >> (8 * e)) & 0xFFu, nq, sld);
          const float4* wq = wq0;
#pragma unroll
          for (int r = 0; r < BH; ++r) {
            if ((rm >> r) & 1u) {
              const float4 w = *wq;
              wq += 2;
              // two chains of two instead of one of four: rows cannot overlap (each sits behind its own branch)
              const float t = fmaf(w.y, x[1], w.x * x[0]);
              const float u = fmaf(w.w, x[3], w.z * x[2]);
              nacc[b][NARROW ? r : 0] += t + u;
            }
          }
          wq0 += 2 * kr;
        }
        continue;
      }
      constexpr int KS = kRcChunk / (NARROW ? 1 : CW);
      for (int ch = 0; ch < nch; ++ch) {
        const uint2 cc = *reinterpret_cast<const uint2*>(cols + ch * kRcChunk);
#pragma unroll
        for (int hs = 0; hs < kRcChunk / KS; ++hs) {
          ulonglong2 x[KS][NARROW ? 1 : CW];
#pragma unroll
          for (int e = 0; e < KS; ++e) {
            const int idx = hs * KS + e;
            const unsigned col = ((idx < 4 ? cc.x : cc.y) >> (8 * (idx & 3))) & 0xFFu;
#pragma unroll
            for (int c = 0; c < CW; ++c) x[e][c] = ld_x4(slab + c * kTN, col, lane4, sld);
          }
          // one test per row of the band; a kept row owns the next eight weights of the chunk
          const float4* wq = wp;
#pragma unroll
          for (int r = 0; r < BH; ++r) {
            if ((rm >> r) & 1u) {
#pragma unroll
              for (int g = 0; g < KS / 4; ++g) {
                const float4 w = wq[KS == kRcChunk ? g : hs];
                const float wv[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  const unsigned long long w2 = dup2(wv[j]);
#pragma unroll
                  for (int c = 0; c < CW; ++c) {
                    ffma2(acc[b][r][2 * c], w2, x[4 * g + j][c].x);
                    ffma2(acc[b][r][2 * c + 1], w2, x[4 * g + j][c].y);
                  }
                }
              }
              wq += 2;
            }
          }
        }
        wp += 2 * kr;
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(empty + slot);
  }

  if (failed) {
    // a bounded wait ran out: tell every warp, record it, let copies that were requested land, leave
    *s_abort = 1;
    if (lane == 0) atomicExch(p.status, (unsigned)GRIM_ERR_TIMEOUT);
  }
  __syncthreads();
  if (*s_abort) {
    if (tid == 0)
      for (int s = 0; s < NS; ++s)
        for (unsigned i = 0; i < 4096u && !mbar_try_wait(full + s, 0) && !mbar_try_wait(full + s, 1); ++i) {}
    return;
  }

  // ---- epilogue: bias, activation, store every row of the band (rows kept by no block are +0)
  const int64_t ohw = (int64_t)a.OH * a.OW;
  if constexpr (NARROW) {
    const int64_t q = q0 + nq;
    int64_t qbase = 0;  // offset of column q in row 0 of the output
    if (q < a.ncols) {
      if (a.conv) {
        const int64_t img = q / ohw;
        qbase = img * p.M * ohw + (q - img * ohw);
      } else {
        qbase = q * a.y_sq;
      }
    }
    const int64_t rstride = a.conv ? ohw : a.y_sr;
#pragma unroll
    for (int b = 0; b < BPW; ++b) {
      const int pos = (g0 + b) * kRcBands + warp;
      if (pos >= p.nbr) continue;  // (uniform over the warp: the shuffles below are taken by all lanes or none)
      const int band = p.band_order[pos];
#pragma unroll
      for (int r = 0; r < BH; ++r) {
        float t = nacc[b][NARROW ? r : 0];
        t += __shfl_xor_sync(0xffffffffu, t, 16);
        const int64_t row = (int64_t)band * p.bh + r;
        if (r >= p.bh || row >= p.M || nhalf != 0 || q >= a.ncols) continue;
        const int64_t off = row * rstride + qbase;
        if (p.ksplit > 1) {
          if (t != 0.f) atomicAdd(static_cast<float*>(a.Y) + off, t);
          continue;
        }
        t += a.bias ? __ldg(a.bias + row) : 0.f;
        if (a.relu) t = fmaxf(t, 0.f);
        if (a.y_dtype == GRIM_F32) static_cast<float*>(a.Y)[off] = t;
        else static_cast<__nv_bfloat16*>(a.Y)[off] = __float2bfloat16_rn(t);
      }
    }
  } else {
#pragma unroll
  for (int cp = 0; cp < CW; ++cp) {
  const int64_t q = q0 + cp * kTN + lane4;
  if (q >= a.ncols) continue;
#pragma unroll
  for (int b = 0; b < BPW; ++b) {
    const int pos = (g0 + b) * kRcBands + warp;
    if (pos >= p.nbr) continue;
    const int band = p.band_order[pos];
#pragma unroll
    for (int r = 0; r < BH; ++r) {
      const int64_t row = (int64_t)band * p.bh + r;
      if (r >= p.bh || row >= p.M) continue;
      const float2 t01 = unpack2(acc[b][r][2 * cp]), t23 = unpack2(acc[b][r][2 * cp + 1]);
      float t[4] = {t01.x, t01.y, t23.x, t23.y};
      if (p.ksplit > 1) {
        // partial sums of one share of the block columns: added into Y (fp32, zeroed before the launch);
        // bias and activation follow in a separate pass
        float* y = static_cast<float*>(a.Y);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          if (q + e >= a.ncols) break;
          int64_t off;
          if (a.conv) {
            const int64_t img = (q + e) / ohw;
            off = (img * p.M + row) * ohw + ((q + e) - img * ohw);
          } else {
            off = row * a.y_sr + (q + e) * a.y_sq;
          }
          if (t[e] != 0.f) atomicAdd(y + off, t[e]);
        }
        continue;
      }
      const float bias = a.bias ? __ldg(a.bias + row) : 0.f;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        t[e] += bias;
        if (a.relu) t[e] = fmaxf(t[e], 0.f);
      }
      int64_t off0;
      bool contiguous;
      if (a.conv) {
        const int64_t img = q / ohw;
        const int64_t pix = q - img * ohw;
        off0 = (img * p.M + row) * ohw + pix;
        contiguous = (pix + 3 < ohw) && (q + 3 < a.ncols);
      } else {
        off0 = row * a.y_sr + q * a.y_sq;
        contiguous = a.y_sq == 1 && (q + 3 < a.ncols);
      }
      if (a.y_dtype == GRIM_F32) {
        float* y = static_cast<float*>(a.Y);
        if (contiguous && ((reinterpret_cast<uintptr_t>(y + off0) & 15) == 0)) {
          *reinterpret_cast<float4*>(y + off0) = make_float4(t[0], t[1], t[2], t[3]);
          continue;
        }
      } else {
        __nv_bfloat16* y = static_cast<__nv_bfloat16*>(a.Y);
        if (contiguous && ((reinterpret_cast<uintptr_t>(y + off0) & 7) == 0)) {
          __nv_bfloat162 lo = __floats2bfloat162_rn(t[0], t[1]);
          __nv_bfloat162 hi = __floats2bfloat162_rn(t[2], t[3]);
          uint2 u;
          u.x = *reinterpret_cast<unsigned*>(&lo);
          u.y = *reinterpret_cast<unsigned*>(&hi);
          *reinterpret_cast<uint2*>(y + off0) = u;
          continue;
        }
      }
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        if (q + e >= a.ncols) break;
        int64_t off;
        if (a.conv) {
          const int64_t img = (q + e) / ohw;
          const int64_t pix = (q + e) - img * ohw;
          off = (img * p.M + row) * ohw + pix;
        } else {
          off = row * a.y_sr + (q + e) * a.y_sq;
        }
        if (a.y_dtype == GRIM_F32) static_cast<float*>(a.Y)[off] = t[e];
        else static_cast<__nv_bfloat16*>(a.Y)[off] = __float2bfloat16_rn(t[e]);
      }
    }
  }
  }  // pieces
  }
}

// The driver's tensor-map encoder, looked up through the runtime so that the library does not link
// against the driver (it must load on machines without one).
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

// Second pass of a split multiply: Y = act(Y + bias) in place.
__global__ void bcr_finalize_kernel(const SpmmArgs a, int M) {
  const int64_t total = (int64_t)M * a.ncols;
  const int64_t ohw = (int64_t)a.OH * a.OW;
  float* y = static_cast<float*>(a.Y);
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    int64_t off, row;
    if (a.conv) {  // i runs over the NCHW output
      off = i;
      row = (i / ohw) % M;
    } else if (a.y_sq == 1) {
      row = i / a.ncols;
      off = row * a.y_sr + (i - row * a.ncols);
    } else {
      const int64_t q = i / M;
      row = i - q * M;
      off = row * a.y_sr + q * a.y_sq;
    }
    float v = y[off] + (a.bias ? __ldg(a.bias + row) : 0.f);
    if (a.relu) v = fmaxf(v, 0.f);
    y[off] = v;
  }
}

bool tma_eligible(const SpmmArgs& a) {
  if (a.conv || a.x_sq != 1) return false;
  const int esz = a.x_dtype == GRIM_F32 ? 4 : 2;
  return (reinterpret_cast<uintptr_t>(a.X) % 16 == 0) && ((a.x_sk * esz) % 16 == 0) && a.ncols < (int64_t(1) << 31);
}

// Zeroes the M x ncols region of Y that a split multiply accumulates into.
cudaError_t zero_output(const SpmmArgs& a, int64_t M, cudaStream_t s) {
  float* y = static_cast<float*>(a.Y);
  if (a.conv) return cudaMemsetAsync(y, 0, (size_t)M * a.ncols * 4, s);
  if (a.y_sq == 1) return cudaMemset2DAsync(y, (size_t)a.y_sr * 4, 0, (size_t)a.ncols * 4, (size_t)M, s);
  if (a.y_sr == 1) return cudaMemset2DAsync(y, (size_t)a.y_sq * 4, 0, (size_t)M * 4, (size_t)a.ncols, s);
  return cudaErrorInvalidValue;
}

template <int BH, int BPW, int CW, typename XT, int MODE>
cudaError_t launch_variant(const CUtensorMap& tm, const FParams& p, size_t smem, dim3 grid, cudaStream_t s) {
  auto kern = bcr_ffma_kernel<BH, BPW, CW, XT, MODE>;
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), smem);
  if (e != cudaSuccess) return e;
  return launch_pdl(kern, grid, dim3(kFThreads), smem, s, tm, p);
}

// The accumulators of a lane take BH * BPW * CW * 4 registers: at most 64.
template <int BH, typename XT, int MODE>
cudaError_t launch_bpw(int bpw, int cw, const CUtensorMap& tm, const FParams& p, size_t smem, dim3 grid, cudaStream_t s) {
  if (cw == 0) {
    if (BH <= 8 && bpw == 4) return launch_variant<BH, (BH <= 8 ? 4 : 1), 0, XT, MODE>(tm, p, smem, grid, s);
    if (bpw == 2) return launch_variant<BH, 2, 0, XT, MODE>(tm, p, smem, grid, s);
    return launch_variant<BH, 1, 0, XT, MODE>(tm, p, smem, grid, s);
  }
  if (cw == 2) {
    if (BH <= 4 && bpw == 2) return launch_variant<BH, (BH <= 4 ? 2 : 1), (BH <= 4 ? 2 : 1), XT, MODE>(tm, p, smem, grid, s);
    if (BH <= 8) return launch_variant<BH, 1, (BH <= 8 ? 2 : 1), XT, MODE>(tm, p, smem, grid, s);
    return cudaErrorInvalidValue;
  }
  if (BH <= 8 && bpw == 2) return launch_variant<BH, (BH <= 8 ? 2 : 1), 1, XT, MODE>(tm, p, smem, grid, s);
  if (BH <= 4 && bpw == 4) return launch_variant<BH, (BH <= 4 ? 4 : 1), 1, XT, MODE>(tm, p, smem, grid, s);
  return launch_variant<BH, 1, 1, XT, MODE>(tm, p, smem, grid, s);
}

template <typename XT, int MODE>
cudaError_t launch_bh(int BHc, int bpw, int cw, const CUtensorMap& tm, const FParams& p, size_t smem, dim3 grid, cudaStream_t s) {
  if (BHc == 4) return launch_bpw<4, XT, MODE>(bpw, cw, tm, p, smem, grid, s);
  if (BHc == 8) return launch_bpw<8, XT, MODE>(bpw, cw, tm, p, smem, grid, s);
  return launch_bpw<16, XT, MODE>(bpw, cw, tm, p, smem, grid, s);
}

constexpr size_t kSmemBudget = 220 * 1024;

int tile_cols(int cw) { return cw ? kTN * cw : kNarrowTN; }
int slab_ld_for(const SpmmArgs& a, bool tma, int cw) { return (!tma && !a.conv && a.x_sq != 1) ? tile_cols(cw) + 4 : tile_cols(cw); }
size_t slab_bytes_for(const grim_bcr* h, int sld, int esz) { return ((size_t)h->bw * sld * esz + 127) & ~size_t(127); }
size_t smem_need(const grim_bcr* h, int bpw, int esz, int sld = kTN + 4, int stages = kStages) {
  const size_t blob_stride = ((size_t)h->rc_max_blob + 127) & ~size_t(127);
  return kHdrBytes + (size_t)stages * (slab_bytes_for(h, sld, esz) + bpw * blob_stride);
}

}  // namespace

bool ffma_path_supported(const grim_bcr* h, const SpmmArgs& a) {
  if (h->device < 0 || !h->d_rc_stage || !h->d_status) return false;
  if (h->nbc > kJlistCap || h->rc_max_blob == 0 || h->rc_max_blob > 0xFFFF * 16u) return false;
  if (a.ncols <= 0 || a.ncols > (int64_t(1) << 31) - 2 * kTN) return false;
  const bool tma = tma_eligible(a);
  return smem_need(h, 1, (tma && a.x_dtype == GRIM_BF16) ? 2 : 4) <= kSmemBudget;
}

grim_status_t launch_ffma(const grim_bcr* h, const SpmmArgs& a, cudaStream_t s) {
  if (!ffma_path_supported(h, a)) return GRIM_ERR_UNSUPPORTED;
  const bool tma = tma_eligible(a);
  const int esz = (tma && a.x_dtype == GRIM_BF16) ? 2 : 4;  // bytes per slab element (the gather loader widens bf16)
  const int BHc = h->bh <= 4 ? 4 : (h->bh <= 8 ? 8 : 16);
  const int sms = sm_count(h->device);
  // band groups per warp (bpw) and 128-column pieces per lane (cw): as much as the 64 accumulator registers of a
  // lane allow, less when the grid would not fill the GPU.  Two pieces per lane are preferred over two bands per
  // warp: the slab addresses, the weight loads and the row tests of a block are then shared by twice the FMAs.
  int bpw = BHc == 4 ? 4 : (BHc == 8 ? 2 : 1), cw = 1;
  const int tn = a.tile_n % 256;
  auto tiles_of = [&](int bpw_, int cw_) { return ((a.ncols + tile_cols(cw_) - 1) / tile_cols(cw_)) * ((h->rc_groups + bpw_ - 1) / bpw_); };
  auto fits = [&](int bpw_, int cw_) { return smem_need(h, bpw_, esz, tile_cols(cw_) + 4, cw_ ? kStages : kNarrowStages) <= kSmemBudget; };
  if (tn == 1 || tn == 2 || tn == 4) {
    bpw = std::min(tn, bpw);
  } else if (tn == 8 && BHc <= 8) {
    cw = 2; bpw = 1;
  } else if (tn == 9 && BHc <= 4) {
    cw = 2; bpw = 2;
  } else if (tn == 17 || tn == 18 || tn == 20) {
    cw = 0; bpw = std::min(tn - 16, BHc <= 8 ? 4 : 2);
  } else if (a.ncols <= kNarrowTN) {
    cw = 0; bpw = 1;
  } else {
    // (measured at 8192 x 8192 and 4096 x 4096, N = 256 and 1024: two pieces per lane are 10 - 20 % faster than
    // any one-piece variant, also where they leave the grid smaller than the GPU - the split below then applies)
    if (BHc <= 8 && a.ncols > kTN && fits(1, 2)) {
      cw = 2;
      bpw = (BHc == 4 && fits(2, 2) && tiles_of(2, 2) >= sms) ? 2 : 1;
    } else {
      while (bpw > 1 && (!fits(bpw, 1) || tiles_of(bpw, 1) < sms)) bpw >>= 1;
    }
  }
  if (!fits(bpw, cw)) return GRIM_ERR_UNSUPPORTED;
  const int64_t qtiles = (a.ncols + tile_cols(cw) - 1) / tile_cols(cw);
  const int64_t gy = (h->rc_groups + bpw - 1) / bpw;
  if (gy > 65535) return GRIM_ERR_UNSUPPORTED;
  // too few tiles for the GPU: split the block columns over several thread blocks (fp32 output only)
  int ksplit = 1;
  const bool split_ok = a.y_dtype == GRIM_F32 && (a.conv || a.y_sq == 1 || a.y_sr == 1);
  if (split_ok && qtiles * gy * 2 <= sms) {
    ksplit = (int)std::min<int64_t>(std::min<int64_t>(8, sms / (qtiles * gy)), std::max<int64_t>(1, h->nbc / 4));
    if (ksplit < 1) ksplit = 1;
  }
  // narrow tiles are light (two thread blocks share an SM): as many parts as still run in one wave
  if (cw == 0 && split_ok && qtiles * gy < 2 * sms)
    ksplit = (int)std::max<int64_t>(1, std::min<int64_t>(std::min<int64_t>(8, 2 * sms / (qtiles * gy)), h->nbc / 4));
  if (a.tile_n >= 256) ksplit = split_ok ? std::max(1, std::min(8, a.tile_n / 256)) : 1;  // test / tuning override

  FParams p;
  p.stage = h->d_rc_stage; p.blob = h->d_rc_blob; p.band_order = h->d_band_order; p.status = h->d_status;
  p.nbr = (int)h->nbr; p.nbc = (int)h->nbc; p.M = (int)h->M; p.K = (int)h->K; p.bh = h->bh; p.bw = h->bw;
  p.ngroups = (int)h->rc_groups;
  p.blob_stride = (h->rc_max_blob + 127u) & ~127u;
  p.slab_ld = slab_ld_for(a, tma, cw);
  p.slab_bytes = (uint32_t)slab_bytes_for(h, p.slab_ld, esz);
  p.spin_limit = 1u << 20;
  p.ksplit = ksplit;
  p.a = a;

  CUtensorMap tm;
  memset(&tm, 0, sizeof(tm));
  if (tma) {
    const cuuint64_t dims[2] = {(cuuint64_t)a.ncols, (cuuint64_t)h->K};
    const cuuint64_t strides[1] = {(cuuint64_t)(a.x_sk * esz)};
    const cuuint32_t box[2] = {(cuuint32_t)tile_cols(cw), (cuuint32_t)h->bw};
    const cuuint32_t estr[2] = {1, 1};
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return GRIM_ERR_CUDA;
    const CUresult r = encode(&tm, esz == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
                                              2, const_cast<void*>(a.X), dims, strides, box, estr,
                                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                                              CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return GRIM_ERR_CUDA;
  }
  const size_t smem = smem_need(h, bpw, esz, p.slab_ld, cw ? kStages : kNarrowStages);
  dim3 grid((unsigned)qtiles, (unsigned)gy, (unsigned)ksplit);
  cudaError_t e = cudaSuccess;
  if (ksplit > 1 && !(a.y_prefilled && !a.relu)) {
    e = zero_output(a, h->M, s);
    if (e != cudaSuccess) return GRIM_ERR_CUDA;
  }
  if (tma) {
    e = esz == 4 ? launch_bh<float, kModeTma>(BHc, bpw, cw, tm, p, smem, grid, s)
                 : launch_bh<__nv_bfloat16, kModeTma>(BHc, bpw, cw, tm, p, smem, grid, s);
  } else {
    e = launch_bh<float, kModeGather>(BHc, bpw, cw, tm, p, smem, grid, s);
  }
  count_launch();
  if (e == cudaSuccess && ksplit > 1 && (a.bias || a.relu) && !(a.y_prefilled && !a.relu)) {
    const int64_t total = h->M * a.ncols;
    bcr_finalize_kernel<<<(unsigned)std::min<int64_t>((total + 255) / 256, (int64_t)sm_count(h->device) * 8), 256, 0, s>>>(a, (int)h->M);
    count_launch();
    e = cudaGetLastError();
  }
  return e == cudaSuccess ? GRIM_OK : GRIM_ERR_CUDA;
}

}  // namespace grim
