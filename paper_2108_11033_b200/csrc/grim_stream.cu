// Streaming kernel for N <= 16 right-hand sides (N = 1: matrix-vector product; Sections 3.1, 4.2, 4.4).
//
// The multiply reads every kept weight exactly once, so it is bound by how fast the packed matrix can be
// streamed.  One persistent thread block per SM walks its share of the row bands; all warps of the block work
// on the same band, each on its own runs (up to four consecutive chunks, cut by the packer so that a run's values
// fit a stage).  A warp keeps a private ring of stages in
// shared memory and fills it with bulk asynchronous copies (one for the column words of a run, one for its
// values), several stages ahead of the multiply, so the global-memory latency is paid by the copy engine and
// not by the warp.  The multiply then reads column words, values and (for N = 1) the activation vector from
// shared memory only: a lane owns one kept column of a chunk and walks the block's row mask.
//
// Runs of a band are dealt to the warps round-robin, and the deal continues where the previous band stopped,
// so over a few bands every warp gets the same number of runs.  Partial sums of a batch of bands are combined
// through shared memory once per batch (one block barrier pair per batch, not per band).
#include <cuda_bf16.h>

#include "grim_device.cuh"
#include "grim_internal.h"

namespace grim {

namespace {

constexpr int kSRun = kRunChunks;   // chunks per stage at most (one bulk copy for their column words, one for their values)
constexpr int kSMaxSlots = 4;      // ring slots per warp
constexpr int kSPartBytes = 8192;  // shared memory for the partial sums of one batch of bands
constexpr int kSMaxBands = 2048;   // bands one thread block can list
constexpr int kSMaxXBytes = 81920; // most bytes of activations staged in shared memory (N = 1: the vector; N > 1: a K slice)

// shared memory for the partial sums of one batch of bands
__host__ __device__ constexpr int part_bytes(bool staged) { return staged ? 4 * kSPartBytes : kSPartBytes; }
// bytes between staged rows of X (see the kernel)
__host__ __device__ constexpr int x_row_stride(int nq, int esz) { return nq * esz + (nq * esz >= 32 ? 16 : 0); }

struct StreamParams {
  const uint32_t* run_ptr;
  const RunDesc* runs;
  const uint32_t* colwords;
  const uint8_t* vals;
  const uint32_t* band_order;
  const void* X;
  void* Y;
  unsigned* status;
  int64_t ldx, ldy;
  int N, nbr, M, K, bh, y_dtype, vec_ok;
  int stage_vec;  // the staged rows of X can be copied in aligned 16-byte (8-byte for rows of 8 bytes) pieces
  int nslots, nk_max;
  uint32_t stage_bytes, off_band, off_part, off_x, off_ring;
  unsigned spin_limit;
  // K-sliced mode (2 <= N <= 16): the "bands" above are virtual bands (one band restricted to one K slice); slice_of
  // gives each one's slice (null: everything is slice 0), sl_rows the rows of X per slice, accumulate = 1 when a row
  // of Y gets contributions from several virtual bands (added atomically into a zeroed Y)
  const uint32_t* slice_of;
  int sl_rows, accumulate;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false when the limit ran out or another warp raised the abort flag.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, unsigned parity, unsigned limit, const volatile int* abort_flag) {
  for (unsigned i = 0; i < limit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 63u) == 63u && *abort_flag) return false;
  }
  return false;
}
__device__ __forceinline__ void bulk_load(void* dst, const void* src, unsigned bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

// acc += w * x and at += step when (rm & bit) != 0, with w the value at shared-window address at.
template <typename VT>
__device__ __forceinline__ void row_step(unsigned rm, unsigned bit, float x, unsigned step, float& acc, uint32_t& at) {
  if (sizeof(VT) == 4) {
    asm("{\n.reg .pred p;\n.reg .b32 t;\n.reg .f32 w;\n"
        "and.b32 t, %2, %3;\nsetp.ne.u32 p, t, 0;\n"
        "ld.shared.f32 w, [%1];\n"
        "@p fma.rn.f32 %0, w, %4, %0;\n"
        "@p add.u32 %1, %1, %5;\n}"
        : "+f"(acc), "+r"(at)
        : "r"(rm), "r"(bit), "f"(x), "r"(step));
  } else {
    asm("{\n.reg .pred p;\n.reg .b32 t;\n.reg .b16 h, z;\n.reg .f32 w;\n"
        "and.b32 t, %2, %3;\nsetp.ne.u32 p, t, 0;\n"
        "ld.shared.b16 h, [%1];\nmov.b16 z, 0;\nmov.b32 w, {z, h};\n"
        "@p fma.rn.f32 %0, w, %4, %0;\n"
        "@p add.u32 %1, %1, %5;\n}"
        : "+f"(acc), "+r"(at)
        : "r"(rm), "r"(bit), "f"(x), "r"(step));
  }
}

template <int NQ, typename XT>
__device__ __forceinline__ void load_x(const StreamParams& p, uint32_t col, int q0, float (&x)[NQ]) {
  const XT* row = static_cast<const XT*>(p.X) + (int64_t)col * p.ldx + q0;
  if (NQ >= 4 && p.vec_ok) {
    if (sizeof(XT) == 4) {
#pragma unroll
      for (int i = 0; i < NQ / 4; ++i) {
        const float4 v = __ldg(reinterpret_cast<const float4*>(row) + i);
        x[4 * i] = v.x; x[4 * i + 1] = v.y; x[4 * i + 2] = v.z; x[4 * i + 3] = v.w;
      }
    } else {
#pragma unroll
      for (int i = 0; i < NQ / 4; ++i) {
        const uint2 u = __ldg(reinterpret_cast<const uint2*>(row) + i);
        x[4 * i] = __uint_as_float(u.x << 16); x[4 * i + 1] = __uint_as_float(u.x & 0xFFFF0000u);
        x[4 * i + 2] = __uint_as_float(u.y << 16); x[4 * i + 3] = __uint_as_float(u.y & 0xFFFF0000u);
      }
    }
  } else {
#pragma unroll
    for (int i = 0; i < NQ; ++i) x[i] = (q0 + i < p.N) ? to_f32(row[i]) : 0.f;
  }
}

// Walks the runs of one warp: band after band of the thread block's list, inside a band every NW-th run,
// the first one chosen so that the round-robin deal continues across bands.
template <int NW>
struct RunWalk {
  int k = -1, rot = 0;
  uint32_t beg = 0, r = 0, end = 0;
  // moves to the next band; false after the last one
  __device__ __forceinline__ bool next_band(const uint2* s_band, int nk, int warp) {
    if (k >= nk) return false;
    if (k >= 0) rot = (int)((rot + (end - beg)) % NW);
    if (++k >= nk) { r = end = beg = 0; return false; }
    const uint2 b = s_band[k];
    beg = b.x; end = b.y;
    r = beg + (uint32_t)((warp - rot + NW) % NW);
    return true;
  }
  // next run of this warp; false when the warp has no run left
  __device__ __forceinline__ bool next_run(const uint2* s_band, int nk, int warp, uint32_t& run) {
    for (;;) {
      if (r < end) {
        run = r;
        r += NW;
        return true;
      }
      if (!next_band(s_band, nk, warp)) return false;
    }
  }
};

// What a bulk copy pair needs to know about a run: its table entry and the next one.
struct RunFetch {
  uint2 a = make_uint2(0, 0), b = make_uint2(0, 0);
  int valid = 0;
};

// XS: the activations are staged in shared memory - the whole vector for N = 1; for N > 1 the rows of the current K
// slice (NQ columns of them), reloaded by the whole block when its next band lies in another slice.
template <int BH, int NQ, int NW, bool XS, typename VT, typename XT>
__global__ void __launch_bounds__(NW * 32, 1) bcr_stream_kernel(const StreamParams p) {
  // bands per batch (between two block-wide meetings).  In the staged mode a band is only one K slice of a band and
  // has a few runs, i.e. work for a few warps: the batch is what keeps all warps busy, so it is larger there.
  constexpr int kPart = part_bytes(XS && NQ > 1);
  constexpr int PB = (kPart / (NW * BH * NQ * 4)) > 0 ? (kPart / (NW * BH * NQ * 4)) : 1;
  // staged rows of X (N > 1): NQ elements, 16 bytes apart from the next row when a row is 32 bytes or longer, so that
  // the 32 lanes' rows (any 32 of the slice) spread over the shared-memory banks instead of two or four groups of them
  constexpr int kRowBytes = NQ * (int)sizeof(XT);
  constexpr int kRowStride = x_row_stride(NQ, (int)sizeof(XT));
  extern __shared__ __align__(128) uint8_t smem[];
  uint64_t* full = reinterpret_cast<uint64_t*>(smem);                            // [NW][kSMaxSlots]
  uint32_t* s_slack = reinterpret_cast<uint32_t*>(smem + NW * kSMaxSlots * 8);   // [NW][kSMaxSlots]
  int* s_abort = reinterpret_cast<int*>(s_slack + NW * kSMaxSlots);
  uint2* s_band = reinterpret_cast<uint2*>(smem + p.off_band);                   // [nk] runs of each band
  uint32_t* s_first_row = reinterpret_cast<uint32_t*>(s_band + p.nk_max);        // [nk] first matrix row of each band
  uint32_t* s_slice = s_first_row + p.nk_max;                                    // [nk] K slice of each band (sliced mode)
  float* part = reinterpret_cast<float*>(smem + p.off_part);                     // [PB][NW][BH * NQ]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t ring_off = p.off_ring + (uint32_t)warp * p.nslots * p.stage_bytes;  // this warp's ring, from the base
  uint8_t* ring = smem + ring_off;
  uint64_t* my_full = full + warp * kSMaxSlots;
  // Bands are scheduled heaviest first; thread blocks take them in rounds of gridDim.x, forwards in even rounds and
  // backwards in odd ones, so that no block collects the heaviest band of every round.
  const int grid = (int)gridDim.x, bid = (int)blockIdx.x;
  const int nfull = p.nbr / grid, rem = p.nbr - nfull * grid;
  const int nk = nfull + ((((nfull & 1) ? grid - 1 - bid : bid) < rem) ? 1 : 0);  // bands of this thread block
  const int q0 = blockIdx.y * NQ;
  const int nslots = p.nslots;

  // Programmatic dependent launch: the launch that follows in the stream may start as soon as SMs free up (this
  // kernel reads nothing an earlier launch wrote until the wait below), and this one, if it was launched that way
  // itself, has come this far while its predecessor was still running.  Until the wait it touches only the packed
  // matrix (immutable) and its own shared memory: tables, barriers and the first weight copies are under way when
  // the predecessor ends, which hides most of a launch's fixed cost in a chain of back-to-back products.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (threadIdx.x == 0) *s_abort = 0;
  if (lane == 0) {
    for (int s = 0; s < kSMaxSlots; ++s) mbar_init(my_full + s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int k = threadIdx.x; k < nk; k += NW * 32) {
    const int pos = k * grid + ((k & 1) ? grid - 1 - bid : bid);
    s_band[k] = make_uint2(p.run_ptr[pos], p.run_ptr[pos + 1]);
    s_first_row[k] = p.band_order[pos] * (uint32_t)p.bh;
    s_slice[k] = p.slice_of ? p.slice_of[pos] : 0u;
  }
  __syncthreads();
  // The run table entries of this block's bands are pulled into L2 now, while the memory system is idle: the
  // loads that read them later would otherwise queue behind the bulk copies of the whole GPU.
  for (int k = 0; k < nk; ++k) {
    const uint2 b = s_band[k];
    const uint64_t lo = (uint64_t)b.x * sizeof(RunDesc) & ~(uint64_t)31, hi = ((uint64_t)b.y + 1) * sizeof(RunDesc);
    const uint8_t* base = reinterpret_cast<const uint8_t*>(p.runs);
    for (uint64_t a = lo + (uint64_t)threadIdx.x * 32; a < hi; a += (uint64_t)NW * 32 * 32)
      asm volatile("prefetch.global.L2 [%0];" ::"l"(base + a));
  }

  RunWalk<NW> fw;  // the copies run ahead of the multiply with a walk of their own
  auto prepare = [&]() {
    RunFetch f;
    uint32_t run;
    if (fw.next_run(s_band, nk, warp, run)) {
      // only loaded here; the first use is in issue(), two multiplies later, so the loads' latency stays hidden
      f.a = __ldg(reinterpret_cast<const uint2*>(p.runs) + run);
      f.b = __ldg(reinterpret_cast<const uint2*>(p.runs) + run + 1);
      f.valid = 1;
    }
    return f;
  };
  // The values of a run are contiguous but start anywhere: the copy starts at the 16-byte boundary below them and
  // the number of elements skipped that way ("slack") is left beside the barrier for the multiply, with the run's
  // chunk count above it.
  auto issue = [&](const RunFetch& f, int slot) {
    if (lane == 0 && f.valid) {
      uint8_t* st = ring + (size_t)slot * p.stage_bytes;
      const uint64_t a0 = (uint64_t)f.a.y * sizeof(VT), a1 = (uint64_t)f.b.y * sizeof(VT);
      const uint64_t al = a0 & ~(uint64_t)15;
      const unsigned vbytes = (unsigned)((a1 - al + 15) & ~(uint64_t)15);
      const unsigned n = f.b.x - f.a.x;
      const unsigned cbytes = n * 128u;
      s_slack[warp * kSMaxSlots + slot] = (uint32_t)((a0 - al) / sizeof(VT)) | (n << 16);
      mbar_arrive_expect_tx(my_full + slot, cbytes + vbytes);
      bulk_load(st, p.colwords + (size_t)f.a.x * 32, cbytes, my_full + slot);
      bulk_load(st + kSRun * 128, p.vals + al, vbytes, my_full + slot);
    }
  };

  {
    RunFetch first[kSMaxSlots];
#pragma unroll
    for (int s = 0; s < kSMaxSlots; ++s)
      if (s < nslots) first[s] = prepare();
#pragma unroll
    for (int s = 0; s < kSMaxSlots; ++s)
      if (s < nslots) issue(first[s], s);
  }
  RunFetch pend0 = prepare(), pend1 = prepare();

  // everything earlier launches in the stream wrote (X, a cleared Y) is complete and visible from here on
  asm volatile("griddepcontrol.wait;" ::: "memory");

  if (XS && NQ == 1) {
    XT* sx = reinterpret_cast<XT*>(smem + p.off_x);
    const XT* X = static_cast<const XT*>(p.X);
    for (int k = threadIdx.x; k < p.K; k += NW * 32) sx[k] = X[(int64_t)k * p.ldx];
    __syncthreads();
  }
  int cur_slice = -1;  // (N > 1) slice whose rows of X are in shared memory

  bool failed = false;
  int slot = 0;
  unsigned phase = 0;
  const int myrow = warp_row<BH>(lane);
  RunWalk<NW> cw_walk;
  for (int kb = 0; kb < nk; kb += PB) {
    const int nb = min(PB, nk - kb);
    if (XS && NQ > 1) {
      // warps without a run in a band leave its slot alone: the slots start at zero
      for (int i = threadIdx.x; i < nb * NW * BH * NQ; i += NW * 32) part[i] = 0.f;
      __syncthreads();
    }
    for (int b = 0; b < nb; ++b) {
      float acc[BH][NQ];
#pragma unroll
      for (int r = 0; r < BH; ++r)
#pragma unroll
        for (int q = 0; q < NQ; ++q) acc[r][q] = 0.f;
      if (XS && NQ > 1 && (int)s_slice[kb + b] != cur_slice) {
        // every warp walks the same bands in the same order, so all of them arrive here together: the rows of the new
        // slice replace the old ones once nobody reads those any more
        cur_slice = (int)s_slice[kb + b];
        __syncthreads();
        uint8_t* sx = smem + p.off_x;
        const XT* X = static_cast<const XT*>(p.X);
        const int64_t base = (int64_t)cur_slice * p.sl_rows;
        if (p.stage_vec) {
          // asynchronous copies in pieces of PIECE bytes (the weight rings keep filling meanwhile)
          constexpr int PIECE = kRowBytes >= 16 ? 16 : 8, PPR = kRowBytes / PIECE;
          for (int e = threadIdx.x; e < p.sl_rows * PPR; e += NW * 32) {
            const int r = e / PPR, pc = e - r * PPR;
            uint8_t* dst = sx + (size_t)r * kRowStride + pc * PIECE;
            if (base + r < p.K) {
              const uint8_t* src = reinterpret_cast<const uint8_t*>(X + (base + r) * p.ldx + q0) + pc * PIECE;
              if (PIECE == 16) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
              else asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
            } else if (PIECE == 16) {
              *reinterpret_cast<uint4*>(dst) = make_uint4(0u, 0u, 0u, 0u);
            } else {
              *reinterpret_cast<uint2*>(dst) = make_uint2(0u, 0u);
            }
          }
          asm volatile("cp.async.wait_all;" ::: "memory");
        } else {
          for (int e = threadIdx.x; e < p.sl_rows * NQ; e += NW * 32) {
            const int r = e / NQ, q = e - r * NQ;
            reinterpret_cast<XT*>(sx + (size_t)r * kRowStride)[q] =
                (base + r < p.K && q0 + q < p.N) ? X[(base + r) * p.ldx + q0 + q] : XT(0.f);
          }
        }
        __syncthreads();
      }
      cw_walk.next_band(s_band, nk, warp);
      bool had_run = false;
      for (uint32_t run = cw_walk.r; run < cw_walk.end && !failed; run += NW) {
        had_run = true;
        if (!__all_sync(0xffffffffu, mbar_wait(my_full + slot, phase, p.spin_limit, s_abort))) {
          failed = true;
          if (lane == 0) {
            atomicExch(s_abort, 1);
            atomicOr(p.status, (unsigned)GRIM_ERR_TIMEOUT);
          }
          break;
        }
        // everything below addresses shared memory by 32-bit byte offsets from its base
        const uint32_t st = ring_off + (uint32_t)slot * p.stage_bytes;
        const uint32_t cw_at = st + (uint32_t)lane * 4u;
        const uint32_t note = s_slack[warp * kSMaxSlots + slot];
        const int n = (int)(note >> 16);
        uint32_t v_at = st + kSRun * 128u + ((note & 0xFFFFu) + (uint32_t)lane) * (uint32_t)sizeof(VT);
        // chunks past the end of a short run read column words of 0 ("no row kept") and multiply nothing, so the
        // run is straight-line code and its chunks overlap
        uint32_t words[kSRun];
        float x[kSRun][NQ];
#pragma unroll
        for (int u = 0; u < kSRun; ++u) {
          const uint32_t wd = *reinterpret_cast<const uint32_t*>(smem + cw_at + u * 128);
          words[u] = u < n ? wd : 0u;
          if (XS && NQ == 1) {
            const float xv = to_f32(*reinterpret_cast<const XT*>(smem + p.off_x + (words[u] & 0xFFFFu) * (uint32_t)sizeof(XT)));
            x[u][0] = (words[u] >> 16) ? xv : 0.f;
          } else if (XS) {
            // this column's row of the staged slice: NQ consecutive elements (unused lanes read row 0 and multiply nothing)
            const uint32_t rl = (words[u] >> 16) ? (words[u] & 0xFFFFu) - (uint32_t)(cur_slice * p.sl_rows) : 0u;
            const XT* xr = reinterpret_cast<const XT*>(smem + p.off_x + rl * (uint32_t)kRowStride);
            if (sizeof(XT) == 4) {
#pragma unroll
              for (int i = 0; i < NQ / 4; ++i) {
                const float4 v = reinterpret_cast<const float4*>(xr)[i];
                x[u][4 * i] = v.x; x[u][4 * i + 1] = v.y; x[u][4 * i + 2] = v.z; x[u][4 * i + 3] = v.w;
              }
            } else {
#pragma unroll
              for (int i = 0; i < NQ / 4; ++i) {
                const uint2 w2 = reinterpret_cast<const uint2*>(xr)[i];
                x[u][4 * i] = __uint_as_float(w2.x << 16); x[u][4 * i + 1] = __uint_as_float(w2.x & 0xFFFF0000u);
                x[u][4 * i + 2] = __uint_as_float(w2.y << 16); x[u][4 * i + 3] = __uint_as_float(w2.y & 0xFFFF0000u);
              }
            }
          } else if (words[u] >> 16) {
            load_x<NQ, XT>(p, words[u] & 0xFFFFu, q0, x[u]);
          } else {
#pragma unroll
            for (int q = 0; q < NQ; ++q) x[u][q] = 0.f;
          }
        }
        auto multiply_chunk = [&](int u) {
          const unsigned rm = words[u] >> 16;
          const unsigned step = __popc(__ballot_sync(0xffffffffu, rm != 0)) * (unsigned)sizeof(VT);  // bytes between a column's values
          const unsigned kr = __popc(__shfl_sync(0xffffffffu, rm, 0));  // equal in every column of a chunk
          uint32_t at = NQ == 1 ? smem_base + v_at : v_at;  // N = 1 walks shared-window addresses, the rest offsets
#pragma unroll
          for (int r = 0; r < BH; ++r) {
            const bool kept = (rm >> r) & 1u;
            if (NQ == 1) {
              // one row of one column: the load stays inside the stage whether the row is kept or not, so only the
              // multiply-add and the step to the column's next value are predicated
              row_step<VT>(rm, 1u << r, x[u][0], step, acc[r][0], at);
              continue;
            } else if (kept) {
              const float w = to_f32(*reinterpret_cast<const VT*>(smem + at));
#pragma unroll
              for (int q = 0; q < NQ; ++q) acc[r][q] = fmaf(w, x[u][q], acc[r][q]);
            }
            at += kept ? step : 0u;
          }
          v_at += kr * step;
        };
        const bool long_run = n > kSRun / 2;  // a short run holds nothing in its second half
#pragma unroll
        for (int u = 0; u < kSRun; ++u)
          if (u < kSRun / 2 || long_run) multiply_chunk(u);
        __syncwarp();  // every lane is done with the stage before it is filled again
        issue(pend0, slot);
        pend0 = pend1;
        pend1 = prepare();
        if (++slot == nslots) { slot = 0; phase ^= 1u; }
      }
      float* mine = part + ((size_t)b * NW + warp) * (BH * NQ);
      if (XS && NQ > 1 && !had_run) continue;  // (the same in every lane) this warp had no run of the band
#pragma unroll
      for (int q = 0; q < NQ; ++q) {
        float t[BH];
#pragma unroll
        for (int r = 0; r < BH; ++r) t[r] = acc[r][q];
        warp_reduce_rows<BH>(t, lane);
        mine[myrow * NQ + q] = t[0];  // lanes that share a row hold the same total
      }
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < nb * BH * NQ; idx += NW * 32) {
      const int b = idx / (BH * NQ), rq = idx % (BH * NQ);
      const int r = rq / NQ, q = rq % NQ;
      const int64_t row = (int64_t)s_first_row[kb + b] + r;
      if (r >= p.bh || row >= p.M || q0 + q >= p.N) continue;
      float s = 0.f;
#pragma unroll 4
      for (int w = 0; w < NW; ++w) s += part[((size_t)b * NW + w) * (BH * NQ) + rq];
      if (p.accumulate) {  // (fp32 only) one of several slices' share of this element; Y was cleared before the launch
        if (s != 0.f) atomicAdd(static_cast<float*>(p.Y) + row * p.ldy + q0 + q, s);
      } else if (p.y_dtype == GRIM_F32) static_cast<float*>(p.Y)[row * p.ldy + q0 + q] = s;
      else static_cast<__nv_bfloat16*>(p.Y)[row * p.ldy + q0 + q] = __float2bfloat16_rn(s);
    }
    __syncthreads();
  }
  if (failed) {
    // copies that were requested still land in this block's shared memory: give them a bounded time to finish
    for (int s = 0; s < nslots; ++s)
      for (unsigned i = 0; i < 4096u && !mbar_try_wait(my_full + s, 0) && !mbar_try_wait(my_full + s, 1); ++i) {}
  }
}

struct StreamPlan {
  int nq, nw, passes, nslots, grid_x, nk_max;
  bool xs;
  uint32_t stage_bytes, off_band, off_part, off_x, off_ring;
  size_t smem;
};

// staged: N > 1 with the current K slice of X in shared memory; nv = number of (virtual) bands the launch walks
bool make_plan(const grim_bcr* h, int64_t N, StreamPlan& pl, bool staged = false, int64_t nv = 0) {
  if (h->device < 0 || !h->gemv_ok || !h->d_status || !h->d_runs || N < 1 || N > kSkinnyMaxN || h->nchunks == 0) return false;
  if (nv <= 0) nv = h->nbr;
  const int BHc = h->bh <= 4 ? 4 : (h->bh <= 8 ? 8 : 16);
  const int esz = h->dtype == GRIM_F32 ? 4 : 2;
  pl.nq = N == 1 ? 1 : (N <= 4 ? 4 : (N <= 8 ? 8 : 16));
  if (BHc == 16 && pl.nq == 16) pl.nq = 8;  // 16 x 16 accumulators do not fit the register file: two passes of 8
  // the wide right-hand sides hold more accumulators: fewer warps
  pl.nw = pl.nq <= 4 ? 16 : 8;
  pl.passes = (int)((N + pl.nq - 1) / pl.nq);
  pl.grid_x = (int)std::min<int64_t>(nv, sm_count(h->device));
  pl.nk_max = (int)((nv + pl.grid_x - 1) / pl.grid_x);
  if (pl.nk_max > kSMaxBands) return false;
  const int pb = std::max(1, part_bytes(staged) / (pl.nw * BHc * pl.nq * 4));
  auto up = [](size_t v, size_t a) { return (v + a - 1) / a * a; };
  // column words of a run, its values, the skipped elements in front, the rounding behind, and one warp's width
  // that a lane of a pruned row may read and discard
  pl.stage_bytes = (uint32_t)up((size_t)kSRun * 128 + (size_t)kRunValueBytes + 32 + 32 * esz, 128);
  const size_t budget = 227 * 1024;
  // the activation vector is staged in shared memory when it fits beside two stages per warp
  const size_t x_bytes = pl.nq == 1 ? (size_t)h->K * esz : (size_t)h->sl_rows * x_row_stride(pl.nq, esz);
  if (staged && (pl.nq == 1 || x_bytes > (size_t)kSMaxXBytes)) return false;
  for (int xs = ((staged || pl.nq == 1) && x_bytes <= (size_t)kSMaxXBytes) ? 1 : 0; xs >= (staged ? 1 : 0); --xs) {
    size_t off = up((size_t)pl.nw * kSMaxSlots * 12 + 16, 128);
    pl.off_band = (uint32_t)off;
    off = up(off + (size_t)pl.nk_max * 16, 16);
    pl.off_part = (uint32_t)off;
    off = up(off + (size_t)pb * pl.nw * BHc * pl.nq * 4, 16);
    pl.off_x = (uint32_t)off;
    if (xs) off += x_bytes;
    off = up(off, 128);
    pl.off_ring = (uint32_t)off;
    if (off + (size_t)2 * pl.nw * pl.stage_bytes > budget) continue;
    pl.xs = xs != 0;
    pl.nslots = (int)std::min<size_t>(kSMaxSlots, (budget - off) / ((size_t)pl.nw * pl.stage_bytes));
    pl.smem = off + (size_t)pl.nslots * pl.nw * pl.stage_bytes;
    return true;
  }
  return false;
}

template <int BH, int NQ, int NW, bool XS, typename VT>
cudaError_t launch_kernel(const StreamParams& p, const StreamPlan& pl, cudaStream_t s) {
  auto kern = bcr_stream_kernel<BH, NQ, NW, XS, VT, VT>;
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), pl.smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)pl.grid_x, (unsigned)pl.passes);
  cfg.blockDim = dim3(NW * 32);
  cfg.dynamicSmemBytes = pl.smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // may overlap the tail of the launch before it
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, p);
}

template <int BH, typename VT>
cudaError_t launch_nq(const StreamParams& p, const StreamPlan& pl, cudaStream_t s) {
  constexpr int NWS = 16;  // warps of the N <= 4 variants
  constexpr int NW1 = 16;  // warps of the N = 1 variants
  switch (pl.nq) {
    case 1:
      return pl.xs ? launch_kernel<BH, 1, NW1, true, VT>(p, pl, s) : launch_kernel<BH, 1, NW1, false, VT>(p, pl, s);
    case 4:
      return pl.xs ? launch_kernel<BH, 4, NWS, true, VT>(p, pl, s) : launch_kernel<BH, 4, NWS, false, VT>(p, pl, s);
    case 8: return pl.xs ? launch_kernel<BH, 8, 8, true, VT>(p, pl, s) : launch_kernel<BH, 8, 8, false, VT>(p, pl, s);
    default:
      if (BH > 8) return cudaErrorInvalidValue;
      return pl.xs ? launch_kernel<(BH <= 8 ? BH : 8), 16, 8, true, VT>(p, pl, s)
                   : launch_kernel<(BH <= 8 ? BH : 8), 16, 8, false, VT>(p, pl, s);
  }
}

template <typename VT>
cudaError_t launch_bh(const StreamParams& p, const StreamPlan& pl, int BHc, cudaStream_t s) {
  if (BHc == 4) return launch_nq<4, VT>(p, pl, s);
  if (BHc == 8) return launch_nq<8, VT>(p, pl, s);
  return launch_nq<16, VT>(p, pl, s);
}

}  // namespace

bool stream_path_supported(const grim_bcr* h, int64_t N) {
  StreamPlan pl;
  return make_plan(h, N, pl);
}

grim_status_t launch_stream(const grim_bcr* h, const void* X, int x_dtype, int64_t ldx, int64_t N, void* Y, int y_dtype,
                            int64_t ldy, cudaStream_t s) {
  StreamPlan pl;
  if (x_dtype != h->dtype) return GRIM_ERR_DTYPE;
  StreamParams p;
  p.run_ptr = h->d_run_ptr; p.runs = h->d_runs; p.colwords = h->d_colwords;
  p.vals = static_cast<const uint8_t*>(h->d_gemv_vals);
  p.band_order = h->d_band_order; p.X = X; p.Y = Y; p.status = h->d_status; p.ldx = ldx; p.ldy = ldy;
  p.N = (int)N; p.nbr = (int)h->nbr; p.M = (int)h->M; p.K = (int)h->K; p.bh = h->bh; p.y_dtype = y_dtype;
  p.slice_of = nullptr; p.sl_rows = h->sl_rows; p.accumulate = 0;
  // 2 <= N <= 16: the rows of X a thread block needs are staged in shared memory - all of them when K is a single
  // slice, else slice by slice on the slice-major copy of the layout, the slices' shares of Y added atomically
  // (fp32 outputs; others gather the activations from L2 per band as before)
  // (measured at 8192 x 8192, c = 4, fp32: N = 4: 68 us staged against 87 us gathered, N = 8: 122 against 150; at
  // N = 16 the slices leave each band too few runs per warp and the gathered walk is faster: 94 against 165 us)
  bool staged = false;
  if (N >= 2 && N <= 8 && h->sl_rows > 0) {
    if (h->sl_nslices <= 1) {
      staged = make_plan(h, N, pl, true, h->nbr);
    } else if (h->d_sl_runs && y_dtype == GRIM_F32 && make_plan(h, N, pl, true, h->sl_nslices * h->nbr)) {
      staged = true;
      p.run_ptr = h->d_sl_run_ptr; p.runs = h->d_sl_runs; p.colwords = h->d_sl_colwords;
      p.vals = static_cast<const uint8_t*>(h->d_sl_vals);
      p.band_order = h->d_sl_band_of; p.slice_of = h->d_sl_slice_of;
      p.nbr = (int)(h->sl_nslices * h->nbr);
      p.accumulate = 1;
      if (cudaMemset2DAsync(Y, (size_t)ldy * 4, 0, (size_t)N * 4, (size_t)h->M, s) != cudaSuccess) return GRIM_ERR_CUDA;
    }
  }
  if (!staged && !make_plan(h, N, pl)) return GRIM_ERR_UNSUPPORTED;
  const int esz = x_dtype == GRIM_F32 ? 4 : 2;
  p.vec_ok = (N % pl.nq == 0) && ldx % 4 == 0 && (reinterpret_cast<uintptr_t>(X) % (4 * esz)) == 0;
  const int piece = pl.nq * esz >= 16 ? 16 : 8;
  p.stage_vec = (N % pl.nq == 0) && pl.nq * esz >= 8 && (ldx * esz) % piece == 0 && (reinterpret_cast<uintptr_t>(X) % piece) == 0;
  p.nslots = pl.nslots; p.nk_max = pl.nk_max; p.stage_bytes = pl.stage_bytes;
  p.off_band = pl.off_band; p.off_part = pl.off_part; p.off_x = pl.off_x; p.off_ring = pl.off_ring;
  p.spin_limit = 1u << 22;
  const int BHc = h->bh <= 4 ? 4 : (h->bh <= 8 ? 8 : 16);
  cudaError_t e = h->dtype == GRIM_F32 ? launch_bh<float>(p, pl, BHc, s) : launch_bh<__nv_bfloat16>(p, pl, BHc, s);
  count_launch();
  return e == cudaSuccess ? GRIM_OK : GRIM_ERR_CUDA;
}

}  // namespace grim
