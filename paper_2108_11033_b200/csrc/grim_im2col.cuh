// Implicit im2col for the tensor-core kernels (Section 3.1: a convolution is a GEMM whose right-hand side is the
// expanded input; Section 4.5: that matrix is never produced in memory).  Same-size 3 x 3 convolutions, stride 1,
// pad 1, bf16, NCHW: with W = OW the input element of tap (kh, kw) for output pixel pix is
// plane[pix + (kh - 1) * W + (kw - 1)], so a row of the X tile (one k = (c, kh, kw), 256 consecutive pixels) is a
// shifted copy of the input plane with zeros where the tap leaves the image.
//
// Two pieces, shared by the single-block and the paired kernel:
//   conv_copy_planes  (one warp)   stages, per K tile, the stretch of every input plane the tile touches in a ring of
//                                  shared-memory segments (variants 2 and 3),
//   conv_build_tiles  (a group of  builds the 64 x 256 tile in the tensor core's N-major 128-byte-swizzled layout from
//                     four warps)  those segments (2, 3) or straight from global memory (1).
// Variant 1 = planes read from global memory; 2 = planes staged by bulk copies (plane size a multiple of 8 pixels);
// 3 = planes staged by 8-byte asynchronous copies (a multiple of 4: plane starts are not all 16-byte aligned).
#pragma once
#include <cuda_bf16.h>

#include "grim_device.cuh"
#include "grim_internal.h"

namespace grim {

constexpr int kImTileCols = 256;  // pixels (GEMM columns) per tile
constexpr int kImTileK = 64;      // k per tile
constexpr int kImBuildWarps = 4;  // warps of a builder group

struct Im2colCtx {
  const SpmmArgs* a;
  int K;               // C * 9
  int in_elems;        // elements of the input tensor (< 2^31)
  int seg_off, seg_len, nseg;
  uint32_t seg_bytes;
  int64_t q0;          // first pixel column of this block's tile
  int nkt, kbase;      // K tiles this block walks, and the first of them
  int ns;              // tile slots
  uint8_t* stages;     // X tile of slot s at stages + s * stage_bytes + b_off
  uint32_t stage_bytes, b_off;
  uint8_t* segs;
  uint64_t *empty, *seg_full, *seg_free, *built;
  int built_rank;      // -1: arrive on built[slot] of this block; r >= 0: on built[slot] of block r of the cluster
  bool cluster_waits;  // the `empty` barriers are completed from another block (wait with cluster-scope acquire)
  unsigned spin_limit;
  const volatile int* s_abort;
};

// Staged variants: elements kept in front of the tile's first pixel in a channel segment (a row and a pixel, rounded
// to vectors, plus one vector), the segment's length, and the bytes of one slot of the ring of planes (eight channels
// at most touch a K tile of 64).  Needs planes whose size is a multiple of 4 pixels (8-byte copies; multiples of 8 take
// 16-byte-aligned bulk copies) and tiles that meet at most three images.
constexpr int kImSegSlots = 4;  // slots of the ring of staged planes at most
inline bool conv_staging(const SpmmArgs& a, int* seg_off, int* seg_len, size_t* seg_bytes) {
  const int64_t ohw = (int64_t)a.OH * a.OW;
  if (!a.conv || ohw % 4 != 0 || ohw < kImTileCols / 2) return false;  // multiples of 8: bulk copies, of 4: 8-byte copies
  if (ohw % 8 != 0 && (kImTileCols + 2 * ((a.W + 1 + 7) / 8 * 8 + 8)) * 2 / 8 > 8 * 32) return false;  // 8 pieces per lane at most
  *seg_off = (a.W + 1 + 7) / 8 * 8 + 8;
  *seg_len = kImTileCols + 2 * *seg_off;
  *seg_bytes = ((size_t)8 * *seg_len * 2 + 16 + 127) / 128 * 128;
  return true;
}
// The tile builders cover the common same-size 3 x 3 convolution on tensors of fewer than 2^31 elements.
inline bool conv_tiles_supported(const SpmmArgs& a) {
  if (a.KH != 3 || a.KW != 3 || a.stride != 1 || a.pad != 1 || a.OH != a.H || a.OW != a.W) return false;
  return a.ncols / ((int64_t)a.OH * a.OW) * a.C * a.H * a.W < (int64_t(1) << 31) - 64;
}

__device__ __forceinline__ bool im_wait(const Im2colCtx& c, uint64_t* bar, unsigned parity, bool cluster) {
  return cluster ? ptx::mbar_wait<true>(bar, parity, c.spin_limit, c.s_abort) : ptx::mbar_wait<false>(bar, parity, c.spin_limit, c.s_abort);
}

// Staged variants: per K tile the (at most eight) input channels it touches, and of each the stretch of the plane
// that the tile's 256 pixels and their 3 x 3 neighbourhoods cover, one copy per channel and image.  A channel's
// segment holds tile pixel q at element seg_off + q; where the tile runs into the next image that image's plane
// follows directly (taps that would cross the boundary are masked anyway).  The ring of segments is freed by the
// builders, long before the tensor core is done with the tile built from them, so the copies run several K tiles
// ahead.  Whole warp; returns false when a bounded wait gave up.
template <int CONV>
__device__ __forceinline__ bool conv_copy_planes(const Im2colCtx& c, int lane) {
  const SpmmArgs& a = *c.a;
  const int ohw = a.OH * a.OW;
  const __nv_bfloat16* in = static_cast<const __nv_bfloat16*>(a.X);
  const int64_t q0 = c.q0;
  const int64_t q_end = q0 + kImTileCols < a.ncols ? q0 + kImTileCols : a.ncols;
  if (q0 >= a.ncols) {
    // nothing of this tile exists: the segments still have to be reported, or the builders would wait for ever
    for (int kt = 0; kt < c.nkt; ++kt) {
      const int ss = kt % c.nseg;
      if (kt >= c.nseg && !__all_sync(0xffffffffu, im_wait(c, c.seg_free + ss, (unsigned)((kt / c.nseg - 1) & 1), false))) return false;
      if (CONV == 3) ptx::mbar_arrive(c.seg_full + ss);
      else if (lane == 0) ptx::mbar_arrive(c.seg_full + ss);
    }
    return true;
  }
  const int n0 = (int)(q0 / ohw), n1 = (int)((q_end - 1) / ohw);
  int src_lo[3], dst_idx[3];
  unsigned nbytes[3], per_channel = 0;
  const int nimg = n1 - n0 + 1;  // <= 3 (checked on the host)
  for (int i = 0; i < nimg; ++i) {
    const int64_t img0 = (int64_t)(n0 + i) * ohw;
    const int qa = (int)((q0 > img0 ? q0 : img0) - q0);
    const int qb = (int)((q_end < img0 + ohw ? q_end : img0 + ohw) - q0);
    const int pa = (int)(q0 + qa - img0), pb = pa + (qb - qa);
    const int lo = pa - c.seg_off > 0 ? pa - c.seg_off : 0;
    const int hi = pb + c.seg_off < ohw ? pb + c.seg_off : ohw;
    src_lo[i] = lo;
    dst_idx[i] = lo - pa + qa + c.seg_off;
    nbytes[i] = (unsigned)(hi - lo) * 2u;
    per_channel += nbytes[i];
  }
  // 8-byte variant: the pieces of a channel's segment this lane copies (pieces lane, lane + 32, ...): byte offset
  // in the segment and element offset in the input relative to channel 0 of image 0; -1: none
  constexpr int kPiecesPerLane = 8;
  int piece_dst[kPiecesPerLane], piece_src[kPiecesPerLane];
  if (CONV == 3) {
#pragma unroll
    for (int t = 0; t < kPiecesPerLane; ++t) {
      int rem = lane + 32 * t, i = 0;
      while (i + 1 < nimg && rem >= (int)(nbytes[i] >> 3)) { rem -= (int)(nbytes[i] >> 3); ++i; }
      const bool ok = rem < (int)(nbytes[i] >> 3);
      piece_dst[t] = ok ? dst_idx[i] * 2 + rem * 8 : -1;
      piece_src[t] = ok ? (n0 + i) * a.C * ohw + src_lo[i] + rem * 4 : 0;
    }
  }
  for (int kt = 0; kt < c.nkt; ++kt) {
    const int ss = kt % c.nseg;
    if (kt >= c.nseg && !__all_sync(0xffffffffu, im_wait(c, c.seg_free + ss, (unsigned)((kt / c.nseg - 1) & 1), false))) return false;
    uint8_t* seg = c.segs + (size_t)ss * c.seg_bytes;
    const int c_lo = (c.kbase + kt) * kImTileK / 9;
    const int k_hi = (c.kbase + kt + 1) * kImTileK < c.K ? (c.kbase + kt + 1) * kImTileK - 1 : c.K - 1;
    const int nch = k_hi / 9 - c_lo + 1;
    if (CONV == 3) {
      // 8-byte pieces: a lane copies the same pieces of every channel (worked out once, above); its arrival is
      // deferred until its copies have landed
      for (int ci = 0; ci < nch; ++ci) {
        uint8_t* dch = seg + (size_t)ci * c.seg_len * 2;
        const __nv_bfloat16* sch = in + (int64_t)(c_lo + ci) * ohw;
#pragma unroll
        for (int t = 0; t < kPiecesPerLane; ++t)
          if (piece_dst[t] >= 0) ptx::cp_async8(dch + piece_dst[t], sch + piece_src[t]);
      }
      ptx::cp_async_arrive_noinc(c.seg_full + ss);
      continue;
    }
    if (lane == 0) ptx::mbar_arrive_expect_tx(c.seg_full + ss, per_channel * (unsigned)nch);
    __syncwarp();  // the byte count is announced before any copy can complete
    // one copy per lane: a single thread needs several hundred cycles per copy it issues
    for (int idx = lane; idx < nch * nimg; idx += 32) {
      const int ci = idx / nimg, i = idx - ci * nimg;
      ptx::bulk_load(seg + ((size_t)ci * c.seg_len + dst_idx[i]) * 2,
                     in + ((int64_t)(n0 + i) * a.C + c_lo + ci) * ohw + src_lo[i], nbytes[i], c.seg_full + ss);
    }
  }
  return true;
}

// Element-wise construction of one 8-pixel piece of an im2col row (pieces that cross into the next image or touch
// the end of the tensor).  Kept out of line so that the common vector path stays short.
static __device__ __noinline__ uint4 im2col_piece_slow(const unsigned short* in1, int in_elems, int plane0, int plane1, int c_off,
                                                int pix0, int split, int shift, uint32_t bad) {
  uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    const int ee = (e < split ? plane0 + pix0 + e : plane1 + e - split) + c_off + shift;
    const uint32_t val = (!((bad >> e) & 1u) && ee >= 0 && ee < in_elems) ? in1[ee] : 0u;
    w[e >> 1] |= val << ((e & 1) * 16);
  }
  return make_uint4(w[0], w[1], w[2], w[3]);
}

// The 16-byte piece that starts `rb & 7` elements into the vector pair (l, h).
__device__ __forceinline__ uint4 im_shift_pair(const uint4& l, const uint4& h, int rb) {
  const int sb = (rb & 1) * 16;
  switch ((rb >> 1) & 3) {  // 32-bit word of the vector pair at which the piece starts
    case 0: return make_uint4(__funnelshift_r(l.x, l.y, sb), __funnelshift_r(l.y, l.z, sb), __funnelshift_r(l.z, l.w, sb), __funnelshift_r(l.w, h.x, sb));
    case 1: return make_uint4(__funnelshift_r(l.y, l.z, sb), __funnelshift_r(l.z, l.w, sb), __funnelshift_r(l.w, h.x, sb), __funnelshift_r(h.x, h.y, sb));
    case 2: return make_uint4(__funnelshift_r(l.z, l.w, sb), __funnelshift_r(l.w, h.x, sb), __funnelshift_r(h.x, h.y, sb), __funnelshift_r(h.y, h.z, sb));
    default: return make_uint4(__funnelshift_r(l.w, h.x, sb), __funnelshift_r(h.x, h.y, sb), __funnelshift_r(h.y, h.z, sb), __funnelshift_r(h.z, h.w, sb));
  }
}
// Clears the pixels (16-bit elements) of a piece whose bit is set in `bad`.
__device__ __forceinline__ uint4 im_clear(uint4 out, uint32_t bad) {
  uint32_t w[4] = {out.x, out.y, out.z, out.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint32_t b2 = (bad >> (2 * i)) & 3u;
    w[i] &= ~((b2 & 1u ? 0xFFFFu : 0u) | (b2 & 2u ? 0xFFFF0000u : 0u));
  }
  return make_uint4(w[0], w[1], w[2], w[3]);
}

// A builder group (kImBuildWarps warps, thread bt = 0 .. 127 inside it) takes K tiles bgrp, bgrp + ngroups, ... and
// writes each as the 64 x 256 X tile of its slot.  A thread owns one 16-byte piece (8 pixels) of a row: it reads the
// two aligned 16-byte vectors that cover it, shifts, clears the out-of-image pixels (four masks that are fixed per
// thread: pixel on the left / right / top / bottom edge) and stores the piece where the 128-byte swizzled N-major
// layout wants it.  Returns false when a bounded wait gave up (fail_site says which).
template <int CONV>
__device__ __forceinline__ bool conv_build_tiles(const Im2colCtx& c, int bgrp, int ngroups, int bt, int lane, int& fail_site) {
  const SpmmArgs& a = *c.a;
  const int cq = bt & 31;  // this thread's piece of the row
  const int64_t qc = c.q0 + cq * 8;
  const int ohw = a.OH * a.OW;
  const __nv_bfloat16* in = static_cast<const __nv_bfloat16*>(a.X);
  const int in_elems = c.in_elems;
  uint32_t m_left = 0, m_right = 0, m_top = 0, m_bottom = 0, m_off = 0;  // bit e: pixel e of the piece
  int plane0, plane1, pix0;  // element offsets of channel 0 of the image of the first / last pixel; first pixel
  {
    const int64_t img = qc / ohw, img1 = (qc + 7) / ohw;
    pix0 = (int)(qc - img * ohw);
    plane0 = (int)(img * a.C * ohw);
    plane1 = (int)(img1 * a.C * ohw);
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int64_t q = qc + e;
      if (q >= a.ncols) { m_off |= 1u << e; continue; }
      const int pe = (int)(q - (q / ohw) * ohw);
      const int oh = pe / a.OW, ow = pe - oh * a.OW;
      if (ow == 0) m_left |= 1u << e;
      if (ow == a.OW - 1) m_right |= 1u << e;
      if (oh == 0) m_top |= 1u << e;
      if (oh == a.OH - 1) m_bottom |= 1u << e;
    }
    if (qc >= a.ncols) { plane0 = plane1 = 0; pix0 = 0; }
  }
  const int split = (plane1 != plane0) ? (ohw - pix0) : 8;  // pixels of the piece that lie in the first image
  const uint32_t panel_off = (uint32_t)(cq >> 3) * (64 * kImTileK * 2);  // 64-pixel panel of the tile
  const uint32_t piece = (uint32_t)(cq & 7);
  const uint4* in16 = reinterpret_cast<const uint4*>(in);
  const unsigned short* in1 = reinterpret_cast<const unsigned short*>(in);
  const int nvec = in_elems >> 3;  // complete 16-byte vectors of the tensor
  for (int kt = bgrp; kt < c.nkt; kt += ngroups) {
    const int slot = kt % c.ns;
    const int ss = CONV >= 2 ? kt % c.nseg : 0;
    if (kt >= c.ns && !__all_sync(0xffffffffu, im_wait(c, c.empty + slot, (unsigned)((kt / c.ns - 1) & 1), c.cluster_waits))) { fail_site = 3; return false; }
    // staged variants: the planes of this K tile have landed (their copies were requested several tiles ago)
    if (CONV >= 2 && !__all_sync(0xffffffffu, im_wait(c, c.seg_full + ss, (unsigned)((kt / c.nseg) & 1), false))) { fail_site = 7; return false; }
    uint8_t* bt_base = c.stages + (size_t)slot * c.stage_bytes + c.b_off + panel_off;
    if (CONV >= 2) {
      // Row kk of the tile is k = (c, kh, kw); the warp takes rows w, w + 4, ... and keeps (c, tap) up to date without
      // dividing.  Everything that depends on the row only is the same in all lanes: the first element of the row in
      // the channel's segment (rb), hence the shift inside a vector; a lane adds its piece.
      const int w0 = bt >> 5;
      const uint32_t seg_s = ptx::smem_u32(c.segs + (size_t)ss * c.seg_bytes), bt_s = ptx::smem_u32(bt_base);
      const int k0 = (c.kbase + kt) * kImTileK;  // first k of this tile
      int c_rel = (k0 + w0) / 9 - k0 / 9;        // channel relative to the first one staged for this K tile
      int tap = (k0 + w0) % 9;
      // rows in batches: first the shared-memory loads of the whole batch (so that their latencies overlap), then
      // shifting, masking and storing
      constexpr int kRows = 4;
      for (int kk0 = w0; kk0 < kImTileK; kk0 += kImBuildWarps * kRows) {
        uint4 lo[kRows], hi[kRows];
        int rbs[kRows], taps[kRows];
#pragma unroll
        for (int bb = 0; bb < kRows; ++bb) {
          const int kh = tap >= 6 ? 2 : (tap >= 3 ? 1 : 0), kw = tap - 3 * kh;
          const int rb = c_rel * c.seg_len + c.seg_off + (kh - 1) * a.W + (kw - 1);
          rbs[bb] = rb;
          taps[bb] = kh * 4 + kw;
          lo[bb] = ptx::lds128(seg_s + (uint32_t)((rb >> 3) + cq) * 16u);
          hi[bb] = ptx::lds128(seg_s + (uint32_t)((rb >> 3) + cq + 1) * 16u);
          tap += kImBuildWarps;
          if (tap >= 9) { tap -= 9; ++c_rel; }
        }
#pragma unroll
        for (int bb = 0; bb < kRows; ++bb) {
          const int kk = kk0 + bb * kImBuildWarps;
          uint4 out = make_uint4(0u, 0u, 0u, 0u);
          if (k0 + kk < c.K) {
            const int kh = taps[bb] >> 2, kw = taps[bb] & 3;
            out = im_shift_pair(lo[bb], hi[bb], rbs[bb]);
            const uint32_t bad = m_off | (kw == 0 ? m_left : 0u) | (kw == 2 ? m_right : 0u) | (kh == 0 ? m_top : 0u) | (kh == 2 ? m_bottom : 0u);
            if (bad) out = im_clear(out, bad);  // pixels whose tap lies outside the image
          }
          ptx::sts128(bt_s + (uint32_t)kk * 128u + ((piece ^ ((uint32_t)kk & 7u)) << 4), out.x, out.y, out.z, out.w);
        }
      }
    } else {
      // The thread's 16 rows of the stage are taken in batches: first the address arithmetic and the vector loads
      // of the whole batch (so that they are in flight together), then shifting, masking, storing.
      constexpr int kBatch = 4;
      for (int kk0 = bt >> 5; kk0 < kImTileK; kk0 += kImBuildWarps * kBatch) {
        uint4 lo[kBatch], hi[kBatch];
        uint32_t info[kBatch];  // bits 0-7: pixels to clear, 8-10: shift inside the vector, 12-13: 0 zeros / 1 vectors / 2 element-wise
#pragma unroll
        for (int bb = 0; bb < kBatch; ++bb) {
          const int kk = kk0 + bb * kImBuildWarps;
          const int kg = (c.kbase + kt) * kImTileK + kk;
          lo[bb] = make_uint4(0u, 0u, 0u, 0u);
          hi[bb] = make_uint4(0u, 0u, 0u, 0u);
          info[bb] = 0;
          if (kg >= c.K || m_off == 0xFFu) continue;
          const int ch = kg / 9, tap = kg - ch * 9;
          const int kh = tap / 3, kw = tap - kh * 3;
          const uint32_t bad = m_off | (kw == 0 ? m_left : 0u) | (kw == 2 ? m_right : 0u) | (kh == 0 ? m_top : 0u) | (kh == 2 ? m_bottom : 0u);
          if (bad == 0xFFu) continue;
          const int e0 = plane0 + ch * ohw + pix0 + (kh - 1) * a.W + (kw - 1);
          const int v0 = e0 >> 3;  // floor: the vector that holds the first pixel (negative at the very start)
          const int sh = e0 & 7;
          // pieces that cross into the next image, or whose vectors are not both complete vectors of the tensor
          // (its very end), are built element by element
          if (split != 8 || v0 + 1 >= nvec) { info[bb] = bad | (2u << 12); continue; }
          if (v0 >= 0) lo[bb] = __ldg(in16 + v0);
          if (sh != 0 && v0 + 1 >= 0) hi[bb] = __ldg(in16 + v0 + 1);
          info[bb] = bad | ((uint32_t)sh << 8) | (1u << 12);
        }
#pragma unroll
        for (int bb = 0; bb < kBatch; ++bb) {
          const int kk = kk0 + bb * kImBuildWarps;
          const uint32_t bad = info[bb] & 0xFFu, mode = info[bb] >> 12;
          uint4 out = make_uint4(0u, 0u, 0u, 0u);
          if (mode == 1u) {
            out = im_shift_pair(lo[bb], hi[bb], (int)((info[bb] >> 8) & 7u));
            if (bad) out = im_clear(out, bad);
          } else if (mode == 2u) {
            const int kg = (c.kbase + kt) * kImTileK + kk;
            const int ch = kg / 9, tap = kg - ch * 9;
            const int kh = tap / 3, kw = tap - kh * 3;
            out = im2col_piece_slow(in1, in_elems, plane0, plane1, ch * ohw, pix0, split, (kh - 1) * a.W + (kw - 1), bad);
          }
          *reinterpret_cast<uint4*>(bt_base + (uint32_t)kk * 128u + ((piece ^ ((uint32_t)kk & 7u)) << 4)) = out;
        }
      }
    }
    ptx::fence_proxy_async();
    __syncwarp();
    if (lane == 0) {
      if (c.built_rank < 0) ptx::mbar_arrive(c.built + slot);
      else ptx::mbar_arrive_remote(c.built + slot, (uint32_t)c.built_rank);
      if (CONV >= 2) ptx::mbar_arrive(c.seg_free + ss);
    }
  }
  return true;
}

}  // namespace grim
