// CUDA-core kernels for Y = W * X with W in packed BCR form (Sections 3.1, 4.2, 4.4, 4.5).
//
//  bcr_spmm_kernel  N > 1.  One thread block owns a group of G row bands and a tile of output columns and
//                   walks the block columns.  Per block column the needed slab of X (bw rows x tile) is
//                   staged once in shared memory and reused by every band of the group and by every kept
//                   row of every block (each input row is loaded once and reused - the load-redundancy
//                   idea of Section 4.4, at shared-memory level); the group's descriptors and kept values
//                   arrive as one contiguous piece ("blob") through cp.async.  With CONV the slab is
//                   produced on the fly from the NCHW input (implicit im2col, Section 4.5); rows whose
//                   column is kept by no block of the group are not read.
//  bcr_skinny_kernel  N <= 16 (N = 1: matrix-vector).  A warp owns (part of) a band; a lane owns one kept
//                   column of one block, reads its activations once and multiplies them with that column's
//                   kr kept values (coalesced across lanes), accumulating into per-row registers selected
//                   by the block's row mask.
#include <cuda_bf16.h>

#include <atomic>

#include "grim_device.cuh"
#include <mutex>
#include <unordered_map>

#include "grim_internal.h"

namespace grim {

static std::atomic<long long> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

cudaError_t ensure_dynamic_smem(const void* kernel, size_t bytes) {
  static std::mutex mu;
  static std::unordered_map<const void*, size_t> have;
  std::lock_guard<std::mutex> lock(mu);
  size_t& h = have[kernel];
  if (h >= bytes) return cudaSuccess;
  const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess) h = bytes;
  return e;
}

int sm_count(int device) {
  constexpr int kFallback = 148;  // B200; used only when the attribute cannot be read
  static int cached[64] = {0};
  if (device < 0 || device >= 64) return kFallback;
  if (!cached[device]) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || n <= 0) {
      cudaGetLastError();
      n = kFallback;
    }
    cached[device] = n;
  }
  return cached[device];
}
long long launches() { return g_launches.load(std::memory_order_relaxed); }
void launches_reset() { g_launches.store(0, std::memory_order_relaxed); }

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxUnits = 8;  // float4 slab units per thread (bw <= 64, tile <= 128)

struct KParams {
  const StageEntry* stage;
  const uint8_t* blob;
  const uint32_t* band_order;
  int nbr, nbc, M, K, bh, bw, G;
  uint32_t blob_stride;  // bytes reserved per blob buffer in shared memory
  SpmmArgs a;
};

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
  unsigned s = (unsigned)__cvta_generic_to_shared(smem);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit_wait_all() {
  asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;\n" ::: "memory");
}

// Loads one slab unit: 4 consecutive output columns of slab row kk of block column j.
template <bool CONV>
__device__ __forceinline__ float4 load_unit(const KParams& p, int64_t k, int64_t q, const int64_t* qbase,
                                            const int* ih0, const int* iw0, bool vec_ok) {
  float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
  if (k >= p.K) return r;
  const SpmmArgs& a = p.a;
  if (!CONV) {
    if (vec_ok && q + 3 < a.ncols) {
      if (a.x_dtype == GRIM_F32) {
        r = __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(a.X) + k * a.x_sk + q));
      } else {
        uint2 u = __ldg(reinterpret_cast<const uint2*>(static_cast<const __nv_bfloat16*>(a.X) + k * a.x_sk + q));
        r.x = __uint_as_float(u.x << 16);
        r.y = __uint_as_float(u.x & 0xFFFF0000u);
        r.z = __uint_as_float(u.y << 16);
        r.w = __uint_as_float(u.y & 0xFFFF0000u);
      }
      return r;
    }
    float t[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      t[e] = 0.f;
      if (q + e < a.ncols) {
        const int64_t off = k * a.x_sk + (q + e) * a.x_sq;
        t[e] = a.x_dtype == GRIM_F32 ? __ldg(static_cast<const float*>(a.X) + off)
                                     : __bfloat162float(static_cast<const __nv_bfloat16*>(a.X)[off]);
      }
    }
    return make_float4(t[0], t[1], t[2], t[3]);
  } else {
    const int khw = a.KH * a.KW;
    const int c = (int)(k / khw);
    const int rem = (int)(k - (int64_t)c * khw);
    const int kh = rem / a.KW;
    const int kw = rem - kh * a.KW;
    const int64_t koff = ((int64_t)c * a.H + kh) * a.W + kw;
    float t[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      t[e] = 0.f;
      const int ih = ih0[e] + kh, iw = iw0[e] + kw;
      if (q + e < a.ncols && ih >= 0 && ih < a.H && iw >= 0 && iw < a.W) {
        const int64_t off = qbase[e] + koff;
        t[e] = a.x_dtype == GRIM_F32 ? __ldg(static_cast<const float*>(a.X) + off)
                                     : __bfloat162float(static_cast<const __nv_bfloat16*>(a.X)[off]);
      }
    }
    return make_float4(t[0], t[1], t[2], t[3]);
  }
}

template <int BH, int BPW, int NQL, typename VT, bool CONV>
__global__ void __launch_bounds__(kThreads) bcr_spmm_kernel(const KParams p) {
  constexpr int TN = NQL * 4;
  constexpr int KQ = 32 / NQL;
  extern __shared__ __align__(16) uint8_t smem[];
  const int bw = p.bw;
  float* slab0 = reinterpret_cast<float*>(smem);
  float* slab1 = slab0 + bw * TN;
  uint8_t* blob0 = reinterpret_cast<uint8_t*>(slab1 + bw * TN);
  uint8_t* blob1 = blob0 + p.blob_stride;
  __shared__ uint8_t cols_s[kWarps][64];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nq = lane % NQL, kq = lane / NQL;
  const int64_t q0 = (int64_t)blockIdx.x * TN;
  const int group = blockIdx.y;
  const SpmmArgs& a = p.a;
  const StageEntry* st = p.stage + (int64_t)group * p.nbc;

  // slab units owned by this thread: unit u = tid + i * kThreads -> row u / NQL, column quad u % NQL
  const int units = bw * NQL;
  const int my_qq = (tid % NQL) * 4;  // constant per thread because kThreads % NQL == 0
  bool vec_ok = false;
  int64_t qbase[4] = {0, 0, 0, 0};
  int ih0[4] = {0, 0, 0, 0}, iw0[4] = {0, 0, 0, 0};
  if (!CONV) {
    const int al = a.x_dtype == GRIM_F32 ? 16 : 8;
    vec_ok = a.x_sq == 1 && (a.x_sk % 4 == 0) && (reinterpret_cast<uintptr_t>(a.X) % al == 0);
  } else {
    const int64_t ohw = (int64_t)a.OH * a.OW;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int64_t q = q0 + my_qq + e;
      const int64_t img = q / ohw;
      const int pix = (int)(q - img * ohw);
      const int oh = pix / a.OW, ow = pix - oh * a.OW;
      ih0[e] = oh * a.stride - a.pad;
      iw0[e] = ow * a.stride - a.pad;
      qbase[e] = img * a.C * a.H * a.W + (int64_t)ih0[e] * a.W + iw0[e];
    }
  }

  float4 acc[BPW][BH];
#pragma unroll
  for (int b = 0; b < BPW; ++b)
#pragma unroll
    for (int r = 0; r < BH; ++r) acc[b][r] = make_float4(0.f, 0.f, 0.f, 0.f);

  float4 stg[kMaxUnits];
  auto fetch = [&](int j) {
    const unsigned long long um = st[j].union_colmask;
#pragma unroll
    for (int i = 0; i < kMaxUnits; ++i) {
      const int u = tid + i * kThreads;
      stg[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (u < units) {
        const int kk = u / NQL;
        if ((um >> kk) & 1ull) stg[i] = load_unit<CONV>(p, (int64_t)j * bw + kk, q0 + my_qq, qbase, ih0, iw0, vec_ok);
      }
    }
  };
  auto stash = [&](float* slab) {
#pragma unroll
    for (int i = 0; i < kMaxUnits; ++i) {
      const int u = tid + i * kThreads;
      if (u < units) *reinterpret_cast<float4*>(slab + (u / NQL) * TN + my_qq) = stg[i];
    }
  };
  auto fetch_blob = [&](int j, uint8_t* dst) {
    const uint8_t* src = p.blob + (size_t)st[j].blob_off16 * 16;
    const int n16 = st[j].blob_bytes >> 4;
    for (int i = tid; i < n16; i += kThreads) cp_async16(dst + i * 16, src + i * 16);
  };
  auto next_stage = [&](int j) {
    while (j < p.nbc && st[j].blob_bytes == 0) ++j;
    return j;
  };

  int j = next_stage(0);
  if (j < p.nbc) {
    fetch_blob(j, blob0);
    fetch(j);
    stash(slab0);
    cp_async_commit_wait_all();
  }
  __syncthreads();
  int buf = 0;
  while (j < p.nbc) {
    const int jn = next_stage(j + 1);
    float* slab = buf ? slab1 : slab0;
    const uint8_t* blob = buf ? blob1 : blob0;
    if (jn < p.nbc) {
      fetch_blob(jn, buf ? blob0 : blob1);
      fetch(jn);
    }
    // ---- multiply the staged slab with this warp's blocks
    const BlockDesc* descs = reinterpret_cast<const BlockDesc*>(blob);
    const VT* vals = reinterpret_cast<const VT*>(blob + p.G * sizeof(BlockDesc));
#pragma unroll
    for (int b = 0; b < BPW; ++b) {
      const BlockDesc d = descs[warp * BPW + b];
      if (d.rowmask == 0) continue;
      const unsigned rm = d.rowmask;
      const int kc = d.kc;
      const VT* v = vals + d.val_off;
      __syncwarp();
      for (int c = lane; c < 64; c += 32)
        if ((d.colmask >> c) & 1ull) cols_s[warp][__popcll(d.colmask & ((1ull << c) - 1ull))] = (uint8_t)c;
      __syncwarp();
      for (int pcol = kq; pcol < kc; pcol += KQ) {
        const int c = cols_s[warp][pcol];
        const float4 xv = *reinterpret_cast<const float4*>(slab + c * TN + nq * 4);
        int ai = 0;
#pragma unroll
        for (int r = 0; r < BH; ++r) {
          if ((rm >> r) & 1u) {
            const float w = to_f32(v[ai * kc + pcol]);
            ++ai;
            acc[b][r].x = fmaf(w, xv.x, acc[b][r].x);
            acc[b][r].y = fmaf(w, xv.y, acc[b][r].y);
            acc[b][r].z = fmaf(w, xv.z, acc[b][r].z);
            acc[b][r].w = fmaf(w, xv.w, acc[b][r].w);
          }
        }
      }
    }
    if (jn < p.nbc) stash(buf ? slab0 : slab1);
    cp_async_commit_wait_all();
    __syncthreads();
    buf ^= 1;
    j = jn;
  }

  // ---- epilogue: combine the k-split lanes, add bias, activation, store every row of the band
  if (KQ > 1) {
#pragma unroll
    for (int b = 0; b < BPW; ++b)
#pragma unroll
      for (int r = 0; r < BH; ++r)
#pragma unroll
        for (int o = NQL; o < 32; o <<= 1) {
          acc[b][r].x += __shfl_xor_sync(0xffffffffu, acc[b][r].x, o);
          acc[b][r].y += __shfl_xor_sync(0xffffffffu, acc[b][r].y, o);
          acc[b][r].z += __shfl_xor_sync(0xffffffffu, acc[b][r].z, o);
          acc[b][r].w += __shfl_xor_sync(0xffffffffu, acc[b][r].w, o);
        }
    if (kq != 0) return;
  }
  const int64_t q = q0 + nq * 4;
  if (q >= a.ncols) return;
  const int64_t ohw = (int64_t)a.OH * a.OW;
#pragma unroll
  for (int b = 0; b < BPW; ++b) {
    const int pos = group * p.G + warp * BPW + b;
    if (pos >= p.nbr) continue;
    const int band = p.band_order[pos];
#pragma unroll
    for (int r = 0; r < BH; ++r) {
      const int64_t row = (int64_t)band * p.bh + r;
      if (r >= p.bh || row >= p.M) continue;
      float t[4] = {acc[b][r].x, acc[b][r].y, acc[b][r].z, acc[b][r].w};
      const float bias = a.bias ? __ldg(a.bias + row) : 0.f;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        t[e] += bias;
        if (a.relu) t[e] = fmaxf(t[e], 0.f);
      }
      int64_t off0;
      bool contiguous;
      if (CONV) {
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
        if (CONV) {
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
}

// ---------------------------------------------------------------------------------------------
// N <= 16 ("skinny" right-hand side, N = 1 is the matrix-vector product)
//
// A warp owns a contiguous run of a band's chunks, a lane one kept column of a chunk.  The lane reads
// the NQ activations of its column once and multiplies them with the column's kr kept values, which are
// read straight from global memory (coalesced across lanes, each value used NQ times) and accumulated
// into per-row registers selected by the block's row mask.  U chunks are processed per pass so that
// their loads are in flight together; column words have a fixed place (32 per chunk), so a pass starts
// with two independent loads (words and value offsets) instead of a dependent chain.
// ---------------------------------------------------------------------------------------------
struct SkinnyParams {
  const uint32_t* band_ptr;
  const ChunkDesc* chunks;
  const uint32_t* colwords;
  const void* vals;
  const uint32_t* band_order;
  const void* X;
  void* Y;
  int64_t ldx, ldy;
  int N, nbr, M, bh, wpb, y_dtype, vec_ok;
};

template <int NQ, typename XT>
__device__ __forceinline__ void load_x_row(const SkinnyParams& p, uint32_t col, int q0, float (&x)[NQ]) {
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

template <int BH, int NQ, int U, typename VT, typename XT>
__global__ void __launch_bounds__(kThreads) bcr_skinny_kernel(const SkinnyParams p) {
  __shared__ float part[kWarps][BH][NQ];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int wpb = p.wpb, bpc = kWarps / wpb;
  const int bi = warp / wpb, ks = warp % wpb;
  const int pos = blockIdx.x * bpc + bi;
  const int q0 = blockIdx.y * NQ;
  const VT* __restrict__ vals = static_cast<const VT*>(p.vals);
  float acc[BH][NQ];
#pragma unroll
  for (int r = 0; r < BH; ++r)
#pragma unroll
    for (int q = 0; q < NQ; ++q) acc[r][q] = 0.f;
  if (pos < p.nbr) {
    const uint32_t cbeg = p.band_ptr[pos], cend = p.band_ptr[pos + 1];
    // warp ks takes chunks cbeg + ks, cbeg + ks + wpb, ...: chunks are sorted by kept-row count, so a strided
    // share gives every warp of the band the same mix of heavy and light chunks
    const uint32_t my_beg = cbeg + ks, my_end = cend;
    // column words and value offsets of a pass are requested one pass ahead of their use
    uint32_t cw_n[U], voff_n[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const uint32_t c = my_beg + u * wpb;
      const bool live = c < my_end;
      cw_n[u] = live ? __ldg(p.colwords + (size_t)c * 32 + lane) : 0u;
      voff_n[u] = live ? __ldg(&p.chunks[c].val_off) : 0u;
    }
    for (uint32_t base = my_beg; base < my_end; base += U * wpb) {
      uint32_t cw[U], voff[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        cw[u] = cw_n[u];
        voff[u] = voff_n[u];
        const uint32_t c = base + (U + u) * wpb;
        const bool live = c < my_end;
        cw_n[u] = live ? __ldg(p.colwords + (size_t)c * 32 + lane) : 0u;
        voff_n[u] = live ? __ldg(&p.chunks[c].val_off) : 0u;
      }
      // all loads of the pass first (values land in their row's slot, 0 for rows the block does not keep),
      // so that they are in flight together; the multiplies follow
      float w[U][BH], x[U][NQ];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const unsigned rm = cw[u] >> 16;
        const int ncols = __popc(__ballot_sync(0xffffffffu, rm != 0));
        if (rm) load_x_row<NQ, XT>(p, cw[u] & 0xFFFFu, q0, x[u]);
        else {
#pragma unroll
          for (int q = 0; q < NQ; ++q) x[u][q] = 0.f;
        }
        const VT* v = vals + voff[u] + lane;
        int cnt = 0;
#pragma unroll
        for (int r = 0; r < BH; ++r) {
          // unconditional load (a pruned row re-reads the chunk's first line) + select: no branch, so every
          // load of the pass is issued before the first use
          const bool kept = (rm >> r) & 1u;
          const float val = to_f32(v[kept ? cnt * ncols : 0]);
          w[u][r] = kept ? val : 0.f;
          cnt += kept ? 1 : 0;
        }
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
#pragma unroll
        for (int r = 0; r < BH; ++r) {
          if (NQ == 1) {
            acc[r][0] = fmaf(w[u][r], x[u][0], acc[r][0]);
          } else if ((cw[u] >> (16 + r)) & 1u) {
#pragma unroll
            for (int q = 0; q < NQ; ++q) acc[r][q] = fmaf(w[u][r], x[u][q], acc[r][q]);
          }
        }
      }
    }
  }
  const int myrow = warp_row<BH>(lane);
#pragma unroll
  for (int q = 0; q < NQ; ++q) {
    float t[BH];
#pragma unroll
    for (int r = 0; r < BH; ++r) t[r] = acc[r][q];
    warp_reduce_rows<BH>(t, lane);
    part[warp][myrow][q] = t[0];  // lanes that share a row hold the same total
  }
  __syncthreads();
  if (pos < p.nbr && ks == 0) {
    for (int idx = lane; idx < BH * NQ; idx += 32) {
      const int r = idx / NQ, q = idx % NQ;
      const int64_t row = (int64_t)p.band_order[pos] * p.bh + r;
      if (r >= p.bh || row >= p.M || q0 + q >= p.N) continue;
      float s = 0.f;
      for (int w = 0; w < wpb; ++w) s += part[bi * wpb + w][r][q];
      if (p.y_dtype == GRIM_F32) static_cast<float*>(p.Y)[row * p.ldy + q0 + q] = s;
      else static_cast<__nv_bfloat16*>(p.Y)[row * p.ldy + q0 + q] = __float2bfloat16_rn(s);
    }
  }
}

template <int BH, int BPW, int NQL, typename VT, bool CONV>
cudaError_t launch_one(const KParams& p, cudaStream_t s) {
  constexpr int TN = NQL * 4;
  KParams q = p;
  q.blob_stride = (p.blob_stride + 15u) & ~15u;
  const size_t smem = (size_t)2 * p.bw * TN * 4 + (size_t)2 * q.blob_stride;
  auto kern = bcr_spmm_kernel<BH, BPW, NQL, VT, CONV>;
  if (smem > 48 * 1024) {
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), smem);
    if (e != cudaSuccess) return e;
  }
  const int64_t ntiles = (p.a.ncols + TN - 1) / TN;
  const int64_t ngroups = (p.nbr + p.G - 1) / p.G;
  if (ntiles > 0x7FFFFFFF || ngroups > 65535) return cudaErrorInvalidConfiguration;
  dim3 grid((unsigned)ntiles, (unsigned)ngroups);
  kern<<<grid, kThreads, smem, s>>>(q);
  count_launch();
  return cudaGetLastError();
}

template <int BH, int BPW, typename VT, bool CONV>
cudaError_t launch_by_tile(const KParams& p, int tile_n, cudaStream_t s) {
  switch (tile_n) {
    case 16: return launch_one<BH, BPW, 4, VT, CONV>(p, s);
    case 32: return launch_one<BH, BPW, 8, VT, CONV>(p, s);
    case 64: return launch_one<BH, BPW, 16, VT, CONV>(p, s);
    default: return launch_one<BH, BPW, 32, VT, CONV>(p, s);
  }
}

template <typename VT, bool CONV>
cudaError_t launch_by_bh(const KParams& p, int tile_n, cudaStream_t s) {
  if (p.bh <= 4) return launch_by_tile<4, 4, VT, CONV>(p, tile_n, s);
  if (p.bh <= 8) return launch_by_tile<8, 2, VT, CONV>(p, tile_n, s);
  return launch_by_tile<16, 1, VT, CONV>(p, tile_n, s);
}

int default_tile_n(int64_t ncols) {
  if (ncols <= 16) return 16;
  if (ncols <= 32) return 32;
  if (ncols <= 64) return 64;
  return 128;
}

}  // namespace

grim_status_t launch_spmm(const grim_bcr* h, const SpmmArgs& a, cudaStream_t s) {
  if (h->device < 0) return GRIM_ERR_INVALID_ARG;
  if (!h->d_stage) return GRIM_ERR_UNSUPPORTED;  // packed for narrow right-hand sides only
  KParams p;
  p.stage = h->d_stage; p.blob = h->d_blob; p.band_order = h->d_band_order;
  p.nbr = (int)h->nbr; p.nbc = (int)h->nbc; p.M = (int)h->M; p.K = (int)h->K; p.bh = h->bh; p.bw = h->bw; p.G = h->G;
  p.blob_stride = h->max_blob_bytes ? h->max_blob_bytes : 16;
  p.a = a;
  int tn = a.tile_n ? a.tile_n : default_tile_n(a.ncols);
  if (tn != 16 && tn != 32 && tn != 64 && tn != 128) return GRIM_ERR_INVALID_ARG;
  cudaError_t e;
  if (h->dtype == GRIM_F32) e = a.conv ? launch_by_bh<float, true>(p, tn, s) : launch_by_bh<float, false>(p, tn, s);
  else e = a.conv ? launch_by_bh<__nv_bfloat16, true>(p, tn, s) : launch_by_bh<__nv_bfloat16, false>(p, tn, s);
  return e == cudaSuccess ? GRIM_OK : GRIM_ERR_CUDA;
}

namespace {

template <int BH, typename VT, typename XT>
cudaError_t launch_skinny_nq(const SkinnyParams& p, int nq, dim3 grid, cudaStream_t s) {
  switch (nq) {
    case 1: bcr_skinny_kernel<BH, 1, 4, VT, XT><<<grid, kThreads, 0, s>>>(p); break;
    case 4: bcr_skinny_kernel<BH, 4, 4, VT, XT><<<grid, kThreads, 0, s>>>(p); break;
    case 8: bcr_skinny_kernel<BH, 8, 2, VT, XT><<<grid, kThreads, 0, s>>>(p); break;
    default:
      if (BH > 8) return cudaErrorInvalidValue;
      bcr_skinny_kernel<(BH <= 8 ? BH : 8), 16, 2, VT, XT><<<grid, kThreads, 0, s>>>(p);
  }
  return cudaGetLastError();
}

template <typename VT, typename XT>
cudaError_t launch_skinny_bh(const SkinnyParams& p, int BHc, int nq, dim3 grid, cudaStream_t s) {
  if (BHc == 4) return launch_skinny_nq<4, VT, XT>(p, nq, grid, s);
  if (BHc == 8) return launch_skinny_nq<8, VT, XT>(p, nq, grid, s);
  return launch_skinny_nq<16, VT, XT>(p, nq, grid, s);
}

}  // namespace

grim_status_t launch_skinny(const grim_bcr* h, const void* X, int x_dtype, int64_t ldx, int64_t N, void* Y, int y_dtype,
                            int64_t ldy, cudaStream_t s) {
  if (h->device < 0 || !h->gemv_ok || !h->d_chunks || N < 1 || N > kSkinnyMaxN) return GRIM_ERR_UNSUPPORTED;
  if (x_dtype != h->dtype) return GRIM_ERR_DTYPE;
  const int nbr = (int)h->nbr;
  const int BHc = h->bh <= 4 ? 4 : (h->bh <= 8 ? 8 : 16);
  int nq = N == 1 ? 1 : (N <= 4 ? 4 : (N <= 8 ? 8 : 16));
  if (BHc == 16 && nq == 16) nq = 8;  // 16 x 16 accumulators do not fit the register file: two passes of 8
  const int passes = (int)((N + nq - 1) / nq);
  // enough warps to keep every SM's memory pipeline busy: split a band over several warps when bands are few
  int wpb = 1;
  const int64_t want_warps = (int64_t)sm_count(h->device) * 20;
  while (wpb < 8 && (int64_t)nbr * passes * wpb < want_warps && (int64_t)nbr * wpb * 8 <= h->nchunks) wpb *= 2;
  const int bpc = kWarps / wpb;
  SkinnyParams p;
  p.band_ptr = h->d_gemv_band_ptr; p.chunks = h->d_chunks; p.colwords = h->d_colwords; p.vals = h->d_gemv_vals;
  p.band_order = h->d_band_order; p.X = X; p.Y = Y; p.ldx = ldx; p.ldy = ldy;
  p.N = (int)N; p.nbr = nbr; p.M = (int)h->M; p.bh = h->bh; p.wpb = wpb; p.y_dtype = y_dtype;
  const int esz = x_dtype == GRIM_F32 ? 4 : 2;
  p.vec_ok = (N % nq == 0) && ldx % 4 == 0 && (reinterpret_cast<uintptr_t>(X) % (4 * esz)) == 0;
  dim3 grid((unsigned)((nbr + bpc - 1) / bpc), (unsigned)passes);
  cudaError_t e = h->dtype == GRIM_F32 ? launch_skinny_bh<float, float>(p, BHc, nq, grid, s)
                                       : launch_skinny_bh<__nv_bfloat16, __nv_bfloat16>(p, BHc, nq, grid, s);
  count_launch();
  return e == cudaSuccess ? GRIM_OK : GRIM_ERR_CUDA;
}

}  // namespace grim

extern "C" int64_t grim_launch_count(void) { return grim::launches(); }
extern "C" void grim_launch_count_reset(void) { grim::launches_reset(); }
