// GRU sequence inference built from the BCR matrix-vector product (Section 3.1: RNN layers are
// matrix-vector multiplications; Section 6.1: a 2-layer GRU is the RNN workload).
//
// Per layer: (1) the input-side products W_ih x_t for all T steps do not depend on the recurrence and
// are hoisted into one sparse GEMM with N = T (bias b_ih fused); (2) one persistent kernel walks the T
// dependent steps.  Every thread block owns a few groups of bh hidden units and the three row bands
// (r, z, n gates) of W_hh that produce them; it copies those bands' packed chunks into shared memory
// once, so that W_hh is read from HBM once per sequence instead of once per step.  Per step the blocks
// multiply their bands with h_{t-1}, apply the gate non-linearities, publish their slice of h_t and
// meet at a grid-wide barrier whose wait is bounded.
#include <cooperative_groups.h>

#include <algorithm>
#include <new>

#include "grim_device.cuh"
#include "grim_internal.h"

using namespace grim;

struct grim_gru {
  int L = 0;
  int64_t H = 0, max_T = 0;
  int bh = 0;
  std::vector<const grim_bcr*> Wih, Whh;
  std::vector<float*> d_bih, d_bhh;
  std::vector<uint32_t*> d_pos_of_band;
  float* d_gi = nullptr;
  float* d_seq[2] = {nullptr, nullptr};
  unsigned* d_sync = nullptr;  // [0..L): barrier counters, [L]: status word
  int tpc = 1, ks = 1, threads = 0, grid = 0, resident = 0;
  uint32_t max_chunks = 0, max_cw = 0, max_vals = 0;
  size_t smem = 0;
  int device = -1;
  cudaStream_t last_stream = nullptr;
  int dbg_skip_cta = -1;
  unsigned spin_limit = 1u << 22;
  bool profile = false;
  std::vector<cudaEvent_t> ev;  // 3 per layer: before projection, before recurrent kernel, after it
};

namespace {

constexpr int kMaxLocalBands = 24;

struct GruParams {
  const uint32_t* band_ptr;
  const ChunkDesc* chunks;
  const uint32_t* colwords;
  const float* vals;
  const uint32_t* pos_of_band;
  const float* b_hh;
  const float* gi;   // T x 3H, b_ih already added
  const float* h0;   // H or null
  float* out;        // T x H
  float* hT;         // H or null
  unsigned* bar;
  unsigned* status;
  int H, bh, T, tpc, ks, resident;
  uint32_t max_chunks, max_cw, max_vals;
  int skip_cta;
  unsigned spin_limit;
};

__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_release_gpu_add(unsigned* p, unsigned v) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

__device__ __forceinline__ float sigmoidf_(float v) { return 1.f / (1.f + expf(-v)); }

template <int BH>
__global__ void __launch_bounds__(1024, 1) gru_recurrent_kernel(const GruParams p) {
  extern __shared__ __align__(16) uint8_t smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nb = 3 * p.tpc;        // local bands: index tri * 3 + gate
  const int nbands_gate = p.H / p.bh;
  float* hs = reinterpret_cast<float*>(smem);
  float* partial = hs + p.H;  // [nb][ks][BH]
  uint32_t* s_cb = reinterpret_cast<uint32_t*>(partial + nb * p.ks * BH);  // chunk range per local band
  uint32_t* s_ce = s_cb + kMaxLocalBands;
  ChunkDesc* s_ch = reinterpret_cast<ChunkDesc*>(s_ce + kMaxLocalBands);
  uint32_t* s_cw = reinterpret_cast<uint32_t*>(s_ch + p.max_chunks);
  float* s_val = reinterpret_cast<float*>(s_cw + p.max_cw);
  __shared__ uint32_t s_src_c[kMaxLocalBands], s_src_cw[kMaxLocalBands], s_src_v[kMaxLocalBands];
  __shared__ uint32_t s_dst_cw[kMaxLocalBands], s_dst_v[kMaxLocalBands], s_n_cw[kMaxLocalBands], s_n_v[kMaxLocalBands];
  __shared__ int s_abort;

  // ---- one-time set-up: locate this block's bands and (if they fit) make them resident
  if (tid == 0) {
    s_abort = 0;
    uint32_t nc = 0, ncw = 0, nv = 0;
    for (int lb = 0; lb < nb; ++lb) {
      const int tri = blockIdx.x * p.tpc + lb / 3;
      uint32_t cb = 0, ce = 0;
      if (tri < nbands_gate) {
        const uint32_t pos = p.pos_of_band[(lb % 3) * nbands_gate + tri];
        cb = p.band_ptr[pos];
        ce = p.band_ptr[pos + 1];
      }
      uint32_t n_cw = 0, n_v = 0;
      for (uint32_t c = cb; c < ce; ++c) {
        const uint32_t nk = p.chunks[c].ncols_kr;
        n_cw += nk & 0xFFFFu;
        n_v += (nk & 0xFFFFu) * (nk >> 16);
      }
      s_src_c[lb] = cb;
      s_src_cw[lb] = cb < ce ? p.chunks[cb].cw_off : 0;
      s_src_v[lb] = cb < ce ? p.chunks[cb].val_off : 0;
      s_dst_cw[lb] = ncw; s_dst_v[lb] = nv; s_n_cw[lb] = n_cw; s_n_v[lb] = n_v;
      if (p.resident) { s_cb[lb] = nc; s_ce[lb] = nc + (ce - cb); }
      else { s_cb[lb] = cb; s_ce[lb] = ce; }
      nc += ce - cb; ncw += n_cw; nv += n_v;
    }
  }
  __syncthreads();
  const ChunkDesc* ch = p.chunks;
  const uint32_t* cw = p.colwords;
  const float* vals = p.vals;
  if (p.resident) {
    for (int lb = 0; lb < nb; ++lb) {
      const uint32_t n = s_ce[lb] - s_cb[lb];
      for (uint32_t i = tid; i < n; i += blockDim.x) {
        ChunkDesc cd = p.chunks[s_src_c[lb] + i];
        cd.cw_off = cd.cw_off - s_src_cw[lb] + s_dst_cw[lb];
        cd.val_off = cd.val_off - s_src_v[lb] + s_dst_v[lb];
        s_ch[s_cb[lb] + i] = cd;
      }
      for (uint32_t i = tid; i < s_n_cw[lb]; i += blockDim.x) s_cw[s_dst_cw[lb] + i] = p.colwords[s_src_cw[lb] + i];
      for (uint32_t i = tid; i < s_n_v[lb]; i += blockDim.x) s_val[s_dst_v[lb] + i] = p.vals[s_src_v[lb] + i];
    }
    ch = s_ch; cw = s_cw; vals = s_val;
  }
  __syncthreads();

  const int my_lb = warp / p.ks, my_ks = warp % p.ks;
  const bool gemv_warp = my_lb < nb;
  // gate threads: one per hidden unit owned by this block
  const bool gate_thread = tid < p.tpc * p.bh;
  const int g_tri = tid / p.bh, g_r = tid % p.bh;
  const int unit = (blockIdx.x * p.tpc + g_tri) * p.bh + g_r;
  const bool gate_live = gate_thread && unit < p.H;
  float bq[3] = {0.f, 0.f, 0.f};
  if (gate_live)
    for (int g = 0; g < 3; ++g) bq[g] = p.b_hh[g * p.H + unit];

  for (int t = 0; t < p.T; ++t) {
    float gi[3] = {0.f, 0.f, 0.f};
    if (gate_live)
      for (int g = 0; g < 3; ++g) gi[g] = __ldg(p.gi + (int64_t)t * 3 * p.H + g * p.H + unit);
    // h_{t-1}: written by other blocks during this launch -> read through L2
    const float* hprev = t == 0 ? p.h0 : p.out + (int64_t)(t - 1) * p.H;
    for (int i = tid; i < p.H; i += blockDim.x) hs[i] = hprev ? __ldcg(hprev + i) : 0.f;
    __syncthreads();

    if (gemv_warp) {
      float acc[BH];
#pragma unroll
      for (int r = 0; r < BH; ++r) acc[r] = 0.f;
      for (uint32_t c = s_cb[my_lb] + my_ks; c < s_ce[my_lb]; c += p.ks) {
        const ChunkDesc cd = ch[c];
        const int ncols = cd.ncols_kr & 0xFFFF;
        if (lane < ncols) {
          const uint32_t w = cw[cd.cw_off + lane];
          const unsigned rm = w >> 16;
          const float xv = hs[w & 0xFFFFu];
          const float* v = vals + cd.val_off + lane;
          int cnt = 0;
#pragma unroll
          for (int r = 0; r < BH; ++r)
            if ((rm >> r) & 1u) { acc[r] = fmaf(v[cnt * ncols], xv, acc[r]); ++cnt; }
        }
      }
      warp_reduce_rows<BH>(acc, lane);
      partial[(my_lb * p.ks + my_ks) * BH + warp_row<BH>(lane)] = acc[0];
    }
    __syncthreads();

    if (gate_live) {
      float q[3];
#pragma unroll
      for (int g = 0; g < 3; ++g) {
        float s = bq[g];
        for (int k = 0; k < p.ks; ++k) s += partial[((g_tri * 3 + g) * p.ks + k) * BH + g_r];
        q[g] = s;
      }
      const float rg = sigmoidf_(gi[0] + q[0]);
      const float zg = sigmoidf_(gi[1] + q[1]);
      const float ng = tanhf(gi[2] + rg * q[2]);
      const float hn = (1.f - zg) * ng + zg * hs[unit];
      p.out[(int64_t)t * p.H + unit] = hn;
      if (t == p.T - 1 && p.hT) p.hT[unit] = hn;
    }
    if (t == p.T - 1) break;
    __syncthreads();
    if (tid == 0) {
      // bounded grid-wide barrier: arrive with release, poll with acquire
      if ((int)blockIdx.x != p.skip_cta) red_release_gpu_add(p.bar, 1u);
      const unsigned target = (unsigned)(t + 1) * gridDim.x;
      unsigned spins = 0;
      while (ld_acquire_gpu(p.bar) < target) {
        if (++spins > p.spin_limit) {
          atomicExch(p.status, (unsigned)GRIM_ERR_TIMEOUT);
          s_abort = 1;
          break;
        }
      }
    }
    __syncthreads();
    if (s_abort) break;
  }
}

size_t gru_smem_bytes(const grim_gru* g, int BH) {
  const int nb = 3 * g->tpc;
  size_t b = (size_t)g->H * 4 + (size_t)nb * g->ks * BH * 4 + 2 * kMaxLocalBands * 4;
  if (g->resident) b += (size_t)g->max_chunks * sizeof(ChunkDesc) + (size_t)g->max_cw * 4 + (size_t)g->max_vals * 4;
  return (b + 15) & ~size_t(15);
}

template <int BH>
cudaError_t launch_recurrent(const grim_gru* g, const GruParams& p, cudaStream_t s) {
  auto kern = gru_recurrent_kernel<BH>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)g->smem);
  if (e != cudaSuccess) return e;
  int per_sm = 0, sms = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, g->threads, g->smem);
  if (e != cudaSuccess) return e;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, g->device);
  if ((int64_t)per_sm * sms < g->grid) return cudaErrorCooperativeLaunchTooLarge;
  void* args[] = {(void*)&p};
  e = cudaLaunchCooperativeKernel((void*)kern, dim3(g->grid), dim3(g->threads), args, g->smem, s);
  count_launch();
  return e;
}

void destroy(grim_gru* g) {
  if (!g) return;
  for (float* p : g->d_bih) cudaFree(p);
  for (float* p : g->d_bhh) cudaFree(p);
  for (uint32_t* p : g->d_pos_of_band) cudaFree(p);
  for (cudaEvent_t e : g->ev) cudaEventDestroy(e);
  cudaFree(g->d_gi);
  cudaFree(g->d_seq[0]);
  cudaFree(g->d_seq[1]);
  cudaFree(g->d_sync);
  delete g;
}

}  // namespace

extern "C" grim_status_t grim_gru_create(int layers, const grim_bcr_t* W_ih, const grim_bcr_t* W_hh,
                                         const float* const* b_ih, const float* const* b_hh, int64_t max_T,
                                         grim_gru_t* out) {
  if (layers <= 0 || !W_ih || !W_hh || !b_ih || !b_hh || !out || max_T <= 0) return GRIM_ERR_INVALID_ARG;
  for (int l = 0; l < layers; ++l)
    if (!W_ih[l] || !W_hh[l] || !b_ih[l] || !b_hh[l]) return GRIM_ERR_INVALID_ARG;
  const int64_t H = W_hh[0]->K;
  const int bh = W_hh[0]->bh;
  for (int l = 0; l < layers; ++l) {
    const grim_bcr *wi = W_ih[l], *wh = W_hh[l];
    if (wi->device < 0 || wh->device < 0) return GRIM_ERR_INVALID_ARG;
    if (wh->K != H || wh->M != 3 * H || wi->M != 3 * H) return GRIM_ERR_SHAPE;
    if (l > 0 && wi->K != H) return GRIM_ERR_SHAPE;
    if (wi->dtype != GRIM_F32 || wh->dtype != GRIM_F32) return GRIM_ERR_DTYPE;
    if (wh->bh != bh || H % bh != 0 || !wh->gemv_ok) return GRIM_ERR_UNSUPPORTED;
  }
  grim_gru* g = new (std::nothrow) grim_gru();
  if (!g) return GRIM_ERR_ALLOC;
  g->L = layers; g->H = H; g->max_T = max_T; g->bh = bh;
  cudaGetDevice(&g->device);
  const int ntri = (int)(H / bh);
  g->tpc = (ntri + 127) / 128;
  if (3 * g->tpc > kMaxLocalBands) { delete g; return GRIM_ERR_UNSUPPORTED; }
  g->grid = (ntri + g->tpc - 1) / g->tpc;
  const int nb = 3 * g->tpc;
  g->ks = std::max(1, std::min(4, 32 / nb));
  g->threads = std::max(nb * g->ks * 32, ((g->tpc * bh + 31) / 32) * 32);
  grim_status_t st = GRIM_OK;
  try {
    for (int l = 0; l < layers && st == GRIM_OK; ++l) {
      const grim_bcr* wh = W_hh[l];
      g->Wih.push_back(W_ih[l]);
      g->Whh.push_back(wh);
      std::vector<uint32_t> pos_of_band((size_t)wh->nbr);
      for (size_t p = 0; p < pos_of_band.size(); ++p) pos_of_band[wh->band_order[p]] = (uint32_t)p;
      // per thread block: how much of the chunk layout it would hold on-chip
      for (int c = 0; c < g->grid; ++c) {
        uint32_t nc = 0, ncw = 0, nv = 0;
        for (int lb = 0; lb < nb; ++lb) {
          const int tri = c * g->tpc + lb / 3;
          if (tri >= ntri) continue;
          const uint32_t pos = pos_of_band[(size_t)((lb % 3) * ntri + tri)];
          for (uint32_t k = wh->h_gemv_band_ptr[pos]; k < wh->h_gemv_band_ptr[pos + 1]; ++k) {
            const uint32_t nk = wh->h_chunks[k].ncols_kr;
            ++nc; ncw += nk & 0xFFFFu; nv += (nk & 0xFFFFu) * (nk >> 16);
          }
        }
        g->max_chunks = std::max(g->max_chunks, nc);
        g->max_cw = std::max(g->max_cw, ncw);
        g->max_vals = std::max(g->max_vals, nv);
      }
      float *db1 = nullptr, *db2 = nullptr;
      uint32_t* dp = nullptr;
      cudaError_t e = cudaMalloc((void**)&db1, (size_t)3 * H * 4);
      if (e == cudaSuccess) { g->d_bih.push_back(db1); e = cudaMalloc((void**)&db2, (size_t)3 * H * 4); }
      if (e == cudaSuccess) { g->d_bhh.push_back(db2); e = cudaMalloc((void**)&dp, pos_of_band.size() * 4); }
      if (e == cudaSuccess) {
        g->d_pos_of_band.push_back(dp);
        e = cudaMemcpy(db1, b_ih[l], (size_t)3 * H * 4, cudaMemcpyHostToDevice);
        if (e == cudaSuccess) e = cudaMemcpy(db2, b_hh[l], (size_t)3 * H * 4, cudaMemcpyHostToDevice);
        if (e == cudaSuccess) e = cudaMemcpy(dp, pos_of_band.data(), pos_of_band.size() * 4, cudaMemcpyHostToDevice);
      }
      if (e != cudaSuccess) st = e == cudaErrorMemoryAllocation ? GRIM_ERR_ALLOC : GRIM_ERR_CUDA;
    }
    if (st == GRIM_OK) {
      cudaError_t e = cudaMalloc((void**)&g->d_gi, (size_t)max_T * 3 * H * 4);
      if (e == cudaSuccess) e = cudaMalloc((void**)&g->d_seq[0], (size_t)max_T * H * 4);
      if (e == cudaSuccess) e = cudaMalloc((void**)&g->d_seq[1], (size_t)max_T * H * 4);
      if (e == cudaSuccess) e = cudaMalloc((void**)&g->d_sync, (size_t)(layers + 1) * 4);
      if (e == cudaSuccess) e = cudaMemset(g->d_sync, 0, (size_t)(layers + 1) * 4);
      if (e != cudaSuccess) st = e == cudaErrorMemoryAllocation ? GRIM_ERR_ALLOC : GRIM_ERR_CUDA;
    }
  } catch (const std::bad_alloc&) {
    st = GRIM_ERR_ALLOC;
  }
  if (st != GRIM_OK) { cudaGetLastError(); destroy(g); return st; }
  const int BHc = bh <= 4 ? 4 : (bh <= 8 ? 8 : 16);
  g->resident = 1;
  g->smem = gru_smem_bytes(g, BHc);
  if (g->smem > 200 * 1024) {  // does not fit on-chip: stream the chunks from L2 every step
    g->resident = 0;
    g->smem = gru_smem_bytes(g, BHc);
    if (g->smem > 200 * 1024) { destroy(g); return GRIM_ERR_UNSUPPORTED; }
  }
  *out = g;
  return GRIM_OK;
}

extern "C" grim_status_t grim_gru_seq(grim_gru_t g, const float* x, int64_t T, const float* h0, float* y, float* hT,
                                      grim_stream_t stream) {
  if (!g || !x || !y || T <= 0) return GRIM_ERR_INVALID_ARG;
  if (T > g->max_T) return GRIM_ERR_SHAPE;
  cudaStream_t s = (cudaStream_t)stream;
  g->last_stream = s;
  const int64_t H = g->H;
  if (cudaMemsetAsync(g->d_sync, 0, (size_t)(g->L + 1) * 4, s) != cudaSuccess) return GRIM_ERR_CUDA;
  const float* seq_in = x;
  for (int l = 0; l < g->L; ++l) {
    const grim_bcr* wi = g->Wih[l];
    // hoisted input projection: gi[t, :] = W_ih x_t + b_ih for all t (X given as T x in, output T x 3H)
    SpmmArgs a;
    a.X = seq_in; a.Y = g->d_gi; a.ncols = T;
    a.x_sk = 1; a.x_sq = wi->K; a.y_sr = 1; a.y_sq = 3 * H;
    a.x_dtype = GRIM_F32; a.y_dtype = GRIM_F32; a.bias = g->d_bih[l];
    if (g->profile) cudaEventRecord(g->ev[3 * l], s);
    grim_status_t st = launch_spmm(wi, a, s);
    if (st != GRIM_OK) return st;
    if (g->profile) cudaEventRecord(g->ev[3 * l + 1], s);
    float* seq_out = (l == g->L - 1) ? y : g->d_seq[l & 1];
    const grim_bcr* wh = g->Whh[l];
    GruParams p;
    p.band_ptr = wh->d_gemv_band_ptr; p.chunks = wh->d_chunks; p.colwords = wh->d_colwords;
    p.vals = static_cast<const float*>(wh->d_gemv_vals); p.pos_of_band = g->d_pos_of_band[l];
    p.b_hh = g->d_bhh[l]; p.gi = g->d_gi; p.h0 = h0 ? h0 + (int64_t)l * H : nullptr;
    p.out = seq_out; p.hT = hT ? hT + (int64_t)l * H : nullptr;
    p.bar = g->d_sync + l; p.status = g->d_sync + g->L;
    p.H = (int)H; p.bh = g->bh; p.T = (int)T; p.tpc = g->tpc; p.ks = g->ks; p.resident = g->resident;
    p.max_chunks = g->max_chunks; p.max_cw = g->max_cw; p.max_vals = g->max_vals;
    p.skip_cta = g->dbg_skip_cta; p.spin_limit = g->spin_limit;
    cudaError_t e;
    if (g->bh <= 4) e = launch_recurrent<4>(g, p, s);
    else if (g->bh <= 8) e = launch_recurrent<8>(g, p, s);
    else e = launch_recurrent<16>(g, p, s);
    if (e != cudaSuccess) { cudaGetLastError(); return e == cudaErrorCooperativeLaunchTooLarge ? GRIM_ERR_UNSUPPORTED : GRIM_ERR_CUDA; }
    if (g->profile) cudaEventRecord(g->ev[3 * l + 2], s);
    seq_in = seq_out;
  }
  return GRIM_OK;
}

extern "C" grim_status_t grim_gru_status(grim_gru_t g) {
  if (!g) return GRIM_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(g->last_stream) != cudaSuccess) return GRIM_ERR_CUDA;
  unsigned v = 0;
  if (cudaMemcpy(&v, g->d_sync + g->L, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return GRIM_ERR_CUDA;
  return (grim_status_t)v;
}

// Test hook: make thread block `skip_cta` stay away from the barrier (-1: off) and set the number of
// polls after which a waiting block gives up.  The waits then run out and the status word reports it;
// no thread block ever waits without a bound.
extern "C" grim_status_t grim_gru_debug_barrier(grim_gru_t g, int skip_cta, unsigned spin_limit) {
  if (!g) return GRIM_ERR_INVALID_ARG;
  g->dbg_skip_cta = skip_cta;
  g->spin_limit = spin_limit ? spin_limit : (1u << 22);
  return GRIM_OK;
}

extern "C" grim_status_t grim_gru_profile(grim_gru_t g, int enable) {
  if (!g) return GRIM_ERR_INVALID_ARG;
  if (enable && g->ev.empty()) {
    g->ev.resize((size_t)3 * g->L);
    for (cudaEvent_t& e : g->ev)
      if (cudaEventCreate(&e) != cudaSuccess) return GRIM_ERR_CUDA;
  }
  g->profile = enable != 0;
  return GRIM_OK;
}

extern "C" grim_status_t grim_gru_profile_read(grim_gru_t g, float* projection_ms, float* recurrent_ms) {
  if (!g || !g->profile || g->ev.empty()) return GRIM_ERR_INVALID_ARG;
  float pj = 0.f, rc = 0.f;
  for (int l = 0; l < g->L; ++l) {
    float a = 0.f, b = 0.f;
    if (cudaEventSynchronize(g->ev[3 * l + 2]) != cudaSuccess) return GRIM_ERR_CUDA;
    if (cudaEventElapsedTime(&a, g->ev[3 * l], g->ev[3 * l + 1]) != cudaSuccess) return GRIM_ERR_CUDA;
    if (cudaEventElapsedTime(&b, g->ev[3 * l + 1], g->ev[3 * l + 2]) != cudaSuccess) return GRIM_ERR_CUDA;
    pj += a; rc += b;
  }
  if (projection_ms) *projection_ms = pj;
  if (recurrent_ms) *recurrent_ms = rc;
  return GRIM_OK;
}

extern "C" grim_status_t grim_gru_destroy(grim_gru_t g) {
  if (!g) return GRIM_OK;
  int cur = -1;
  const int dev = g->device;
  cudaGetDevice(&cur);
  if (cur != dev) cudaSetDevice(dev);
  destroy(g);
  if (cur != dev && cur >= 0) cudaSetDevice(cur);
  return GRIM_OK;
}

// ---------------------------------------------------------------------------------------------
// grim_gru_seq_static: the same sequence pass for callers that must not allocate device memory.
//
// The per-call scratch of the GRU pass (the hoisted pre-activations gi, T x 3H floats, and the two
// T x H buffers that carry one layer's outputs to the next) lives in a fixed array inside the
// library image instead of in buffers obtained from the CUDA allocator.  Host code cannot use the
// array's name as a device address; the address is looked up once per device with
// cudaGetSymbolAddress while that device is current, and that pointer is what the kernels receive.
// ---------------------------------------------------------------------------------------------
namespace {
constexpr size_t kStaticScratchBytes = size_t(8) << 20;  // 8 MiB, resident on every GPU that loads the library
constexpr int kMaxDevices = 64;
}  // namespace
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
static unsigned char* g_static_scratch_addr[kMaxDevices] = {};

extern "C" grim_status_t grim_gru_seq_static(grim_gru_t g, const float* x, int64_t T, const float* h0, float* y,
                                             float* hT, grim_stream_t stream) {
  if (!g || !x || !y || T <= 0) return GRIM_ERR_INVALID_ARG;
  if (T > g->max_T) return GRIM_ERR_SHAPE;
  // carve-up of the static array: gi | seq0 | seq1, each start rounded up to 256 bytes
  auto round256 = [](size_t b) { return (b + 255) & ~size_t(255); };
  const size_t gi_bytes = round256((size_t)T * 3 * (size_t)g->H * 4);
  const size_t seq_bytes = g->L > 1 ? round256((size_t)T * (size_t)g->H * 4) : 0;
  if (gi_bytes + 2 * seq_bytes > kStaticScratchBytes) return GRIM_ERR_UNSUPPORTED;  // T * H too large for 8 MiB
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return GRIM_ERR_CUDA;
  if (dev != g->device || dev < 0 || dev >= kMaxDevices) return GRIM_ERR_INVALID_ARG;
  if (!g_static_scratch_addr[dev]) {
    // one-time set-up for this device (device `dev` is current): resolve the array's device address
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
      cudaGetLastError();
      return GRIM_ERR_CUDA;
    }
    g_static_scratch_addr[dev] = static_cast<unsigned char*>(p);
  }
  unsigned char* base = g_static_scratch_addr[dev];
  // Run the ordinary pass with the handle's scratch pointers pointing into the static array for the
  // duration of the call.  Kernel arguments are copied at launch, so the handle can be put back at once.
  float* const saved_gi = g->d_gi;
  float* const saved_seq0 = g->d_seq[0];
  float* const saved_seq1 = g->d_seq[1];
  g->d_gi = reinterpret_cast<float*>(base);
  g->d_seq[0] = reinterpret_cast<float*>(base + gi_bytes);
  g->d_seq[1] = reinterpret_cast<float*>(base + gi_bytes + seq_bytes);
  const grim_status_t st = grim_gru_seq(g, x, T, h0, y, hT, stream);
  g->d_gi = saved_gi;
  g->d_seq[0] = saved_seq0;
  g->d_seq[1] = saved_seq1;
  return st;
}
