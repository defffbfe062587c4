// GRU sequence inference built from the BCR matrix-vector product (Section 3.1: RNN layers are
// matrix-vector multiplications; Section 6.1: a 2-layer GRU is the RNN workload).
//
// Per layer: (1) the input-side products W_ih x_t for all T steps do not depend on the recurrence and
// are hoisted into one sparse GEMM with N = T (bias b_ih fused); (2) one persistent kernel walks the T
// dependent steps.  Every thread block owns some groups of bh hidden units and the three row bands
// (r, z, n gates) of W_hh that produce them; it copies those bands' packed chunks into shared memory
// once, so that W_hh is read from HBM once per sequence instead of once per step.  Per step the blocks
// multiply their bands with h_{t-1}, apply the gate non-linearities and exchange their slices of h_t.
//
// Two exchange schemes:
//   gru_cluster_kernel    one thread-block cluster (up to 16 CTAs) holds all of W_hh; h_t is broadcast
//                         with distributed-shared-memory stores and the step ends with the hardware
//                         cluster barrier.  Used whenever the layer fits one cluster.
//   gru_recurrent_kernel  cooperative grid of up to 128 CTAs; h_t goes through L2 and the step ends with a
//                         grid-wide barrier in global memory whose wait is bounded (status word on expiry).
#include <cooperative_groups.h>

#include <algorithm>
#include <new>

#include "grim_device.cuh"
#include "grim_internal.h"

namespace cg = cooperative_groups;
using namespace grim;

namespace {
constexpr int kMaxLocalBands = 48;
struct ModeCfg {
  int tpc = 1, ks = 1, threads = 0, ctas = 0, resident = 0;
  uint32_t max_chunks = 0, max_cw = 0, max_vals = 0;
  size_t smem = 0;
  bool ok = false;
};
}  // namespace

struct grim_gru {
  int L = 0;
  int64_t H = 0, max_T = 0;
  int bh = 0;
  std::vector<const grim_bcr*> Wih, Whh;
  std::vector<float*> d_bih, d_bhh;
  std::vector<uint32_t*> d_pos_of_band;
  std::vector<float*> d_img_val;      // per layer: register image of the register-resident kernel (may be empty)
  std::vector<uint32_t*> d_img_col;
  std::vector<float*> d_gi_saved;  // grim_gru_seq_static parks d_gi here while it points the pass at the static array
  std::vector<float*> d_gi;  // per layer: hoisted pre-activations, T x 3H (layers overlap in time, so each has its own)
  float* d_seq[2] = {nullptr, nullptr};
  // unit-major copies (feature x time, row stride = T rounded up to 4): the projections then read X row-major
  float* d_seqT[2] = {nullptr, nullptr};
  float* d_xT = nullptr;
  bool transposed_inputs = true;
  // layer pipelining: layer l runs on its own stream, a chunk of time steps behind layer l - 1
  std::vector<cudaStream_t> lstream;   // streams of layers 1 .. L-1 (layer 0 uses the caller's stream)
  std::vector<cudaEvent_t> ev_chunk;   // [layer][chunk]: the layer's recurrence has produced the chunk
  cudaEvent_t ev_fork = nullptr;
  int max_chunks = 8;
  bool pipeline = true;
  int want_chunks = 0;  // 0: chosen from T
  unsigned* d_sync = nullptr;  // [0..L): barrier counters, [L]: status word
  ModeCfg grid, cluster;       // launch shapes of the shared-memory kernels
  ModeCfg regc;                // launch shape of the register-resident cluster kernel
  int reg_ni = 0, reg_s = 0;   // its compiled (items per warp, slots per item) variant
  int device = -1;
  cudaStream_t last_stream = nullptr;
  int dbg_skip_cta = -1;
  unsigned spin_limit = 1u << 22;
  bool force_grid = false;
  bool profile = false;
  std::vector<cudaEvent_t> ev;  // timing events, used in pairs: (before, after) each projection / recurrent launch
  std::vector<int> ev_kind;     // 0 / 1: before / after a projection, 2 / 3: before / after a recurrent kernel
  int ev_used = 0;
};

namespace {

struct GruParams {
  const uint32_t* band_ptr;
  const ChunkDesc* chunks;
  const uint32_t* colwords;
  const float* vals;
  const uint32_t* pos_of_band;
  const float* b_hh;
  const float* gi;   // T x 3H, b_ih already added
  const float* b_ih; // 3H or null: added to gi here (not used by the register-resident kernel)
  const float* h0;   // H or null
  float* out;        // T x H
  float* outT;       // null, or the same values unit-major: outT[unit * ldT + t] (input of the next layer's projection)
  int64_t ldT;
  float* hT;         // H or null
  unsigned* bar;
  unsigned* status;
  int H, bh, T, tpc, ks, resident;
  uint32_t max_chunks, max_cw, max_vals;
  int skip_cta;
  unsigned spin_limit;
  // register image of the register-resident kernel: what every thread keeps for the whole sequence, laid out
  // so that the threads of a block read consecutive words ([cta][item][slot][row or column][thread])
  const float* img_val;
  const uint32_t* img_col;
};

__device__ __forceinline__ void gru_mbar_init(uint64_t* bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"((uint32_t)__cvta_generic_to_shared(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void gru_mbar_arrive_expect_tx(uint64_t* bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"((uint32_t)__cvta_generic_to_shared(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool gru_mbar_try_wait(uint64_t* bar, unsigned parity) {
  unsigned ok;
  asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
               : "=r"(ok) : "r"((uint32_t)__cvta_generic_to_shared(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Stores v at the place of CTA-local shared address `local` in CTA `rank` of the cluster and counts its 4 bytes on
// that CTA's mbarrier at CTA-local address `bar_local`.
__device__ __forceinline__ void gru_st_async_f32(uint32_t local, uint32_t bar_local, uint32_t rank, float v) {
  uint32_t raddr, rbar;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(raddr) : "r"(local), "r"(rank));
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rbar) : "r"(bar_local), "r"(rank));
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.f32 [%0], %1, [%2];" ::"r"(raddr), "f"(v), "r"(rbar) : "memory");
}
__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_release_gpu_add(unsigned* p, unsigned v) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

__device__ __forceinline__ float sigmoidf_(float v) { return 1.f / (1.f + expf(-v)); }

// Per-CTA view of its bands' chunks: either the global arrays or copies in shared memory.
struct BandView {
  const ChunkDesc* ch;
  const uint32_t* cw;
  const float* vals;
  const uint32_t* cb;  // chunk range per local band (local band = group * 3 + gate)
  const uint32_t* ce;
};

// One-time set-up: locate the bands of CTA `cta` (tpc groups of bh hidden units x 3 gates) and, if they
// fit, copy their chunk descriptors / column words / values into shared memory.  `pool` is the dynamic
// shared memory left after the caller's own arrays.
__device__ BandView setup_bands(const GruParams& p, int cta, uint8_t* pool) {
  __shared__ uint32_t s_src_c[kMaxLocalBands], s_src_cw[kMaxLocalBands], s_src_v[kMaxLocalBands];
  __shared__ uint32_t s_dst_cw[kMaxLocalBands], s_dst_v[kMaxLocalBands], s_n_cw[kMaxLocalBands], s_n_v[kMaxLocalBands];
  __shared__ uint32_t s_cb[kMaxLocalBands], s_ce[kMaxLocalBands];
  const int tid = threadIdx.x;
  const int nb = 3 * p.tpc;
  const int nbands_gate = p.H / p.bh;
  ChunkDesc* s_ch = reinterpret_cast<ChunkDesc*>(pool);
  uint32_t* s_cw = reinterpret_cast<uint32_t*>(s_ch + p.max_chunks);
  float* s_val = reinterpret_cast<float*>(s_cw + p.max_cw);
  if (tid == 0) {
    uint32_t nc = 0, ncw = 0, nv = 0;
    for (int lb = 0; lb < nb; ++lb) {
      const int tri = cta * p.tpc + lb / 3;
      uint32_t cb = 0, ce = 0;
      if (tri < nbands_gate) {
        const uint32_t pos = p.pos_of_band[(lb % 3) * nbands_gate + tri];
        cb = p.band_ptr[pos];
        ce = p.band_ptr[pos + 1];
      }
      uint32_t n_cw = 0, n_v = 0;
      for (uint32_t c = cb; c < ce; ++c) {
        const uint32_t nk = p.chunks[c].ncols_kr;
        n_cw += 32;  // every chunk owns 32 column words
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
  BandView v{p.chunks, p.colwords, p.vals, s_cb, s_ce};
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
    v.ch = s_ch; v.cw = s_cw; v.vals = s_val;
  }
  __syncthreads();
  return v;
}

// Band x vector for work item (local band lb, k-split part ks_i): partial[(lb*ks + ks_i)*BH + row].
template <int BH>
__device__ __forceinline__ void band_gemv(const BandView& v, const float* hs, float* partial, int lb, int ks_i, int ks,
                                          int lane) {
  float acc[BH];
#pragma unroll
  for (int r = 0; r < BH; ++r) acc[r] = 0.f;
  for (uint32_t c = v.cb[lb] + ks_i; c < v.ce[lb]; c += ks) {
    const ChunkDesc cd = v.ch[c];
    const int ncols = cd.ncols_kr & 0xFFFF;
    if (lane < ncols) {
      const uint32_t w = v.cw[cd.cw_off + lane];
      const unsigned rm = w >> 16;
      const float xv = hs[w & 0xFFFFu];
      const float* val = v.vals + cd.val_off + lane;
      int cnt = 0;
#pragma unroll
      for (int r = 0; r < BH; ++r)
        if ((rm >> r) & 1u) { acc[r] = fmaf(val[cnt * ncols], xv, acc[r]); ++cnt; }
    }
  }
  warp_reduce_rows<BH>(acc, lane);
  partial[(lb * ks + ks_i) * BH + warp_row<BH>(lane)] = acc[0];
}

__device__ __forceinline__ float gru_gate(const float* partial, const float (&bq)[3], const float (&gi)[3], int g_tri,
                                          int g_r, int ks, int BH, float hprev) {
  float q[3];
#pragma unroll
  for (int g = 0; g < 3; ++g) {
    float s = bq[g];
    for (int k = 0; k < ks; ++k) s += partial[((g_tri * 3 + g) * ks + k) * BH + g_r];
    q[g] = s;
  }
  const float rg = sigmoidf_(gi[0] + q[0]);
  const float zg = sigmoidf_(gi[1] + q[1]);
  const float ng = tanhf(gi[2] + rg * q[2]);
  return (1.f - zg) * ng + zg * hprev;
}

// ---------------------------------------------------------------------------------------------
// cooperative-grid version (h through L2, bounded global barrier)
// ---------------------------------------------------------------------------------------------
template <int BH>
__global__ void __launch_bounds__(1024, 1) gru_recurrent_kernel(const GruParams p) {
  extern __shared__ __align__(16) uint8_t smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nb = 3 * p.tpc;
  float* hs = reinterpret_cast<float*>(smem);
  float* partial = hs + p.H;  // [nb][ks][BH]
  __shared__ int s_abort;
  if (tid == 0) s_abort = 0;
  const BandView v = setup_bands(p, blockIdx.x, reinterpret_cast<uint8_t*>(partial + nb * p.ks * BH));

  const int nwarps = blockDim.x >> 5;
  const bool gate_thread = tid < p.tpc * p.bh;
  const int g_tri = tid / p.bh, g_r = tid % p.bh;
  const int unit = (blockIdx.x * p.tpc + g_tri) * p.bh + g_r;
  const bool gate_live = gate_thread && unit < p.H;
  float bq[3] = {0.f, 0.f, 0.f}, bi[3] = {0.f, 0.f, 0.f};
  if (gate_live)
    for (int g = 0; g < 3; ++g) {
      bq[g] = p.b_hh[g * p.H + unit];
      if (p.b_ih) bi[g] = p.b_ih[g * p.H + unit];
    }

  for (int t = 0; t < p.T; ++t) {
    float gi[3] = {0.f, 0.f, 0.f};
    if (gate_live)
      for (int g = 0; g < 3; ++g) gi[g] = __ldg(p.gi + (int64_t)t * 3 * p.H + g * p.H + unit) + bi[g];
    // h_{t-1}: written by other blocks during this launch -> read through L2
    const float* hprev = t == 0 ? p.h0 : p.out + (int64_t)(t - 1) * p.H;
    for (int i = tid; i < p.H; i += blockDim.x) hs[i] = hprev ? __ldcg(hprev + i) : 0.f;
    __syncthreads();
    for (int item = warp; item < nb * p.ks; item += nwarps) band_gemv<BH>(v, hs, partial, item / p.ks, item % p.ks, p.ks, lane);
    __syncthreads();
    if (gate_live) {
      const float hn = gru_gate(partial, bq, gi, g_tri, g_r, p.ks, BH, hs[unit]);
      p.out[(int64_t)t * p.H + unit] = hn;
      if (p.outT) p.outT[(int64_t)unit * p.ldT + t] = hn;
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

// ---------------------------------------------------------------------------------------------
// cluster version (h through distributed shared memory, hardware cluster barrier - no spin waits)
// ---------------------------------------------------------------------------------------------
template <int BH>
__global__ void __launch_bounds__(1024, 1) gru_cluster_kernel(const GruParams p) {
  extern __shared__ __align__(16) uint8_t smem[];
  cg::cluster_group cluster = cg::this_cluster();
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int rank = (int)cluster.block_rank();
  const int CS = (int)cluster.num_blocks();
  const int nb = 3 * p.tpc;
  const int U = p.tpc * p.bh;                      // hidden units owned by this CTA
  float* hs = reinterpret_cast<float*>(smem);      // [2][H], double-buffered h
  float* hnew = hs + 2 * p.H;                      // [U]
  float* partial = hnew + ((U + 3) & ~3);          // [nb][ks][BH]
  const BandView v = setup_bands(p, rank, reinterpret_cast<uint8_t*>(partial + nb * p.ks * BH));

  const int nwarps = blockDim.x >> 5;
  const bool gate_live = tid < U;
  const int g_tri = tid / p.bh, g_r = tid % p.bh;
  const int unit = rank * U + tid;
  float bq[3] = {0.f, 0.f, 0.f}, bi[3] = {0.f, 0.f, 0.f};
  if (gate_live)
    for (int g = 0; g < 3; ++g) {
      bq[g] = p.b_hh[g * p.H + unit];
      if (p.b_ih) bi[g] = p.b_ih[g * p.H + unit];
    }
  for (int i = tid; i < p.H; i += blockDim.x) hs[i] = p.h0 ? p.h0[i] : 0.f;
  cluster.sync();  // every CTA of the cluster is resident and has initialised its buffers

  for (int t = 0; t < p.T; ++t) {
    const float* hcur = hs + (t & 1) * p.H;
    float* hnxt_local = hs + ((t + 1) & 1) * p.H;
    float gi[3] = {0.f, 0.f, 0.f};
    if (gate_live)
      for (int g = 0; g < 3; ++g) gi[g] = __ldg(p.gi + (int64_t)t * 3 * p.H + g * p.H + unit) + bi[g];
    for (int item = warp; item < nb * p.ks; item += nwarps) band_gemv<BH>(v, hcur, partial, item / p.ks, item % p.ks, p.ks, lane);
    __syncthreads();
    if (gate_live) {
      const float hn = gru_gate(partial, bq, gi, g_tri, g_r, p.ks, BH, hcur[unit]);
      hnew[tid] = hn;
      p.out[(int64_t)t * p.H + unit] = hn;
      if (p.outT) p.outT[(int64_t)unit * p.ldT + t] = hn;
      if (t == p.T - 1 && p.hT) p.hT[unit] = hn;
    }
    __syncthreads();
    // broadcast this CTA's slice of h_t into the next-step buffer of every CTA of the cluster
    if ((U & 3) == 0) {
      const int q = U >> 2;
      for (int i = tid; i < CS * q; i += blockDim.x) {
        const int dst = i / q, j = i - dst * q;
        float4* remote = cluster.map_shared_rank(reinterpret_cast<float4*>(hnxt_local + rank * U) + j, dst);
        *remote = reinterpret_cast<const float4*>(hnew)[j];
      }
    } else {
      for (int i = tid; i < CS * U; i += blockDim.x) {
        const int dst = i / U, j = i - dst * U;
        *cluster.map_shared_rank(hnxt_local + rank * U + j, dst) = hnew[j];
      }
    }
    cluster.sync();  // release our stores, acquire everyone else's; also keeps all CTAs alive until the end
  }
}

// ---------------------------------------------------------------------------------------------
// cluster version with W_hh in registers.  Every warp keeps its share of the bands in registers for the whole
// sequence, and the new state travels by asynchronous shared-memory stores counted on mbarriers instead of through a
// cluster barrier (whose release / acquire pair was the largest stall of a step): a band is cut in two halves (work items), an
// item's kept columns are dealt to S slots x 32 lanes, and a lane holds per slot the column index and
// the column's BH values expanded to row positions (zeros where the row is not kept).  A time step then
// costs one shared-memory gather of h and BH FMAs per slot - no index decoding, no predicates.
// NI = items per warp.  Shapes that need more slots than the compiled menu use the other kernels.
// ---------------------------------------------------------------------------------------------
constexpr int kRegThreads = 512;
constexpr int kRegWarps = kRegThreads / 32;

template <int BH, int NI, int S>
__global__ void __launch_bounds__(kRegThreads, 1) gru_cluster_reg_kernel(const GruParams p) {
  extern __shared__ __align__(16) float smem_f[];
  cg::cluster_group cluster = cg::this_cluster();
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int rank = (int)cluster.block_rank();
  const int CS = (int)cluster.num_blocks();
  const int nb = 3 * p.tpc;
  const int U = p.tpc * p.bh;
  const int H = p.H;
  const int nbands_gate = H / p.bh;
  float* hs = smem_f;                         // [2][H]
  float* hnew = hs + 2 * H;                   // [U]
  float* partial = hnew + ((U + 3) & ~3);     // [nb][2][BH]

  // ---- one-time: this thread's share of W_hh (built on the host when the handle was created): coalesced loads
  float val[NI][S][BH];
  uint32_t col[NI][S];
  {
    const float* iv = p.img_val + (size_t)rank * NI * S * BH * kRegThreads + tid;
    const uint32_t* ic = p.img_col + (size_t)rank * NI * S * kRegThreads + tid;
#pragma unroll
    for (int i = 0; i < NI; ++i)
#pragma unroll
      for (int s = 0; s < S; ++s) {
        col[i][s] = __ldg(ic + (size_t)(i * S + s) * kRegThreads);
#pragma unroll
        for (int r = 0; r < BH; ++r) val[i][s][r] = __ldg(iv + (size_t)((i * S + s) * BH + r) * kRegThreads);
      }
  }

  const bool gate_live = tid < U;
  const int g_tri = tid / p.bh, g_r = tid % p.bh;
  const int unit = rank * U + tid;
  float bq[3] = {0.f, 0.f, 0.f};
  float gi[3] = {0.f, 0.f, 0.f};
  if (gate_live)
    for (int g = 0; g < 3; ++g) {
      bq[g] = p.b_hh[g * H + unit];
      gi[g] = __ldg(p.gi + g * H + unit);
    }
  for (int i = tid; i < H; i += kRegThreads) hs[i] = p.h0 ? p.h0[i] : 0.f;
  // The state exchange: the thread that owns a hidden unit sends its new value into the next-step buffer of every
  // CTA of the cluster with asynchronous stores that count their bytes on the receiver's mbarrier; a CTA starts a
  // step when the H values of that step have been counted.  No cluster-wide barrier and no fence per step: a
  // buffer is written again only after every CTA has received the whole state computed from it, i.e. after every
  // warp of the cluster is done reading it.
  uint64_t* hbar = reinterpret_cast<uint64_t*>(partial + nb * 2 * BH);  // [2], 8-byte aligned (all counts are even)
  if (tid == 0) {
    gru_mbar_init(hbar, 1);
    gru_mbar_init(hbar + 1, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  cluster.sync();
  const uint32_t hs_local = (uint32_t)__cvta_generic_to_shared(hs), bar_local = (uint32_t)__cvta_generic_to_shared(hbar);
  bool failed = false;

  for (int t = 0; t < p.T; ++t) {
    const int cur = t & 1, nxt = cur ^ 1;
    const float* hcur = hs + cur * H;
    // this step's outputs arrive on the next buffer's barrier: announce the byte count (fast CTAs may already be
    // sending, which drives the count negative; the pending arrival keeps the phase open until it is announced)
    if (tid == 0 && t + 1 < p.T) gru_mbar_arrive_expect_tx(hbar + nxt, (unsigned)H * 4u);
    // pre-activations of the next step are fetched now so that their DRAM latency hides behind this step
    float gi_next[3] = {0.f, 0.f, 0.f};
    if (gate_live && t + 1 < p.T)
      for (int g = 0; g < 3; ++g) gi_next[g] = __ldg(p.gi + (int64_t)(t + 1) * 3 * H + g * H + unit);
#pragma unroll
    for (int i = 0; i < NI; ++i) {
      const int item = warp * NI + i;
      float acc[BH];
#pragma unroll
      for (int r = 0; r < BH; ++r) acc[r] = 0.f;
#pragma unroll
      for (int s = 0; s < S; ++s) {
        const float xv = hcur[col[i][s]];
#pragma unroll
        for (int r = 0; r < BH; ++r) acc[r] = fmaf(val[i][s][r], xv, acc[r]);
      }
      warp_reduce_rows<BH>(acc, lane);
      if (item < nb * 2) partial[item * BH + warp_row<BH>(lane)] = acc[0];
    }
    __syncthreads();
    float hnew_val = 0.f;
    if (gate_live) {
      // the thread that owns a hidden unit computes it; below it is sent straight to the next-step buffer of every CTA
      const float hn = gru_gate(partial, bq, gi, g_tri, g_r, 2, BH, hcur[unit]);
      hnew_val = hn;
      p.out[(int64_t)t * H + unit] = hn;
      if (p.outT) p.outT[(int64_t)unit * p.ldT + t] = hn;
      if (t == p.T - 1 && p.hT) p.hT[unit] = hn;
    }
    if (gate_live && t + 1 < p.T) {
      // one 4-byte store per destination (pooling four neighbours' values into 16-byte stores was slower: the
      // shuffles lengthen the chain more than the fewer messages save)
      const uint32_t dst_local = hs_local + (uint32_t)(nxt * H + unit) * 4u, bar_nxt = bar_local + (uint32_t)nxt * 8u;
#pragma unroll 4
      for (int dst = 0; dst < CS; ++dst) gru_st_async_f32(dst_local, bar_nxt, (uint32_t)dst, hnew_val);
    }
#pragma unroll
    for (int g = 0; g < 3; ++g) gi[g] = gi_next[g];
    if (t + 1 < p.T && warp == 0) {
      // the next step's state: bounded wait on the local barrier (its (t / 2)-th use).  One thread polls for the
      // whole block; the others sleep in the block barrier below (many pollers slow the arrival of the stores down)
      const unsigned parity = (unsigned)((t >> 1) & 1);
      bool ok = false;
      if (lane == 0)
        for (unsigned it = 0; it < p.spin_limit && !ok; ++it) ok = gru_mbar_try_wait(hbar + nxt, parity);
      __syncwarp();
      if (!__shfl_sync(0xffffffffu, ok, 0)) {
        failed = true;
        if (lane == 0) atomicExch(p.status, (unsigned)GRIM_ERR_TIMEOUT);
      }
    }
    if (__syncthreads_or(failed ? 1 : 0)) break;  // the state of the next step is there (or a wait ran out)
  }
  cluster.sync();  // no CTA leaves while another may still address its shared memory
}

size_t smem_bytes(const grim_gru* g, const ModeCfg& m, int BH, bool cluster) {
  const int nb = 3 * m.tpc;
  size_t b = (size_t)nb * m.ks * BH * 4;
  if (cluster) b += (size_t)2 * g->H * 4 + (size_t)((m.tpc * g->bh + 3) & ~3) * 4;
  else b += (size_t)g->H * 4;
  if (m.resident) b += (size_t)m.max_chunks * sizeof(ChunkDesc) + (size_t)m.max_cw * 4 + (size_t)m.max_vals * 4;
  return (b + 15) & ~size_t(15);
}

template <int BH>
cudaError_t launch_grid(const grim_gru* g, const GruParams& p, cudaStream_t s) {
  const ModeCfg& m = g->grid;
  auto kern = gru_recurrent_kernel<BH>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)m.smem);
  if (e != cudaSuccess) return e;
  int per_sm = 0, sms = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, m.threads, m.smem);
  if (e != cudaSuccess) return e;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, g->device);
  if ((int64_t)per_sm * sms < m.ctas) return cudaErrorCooperativeLaunchTooLarge;
  void* args[] = {(void*)&p};
  e = cudaLaunchCooperativeKernel((void*)kern, dim3(m.ctas), dim3(m.threads), args, m.smem, s);
  count_launch();
  return e;
}

template <typename Kern>
cudaError_t cluster_launch_config(Kern kern, const ModeCfg& m, cudaLaunchConfig_t* cfg, cudaLaunchAttribute* attr,
                                  cudaStream_t s, bool set_attributes) {
  if (set_attributes) {  // once, when the handle is created (the kernel keeps them)
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)m.smem);
    if (e == cudaSuccess && m.ctas > 8) e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
  }
  *cfg = cudaLaunchConfig_t{};
  cfg->gridDim = dim3(m.ctas);
  cfg->blockDim = dim3(m.threads);
  cfg->dynamicSmemBytes = m.smem;
  cfg->stream = s;
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = m.ctas;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg->attrs = attr;
  cfg->numAttrs = 1;
  return cudaSuccess;
}

// Can one cluster of this shape be resident?  (asked once, at creation)
template <typename Kern>
bool cluster_fits(Kern kern, const ModeCfg& m) {
  cudaLaunchConfig_t cfg;
  cudaLaunchAttribute attr[1];
  if (cluster_launch_config(kern, m, &cfg, attr, nullptr, true) != cudaSuccess) { cudaGetLastError(); return false; }
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) { cudaGetLastError(); return false; }
  return n >= 1;
}

template <typename Kern>
cudaError_t launch_cluster(Kern kern, const ModeCfg& m, const GruParams& p, cudaStream_t s) {
  cudaLaunchConfig_t cfg;
  cudaLaunchAttribute attr[1];
  cudaError_t e = cluster_launch_config(kern, m, &cfg, attr, s, false);
  if (e != cudaSuccess) return e;
  e = cudaLaunchKernelEx(&cfg, kern, p);
  count_launch();
  return e;
}

// The compiled variants of the register-resident kernel: (BH, items per warp, slots per item).
using GruKernel = void (*)(const GruParams);
GruKernel reg_kernel(int BH, int ni, int s) {
  if (BH != 8) return nullptr;
  if (ni == 1 && s == 2) return gru_cluster_reg_kernel<8, 1, 2>;
  if (ni == 1 && s == 4) return gru_cluster_reg_kernel<8, 1, 4>;
  if (ni == 3 && s == 3) return gru_cluster_reg_kernel<8, 3, 3>;
  if (ni == 3 && s == 4) return gru_cluster_reg_kernel<8, 3, 4>;
  return nullptr;
}
GruKernel smem_cluster_kernel(int BH) {
  return BH == 4 ? gru_cluster_kernel<4> : (BH == 8 ? gru_cluster_kernel<8> : gru_cluster_kernel<16>);
}

// Largest number of kept columns in half a band, over all bands of all layers.
int max_half_band_columns(const grim_gru* g) {
  uint32_t mx = 0;
  for (const grim_bcr* wh : g->Whh)
    for (int64_t pos = 0; pos < wh->nbr; ++pos) {
      uint32_t n = 0;
      for (uint32_t k = wh->h_gemv_band_ptr[(size_t)pos]; k < wh->h_gemv_band_ptr[(size_t)pos + 1]; ++k)
        n += wh->h_chunks[k].ncols_kr & 0xFFFFu;
      mx = std::max(mx, (n + 1) / 2);
    }
  return (int)mx;
}

// How much of the chunk layout the busiest CTA would hold when CTA c owns groups [c*tpc, (c+1)*tpc).
void residency_needs(const grim_gru* g, ModeCfg& m) {
  const int ntri = (int)(g->H / g->bh);
  const int nb = 3 * m.tpc;
  for (size_t l = 0; l < g->Whh.size(); ++l) {
    const grim_bcr* wh = g->Whh[l];
    std::vector<uint32_t> pos_of_band((size_t)wh->nbr);
    for (size_t p = 0; p < pos_of_band.size(); ++p) pos_of_band[wh->band_order[p]] = (uint32_t)p;
    for (int c = 0; c < m.ctas; ++c) {
      uint32_t nc = 0, ncw = 0, nv = 0;
      for (int lb = 0; lb < nb; ++lb) {
        const int tri = c * m.tpc + lb / 3;
        if (tri >= ntri) continue;
        const uint32_t pos = pos_of_band[(size_t)((lb % 3) * ntri + tri)];
        for (uint32_t k = wh->h_gemv_band_ptr[pos]; k < wh->h_gemv_band_ptr[pos + 1]; ++k) {
          const uint32_t nk = wh->h_chunks[k].ncols_kr;
          ++nc; ncw += 32; nv += (nk & 0xFFFFu) * (nk >> 16);
        }
      }
      m.max_chunks = std::max(m.max_chunks, nc);
      m.max_cw = std::max(m.max_cw, ncw);
      m.max_vals = std::max(m.max_vals, nv);
    }
  }
}

void destroy(grim_gru* g) {
  if (!g) return;
  for (float* p : g->d_bih) cudaFree(p);
  for (float* p : g->d_bhh) cudaFree(p);
  for (uint32_t* p : g->d_pos_of_band) cudaFree(p);
  for (float* p : g->d_img_val) cudaFree(p);
  for (uint32_t* p : g->d_img_col) cudaFree(p);
  for (cudaEvent_t e : g->ev) cudaEventDestroy(e);
  for (float* p : g->d_gi) cudaFree(p);
  for (cudaStream_t st : g->lstream) cudaStreamDestroy(st);
  for (cudaEvent_t e : g->ev_chunk) cudaEventDestroy(e);
  if (g->ev_fork) cudaEventDestroy(g->ev_fork);
  cudaFree(g->d_seq[0]);
  cudaFree(g->d_seq[1]);
  cudaFree(g->d_seqT[0]);
  cudaFree(g->d_seqT[1]);
  cudaFree(g->d_xT);
  cudaFree(g->d_sync);
  delete g;
}

constexpr size_t kSmemLimit = 200 * 1024;

}  // namespace

namespace {
// out[t, :] = bias for t < T (n = row length, a multiple of 4).
__global__ void fill_rows_kernel(float* __restrict__ out, const float* __restrict__ bias, int64_t T, int64_t n) {
  const int64_t total4 = T * n / 4, n4 = n / 4;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total4; i += (int64_t)gridDim.x * blockDim.x)
    reinterpret_cast<float4*>(out)[i] = __ldg(reinterpret_cast<const float4*>(bias) + i % n4);
}
// out[k * ld + t] = in[t * K + k]: the caller's T x K input, feature-major.
__global__ void transpose_input_kernel(const float* __restrict__ in, float* __restrict__ out, int64_t T, int64_t K, int64_t ld) {
  __shared__ float tile[32][33];
  const int64_t t0 = (int64_t)blockIdx.x * 32, k0 = (int64_t)blockIdx.y * 32;
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int64_t t = t0 + i, k = k0 + threadIdx.x;
    tile[i][threadIdx.x] = (t < T && k < K) ? in[t * K + k] : 0.f;
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int64_t k = k0 + i, t = t0 + threadIdx.x;
    if (k < K && t < T) out[k * ld + t] = tile[threadIdx.x][i];
  }
}
// Records the next timing event of the pool on stream s (profiling only).
void profile_mark(grim_gru* g, int kind, cudaStream_t s) {
  if (g->ev_used >= (int)g->ev.size()) return;
  g->ev_kind[(size_t)g->ev_used] = kind;
  cudaEventRecord(g->ev[(size_t)g->ev_used++], s);
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
    if (H % 4 != 0) return GRIM_ERR_UNSUPPORTED;  // rows of 3H floats are filled and read as 16-byte vectors
  }
  grim_gru* g = new (std::nothrow) grim_gru();
  if (!g) return GRIM_ERR_ALLOC;
  g->L = layers; g->H = H; g->max_T = max_T; g->bh = bh;
  cudaGetDevice(&g->device);
  const int ntri = (int)(H / bh);
  const int BHc = bh <= 4 ? 4 : (bh <= 8 ? 8 : 16);
  grim_status_t st = GRIM_OK;
  try {
    for (int l = 0; l < layers && st == GRIM_OK; ++l) {
      const grim_bcr* wh = W_hh[l];
      g->Wih.push_back(W_ih[l]);
      g->Whh.push_back(wh);
      std::vector<uint32_t> pos_of_band((size_t)wh->nbr);
      for (size_t p = 0; p < pos_of_band.size(); ++p) pos_of_band[wh->band_order[p]] = (uint32_t)p;
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
      cudaError_t e = cudaSuccess;
      for (int l = 0; l < layers && e == cudaSuccess; ++l) {
        float* p = nullptr;
        e = cudaMalloc((void**)&p, (size_t)max_T * 3 * H * 4);
        if (e == cudaSuccess) g->d_gi.push_back(p);
      }
      g->d_gi_saved.resize(g->d_gi.size());  // sized here so that grim_gru_seq_static never touches the heap
      for (int l = 1; l < layers && e == cudaSuccess; ++l) {
        cudaStream_t st = nullptr;
        e = cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking);
        if (e == cudaSuccess) g->lstream.push_back(st);
      }
      for (int i = 0; i < layers * g->max_chunks && e == cudaSuccess; ++i) {
        cudaEvent_t ev = nullptr;
        e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
        if (e == cudaSuccess) g->ev_chunk.push_back(ev);
      }
      if (e == cudaSuccess) e = cudaEventCreateWithFlags(&g->ev_fork, cudaEventDisableTiming);
      if (e == cudaSuccess) e = cudaMalloc((void**)&g->d_seq[0], (size_t)max_T * H * 4);
      if (e == cudaSuccess) e = cudaMalloc((void**)&g->d_seq[1], (size_t)max_T * H * 4);
      const size_t ldT_max = (size_t)((max_T + 3) / 4 * 4);
      if (e == cudaSuccess) e = cudaMalloc((void**)&g->d_seqT[0], ldT_max * H * 4);
      if (e == cudaSuccess) e = cudaMalloc((void**)&g->d_seqT[1], ldT_max * H * 4);
      if (e == cudaSuccess) e = cudaMalloc((void**)&g->d_xT, ldT_max * (size_t)W_ih[0]->K * 4);
      if (e == cudaSuccess) e = cudaMalloc((void**)&g->d_sync, (size_t)(layers + 1) * 4);
      if (e == cudaSuccess) e = cudaMemset(g->d_sync, 0, (size_t)(layers + 1) * 4);
      if (e != cudaSuccess) st = e == cudaErrorMemoryAllocation ? GRIM_ERR_ALLOC : GRIM_ERR_CUDA;
    }
    if (st == GRIM_OK) {
      // ---- cooperative-grid shape: up to 128 CTAs, weights on-chip if they fit, else streamed from L2
      ModeCfg& m = g->grid;
      m.tpc = (ntri + 127) / 128;
      if (3 * m.tpc <= kMaxLocalBands) {
        m.ctas = (ntri + m.tpc - 1) / m.tpc;
        const int nb = 3 * m.tpc;
        m.ks = std::max(1, std::min(4, 32 / nb));
        m.threads = std::min(1024, std::max(nb * m.ks * 32, ((m.tpc * bh + 31) / 32) * 32));
        residency_needs(g, m);
        m.resident = 1;
        m.smem = smem_bytes(g, m, BHc, false);
        if (m.smem > kSmemLimit) { m.resident = 0; m.smem = smem_bytes(g, m, BHc, false); }
        m.ok = m.smem <= kSmemLimit;
      }
      // ---- cluster shape: the largest cluster (<= 16 CTAs) that divides the unit groups evenly
      for (int cs = 16; cs >= 1 && !g->cluster.ok; cs >>= 1) {
        if (ntri % cs) continue;
        ModeCfg t;
        t.tpc = ntri / cs;
        if (3 * t.tpc > kMaxLocalBands || t.tpc * bh > 1024) continue;
        t.ctas = cs;
        const int nb = 3 * t.tpc;
        t.ks = std::max(1, std::min(4, 32 / nb));
        t.threads = std::min(1024, std::max(std::max(nb * t.ks * 32, ((t.tpc * bh + 31) / 32) * 32), 256));
        residency_needs(g, t);
        t.resident = 1;
        t.smem = smem_bytes(g, t, BHc, true);
        if (t.smem > kSmemLimit) continue;  // the cluster scheme is only used with weights on-chip
        g->cluster = t;
        g->cluster.ok = cluster_fits(smem_cluster_kernel(BHc), g->cluster);
        if (!g->cluster.ok) g->cluster = ModeCfg{};
      }
      // ---- register-resident cluster shape: 16 warps, two work items per band
      const int slots_needed = (max_half_band_columns(g) + 31) / 32;
      for (int cs = 16; cs >= 1 && !g->regc.ok; cs >>= 1) {
        if (ntri % cs) continue;
        ModeCfg t;
        t.tpc = ntri / cs;
        const int nb = 3 * t.tpc;
        if (t.tpc * bh > kRegThreads) continue;
        const int ni_needed = (nb * 2 + kRegWarps - 1) / kRegWarps;
        const int menu[4][2] = {{1, 2}, {1, 4}, {3, 3}, {3, 4}};
        for (const auto& v : menu) {
          if (v[0] < ni_needed || v[1] < slots_needed || !reg_kernel(BHc, v[0], v[1])) continue;
          t.ctas = cs; t.ks = 2; t.threads = kRegThreads; t.resident = 1;
          t.smem = ((((size_t)2 * H + (size_t)((t.tpc * bh + 3) & ~3) + (size_t)nb * 2 * BHc) * 4 + 15) & ~size_t(15)) + 16;  // + the two state barriers
          if (t.smem > kSmemLimit || !cluster_fits(reg_kernel(BHc, v[0], v[1]), t)) continue;
          t.ok = true;
          g->regc = t; g->reg_ni = v[0]; g->reg_s = v[1];
          break;
        }
      }
      if (g->regc.ok) {
        // register image: for every thread of every CTA the columns it owns (global index + values at row positions)
        const int NI = g->reg_ni, S = g->reg_s, tpc = g->regc.tpc, cs = g->regc.ctas, nbb = 3 * tpc;
        const size_t nval = (size_t)cs * NI * S * BHc * kRegThreads, ncol = (size_t)cs * NI * S * kRegThreads;
        std::vector<float> iv(nval);
        std::vector<uint32_t> ic(ncol);
        struct ColRec { uint32_t col; float v[16]; };
        std::vector<ColRec> cols;
        for (int l = 0; l < layers && st == GRIM_OK; ++l) {
          const grim_bcr* wh = W_hh[l];
          std::fill(iv.begin(), iv.end(), 0.f);
          std::fill(ic.begin(), ic.end(), 0u);
          for (int rank = 0; rank < cs; ++rank)
            for (int lb = 0; lb < nbb; ++lb) {
              const int64_t band = (int64_t)(lb % 3) * ntri + (int64_t)rank * tpc + lb / 3;
              cols.clear();
              for (int64_t j = 0; j < wh->nbc; ++j) {
                const HostBlock& hb = wh->blocks[(size_t)(band * wh->nbc + j)];
                if (!(hb.kr && hb.kc)) continue;
                int bidx = 0;
                for (int c = 0; c < wh->bw; ++c) {
                  if (!((hb.colmask >> c) & 1ull)) continue;
                  ColRec cr;
                  cr.col = (uint32_t)(j * wh->bw + c);
                  int a = 0;
                  for (int r = 0; r < 16; ++r) {
                    cr.v[r] = 0.f;
                    if ((hb.rowmask >> r) & 1u) cr.v[r] = wh->vals[(size_t)hb.val_off + (size_t)(a++) * hb.kc + (size_t)bidx];
                  }
                  cols.push_back(cr);
                  ++bidx;
                }
              }
              const size_t n = cols.size(), mid = (n + 1) / 2;
              for (int half = 0; half < 2; ++half) {
                const int item = lb * 2 + half, warp = item / NI, i = item % NI;
                const size_t c0 = half ? mid : 0, c1 = half ? n : mid;
                for (size_t ci = c0; ci < c1; ++ci) {
                  const size_t k = ci - c0;
                  const int sl = (int)(k / 32), lane = (int)(k % 32);
                  if (sl >= S || warp >= kRegWarps) { st = GRIM_ERR_UNSUPPORTED; break; }
                  const int tid = warp * 32 + lane;
                  ic[((size_t)(rank * NI + i) * S + sl) * kRegThreads + tid] = cols[ci].col;
                  for (int r = 0; r < BHc; ++r)
                    iv[(((size_t)(rank * NI + i) * S + sl) * BHc + r) * kRegThreads + tid] = cols[ci].v[r];
                }
              }
            }
          if (st != GRIM_OK) break;
          float* dv = nullptr;
          uint32_t* dc = nullptr;
          cudaError_t e = cudaMalloc((void**)&dv, nval * 4);
          if (e == cudaSuccess) { g->d_img_val.push_back(dv); e = cudaMalloc((void**)&dc, ncol * 4); }
          if (e == cudaSuccess) { g->d_img_col.push_back(dc); e = cudaMemcpy(dv, iv.data(), nval * 4, cudaMemcpyHostToDevice); }
          if (e == cudaSuccess) e = cudaMemcpy(dc, ic.data(), ncol * 4, cudaMemcpyHostToDevice);
          if (e != cudaSuccess) st = e == cudaErrorMemoryAllocation ? GRIM_ERR_ALLOC : GRIM_ERR_CUDA;
        }
      }
      if (st == GRIM_OK && !g->grid.ok && !g->cluster.ok && !g->regc.ok) st = GRIM_ERR_UNSUPPORTED;
    }
  } catch (const std::bad_alloc&) {
    st = GRIM_ERR_ALLOC;
  }
  if (st != GRIM_OK) { cudaGetLastError(); destroy(g); return st; }
  *out = g;
  return GRIM_OK;
}

extern "C" grim_status_t grim_gru_seq(grim_gru_t g, const float* x, int64_t T, const float* h0, float* y, float* hT,
                                      grim_stream_t stream) {
  if (!g || !x || !y || T <= 0) return GRIM_ERR_INVALID_ARG;
  if (T > g->max_T) return GRIM_ERR_SHAPE;
  cudaStream_t s0 = (cudaStream_t)stream;
  g->last_stream = s0;
  const int64_t H = g->H;
  const int L = g->L;
  // preference: weights in registers > cooperative grid > shared-memory cluster
  const bool want_grid = g->force_grid && g->grid.ok;
  const bool use_reg = g->regc.ok && !want_grid;
  const bool use_cluster = !use_reg && g->cluster.ok && !g->grid.ok;
  const ModeCfg& m = use_reg ? g->regc : (use_cluster ? g->cluster : g->grid);
  const int BHc = g->bh <= 4 ? 4 : (g->bh <= 8 ? 8 : 16);
  if (cudaMemsetAsync(g->d_sync, 0, (size_t)(L + 1) * 4, s0) != cudaSuccess) return GRIM_ERR_CUDA;

  // Time is cut into chunks; layer l works on chunk k while layer l - 1 works on chunk k + 1 (each layer on its own
  // stream, ordered by events), so a stack of L layers takes about (1 + (L - 1) / chunks) single-layer times instead
  // of L.  The kernels with a global barrier (fall-back) and single-layer models run as one chunk on one stream.
  int chunks = 1;
  // With four or more layers, layers l and l + 2 share an inter-layer buffer, and layer l reads its chunk-entering
  // state from that buffer while layer l + 2 may already be writing it: such stacks run one layer after the other.
  if (g->pipeline && L > 1 && L <= 3 && (use_reg || use_cluster))
    chunks = g->want_chunks > 0 ? (int)std::min<int64_t>(g->want_chunks, T)
                                : (int)std::max<int64_t>(1, std::min<int64_t>(3, T / 64));
  const int64_t clen = ((T + chunks - 1) / chunks + 3) / 4 * 4;  // a multiple of 4: chunk starts stay 16-byte aligned
  const int64_t ldT = (T + 3) / 4 * 4;
  const bool tin = g->transposed_inputs && g->d_xT != nullptr;
  auto stream_of = [&](int l) { return (chunks > 1 && l > 0) ? g->lstream[(size_t)l - 1] : s0; };
  if (chunks > 1) {
    if (cudaEventRecord(g->ev_fork, s0) != cudaSuccess) return GRIM_ERR_CUDA;
    for (int l = 1; l < L; ++l)
      if (cudaStreamWaitEvent(g->lstream[(size_t)l - 1], g->ev_fork, 0) != cudaSuccess) return GRIM_ERR_CUDA;
  }
  if (g->profile) g->ev_used = 0;
  // every row of a pre-activation buffer starts as b_ih: the projections may add partial sums onto it
  auto prefill = [&](int l, cudaStream_t s) {
    const int64_t total = T * 3 * H;
    fill_rows_kernel<<<(unsigned)std::min<int64_t>((total / 4 + 255) / 256, (int64_t)sm_count(g->device) * 8), 256, 0, s>>>(g->d_gi[(size_t)l], g->d_bih[(size_t)l], T, 3 * H);
    count_launch();
    return cudaGetLastError() == cudaSuccess;
  };
  for (int l = 0; l < L; ++l) {
    if (l > 0 && g->d_gi[(size_t)l] == g->d_gi[0]) break;  // one shared buffer: filled per layer, below
    if (!prefill(l, stream_of(l))) return GRIM_ERR_CUDA;
  }

  auto launch_projection = [&](int l, const float* seq_in, int64_t t0, int64_t n, cudaStream_t s) -> grim_status_t {
    const grim_bcr* wi = g->Wih[(size_t)l];
    // gi[t, :] = W_ih x_t + b_ih for the n steps from t0 (X given q-major as n x in, output n x 3H)
    SpmmArgs a;
    a.Y = g->d_gi[(size_t)l] + t0 * 3 * H; a.ncols = n;
    a.y_sr = 1; a.y_sq = 3 * H;
    if (tin) {  // feature-major copy: a plain row-major K x n operand (fetched by TMA)
      a.X = (l == 0 ? g->d_xT : g->d_seqT[(l - 1) & 1]) + t0;
      a.x_sk = ldT; a.x_sq = 1;
    } else {
      a.X = seq_in + t0 * wi->K;
      a.x_sk = 1; a.x_sq = wi->K;
    }
    a.x_dtype = GRIM_F32; a.y_dtype = GRIM_F32;
    a.bias = g->d_bih[(size_t)l];
    a.y_prefilled = 1;  // every row of the buffer already holds b_ih (below): a split multiply adds onto it and
                        // needs neither its own clearing nor a bias pass; an unsplit one writes sum + bias as usual
    if (g->profile) profile_mark(g, 0, s);
    const grim_status_t st = ffma_path_supported(wi, a) ? launch_ffma(wi, a, s) : launch_spmm(wi, a, s);
    if (g->profile) profile_mark(g, 1, s);
    return st;
  };
  auto launch_recurrence = [&](int l, float* seq_out, int64_t t0, int64_t n, cudaStream_t s) -> grim_status_t {
    const grim_bcr* wh = g->Whh[(size_t)l];
    GruParams p;
    p.band_ptr = wh->d_gemv_band_ptr; p.chunks = wh->d_chunks; p.colwords = wh->d_colwords;
    p.vals = static_cast<const float*>(wh->d_gemv_vals); p.pos_of_band = g->d_pos_of_band[(size_t)l];
    p.b_hh = g->d_bhh[(size_t)l]; p.b_ih = nullptr; p.gi = g->d_gi[(size_t)l] + t0 * 3 * H;
    // the state entering a later chunk is the previous chunk's last output row
    p.h0 = t0 == 0 ? (h0 ? h0 + (int64_t)l * H : nullptr) : seq_out + (t0 - 1) * H;
    p.out = seq_out + t0 * H;
    p.outT = (tin && l < L - 1) ? g->d_seqT[l & 1] + t0 : nullptr;
    p.ldT = ldT;
    p.hT = (hT && t0 + n == T) ? hT + (int64_t)l * H : nullptr;
    p.bar = g->d_sync + l; p.status = g->d_sync + L;
    p.H = (int)H; p.bh = g->bh; p.T = (int)n; p.tpc = m.tpc; p.ks = m.ks; p.resident = m.resident;
    p.max_chunks = m.max_chunks; p.max_cw = m.max_cw; p.max_vals = m.max_vals;
    p.skip_cta = g->dbg_skip_cta; p.spin_limit = g->spin_limit;
    p.img_val = use_reg ? g->d_img_val[(size_t)l] : nullptr;
    p.img_col = use_reg ? g->d_img_col[(size_t)l] : nullptr;
    if (g->profile) profile_mark(g, 2, s);
    cudaError_t e;
    if (use_reg) {
      e = launch_cluster(reg_kernel(BHc, g->reg_ni, g->reg_s), m, p, s);
    } else if (use_cluster) {
      e = launch_cluster(smem_cluster_kernel(BHc), m, p, s);
    } else {
      if (g->bh <= 4) e = launch_grid<4>(g, p, s);
      else if (g->bh <= 8) e = launch_grid<8>(g, p, s);
      else e = launch_grid<16>(g, p, s);
    }
    if (g->profile) profile_mark(g, 3, s);
    if (e != cudaSuccess) { cudaGetLastError(); return e == cudaErrorCooperativeLaunchTooLarge ? GRIM_ERR_UNSUPPORTED : GRIM_ERR_CUDA; }
    return GRIM_OK;
  };

  // issue order: chunk-major over layers (a wavefront), so that every stream always has work queued
  for (int k = 0; k < chunks + L - 1; ++k) {
    for (int l = 0; l < L; ++l) {
      const int c = k - l;  // the chunk layer l handles in this wave
      if (c < 0 || c >= chunks) continue;
      const int64_t t0 = (int64_t)c * clen, n = std::min<int64_t>(clen, T - t0);
      if (n <= 0) continue;
      cudaStream_t s = stream_of(l);
      const float* seq_in = l == 0 ? x : g->d_seq[(l - 1) & 1];
      float* seq_out = (l == L - 1) ? y : g->d_seq[l & 1];
      grim_status_t st = GRIM_OK;
      if (l > 0 && c == 0 && g->d_gi[(size_t)l] == g->d_gi[0] && !prefill(l, s))
        return GRIM_ERR_CUDA;  // layers share one buffer (allocation-free variant): fill it again for this layer
      if (l == 0) {
        if (c == 0) {  // the first layer's input is all there: one launch (after turning it feature-major)
          if (tin) {
            const int64_t K0 = g->Wih[0]->K;
            transpose_input_kernel<<<dim3((unsigned)((T + 31) / 32), (unsigned)((K0 + 31) / 32)), dim3(32, 8), 0, s>>>(x, g->d_xT, T, K0, ldT);
            count_launch();
          }
          st = launch_projection(0, x, 0, T, s);
        }
      } else {
        if (chunks > 1 && cudaStreamWaitEvent(s, g->ev_chunk[(size_t)(l - 1) * g->max_chunks + c], 0) != cudaSuccess) return GRIM_ERR_CUDA;
        st = launch_projection(l, seq_in, t0, n, s);
      }
      if (st != GRIM_OK) return st;
      st = launch_recurrence(l, seq_out, t0, n, s);
      if (st != GRIM_OK) return st;
      if (chunks > 1 && cudaEventRecord(g->ev_chunk[(size_t)l * g->max_chunks + c], s) != cudaSuccess) return GRIM_ERR_CUDA;
    }
  }
  if (chunks > 1) {
    // join: the caller's stream continues when the last layer is done (lower layers finish earlier by construction,
    // but their streams are joined too so that the handle's buffers are quiescent)
    for (int l = 1; l < L; ++l)
      if (cudaStreamWaitEvent(s0, g->ev_chunk[(size_t)l * g->max_chunks + chunks - 1], 0) != cudaSuccess) return GRIM_ERR_CUDA;
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

// Test hook: selects the cooperative-grid kernel (the one with spin waits) whenever skip_cta >= 0 or a
// poll limit is given, makes thread block `skip_cta` stay away from its barrier and sets the number of
// polls after which a waiting block gives up.  The waits then run out and the status word reports it;
// no thread block ever waits without a bound.
extern "C" grim_status_t grim_gru_debug_barrier(grim_gru_t g, int skip_cta, unsigned spin_limit) {
  if (!g) return GRIM_ERR_INVALID_ARG;
  if ((skip_cta >= 0 || spin_limit) && !g->grid.ok) return GRIM_ERR_UNSUPPORTED;
  g->dbg_skip_cta = skip_cta;
  g->spin_limit = spin_limit ? spin_limit : (1u << 22);
  g->force_grid = skip_cta >= 0 || spin_limit != 0;
  return GRIM_OK;
}

extern "C" grim_status_t grim_gru_set_pipeline(grim_gru_t g, int chunks) {
  if (!g || chunks < 0 || chunks > g->max_chunks) return GRIM_ERR_INVALID_ARG;
  g->pipeline = chunks != 1;
  g->want_chunks = chunks;
  return GRIM_OK;
}

extern "C" grim_status_t grim_gru_profile(grim_gru_t g, int enable) {
  if (!g) return GRIM_ERR_INVALID_ARG;
  if (enable && g->ev.empty()) {
    g->ev.resize((size_t)4 * g->L * g->max_chunks);
    g->ev_kind.assign(g->ev.size(), 0);
    for (cudaEvent_t& e : g->ev)
      if (cudaEventCreate(&e) != cudaSuccess) return GRIM_ERR_CUDA;
  }
  g->profile = enable != 0;
  g->ev_used = 0;
  return GRIM_OK;
}

extern "C" grim_status_t grim_gru_profile_read(grim_gru_t g, float* projection_ms, float* recurrent_ms) {
  if (!g || !g->profile || g->ev.empty()) return GRIM_ERR_INVALID_ARG;
  float pj = 0.f, rc = 0.f;
  for (int i = 0; i + 1 < g->ev_used; i += 2) {
    float ms = 0.f;
    if (cudaEventSynchronize(g->ev[(size_t)i + 1]) != cudaSuccess) return GRIM_ERR_CUDA;
    if (cudaEventElapsedTime(&ms, g->ev[(size_t)i], g->ev[(size_t)i + 1]) != cudaSuccess) return GRIM_ERR_CUDA;
    if (g->ev_kind[(size_t)i] == 0) pj += ms; else rc += ms;
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
  // Run the ordinary pass with the handle's scratch pointers pointing into the static array for the duration of
  // the call (kernel arguments are copied at launch, so the handle can be put back at once).  All layers share one
  // pre-activation buffer here, so the layers run one after the other on the caller's stream.
  std::copy(g->d_gi.begin(), g->d_gi.end(), g->d_gi_saved.begin());  // same size since creation: no allocation
  float* const saved_seq0 = g->d_seq[0];
  float* const saved_seq1 = g->d_seq[1];
  const bool saved_pipeline = g->pipeline, saved_tin = g->transposed_inputs;
  g->transposed_inputs = false;  // the feature-major copies live in allocated buffers: not used here
  for (float*& p : g->d_gi) p = reinterpret_cast<float*>(base);
  g->d_seq[0] = reinterpret_cast<float*>(base + gi_bytes);
  g->d_seq[1] = reinterpret_cast<float*>(base + gi_bytes + seq_bytes);
  g->pipeline = false;
  const grim_status_t st = grim_gru_seq(g, x, T, h0, y, hT, stream);
  std::copy(g->d_gi_saved.begin(), g->d_gi_saved.end(), g->d_gi.begin());
  g->d_seq[0] = saved_seq0;
  g->d_seq[1] = saved_seq1;
  g->pipeline = saved_pipeline;
  g->transposed_inputs = saved_tin;
  return st;
}

// -------------------------------------------------------------------------------------------------------------
// One time step for a batch of sequences (Section 6.3 times the GRU at sequence length 1 and batch 32): per layer two
// sparse multiplies with the batch as right-hand side (W_ih x and W_hh h, each with its bias in the epilogue) and one
// fused gate kernel.
// -------------------------------------------------------------------------------------------------------------
namespace {
// h'[b, u] = (1 - z) * n + z * h[b, u] with r, z, n from the two pre-activation buffers (batch-major, 3H per row);
// the state is updated in place and copied to y when given.
__global__ void gru_gate_kernel(const float* __restrict__ gi, const float* __restrict__ gh, float* __restrict__ h,
                                float* __restrict__ y, int64_t B, int64_t H) {
  const int64_t total = B * H;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t b = i / H, u = i - b * H;
    const float* a = gi + b * 3 * H;
    const float* q = gh + b * 3 * H;
    const float r = sigmoidf_(a[u] + q[u]);
    const float z = sigmoidf_(a[H + u] + q[H + u]);
    const float n = tanhf(a[2 * H + u] + r * q[2 * H + u]);
    const float hn = (1.f - z) * n + z * h[i];
    h[i] = hn;
    if (y) y[i] = hn;
  }
}
}  // namespace

extern "C" grim_status_t grim_gru_step(grim_gru_t g, const float* x, int64_t B, float* h, float* y, grim_stream_t stream) {
  if (!g || !x || !h || B <= 0) return GRIM_ERR_INVALID_ARG;
  if (2 * B > g->max_T) return GRIM_ERR_SHAPE;  // both pre-activation buffers of a layer live in its T x 3H scratch
  cudaStream_t s = (cudaStream_t)stream;
  const int64_t H = g->H;
  const float* in = x;
  for (int l = 0; l < g->L; ++l) {
    float* hl = h + (int64_t)l * B * H;
    float* gi = g->d_gi[(size_t)l];
    float* gh = gi + B * 3 * H;
    const grim_bcr* mats[2] = {g->Wih[(size_t)l], g->Whh[(size_t)l]};
    const float* rhs[2] = {in, hl};
    float* outs[2] = {gi, gh};
    const float* bias[2] = {g->d_bih[(size_t)l], g->d_bhh[(size_t)l]};
    for (int t = 0; t < 2; ++t) {
      // batch-major operands: X(k, b) at b * K + k, Y(r, b) at b * 3H + r
      SpmmArgs a;
      a.X = rhs[t]; a.Y = outs[t]; a.ncols = B;
      a.x_sk = 1; a.x_sq = mats[t]->K; a.y_sr = 1; a.y_sq = 3 * H;
      a.x_dtype = GRIM_F32; a.y_dtype = GRIM_F32;
      a.bias = bias[t];
      const grim_status_t st = ffma_path_supported(mats[t], a) ? launch_ffma(mats[t], a, s) : launch_spmm(mats[t], a, s);
      if (st != GRIM_OK) return st;
    }
    const int64_t total = B * H;
    gru_gate_kernel<<<(unsigned)std::min<int64_t>((total + 255) / 256, (int64_t)sm_count(g->device) * 8), 256, 0, s>>>(
        gi, gh, hl, l == g->L - 1 ? y : nullptr, B, H);
    count_launch();
    if (cudaGetLastError() != cudaSuccess) return GRIM_ERR_CUDA;
    in = hl;
  }
  g->last_stream = s;
  return GRIM_OK;
}
