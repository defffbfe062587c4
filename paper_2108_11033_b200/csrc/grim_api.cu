// C-ABI entry points for the multiply, the convolution and small helpers: argument checks and
// marshalling only; all arithmetic runs in the kernels.
#include <cuda_bf16.h>

#include <algorithm>

#include "grim_internal.h"

using namespace grim;

namespace {

grim_status_t check_mats(const grim_bcr* h, const grim_mat_t* X, const grim_mat_t* Y) {
  if (!h || !X || !Y || !X->ptr || !Y->ptr) return GRIM_ERR_INVALID_ARG;
  if (h->device < 0) return GRIM_ERR_INVALID_ARG;
  if (X->rows != h->K || Y->rows != h->M || X->cols != Y->cols || X->cols <= 0) return GRIM_ERR_SHAPE;
  if (X->ld < X->cols || Y->ld < Y->cols) return GRIM_ERR_SHAPE;
  if ((int)X->dtype != h->dtype) return GRIM_ERR_DTYPE;
  if (Y->dtype != GRIM_F32 && !(Y->dtype == GRIM_BF16 && h->dtype == GRIM_BF16)) return GRIM_ERR_DTYPE;
  return GRIM_OK;
}

SpmmArgs mat_args(const grim_mat_t* X, const grim_mat_t* Y) {
  SpmmArgs a;
  a.X = X->ptr; a.Y = Y->ptr; a.ncols = X->cols;
  a.x_sk = X->ld; a.x_sq = 1; a.y_sr = Y->ld; a.y_sq = 1;
  a.x_dtype = X->dtype; a.y_dtype = Y->dtype;
  return a;
}

// Slot of the tune cache for a request: right-hand sides whose widths fall into the same power-of-two bucket share
// an answer (tile choices change with the order of magnitude of N, not with N).
grim_tune_t* tuned_slot(grim_bcr_t h, const grim_mat_t* X, const grim_mat_t* Y) {
  int b = 0;
  while (b < 31 && (int64_t(1) << b) < X->cols) ++b;
  return &h->tuned[b][X->dtype == GRIM_BF16 ? 1 : 0][Y->dtype == GRIM_BF16 ? 1 : 0];
}

grim_status_t run_spmm(grim_bcr_t h, const grim_mat_t* X, grim_mat_t* Y, const grim_tune_t* tune, cudaStream_t s) {
  grim_status_t st = check_mats(h, X, Y);
  if (st != GRIM_OK) return st;
  if (!tune) {  // no explicit choice: an earlier grim_bcr_tune for this kind of request decides
    const grim_tune_t* t = tuned_slot(h, X, Y);
    if (t->path != 0) tune = t;
  }
  int path = tune ? tune->path : 0;
  if (path < 0 || path > 5) return GRIM_ERR_INVALID_ARG;
  if (path == 0 && tune && tune->tile_n >= 16) path = 4;  // a column-tile width only means something to the slab kernel
  SpmmArgs a = mat_args(X, Y);
  a.tile_n = tune ? tune->tile_n : 0;
  if (path == 2) {
    if (!tc_path_supported(h, a)) return GRIM_ERR_UNSUPPORTED;
    return launch_spmm_tc(h, a, s);
  }
  if (path == 5) {
    if (!tc2_path_supported(h, a)) return GRIM_ERR_UNSUPPORTED;
    return launch_spmm_tc2(h, a, s);
  }
  // 8 <= N <= 16, measured at 8192 x 8192 and 4096 x 4096: bf16 handles are fastest on the tensor-core tile (56 us
  // split over K against 102 us on the lane-per-column kernel), fp32 handles with blocks of 8 rows or more on the
  // CUDA-core kernel's 16-column tile (93 against 98 - 124 us); narrower right-hand sides stay on the lane-per-column
  // kernel
  if (path == 0 && X->cols >= 8 && X->cols <= kSkinnyMaxN) {
    if (tc_path_supported(h, a) && h->tc_mtiles >= 8) return launch_spmm_tc(h, a, s);
    if (h->dtype == GRIM_F32 && h->bh >= 8 && ffma_path_supported(h, a)) return launch_ffma(h, a, s);
  }
  if (path == 3 || (path == 0 && X->cols <= kSkinnyMaxN && h->gemv_ok)) {
    // tile_n = 1 under path 3 asks for the register-staged variant; otherwise the streaming one runs when it can
    if (!(path == 3 && a.tile_n == 1) && stream_path_supported(h, X->cols))
      return launch_stream(h, X->ptr, X->dtype, X->ld, X->cols, Y->ptr, Y->dtype, Y->ld, s);
    if (path == 3 && a.tile_n == 2) return GRIM_ERR_UNSUPPORTED;
    return launch_skinny(h, X->ptr, X->dtype, X->ld, X->cols, Y->ptr, Y->dtype, Y->ld, s);
  }
  if (path == 4) return launch_spmm(h, a, s);
  // bf16 handles, wide right-hand sides: tensor cores.  The paired kernel when its 256 x 512 tiles still give most
  // SMs a thread block (measured: with fewer, the single-block kernel's smaller tiles win).
  if (path == 0 && tc2_path_supported(h, a) && a.ncols >= 256 && h->tc_mtiles >= 2 &&
      2 * ((h->tc_mtiles + 1) / 2) * ((a.ncols + 511) / 512) * 3 >= 2 * (int64_t)sm_count(h->device))
    return launch_spmm_tc2(h, a, s);
  // (measured at 8192 x 8192, bf16: from N = 32 up the tensor-core tile is 2.6 times faster than the CUDA-core kernel,
  // which widens bf16 to fp32 on the way in; N <= 16 goes to the lane-per-column kernel above)
  if (path == 0 && tc_path_supported(h, a) && a.ncols > kSkinnyMaxN) return launch_spmm_tc(h, a, s);
  if (ffma_path_supported(h, a)) return launch_ffma(h, a, s);
  if (path == 1) return GRIM_ERR_UNSUPPORTED;
  return launch_spmm(h, a, s);
}

int dev_sms() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) dev = 0;
  return sm_count(dev);
}

// 16 independent chains of dependent fused multiply-adds per thread: enough independent work per warp to keep
// the fp32 pipes full at full occupancy.  The result is stored so that nothing is optimised away.
__global__ void __launch_bounds__(512) ffma_peak_kernel(float* __restrict__ out, int iters, float a, float b) {
  float acc[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) acc[i] = (float)(threadIdx.x + i);
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = fmaf(acc[i], a, b);
  }
  float sum = 0.f;
#pragma unroll
  for (int i = 0; i < 16; ++i) sum += acc[i];
  out[blockIdx.x * (int64_t)blockDim.x + threadIdx.x] = sum;
}

template <typename T>
__global__ void maxpool2x2_kernel(const T* __restrict__ in, T* __restrict__ out, int64_t planes, int H, int W) {
  const int OH = H / 2, OW = W / 2;
  const int64_t total = planes * OH * OW;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int ow = (int)(i % OW);
    const int64_t t = i / OW;
    const int oh = (int)(t % OH);
    const int64_t pl = t / OH;
    const T* p = in + (pl * H + 2 * oh) * W + 2 * ow;
    const float a = (float)p[0], b = (float)p[1], c = (float)p[W], d = (float)p[W + 1];
    out[i] = (T)fmaxf(fmaxf(a, b), fmaxf(c, d));
  }
}

}  // namespace

extern "C" grim_status_t grim_bcr_spmm(grim_bcr_t h, const grim_mat_t* X, grim_mat_t* Y, grim_stream_t stream) {
  return run_spmm(h, X, Y, nullptr, (cudaStream_t)stream);
}

extern "C" grim_status_t grim_bcr_spmm_ex(grim_bcr_t h, const grim_mat_t* X, grim_mat_t* Y, const grim_tune_t* tune,
                                          grim_stream_t stream) {
  return run_spmm(h, X, Y, tune, (cudaStream_t)stream);
}

extern "C" grim_status_t grim_bcr_tune(grim_bcr_t h, const grim_mat_t* X, grim_mat_t* Y, int reps, grim_tune_t* best,
                                       float* best_ms, grim_stream_t stream) {
  if (!best) return GRIM_ERR_INVALID_ARG;
  grim_status_t st = check_mats(h, X, Y);
  if (st != GRIM_OK) return st;
  const bool cold = reps < 0;  // flush the L2 cache before every timed launch
  if (reps < 0) reps = -reps;
  if (reps == 0) reps = 5;
  cudaStream_t s = (cudaStream_t)stream;
  constexpr size_t kFlushBytes = size_t(256) << 20;
  void* flush = nullptr;
  if (cold && cudaMalloc(&flush, kFlushBytes) != cudaSuccess) { cudaGetLastError(); return GRIM_ERR_ALLOC; }
  cudaEvent_t e0, e1;
  if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) { cudaFree(flush); return GRIM_ERR_CUDA; }
  float best_t = -1.f;
  grim_tune_t cand_best{};
  // candidates: (path, tile_n); a candidate that cannot take the request is skipped
  const int cand[][2] = {{1, 1}, {1, 2}, {1, 4}, {1, 8}, {1, 9}, {1, 17}, {1, 18}, {1, 20}, {2, 0}, {5, 0}, {3, 1}, {3, 2}, {4, 16}, {4, 32}, {4, 64}, {4, 128}};
  for (const auto& cd : cand) {
    grim_tune_t c{};
    c.path = cd[0];
    c.tile_n = cd[1];
    if (c.path == 3 && X->cols > kSkinnyMaxN) continue;
    if (c.path == 4 && c.tile_n > 16 && c.tile_n / 2 >= X->cols) continue;  // idle lanes only
    // CUDA-core kernel: 1, 2, 4 = bands per warp; 8, 9 = two 128-column pieces per lane with one or two bands per warp
    if (c.path == 1 && c.tile_n <= 4 && c.tile_n > (h->bh <= 4 ? 4 : (h->bh <= 8 ? 2 : 1))) continue;
    if (c.path == 1 && (c.tile_n == 8 || c.tile_n == 9) && (h->bh > (c.tile_n == 8 ? 8 : 4) || X->cols <= 128)) continue;
    // ... 17, 18, 20 = the narrow tile (at most 16 columns) with 1, 2, 4 bands per warp
    if (c.path == 1 && c.tile_n >= 17 && (X->cols > 16 || c.tile_n - 16 > (h->bh <= 8 ? 4 : 2))) continue;
    if (c.path == 1 && c.tile_n < 17 && X->cols <= 16) continue;
    st = run_spmm(h, X, Y, &c, s);  // warm-up
    if (st == GRIM_ERR_UNSUPPORTED) { st = GRIM_OK; continue; }
    if (st != GRIM_OK) break;
    float ms = 0.f;
    if (!cold) {
      cudaEventRecord(e0, s);
      for (int r = 0; r < reps && st == GRIM_OK; ++r) st = run_spmm(h, X, Y, &c, s);
      cudaEventRecord(e1, s);
      if (st != GRIM_OK || cudaEventSynchronize(e1) != cudaSuccess) { st = st == GRIM_OK ? GRIM_ERR_CUDA : st; break; }
      cudaEventElapsedTime(&ms, e0, e1);
    } else {
      for (int r = 0; r < reps && st == GRIM_OK; ++r) {
        cudaMemsetAsync(flush, r & 1, kFlushBytes, s);
        cudaEventRecord(e0, s);
        st = run_spmm(h, X, Y, &c, s);
        cudaEventRecord(e1, s);
        if (st != GRIM_OK || cudaEventSynchronize(e1) != cudaSuccess) { st = st == GRIM_OK ? GRIM_ERR_CUDA : st; break; }
        float t = 0.f;
        cudaEventElapsedTime(&t, e0, e1);
        ms += t;
      }
      if (st != GRIM_OK) break;
    }
    ms /= reps;
    if (best_t < 0.f || ms < best_t) { best_t = ms; cand_best = c; }
  }
  if (st == GRIM_OK && best_t < 0.f) st = GRIM_ERR_UNSUPPORTED;
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  if (flush) {
    cudaStreamSynchronize(s);
    cudaFree(flush);
  }
  if (st != GRIM_OK) return st;
  *best = cand_best;
  if (best_ms) *best_ms = best_t;
  *tuned_slot(h, X, Y) = cand_best;  // grim_bcr_spmm takes this choice for requests of the same kind from now on
  return GRIM_OK;
}

extern "C" grim_status_t grim_bcr_reserve(grim_bcr_t h, int64_t max_ncols) {
  if (!h || max_ncols < 0) return GRIM_ERR_INVALID_ARG;
  if (h->device < 0) return GRIM_ERR_INVALID_ARG;
  const size_t need = (size_t)h->M * (size_t)max_ncols * 4;
  if (need > ((size_t)1 << 30)) return GRIM_ERR_UNSUPPORTED;  // the split multiply is only used for small outputs
  if (h->tc_acc_bytes >= need && need > 0) return GRIM_OK;
  if (cudaDeviceSynchronize() != cudaSuccess) return GRIM_ERR_CUDA;  // a launch in flight may still use the old scratch
  cudaFree(h->d_tc_acc);
  h->d_tc_acc = nullptr;
  h->tc_acc_bytes = 0;
  if (need == 0) return GRIM_OK;
  if (cudaMalloc((void**)&h->d_tc_acc, need) != cudaSuccess) { cudaGetLastError(); return GRIM_ERR_ALLOC; }
  h->tc_acc_bytes = need;
  return GRIM_OK;
}

extern "C" grim_status_t grim_bcr_conv2d(grim_bcr_t h, const grim_conv_desc_t* d, const void* in, void* out,
                                         grim_stream_t stream) {
  if (!h || !d || !in || !out) return GRIM_ERR_INVALID_ARG;
  if (h->device < 0) return GRIM_ERR_INVALID_ARG;
  if (d->N <= 0 || d->C <= 0 || d->H <= 0 || d->W <= 0 || d->KH <= 0 || d->KW <= 0 || d->stride <= 0 || d->pad < 0)
    return GRIM_ERR_INVALID_ARG;
  if (d->flags & ~(GRIM_CONV_RELU | GRIM_CONV_PAIRED | GRIM_CONV_SINGLE)) return GRIM_ERR_INVALID_ARG;
  if (d->C * (int64_t)d->KH * d->KW != h->K) return GRIM_ERR_SHAPE;
  const int64_t OH = (d->H + 2 * d->pad - d->KH) / d->stride + 1;
  const int64_t OW = (d->W + 2 * d->pad - d->KW) / d->stride + 1;
  if (d->H + 2 * d->pad < d->KH || d->W + 2 * d->pad < d->KW || OH <= 0 || OW <= 0) return GRIM_ERR_SHAPE;
  if ((int)d->in_dtype != h->dtype) return GRIM_ERR_DTYPE;
  if (d->out_dtype != GRIM_F32 && !(d->out_dtype == GRIM_BF16 && h->dtype == GRIM_BF16)) return GRIM_ERR_DTYPE;
  if (d->H > (1 << 20) || d->W > (1 << 20) || d->C > (1 << 24)) return GRIM_ERR_UNSUPPORTED;
  SpmmArgs a;
  a.X = in; a.Y = out; a.ncols = d->N * OH * OW;
  a.x_dtype = d->in_dtype; a.y_dtype = d->out_dtype;
  a.bias = d->bias_dev; a.relu = (d->flags & GRIM_CONV_RELU) ? 1 : 0;
  a.conv = 1; a.C = (int)d->C; a.H = (int)d->H; a.W = (int)d->W; a.KH = d->KH; a.KW = d->KW;
  a.stride = d->stride; a.pad = d->pad; a.OH = (int)OH; a.OW = (int)OW;
  if (d->KH == 1 && d->KW == 1 && d->stride == 1 && d->pad == 0 && !(d->flags & (GRIM_CONV_PAIRED | GRIM_CONV_SINGLE))) {
    // 1 x 1 kernels: the expanded input IS the input - per image a plain Cout x C times C x (H*W) product on the
    // tensors as they lie in memory (row stride H*W), no gather at all; one launch per image
    const int64_t hw = d->H * d->W;
    const size_t in_esz = d->in_dtype == GRIM_BF16 ? 2 : 4, out_esz = d->out_dtype == GRIM_BF16 ? 2 : 4;
    for (int64_t n = 0; n < d->N; ++n) {
      SpmmArgs m;
      m.X = static_cast<const uint8_t*>(in) + (size_t)(n * d->C * hw) * in_esz;
      m.Y = static_cast<uint8_t*>(out) + (size_t)(n * h->M * hw) * out_esz;
      m.ncols = hw; m.x_sk = hw; m.x_sq = 1; m.y_sr = hw; m.y_sq = 1;
      m.x_dtype = d->in_dtype; m.y_dtype = d->out_dtype;
      m.bias = d->bias_dev; m.relu = a.relu;
      grim_status_t st;
      if (tc2_path_supported(h, m) && hw >= 256 && h->tc_mtiles >= 2 &&
          2 * ((h->tc_mtiles + 1) / 2) * ((hw + 511) / 512) * 3 >= 2 * (int64_t)sm_count(h->device))
        st = launch_spmm_tc2(h, m, (cudaStream_t)stream);
      else if (tc_path_supported(h, m) && hw >= 128) st = launch_spmm_tc(h, m, (cudaStream_t)stream);
      else if (ffma_path_supported(h, m)) st = launch_ffma(h, m, (cudaStream_t)stream);
      else st = launch_spmm(h, m, (cudaStream_t)stream);
      if (st != GRIM_OK) return st;
    }
    return GRIM_OK;
  }
  if (d->flags & GRIM_CONV_PAIRED) {
    if (!tc2_path_supported(h, a)) return GRIM_ERR_UNSUPPORTED;
    return launch_spmm_tc2(h, a, (cudaStream_t)stream);
  }
  // bf16 handles: tensor cores; the paired kernel when its 256 x 512 tiles still give most SMs a thread block
  if (!(d->flags & GRIM_CONV_SINGLE) && tc2_path_supported(h, a) && h->tc_mtiles >= 2 &&
      2 * ((h->tc_mtiles + 1) / 2) * ((a.ncols + 511) / 512) * 3 >= 2 * (int64_t)sm_count(h->device))
    return launch_spmm_tc2(h, a, (cudaStream_t)stream);
  if (tc_path_supported(h, a) && a.ncols >= 128) return launch_spmm_tc(h, a, (cudaStream_t)stream);
  if (d->flags & GRIM_CONV_SINGLE) return GRIM_ERR_UNSUPPORTED;
  if (ffma_path_supported(h, a)) return launch_ffma(h, a, (cudaStream_t)stream);
  return launch_spmm(h, a, (cudaStream_t)stream);
}

extern "C" grim_status_t grim_maxpool2x2(const void* in, void* out, int64_t N, int64_t C, int64_t H, int64_t W,
                                         grim_dtype_t dtype, grim_stream_t stream) {
  if (!in || !out || N <= 0 || C <= 0 || H <= 0 || W <= 0) return GRIM_ERR_INVALID_ARG;
  if ((H & 1) || (W & 1)) return GRIM_ERR_SHAPE;
  if (dtype != GRIM_F32 && dtype != GRIM_BF16) return GRIM_ERR_DTYPE;
  const int64_t total = N * C * (H / 2) * (W / 2);
  const int threads = 256;
  const int blocks = (int)std::min<int64_t>((total + threads - 1) / threads, (int64_t)dev_sms() * 16);
  cudaStream_t s = (cudaStream_t)stream;
  if (dtype == GRIM_F32)
    maxpool2x2_kernel<float><<<blocks, threads, 0, s>>>((const float*)in, (float*)out, N * C, (int)H, (int)W);
  else
    maxpool2x2_kernel<__nv_bfloat16><<<blocks, threads, 0, s>>>((const __nv_bfloat16*)in, (__nv_bfloat16*)out, N * C,
                                                                (int)H, (int)W);
  count_launch();
  return cudaGetLastError() == cudaSuccess ? GRIM_OK : GRIM_ERR_CUDA;
}

extern "C" grim_status_t grim_measure_ffma_peak(double* tflops, grim_stream_t stream) {
  if (!tflops) return GRIM_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  const int blocks = dev_sms() * 4, threads = 512, iters = 4096;
  float* out = nullptr;
  if (cudaMalloc((void**)&out, (size_t)blocks * threads * 4) != cudaSuccess) { cudaGetLastError(); return GRIM_ERR_ALLOC; }
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  grim_status_t st = GRIM_OK;
  if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) st = GRIM_ERR_CUDA;
  float best = -1.f;
  for (int rep = 0; rep < 6 && st == GRIM_OK; ++rep) {  // the first repetition is a warm-up
    cudaEventRecord(e0, s);
    ffma_peak_kernel<<<blocks, threads, 0, s>>>(out, iters, 0.999f, 0.001f);
    cudaEventRecord(e1, s);
    count_launch();
    if (cudaEventSynchronize(e1) != cudaSuccess) { st = GRIM_ERR_CUDA; break; }
    float ms = 0.f;
    cudaEventElapsedTime(&ms, e0, e1);
    if (rep > 0 && (best < 0.f || ms < best)) best = ms;
  }
  if (e0) cudaEventDestroy(e0);
  if (e1) cudaEventDestroy(e1);
  cudaFree(out);
  if (st != GRIM_OK || best <= 0.f) return st == GRIM_OK ? GRIM_ERR_CUDA : st;
  *tflops = 2.0 * 16.0 * iters * (double)blocks * threads / (best * 1e-3) / 1e12;
  return GRIM_OK;
}

extern "C" const char* grim_status_string(grim_status_t s) {
  switch (s) {
    case GRIM_OK: return "ok";
    case GRIM_ERR_INVALID_ARG: return "invalid argument";
    case GRIM_ERR_SHAPE: return "shape mismatch";
    case GRIM_ERR_DTYPE: return "dtype mismatch";
    case GRIM_ERR_NOT_BCR: return "mask is not block-wise column-row structured";
    case GRIM_ERR_ALLOC: return "allocation failed";
    case GRIM_ERR_CUDA: return "CUDA error";
    case GRIM_ERR_UNSUPPORTED: return "unsupported";
    case GRIM_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

extern "C" const char* grim_version(void) { return "grim-b200 0.1 (sm_100a)"; }
