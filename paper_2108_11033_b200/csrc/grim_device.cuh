// Small device helpers shared by the kernels.
#pragma once
#include <cuda_bf16.h>

namespace grim {

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }

// Sums acc[0..BH) over the 32 lanes of a warp with a halving exchange: after the call acc[0] of
// every lane holds the warp total of row warp_row<BH>(lane).  BH in {4, 8, 16}.
template <int BH>
__device__ __forceinline__ void warp_reduce_rows(float (&acc)[BH], int lane) {
  int off = 16;
#pragma unroll
  for (int n = BH; n > 1; n >>= 1, off >>= 1) {
    const bool upper = (lane & off) != 0;
#pragma unroll
    for (int i = 0; i < n / 2; ++i) {
      const float send = upper ? acc[i] : acc[i + n / 2];
      const float keep = upper ? acc[i + n / 2] : acc[i];
      acc[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
    }
  }
#pragma unroll
  for (; off > 0; off >>= 1) acc[0] += __shfl_xor_sync(0xffffffffu, acc[0], off);
}

template <int BH>
__device__ __forceinline__ int warp_row(int lane) {
  int row = 0, off = 16;
#pragma unroll
  for (int n = BH; n > 1; n >>= 1, off >>= 1) row += (lane & off) ? n / 2 : 0;
  return row;
}

}  // namespace grim
