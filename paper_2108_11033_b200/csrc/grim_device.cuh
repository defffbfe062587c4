// Small device helpers shared by the kernels.
#pragma once
#include <cuda_bf16.h>

#include <cstdint>

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

// ---------------------------------------------------------------------------------------------
// Thin wrappers over the PTX used by the kernels: shared-memory barriers (mbarrier), bulk asynchronous
// copies, TMA tile loads, cluster addressing.  Every wait is bounded by the caller through mbar_wait.
// ---------------------------------------------------------------------------------------------
namespace grim {
namespace ptx {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Arrives (release, cluster scope) on the barrier at the same CTA-local address in CTA `rank` of the cluster.
__device__ __forceinline__ void mbar_arrive_remote(uint64_t* bar, uint32_t rank) {
  uint32_t raddr;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(raddr) : "r"(smem_u32(bar)), "r"(rank));
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(raddr) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, unsigned parity) {
  unsigned ok;
  asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
               : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// The same with acquire semantics at cluster scope: for barriers that another CTA of the cluster arrives on.
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t* bar, unsigned parity) {
  unsigned ok;
  asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
               : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Non-blocking test of a phase (acquire, cluster scope): returns at once with the current answer.
__device__ __forceinline__ bool mbar_test_wait_cluster(uint64_t* bar, unsigned parity) {
  unsigned ok;
  asm volatile("{\n.reg .pred p;\nmbarrier.test_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
               : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: polls at most `limit` times with a short sleep between polls (most warps of a block wait at any
// time; polling flat out would take issue slots from the working ones) and gives up early when the block's abort
// flag is set.  Returns false when it gave up.
template <bool CLUSTER = false>
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, unsigned parity, unsigned limit, const volatile int* abort_flag,
                                          unsigned sleep_ns = 100) {
  for (unsigned i = 0; i < limit; ++i) {
    if (CLUSTER ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return true;
    if (sleep_ns) __nanosleep(sleep_ns);
    if ((i & 63u) == 63u && *abort_flag) return false;
  }
  return false;
}
__device__ __forceinline__ void bulk_load(void* dst, const void* src, unsigned bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// x = innermost coordinate (must make x * element size a multiple of 16 bytes), y = row
__device__ __forceinline__ void tma_load_2d(void* dst, const void* tensor_map, int x, int y, uint64_t* bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(smem_u32(dst)), "l"(tensor_map), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void cp_async8(void* dst, const void* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
// The executing thread's earlier cp.async copies arrive on the barrier when they have landed (the barrier's count
// must include this arrival).
__device__ __forceinline__ void cp_async_arrive_noinc(uint64_t* bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void sts128(uint32_t saddr, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(saddr), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}

__device__ __forceinline__ uint4 lds128(uint32_t saddr) {
  uint4 v;
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(saddr));
  return v;
}
__device__ __forceinline__ void sts16(uint32_t saddr, uint32_t low_half) {
  asm volatile("st.shared.u16 [%0], %1;" ::"r"(saddr), "h"((unsigned short)low_half) : "memory");
}
// Barrier among `nthreads` threads (a multiple of 32) that all name the same id (1 .. 15; 0 is __syncthreads).
__device__ __forceinline__ void named_barrier(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// Expands one record of the tensor-core scatter layout (32-bit entries: bf16 value | byte offset in the tile << 16,
// `bytes` of them at shared address rec_s, a multiple of 16; 0 = the tile keeps nothing) into the 16 KiB weight
// tile at shared address a_s.  Called by all NT threads of a group (wt = 0 .. NT - 1) that own barrier `bar_id`:
// the tile is cleared, the group meets, and every entry is stored.
template <int NT>
__device__ __forceinline__ void expand_scatter(uint32_t rec_s, uint32_t bytes, uint32_t a_s, int wt, int bar_id) {
#pragma unroll
  for (int i = 0; i < 16384 / 16 / NT; ++i) sts128(a_s + (uint32_t)(wt + i * NT) * 16u, 0u, 0u, 0u, 0u);
  named_barrier(bar_id, NT);
  const uint32_t n16 = bytes >> 4;
  for (uint32_t v = (uint32_t)wt; v < n16; v += NT) {
    const uint4 e = lds128(rec_s + v * 16u);
    sts16(a_s + (e.x >> 16), e.x);
    sts16(a_s + (e.y >> 16), e.y);
    sts16(a_s + (e.z >> 16), e.z);
    sts16(a_s + (e.w >> 16), e.w);
  }
}

}  // namespace ptx
}  // namespace grim
