// Test hook: fills the shared memory and the tensor memory of every SM with a bit pattern.
//
// The tensor-core kernels stage operands in shared memory and multiply padding (unused K halves, rows and
// channels beyond the real extents) by zeros.  That is only harmless while the padding holds finite values:
// a NaN or an infinity times zero is a NaN.  A kernel that reads shared memory no load of its own wrote sees
// whatever an earlier kernel left there, which is almost always finite, so such a read hides from every
// parity test.  Poisoning all shared memory (and tensor memory) with NaN patterns first makes it show.
#include "kernels.h"
#include "umma_common.cuh"

namespace rt3d {
namespace {

constexpr int kPoisonThreads = 128;
constexpr size_t kPoisonSmem = 226 * 1024;     // one CTA per SM takes (almost) all of its shared memory

__global__ void __launch_bounds__(kPoisonThreads, 1) poison_kernel(uint32_t pattern, int* sink) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ unsigned int tmem_base_s;
  uint32_t* words = reinterpret_cast<uint32_t*>(smem_raw);
  for (uint32_t i = threadIdx.x; i < kPoisonSmem / 4; i += blockDim.x) words[i] = pattern;
  const int warp = threadIdx.x >> 5;
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t taddr = tmem_base_s + (uint32_t(warp * 32) << 16);      // each of the four warps owns 32 lanes
  for (uint32_t c = 0; c < 512; c += 8)
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %1, %1, %1, %1, %1, %1, %1};" ::"r"(taddr + c), "r"(pattern) : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
  tc_fence_before();
  __syncthreads();
  if (words[(threadIdx.x * 977u) % (kPoisonSmem / 4)] != pattern) atomicAdd(sink, 1);   // keeps the stores alive
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base_s), "r"(512u) : "memory");
  }
}

}  // namespace

cudaError_t launch_debug_poison(uint32_t pattern, int sm_count, int* sink, cudaStream_t stream) {
  cudaError_t e = cudaFuncSetAttribute(poison_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kPoisonSmem));
  if (e != cudaSuccess) return e;
  // more CTAs than SMs, each holding a whole SM's shared memory: every SM runs at least one
  poison_kernel<<<2 * sm_count, kPoisonThreads, kPoisonSmem, stream>>>(pattern, sink);
  return cudaGetLastError();
}

}  // namespace rt3d
