// Instruction-rate microbenchmarks behind the kernel choices of this library (stand-alone program).
//
// KGS pruning (Section 3 of the paper) removes whole columns of small g_m x g_n group matrices.  Whether a
// mapping that skips exactly those columns can beat multiplying zero-filled tiles on the tensor cores of an
// sm_100a SM is decided by a handful of rates, measured here on a few KB of data:
//   M1  tcgen05.mma (kind::f16, K = 16) clocks per instruction for M in {64, 128}, N in {8 .. 256}, the A
//       operand read from shared memory or from tensor memory, one or two issuing threads;
//   M1p the same for cta_group::2 (M = 256 over a CTA pair);
//   M2  kind::tf32 (K = 8);
//   M3  sustained mma.sync rates per SM (m16n8k16 / m16n8k8 bf16, m16n8k8 / m16n8k4 tf32), operands in
//       registers, 4 to 16 warps;
//   M3g the inner loop an exact-skip kernel for 8-wide groups would run: A fragments by ldmatrix from
//       shared memory, one B fragment per kept group by a shared-memory load, m16n8k8 MMAs.
// Every wait is bounded; nothing here is linked into librt3d.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <vector>
#include <cuda_runtime.h>

#include "umma_common.cuh"
#include "umma_pair.cuh"

using namespace rt3d;

namespace mb {

constexpr uint32_t kARegion = 64 * 1024;      // four 16 KB A tiles (128 rows x 128 bytes, 128-byte swizzle)
constexpr uint32_t kBRegion = 256 * 128;      // one B tile of up to 256 rows

// kind: 0 = f16 (bf16 operands, K = 16), 1 = tf32 (K = 8)
__device__ __forceinline__ uint32_t idesc_any(int kind, int m, int n) {
  const uint32_t fmt = kind == 0 ? 1u : 2u;
  return (1u << 4) | (fmt << 7) | (fmt << 10) | (uint32_t(n >> 3) << 17) | (uint32_t(m >> 4) << 24);
}

template <int kKind, bool kATmem, int kGroup>
__device__ __forceinline__ void mma_any(uint32_t d, uint64_t adesc, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  if (kGroup == 1) {
    if (kKind == 0) {
      if (kATmem)
        asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}\n"
                     ::"r"(d), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
      else
        asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
                     ::"r"(d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
    } else {
      if (kATmem)
        asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n}\n"
                     ::"r"(d), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
      else
        asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n}\n"
                     ::"r"(d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
    }
  } else {
    if (kATmem)
      asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n}\n"
                   ::"r"(d), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
    else
      asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}\n"
                   ::"r"(d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
  }
}

// ------------------------------------------------------------------------------------------ M1 / M2
// A chain of `count` MMAs into one accumulator per issuing thread.  out[2*i] = clocks until thread i had
// issued its share, out[2*i+1] = clocks until its commit arrived.  The A operand rotates over four tiles
// (shared memory) or four 8-column K slices (tensor memory), B over the four K slices of one tile.
template <int kKind, bool kATmem>
__global__ void __launch_bounds__(512, 1)
tc_chain_kernel(long long* out, int m, int n, int count, int issuers, int32_t* err) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  const uint32_t a_smem = base, b_smem = base + kARegion;
  Barriers* bars = reinterpret_cast<Barriers*>(smem_raw + (base - raw) + kARegion + kBRegion);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (uint32_t i = threadIdx.x; i < (kARegion + kBRegion) / 4; i += blockDim.x)
    reinterpret_cast<uint32_t*>(smem_raw + (base - raw))[i] = 0x3c003c00u;
  if (threadIdx.x == 0) {
    for (int q = 0; q < kMaxStages; ++q) { mbar_init(smem_u32(&bars->full[q]), 1); mbar_init(smem_u32(&bars->empty[q]), 1); }
    bars->abort_flag = 0;
    bars->wait_limit = kWaitCycles;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;
  // the A operand in tensor memory: columns 256.. of this warp's 32 lanes, some finite pattern
  if (warp < 4) {
    const uint32_t taddr = tmem_base + (uint32_t(warp * 32) << 16) + 256u;
    for (int c = 0; c < 32; c += 8)
      asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %1, %1, %1, %1, %1, %1, %1};" ::"r"(taddr + c), "r"(0x3c003c00u) : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (lane == 0 && warp < issuers) {
    const uint32_t idesc = idesc_any(kKind, m, n);
    const uint64_t bdesc = smem_desc_sw128(b_smem);
    const uint32_t d = tmem_base + (uint32_t(warp) * uint32_t(n)) % 256u;   // issuers * N <= 256: disjoint accumulators
    const int mine = count / issuers;
    unsigned long long* mybar = warp < kMaxStages ? &bars->full[warp] : &bars->empty[warp - kMaxStages];
    const long long t0 = clock64();
    for (int i = 0; i < mine; ++i) {
      const uint64_t adesc = smem_desc_sw128(a_smem + uint32_t(i & 3) * 16384u) + 2 * (i & 3);
      mma_any<kKind, kATmem, 1>(d, adesc, tmem_base + 256u + uint32_t(i & 3) * 8u, bdesc + 2 * (i & 3), idesc, i ? 1u : 0u);
    }
    const long long t1 = clock64();
    umma_commit(smem_u32(mybar));
    mbar_wait(smem_u32(mybar), 0, bars, err, 1);
    const long long t2 = clock64();
    out[(blockIdx.x * 16 + warp) * 2] = t1 - t0;
    out[(blockIdx.x * 16 + warp) * 2 + 1] = t2 - t0;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// ------------------------------------------------------------------------------------------ M1p
// `issuers` warps of the leader CTA each issue their share of the chain into their own accumulator columns.
template <bool kATmem>
__global__ void __launch_bounds__(256, 1)
tc_chain_pair_kernel(long long* out, int n, int count, int issuers, int32_t* err) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  const uint32_t a_smem = base, b_smem = base + kARegion;
  Barriers* bars = reinterpret_cast<Barriers*>(smem_raw + (base - raw) + kARegion + kBRegion);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  for (uint32_t i = threadIdx.x; i < (kARegion + kBRegion) / 4; i += blockDim.x)
    reinterpret_cast<uint32_t*>(smem_raw + (base - raw))[i] = 0x3c003c00u;
  if (threadIdx.x == 0) {
    for (int q = 0; q < kMaxStages; ++q) mbar_init(smem_u32(&bars->full[q]), 1);
    bars->abort_flag = 0;
    bars->wait_limit = kWaitCycles;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;
  if (warp < 4) {
    const uint32_t taddr = tmem_base + (uint32_t(warp * 32) << 16) + 256u;
    for (int c = 0; c < 32; c += 8)
      asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %1, %1, %1, %1, %1, %1, %1};" ::"r"(taddr + c), "r"(0x3c003c00u) : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  if (lane == 0 && warp < issuers) {
    if (rank == 0) {
      const uint32_t idesc = instr_desc_bf16_pair(n);
      const uint64_t bdesc = smem_desc_sw128(b_smem);
      const uint32_t d = tmem_base + (uint32_t(warp) * uint32_t(n)) % 256u;
      const int mine = count / issuers;
      const long long t0 = clock64();
      for (int i = 0; i < mine; ++i) {
        const uint64_t adesc = smem_desc_sw128(a_smem + uint32_t(i & 3) * 16384u) + 2 * (i & 3);
        mma_any<0, kATmem, 2>(d, adesc, tmem_base + 256u + uint32_t(i & 3) * 8u, bdesc + 2 * (i & 3), idesc, i ? 1u : 0u);
      }
      const long long t1 = clock64();
      umma_commit_pair(smem_u32(&bars->full[warp]));
      mbar_wait(smem_u32(&bars->full[warp]), 0, bars, err, 2);
      const long long t2 = clock64();
      out[((blockIdx.x >> 1) * 16 + warp) * 2] = t1 - t0;
      out[((blockIdx.x >> 1) * 16 + warp) * 2 + 1] = t2 - t0;
    } else {
      mbar_wait(smem_u32(&bars->full[warp]), 0, bars, err, 3);     // the multicast commit arrives here too
    }
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// ------------------------------------------------------------------------------------------ M6
// tcgen05.cp: one 128-row x 64-channel bf16 tile (128-byte rows, 128-byte swizzle, as TMA writes it) copied
// from shared memory into 32 TMEM columns by four 128x256b copies, then (a) read back with tcgen05.ld and
// compared with the logical tile, (b) used as the A operand of an MMA whose result is compared with the
// same MMA fed from shared memory, (c) timed over a chain of copies.
// out[0] = mismatching words of (a), out[1] = mismatching accumulator words of (b), out[2] = clocks of a
// chain of `tiles` tile copies.
__device__ __forceinline__ void tmem_cp_128x256b(uint32_t taddr, uint64_t sdesc) {
  asm volatile("tcgen05.cp.cta_group::1.128x256b [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
__global__ void __launch_bounds__(128, 1)
tc_cp_kernel(long long* out, int tiles, int32_t* err) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* sm = smem_raw + (base - raw);
  const uint32_t a_smem = base, b_smem = base + kARegion;
  Barriers* bars = reinterpret_cast<Barriers*>(sm + kARegion + kBRegion);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // logical A[r][k] = (r * 7 + k * 3) % 251 - 125, B[n][k] = (n * 5 + k) % 13 - 6: small integers, exact in bf16
  for (int i = threadIdx.x; i < 128 * 64; i += blockDim.x) {
    const int r = i >> 6, k = i & 63;
    const uint32_t off = uint32_t(r) * 128u + ((uint32_t(k >> 3) ^ uint32_t(r & 7)) << 4) + uint32_t(k & 7) * 2u;
    *reinterpret_cast<__nv_bfloat16*>(sm + off) = __float2bfloat16(float((r * 7 + k * 3) % 251 - 125));
    if (r < 64) *reinterpret_cast<__nv_bfloat16*>(sm + kARegion + off) = __float2bfloat16(float((r * 5 + k) % 13 - 6));
  }
  if (threadIdx.x == 0) {
    for (int q = 0; q < 4; ++q) mbar_init(smem_u32(&bars->full[q]), 1);
    bars->abort_flag = 0;
    bars->wait_limit = kWaitCycles;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;
  const uint32_t a_tmem = tmem_base + 256u;
  if (threadIdx.x == 0) {
    for (int kk = 0; kk < 4; ++kk) tmem_cp_128x256b(a_tmem + kk * 8, smem_desc_sw128(a_smem) + 2 * kk);
    umma_commit(smem_u32(&bars->full[0]));
    mbar_wait(smem_u32(&bars->full[0]), 0, bars, err, 4);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // (a) read back: lane r = warp*32 + lane, column c holds (A[r][2c], A[r][2c+1]) as (low, high) halves
  int bad = 0;
  {
    uint32_t v[32];
    tmem_ld32(a_tmem + (uint32_t(warp * 32) << 16), v);
    const int r = warp * 32 + lane;
#pragma unroll
    for (int c = 0; c < 32; ++c) {
      const __nv_bfloat162 e = __floats2bfloat162_rn(float((r * 7 + (2 * c) * 3) % 251 - 125), float((r * 7 + (2 * c + 1) * 3) % 251 - 125));
      bad += (*reinterpret_cast<const uint32_t*>(&e) != v[c]);
    }
  }
  // (b) D0 = A(smem) x B^T, D1 = A(tmem) x B^T, N = 64, K = 64
  if (threadIdx.x == 0) {
    const uint32_t idesc = idesc_any(0, 128, 64);
    for (int kk = 0; kk < 4; ++kk)
      mma_any<0, false, 1>(tmem_base, smem_desc_sw128(a_smem) + 2 * kk, 0u, smem_desc_sw128(b_smem) + 2 * kk, idesc, kk ? 1u : 0u);
    for (int kk = 0; kk < 4; ++kk)
      mma_any<0, true, 1>(tmem_base + 64u, 0ull, a_tmem + kk * 8, smem_desc_sw128(b_smem) + 2 * kk, idesc, kk ? 1u : 0u);
    umma_commit(smem_u32(&bars->full[1]));
    mbar_wait(smem_u32(&bars->full[1]), 0, bars, err, 5);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  int bad2 = 0, nonzero = 0;
  {
    uint32_t d0[32], d1[32];
    for (int h = 0; h < 2; ++h) {
      tmem_ld32(tmem_base + (uint32_t(warp * 32) << 16) + h * 32, d0);
      tmem_ld32(tmem_base + (uint32_t(warp * 32) << 16) + 64 + h * 32, d1);
      const int r = warp * 32 + lane;
#pragma unroll
      for (int c = 0; c < 32; ++c) {
        bad2 += d0[c] != d1[c];
        // and against the definition: sum_k A[r][k] * B[n][k], exact in fp32
        float ref = 0.f;
        const int nn = h * 32 + c;
        for (int k = 0; k < 64; ++k) ref += float((r * 7 + k * 3) % 251 - 125) * float((nn * 5 + k) % 13 - 6);
        bad2 += __float_as_uint(ref) != d0[c] && !(ref == 0.f && __uint_as_float(d0[c]) == 0.f);
        nonzero += d0[c] != 0u;
      }
    }
  }
  bad = __reduce_add_sync(0xffffffffu, bad);
  bad2 = __reduce_add_sync(0xffffffffu, bad2);
  nonzero = __reduce_add_sync(0xffffffffu, nonzero);
  if (lane == 0) { atomicAdd(reinterpret_cast<unsigned long long*>(out), (unsigned long long)bad);
                   atomicAdd(reinterpret_cast<unsigned long long*>(out + 1), (unsigned long long)bad2);
                   atomicAdd(reinterpret_cast<unsigned long long*>(out + 3), (unsigned long long)nonzero); }
  // (c) throughput of tile copies
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (threadIdx.x == 0) {
    const long long t0 = clock64();
    for (int t = 0; t < tiles; ++t)
      for (int kk = 0; kk < 4; ++kk)
        tmem_cp_128x256b(a_tmem + uint32_t(t & 3) * 32u + kk * 8, smem_desc_sw128(a_smem + uint32_t(t & 3) * 16384u) + 2 * kk);
    umma_commit(smem_u32(&bars->full[2]));
    mbar_wait(smem_u32(&bars->full[2]), 0, bars, err, 6);
    out[2] = clock64() - t0;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// ------------------------------------------------------------------------------------------ M7
// Shared-memory bandwidth shared between its users.  Up to three streams run at once in one CTA:
//   mma_warps (0..8) warps each issuing a chain of N = 16 MMAs with A in tensor memory (each reads a 512-byte
//             B block from shared memory),
//   cp_warps  (0..4) warps each issuing tcgen05.cp tile copies (16 KB read from shared memory per tile),
//   bulk      one warp streaming 16 KB bulk copies global (L2-resident) -> shared memory, four in flight.
// out[0] = clocks until the MMA chains are done, out[1] = clocks until the copies to tensor memory are done,
// out[2] = clocks until the bulk copies are done (each stream runs a fixed amount of work).
__global__ void __launch_bounds__(448, 1)
smem_share_kernel(long long* out, int mma_warps, int mma_count, int cp_warps, int cp_tiles, int bulk_chunks,
                  const unsigned char* gsrc, int32_t* err) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  const uint32_t a_smem = base, b_smem = base + kARegion, bulk_smem = base + kARegion + kBRegion;   // + 64 KB bulk landing area
  Barriers* bars = reinterpret_cast<Barriers*>(smem_raw + (base - raw) + kARegion + kBRegion + 64 * 1024);
  unsigned long long* bar2 = reinterpret_cast<unsigned long long*>(bars + 1);   // 16 more barriers
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (uint32_t i = threadIdx.x; i < (kARegion + kBRegion) / 4; i += blockDim.x)
    reinterpret_cast<uint32_t*>(smem_raw + (base - raw))[i] = 0x3c003c00u;
  if (threadIdx.x == 0) {
    for (int q = 0; q < kMaxStages; ++q) { mbar_init(smem_u32(&bars->full[q]), 1); mbar_init(smem_u32(&bars->empty[q]), 1); }
    for (int q = 0; q < 16; ++q) mbar_init(smem_u32(&bar2[q]), 1);
    bars->abort_flag = 0;
    bars->wait_limit = kWaitCycles;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;
  if (warp < 4) {
    const uint32_t taddr = tmem_base + (uint32_t(warp * 32) << 16) + 256u;
    for (int c = 0; c < 32; c += 8)
      asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %1, %1, %1, %1, %1, %1, %1};" ::"r"(taddr + c), "r"(0x3c003c00u) : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const long long t0 = clock64();
  if (lane == 0 && warp < mma_warps) {
    const uint32_t idesc = idesc_any(0, 128, 16);
    const uint32_t d = tmem_base + uint32_t(warp) * 16u;
    for (int i = 0; i < mma_count; ++i) {
      // a different 512-byte block of B every time: rows (i % 16) * 16 .. + 16, K slice i & 3
      const uint64_t bdesc = smem_desc_sw128(b_smem + uint32_t((i + warp) & 15) * 2048u) + 2 * (i & 3);
      mma_any<0, true, 1>(d, 0ull, tmem_base + 256u + uint32_t(i & 3) * 8u, bdesc, idesc, i ? 1u : 0u);
    }
    umma_commit(smem_u32(&bars->full[warp]));
    mbar_wait(smem_u32(&bars->full[warp]), 0, bars, err, 7);
    atomicMax(reinterpret_cast<unsigned long long*>(out), (unsigned long long)(clock64() - t0));
  }
  if (lane == 0 && warp >= 8 && warp < 8 + cp_warps) {
    const int w = warp - 8;
    for (int t = 0; t < cp_tiles; ++t)
      for (int kk = 0; kk < 4; ++kk)
        tmem_cp_128x256b(tmem_base + 288u + uint32_t(w) * 32u + kk * 8, smem_desc_sw128(a_smem + uint32_t((t + w) & 3) * 16384u) + 2 * kk);
    umma_commit(smem_u32(&bars->empty[w]));
    mbar_wait(smem_u32(&bars->empty[w]), 0, bars, err, 8);
    atomicMax(reinterpret_cast<unsigned long long*>(out + 1), (unsigned long long)(clock64() - t0));
  }
  if (lane == 0 && warp == 12 && bulk_chunks > 0) {
    // four 16 KB landing buffers, one barrier each; chunk c uses buffer c & 3
    uint32_t ph[4] = {0, 0, 0, 0};
    for (int c = 0; c < bulk_chunks + 4; ++c) {
      const int b = c & 3;
      if (c >= 4) { if (!mbar_wait(smem_u32(&bar2[b]), ph[b], bars, err, 9)) break; ph[b] ^= 1u; }
      if (c < bulk_chunks) {
        mbar_expect_tx(smem_u32(&bar2[b]), 16384u);
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(bulk_smem + uint32_t(b) * 16384u), "l"(gsrc + size_t(c & 63) * 16384), "r"(16384u), "r"(smem_u32(&bar2[b])) : "memory");
      }
    }
    atomicMax(reinterpret_cast<unsigned long long*>(out + 2), (unsigned long long)(clock64() - t0));
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// ------------------------------------------------------------------------------------------ M8
// Tensor-memory traffic next to the MMAs.  Eight warps issue chains of N = 16 MMAs with A in tensor memory;
// B is a 512-byte block in the 128-byte-swizzle layout (b_noswizzle = 0) or in the no-swizzle core-matrix
// layout (1).  Meanwhile `st_warps` (0 or 4) further warps each write 32 lanes x 32 columns (4 KB) per
// iteration with tcgen05.st + wait::st, as a kernel that stages its A operand through registers would, and
// `ld_warps` (0 or 4) read 32 x 32 columns per iteration with tcgen05.ld (an epilogue).
// out[0] = clocks of the MMA chains, out[1] = clocks of the store loops, out[2] = clocks of the load loops.
__global__ void __launch_bounds__(512, 1)
tmem_share_kernel(long long* out, int mma_count, int b_noswizzle, int st_warps, int st_iters, int ld_warps, int ld_iters,
                  float* sink, int32_t* err) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  const uint32_t b_smem = base + kARegion;
  Barriers* bars = reinterpret_cast<Barriers*>(smem_raw + (base - raw) + kARegion + kBRegion);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (uint32_t i = threadIdx.x; i < (kARegion + kBRegion) / 4; i += blockDim.x)
    reinterpret_cast<uint32_t*>(smem_raw + (base - raw))[i] = 0x3c003c00u;
  if (threadIdx.x == 0) {
    for (int q = 0; q < kMaxStages; ++q) mbar_init(smem_u32(&bars->full[q]), 1);
    bars->abort_flag = 0;
    bars->wait_limit = kWaitCycles;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;
  if (warp < 4) {
    const uint32_t taddr = tmem_base + (uint32_t(warp * 32) << 16) + 256u;
    for (int c = 0; c < 32; c += 8)
      asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %1, %1, %1, %1, %1, %1, %1};" ::"r"(taddr + c), "r"(0x3c003c00u) : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const long long t0 = clock64();
  if (warp < 8) {
    if (lane == 0) {
      const uint32_t idesc = idesc_any(0, 128, 16);
      const uint32_t d = tmem_base + uint32_t(warp) * 16u;
      for (int i = 0; i < mma_count; ++i) {
        const uint32_t blk = b_smem + uint32_t((i + warp) & 15) * 2048u;
        const uint64_t bdesc = b_noswizzle ? smem_desc_noswizzle(blk + uint32_t(i & 3) * 512u, 128u, 256u) : smem_desc_sw128(blk) + 2 * (i & 3);
        mma_any<0, true, 1>(d, 0ull, tmem_base + 256u + uint32_t(i & 3) * 8u, bdesc, idesc, i ? 1u : 0u);
      }
      umma_commit(smem_u32(&bars->full[warp]));
      mbar_wait(smem_u32(&bars->full[warp]), 0, bars, err, 10);
      atomicMax(reinterpret_cast<unsigned long long*>(out), (unsigned long long)(clock64() - t0));
    }
  } else if (warp < 8 + st_warps) {
    // columns 320..447 (four 32-column stages), never read by the MMAs
    uint32_t v[32];
#pragma unroll
    for (int q = 0; q < 32; ++q) v[q] = 0x3c003c00u + q + lane;
    const uint32_t lanes = uint32_t((warp & 3) * 32) << 16;
    for (int it = 0; it < st_iters; ++it) {
      const uint32_t taddr = tmem_base + lanes + 320u + uint32_t(it & 3) * 32u;
      asm volatile(
          "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
          "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
          ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]),
            "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]),
            "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]),
            "r"(v[30]), "r"(v[31]) : "memory");
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      v[it & 31] += 1u;
    }
    if (lane == 0) atomicMax(reinterpret_cast<unsigned long long*>(out + 1), (unsigned long long)(clock64() - t0));
  } else if (warp < 12 + ld_warps) {
    float acc = 0.f;
    const uint32_t lanes = uint32_t((warp & 3) * 32) << 16;
    for (int it = 0; it < ld_iters; ++it) {
      uint32_t v[32];
      tmem_ld32(tmem_base + lanes + 128u + uint32_t(it & 3) * 32u, v);
#pragma unroll
      for (int q = 0; q < 32; ++q) acc += __uint_as_float(v[q]);
    }
    if (acc == 123.456f) sink[threadIdx.x] = acc;
    if (lane == 0) atomicMax(reinterpret_cast<unsigned long long*>(out + 2), (unsigned long long)(clock64() - t0));
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// ------------------------------------------------------------------------------------------ M9
// The issue loop of a kernel that works in K steps: eight warps, per step each warp (optionally) executes
// tcgen05.fence::after_thread_sync, issues `per_step` N = 16 MMAs (A in tensor memory, stage step % 8 of an
// eight-stage ring) and (optionally) commits to the step's barrier (count 8); with `ring` the warp first waits
// until the barrier of the step eight earlier has completed.  out[0] = clocks for all steps.
__global__ void __launch_bounds__(256, 1)
stepped_issue_kernel(long long* out, int steps, int per_step, int use_fence, int use_commit, int ring, int a_stages, int d_stride, int n, int32_t* err) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  const uint32_t b_smem = base + kARegion;
  Barriers* bars = reinterpret_cast<Barriers*>(smem_raw + (base - raw) + kARegion + kBRegion);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (uint32_t i = threadIdx.x; i < (kARegion + kBRegion) / 4; i += blockDim.x)
    reinterpret_cast<uint32_t*>(smem_raw + (base - raw))[i] = 0x3c003c00u;
  if (threadIdx.x == 0) {
    for (int q = 0; q < kMaxStages; ++q) { mbar_init(smem_u32(&bars->full[q]), 8); mbar_init(smem_u32(&bars->empty[q]), 1); }
    bars->abort_flag = 0;
    bars->wait_limit = kWaitCycles;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;
  if (warp < 4) {
    for (int c = 0; c < 256; c += 8)
      asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %1, %1, %1, %1, %1, %1, %1};"
                   ::"r"(tmem_base + (uint32_t(warp * 32) << 16) + 256u + c), "r"(0x3c003c00u) : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (lane == 0) {
    const uint32_t idesc = idesc_any(0, 128, n);
    const uint32_t d = tmem_base + uint32_t(warp) * uint32_t(d_stride);
    const long long t0 = clock64();
    for (int st = 0; st < steps; ++st) {
      const int stage = st & 7;
      const int a_stage = st % a_stages;
      if (ring && st >= 8 && !mbar_wait(smem_u32(&bars->full[stage]), uint32_t((st >> 3) - 1) & 1u, bars, err, 11)) break;
      if (use_fence) tc_fence_after();
      for (int i = 0; i < per_step; ++i) {
        const uint64_t bdesc = smem_desc_noswizzle(b_smem + uint32_t((st + warp) & 15) * 2048u + uint32_t(i & 3) * 512u, 128u, 256u);
        mma_any<0, true, 1>(d, 0ull, tmem_base + 256u + uint32_t(a_stage) * 32u + uint32_t(i & 3) * 8u, bdesc, idesc, (st | i) ? 1u : 0u);
      }
      if (use_commit) umma_commit(smem_u32(&bars->full[stage]));
    }
    if (warp == 0) {
      umma_commit(smem_u32(&bars->empty[0]));
      mbar_wait(smem_u32(&bars->empty[0]), 0, bars, err, 12);
    }
    atomicMax(reinterpret_cast<unsigned long long*>(out), (unsigned long long)(clock64() - t0));
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// ------------------------------------------------------------------------------------------ M10
// Several lanes of one warp issuing: lanes 0..L-1 of each of W warps each run their own chain of N = 16 MMAs
// (A in tensor memory) into their own 16 accumulator columns.  out[0] = clocks until all chains are done.
__global__ void __launch_bounds__(512, 1)
lane_issue_kernel(long long* out, int count, int warps, int lanes, int a_slices, int32_t* err) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  const uint32_t b_smem = base + kARegion;
  Barriers* bars = reinterpret_cast<Barriers*>(smem_raw + (base - raw) + kARegion + kBRegion);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (uint32_t i = threadIdx.x; i < (kARegion + kBRegion) / 4; i += blockDim.x)
    reinterpret_cast<uint32_t*>(smem_raw + (base - raw))[i] = 0x3c003c00u;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bars->full[0]), uint32_t(warps * lanes));
    bars->abort_flag = 0;
    bars->wait_limit = kWaitCycles;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;
  if (warp < 4) {
    for (int c = 0; c < 256; c += 8)
      asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %1, %1, %1, %1, %1, %1, %1};"
                   ::"r"(tmem_base + (uint32_t(warp * 32) << 16) + 256u + c), "r"(0x3c003c00u) : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp < warps && lane < lanes) {
    const uint32_t idesc = idesc_any(0, 128, 16);
    const uint32_t d = tmem_base + uint32_t(warp * lanes + lane) * 16u;
    const uint64_t bdesc = smem_desc_noswizzle(b_smem + uint32_t(warp * lanes + lane) * 2048u, 128u, 256u);
    const long long t0 = clock64();
    for (int i = 0; i < count; ++i)
      mma_any<0, true, 1>(d, 0ull, tmem_base + 256u + uint32_t(i & (a_slices - 1)) * 8u, bdesc + uint64_t(i & 3) * 32u, idesc, i ? 1u : 0u);
    umma_commit(smem_u32(&bars->full[0]));
    mbar_wait(smem_u32(&bars->full[0]), 0, bars, err, 13);
    atomicMax(reinterpret_cast<unsigned long long*>(out), (unsigned long long)(clock64() - t0));
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// ------------------------------------------------------------------------------------------ M11
// Two issuing warps with DIFFERENT instruction shapes at once: warp 0 a chain of N = n0 MMAs with A in shared
// memory (a spatial convolution's steps), warp 1 a chain of N = n1 MMAs with A in tensor memory (a temporal
// convolution fed from the intermediate frame).  out[0] / out[1] = clocks until each chain is done.
__global__ void __launch_bounds__(128, 1)
mixed_issue_kernel(long long* out, int n0, int count0, int n1, int count1, int32_t* err) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  const uint32_t a_smem = base, b_smem = base + kARegion;
  Barriers* bars = reinterpret_cast<Barriers*>(smem_raw + (base - raw) + kARegion + kBRegion);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (uint32_t i = threadIdx.x; i < (kARegion + kBRegion) / 4; i += blockDim.x)
    reinterpret_cast<uint32_t*>(smem_raw + (base - raw))[i] = 0x3c003c00u;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bars->full[0]), 1);
    mbar_init(smem_u32(&bars->full[1]), 1);
    bars->abort_flag = 0;
    bars->wait_limit = kWaitCycles;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;
  {
    const uint32_t taddr = tmem_base + (uint32_t(warp * 32) << 16) + 448u;
    for (int c = 0; c < 32; c += 8)
      asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %1, %1, %1, %1, %1, %1, %1};" ::"r"(taddr + c), "r"(0x3c003c00u) : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (lane == 0 && warp < 2) {
    const int n = warp == 0 ? n0 : n1, count = warp == 0 ? count0 : count1;
    const uint32_t idesc = idesc_any(0, 128, n);
    const uint64_t bdesc = smem_desc_sw128(b_smem);
    const uint32_t d = tmem_base + uint32_t(warp) * 256u;          // accumulators at columns 0.. and 256..
    const long long t0 = clock64();
    for (int i = 0; i < count; ++i) {
      const uint64_t adesc = smem_desc_sw128(a_smem + uint32_t(i & 3) * 16384u) + 2 * (i & 3);
      if (warp == 0) mma_any<0, false, 1>(d, adesc, 0u, bdesc + 2 * (i & 3), idesc, i ? 1u : 0u);
      else mma_any<0, true, 1>(d, 0ull, tmem_base + 448u + uint32_t(i & 3) * 8u, bdesc + 2 * (i & 3), idesc, i ? 1u : 0u);
    }
    if (count > 0) {
      umma_commit(smem_u32(&bars->full[warp]));
      mbar_wait(smem_u32(&bars->full[warp]), 0, bars, err, 14);
    }
    out[warp] = clock64() - t0;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// ------------------------------------------------------------------------------------------ M12
// The A operand of the small-C_in kernel: no-swizzle core matrices (8 voxels x 16 bytes) that are windows of a
// staged image whose rows are `sbo` bytes apart, the two K halves of an MMA `lbo` bytes apart (two kernel
// locations), successive MMAs shifted by `shift` bytes (the next kernel column).  M = 128, N = 64, K = 16; B is
// the kernel's weight image (no swizzle, K halves 1 KB apart).  Same timing scheme as M1.
__global__ void __launch_bounds__(128, 1)
ns_window_kernel(long long* out, int count, int issuers, uint32_t sbo, uint32_t lbo, uint32_t shift, int32_t* err) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  const uint32_t a_smem = base, b_smem = base + kARegion;
  Barriers* bars = reinterpret_cast<Barriers*>(smem_raw + (base - raw) + kARegion + kBRegion);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (uint32_t i = threadIdx.x; i < (kARegion + kBRegion) / 4; i += blockDim.x)
    reinterpret_cast<uint32_t*>(smem_raw + (base - raw))[i] = 0x3c003c00u;
  if (threadIdx.x == 0) {
    for (int q = 0; q < kMaxStages; ++q) { mbar_init(smem_u32(&bars->full[q]), 1); mbar_init(smem_u32(&bars->empty[q]), 1); }
    bars->abort_flag = 0;
    bars->wait_limit = kWaitCycles;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)), "r"(256u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;
  if (lane == 0 && warp < issuers) {
    const uint32_t idesc = idesc_any(0, 128, 64);
    const uint32_t d = tmem_base + uint32_t(warp) * 64u;
    const int mine = count / issuers;
    const long long t0 = clock64();
    for (int i = 0; i < mine; ++i) {
      const uint64_t adesc = smem_desc_noswizzle(a_smem + uint32_t(warp) * 8192u + uint32_t(i & 3) * shift, lbo, sbo);
      const uint64_t bdesc = smem_desc_noswizzle(b_smem + uint32_t(i & 3) * 2048u, 1024u, 128u);
      mma_any<0, false, 1>(d, adesc, 0u, bdesc, idesc, i ? 1u : 0u);
    }
    const long long t1 = clock64();
    umma_commit(smem_u32(&bars->full[warp]));
    mbar_wait(smem_u32(&bars->full[warp]), 0, bars, err, 12);
    const long long t2 = clock64();
    out[warp * 2] = t1 - t0;
    out[warp * 2 + 1] = t2 - t0;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(256u) : "memory");
  }
}

// ------------------------------------------------------------------------------------------ M3
// kShape: 0 m16n8k16 bf16, 1 m16n8k8 bf16, 2 m16n8k8 tf32, 3 m16n8k4 tf32.  Eight independent accumulator
// tiles per warp, operands in registers.
template <int kShape>
__device__ __forceinline__ void mma_sync_one(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  if (kShape == 0)
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
  else if (kShape == 1)
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(b[0]));
  else if (kShape == 2)
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
  else
    asm volatile("mma.sync.aligned.m16n8k4.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(b[0]));
}

template <int kShape>
__global__ void mma_sync_rate_kernel(long long* out, float* sink, int iters) {
  float c[8][4];
#pragma unroll
  for (int u = 0; u < 8; ++u)
#pragma unroll
    for (int q = 0; q < 4; ++q) c[u][q] = 0.f;
  uint32_t a[4], b[2];
#pragma unroll
  for (int q = 0; q < 4; ++q) a[q] = 0x3c003c00u + (threadIdx.x & 3u) * 0x10000u + q;
  b[0] = 0x3c003c00u; b[1] = 0x3c013c00u;
  __syncthreads();
  const long long t0 = clock64();
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int u = 0; u < 8; ++u) mma_sync_one<kShape>(c[u], a, b);
  }
  __syncthreads();
  const long long t1 = clock64();
  float s = 0.f;
#pragma unroll
  for (int u = 0; u < 8; ++u) s += c[u][0] + c[u][1] + c[u][2] + c[u][3];
  if (s == 123.456f) sink[threadIdx.x] = s;
  if (threadIdx.x == 0) out[blockIdx.x] = t1 - t0;
}

// ------------------------------------------------------------------------------------------ M3g
// Inner loop of an exact-skip mapping for 8-channel-wide groups: the warp owns kVT voxels; per kept column
// (one kernel location x 8 input channels) it fetches the voxels' A fragments with ldmatrix (kVT/32 x4
// loads, rows of 16 bytes) and, for each of kKpc group rows that keep the column, one B fragment (8 x 8
// weights, one 32-bit shared-memory load per lane) followed by kVT/16 m16n8k8 MMAs.
template <int kVT, int kKpc>
__global__ void mma_sync_gather_kernel(long long* out, float* sink, int iters) {
  extern __shared__ unsigned char smem_raw[];
  constexpr int MT = kVT / 16;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (uint32_t i = threadIdx.x; i < 48 * 1024 / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem_raw)[i] = 0x3c003c00u;
  __syncthreads();
  const uint32_t sbase = smem_u32(smem_raw);
  float c[kKpc][MT][4];
#pragma unroll
  for (int r = 0; r < kKpc; ++r)
#pragma unroll
    for (int t = 0; t < MT; ++t)
#pragma unroll
      for (int q = 0; q < 4; ++q) c[r][t][q] = 0.f;
  // input slab of this warp: 32 KB region walked in steps of kVT rows x 16 bytes; weights: 16 KB region
  const uint32_t a_lane = sbase + uint32_t(lane) * 16u;
  const uint32_t b_lane = sbase + 32 * 1024 + uint32_t(lane) * 4u;
  __syncthreads();
  const long long t0 = clock64();
  uint32_t col = uint32_t(warp) * 7u;
  for (int it = 0; it < iters; ++it) {
    uint32_t af[MT][2];
#pragma unroll
    for (int h = 0; h < kVT / 32; ++h) {
      const uint32_t addr = a_lane + ((col * (kVT * 16u) + h * 512u) & (32 * 1024 - 1));
      asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                   : "=r"(af[2 * h][0]), "=r"(af[2 * h][1]), "=r"(af[2 * h + 1][0]), "=r"(af[2 * h + 1][1]) : "r"(addr));
    }
#pragma unroll
    for (int r = 0; r < kKpc; ++r) {
      uint32_t bf;
      asm volatile("ld.shared.b32 %0, [%1];" : "=r"(bf) : "r"(b_lane + (((col * kKpc + r) * 128u) & (16 * 1024 - 1))));
#pragma unroll
      for (int t = 0; t < MT; ++t)
        asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
                     : "+f"(c[r][t][0]), "+f"(c[r][t][1]), "+f"(c[r][t][2]), "+f"(c[r][t][3]) : "r"(af[t][0]), "r"(af[t][1]), "r"(bf));
    }
    col += 3u;
  }
  __syncthreads();
  const long long t1 = clock64();
  float s = 0.f;
#pragma unroll
  for (int r = 0; r < kKpc; ++r)
#pragma unroll
    for (int t = 0; t < MT; ++t) s += c[r][t][0] + c[r][t][1] + c[r][t][2] + c[r][t][3];
  if (s == 123.456f) sink[threadIdx.x] = s;
  if (threadIdx.x == 0) out[blockIdx.x] = t1 - t0;
}

// ------------------------------------------------------------------------------------------ host side
long long* d_out = nullptr;
float* d_sink = nullptr;
int32_t* d_err = nullptr;
int g_sms = 0;
double g_ghz = 0.0;

bool sync_ok(const char* what) {
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) { printf("CUDA error after %s: %s\n", what, cudaGetErrorString(e)); return false; }
  int32_t err = 0;
  cudaMemcpy(&err, d_err, 4, cudaMemcpyDeviceToHost);
  if (err) { printf("bounded wait gave up in %s (code %d)\n", what, err); return false; }
  return true;
}

template <int kKind, bool kATmem>
bool run_tc(int m, int n, int count, int issuers, int grid, double* issue, double* done) {
  const size_t smem = 1024 + kARegion + kBRegion + sizeof(Barriers) + 64;
  cudaFuncSetAttribute(tc_chain_kernel<kKind, kATmem>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
  for (int rep = 0; rep < 2; ++rep) {
    tc_chain_kernel<kKind, kATmem><<<grid, issuers <= 4 ? 128 : issuers * 32, smem>>>(d_out, m, n, count, issuers, d_err);
    if (!sync_ok("tc_chain")) return false;
  }
  std::vector<long long> h(size_t(grid) * 32);
  cudaMemcpy(h.data(), d_out, h.size() * 8, cudaMemcpyDeviceToHost);
  long long mi = 0, md = 0;
  for (int b = 0; b < grid; ++b)
    for (int w = 0; w < issuers; ++w) {
      mi = h[(b * 16 + w) * 2] > mi ? h[(b * 16 + w) * 2] : mi;
      md = h[(b * 16 + w) * 2 + 1] > md ? h[(b * 16 + w) * 2 + 1] : md;
    }
  *issue = double(mi) / count; *done = double(md) / count;
  return true;
}

template <bool kATmem>
bool run_pair(int n, int count, int issuers, int grid, double* issue, double* done) {
  const size_t smem = 1024 + kARegion + kBRegion + sizeof(Barriers) + 64;
  cudaFuncSetAttribute(tc_chain_pair_kernel<kATmem>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.gridDim = dim3(grid); cfg.blockDim = dim3(issuers <= 4 ? 128 : issuers * 32); cfg.dynamicSmemBytes = smem; cfg.attrs = attr; cfg.numAttrs = 1;
  for (int rep = 0; rep < 2; ++rep) {
    if (cudaLaunchKernelEx(&cfg, tc_chain_pair_kernel<kATmem>, d_out, n, count, issuers, d_err) != cudaSuccess) { printf("launch failed\n"); return false; }
    if (!sync_ok("tc_chain_pair")) return false;
  }
  std::vector<long long> h(size_t(grid) * 16);
  cudaMemcpy(h.data(), d_out, h.size() * 8, cudaMemcpyDeviceToHost);
  long long mi = 0, md = 0;
  for (int b = 0; b < grid / 2; ++b)
    for (int w = 0; w < issuers; ++w) {
      mi = h[(b * 16 + w) * 2] > mi ? h[(b * 16 + w) * 2] : mi;
      md = h[(b * 16 + w) * 2 + 1] > md ? h[(b * 16 + w) * 2 + 1] : md;
    }
  *issue = double(mi) / count; *done = double(md) / count;
  return true;
}

template <int kShape>
bool run_sync(int warps, int grid, int iters, double* mac_per_clk_sm) {
  for (int rep = 0; rep < 2; ++rep) {
    mma_sync_rate_kernel<kShape><<<grid, warps * 32>>>(d_out, d_sink, iters);
    if (!sync_ok("mma_sync_rate")) return false;
  }
  std::vector<long long> h(static_cast<size_t>(grid));
  cudaMemcpy(h.data(), d_out, h.size() * 8, cudaMemcpyDeviceToHost);
  long long mx = 0;
  for (long long v : h) mx = v > mx ? v : mx;
  const int k = kShape == 0 ? 16 : (kShape == 3 ? 4 : 8);
  *mac_per_clk_sm = double(warps) * iters * 8.0 * (16.0 * 8.0 * k) / double(mx);
  return true;
}

template <int kVT, int kKpc>
bool run_gather(int warps, int grid, int iters, double* mac_per_clk_sm, double* smem_b_per_clk) {
  cudaFuncSetAttribute(mma_sync_gather_kernel<kVT, kKpc>, cudaFuncAttributeMaxDynamicSharedMemorySize, 48 * 1024);
  for (int rep = 0; rep < 2; ++rep) {
    mma_sync_gather_kernel<kVT, kKpc><<<grid, warps * 32, 48 * 1024>>>(d_out, d_sink, iters);
    if (!sync_ok("mma_sync_gather")) return false;
  }
  std::vector<long long> h(static_cast<size_t>(grid));
  cudaMemcpy(h.data(), d_out, h.size() * 8, cudaMemcpyDeviceToHost);
  long long mx = 0;
  for (long long v : h) mx = v > mx ? v : mx;
  *mac_per_clk_sm = double(warps) * iters * kKpc * (kVT / 16) * 1024.0 / double(mx);
  *smem_b_per_clk = double(warps) * iters * (kVT * 16.0 + kKpc * 128.0) / double(mx);
  return true;
}

double tflops(double mac_per_clk_sm) { return mac_per_clk_sm * 2.0 * g_sms * g_ghz / 1000.0; }

}  // namespace mb

using namespace mb;

int main(int argc, char** argv) {
  const bool quick = argc > 1 && !strcmp(argv[1], "--quick");
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, 0) != cudaSuccess) { printf("no CUDA device\n"); return 1; }
  if (prop.major != 10) { printf("needs an sm_100 device (found %d.%d)\n", prop.major, prop.minor); return 1; }
  g_sms = prop.multiProcessorCount;
  int khz = 0;
  cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, 0);
  g_ghz = khz / 1e6;
  cudaMalloc(&d_out, 8 * 16 * 1024); cudaMalloc(&d_sink, 4 * 1024); cudaMalloc(&d_err, 4);
  cudaMemset(d_err, 0, 4);
  printf("# MMA microbenchmarks on %s (%d SMs, max SM clock %.3f GHz)\n\n", prop.name, g_sms, g_ghz);
  printf("Clocks are SM clocks (clock64) per instruction over a chain of `count` instructions; `done` includes the\n");
  printf("drain of the chain (commit -> mbarrier), `issue` is the issuing thread alone.  `tensor` = 128*N*K / 4096\n");
  printf("MAC/clk (the dense bf16 rate of one SM; an M = 64 instruction holds the pipe as long as M = 128); `smem` = operand bytes read from shared memory\n");
  printf("per instruction / 128 B/clk.\n\n");

  const int count = 256;
  const int ns[] = {8, 16, 32, 64, 128, 256};
  printf("## M1: tcgen05.mma cta_group::1 kind::f16 (bf16, K = 16), one CTA on one SM\n\n");
  printf("| M | N | A from | issuers | issue clk/MMA | done clk/MMA | tensor clk | smem clk | MAC/clk/SM |\n|---|---|---|---|---|---|---|---|---|\n");
  for (int m : {128, 64})
    for (int a_tmem = 0; a_tmem < 2; ++a_tmem)
      for (int n : ns) {
        if (m == 128 && n < 16) continue;
        for (int issuers = 1; issuers <= 16; issuers *= 2) {
          if (issuers * n > 256) continue;
          if (quick && issuers > 1) continue;
          double is = 0, dn = 0;
          const bool ok = a_tmem ? run_tc<0, true>(m, n, count, issuers, 1, &is, &dn) : run_tc<0, false>(m, n, count, issuers, 1, &is, &dn);
          if (!ok) return 1;
          const double tensor = 128.0 * n * 16 / 4096.0;
          const double smem = ((a_tmem ? 0.0 : m * 32.0) + n * 32.0) / 128.0;
          printf("| %d | %d | %s | %d | %.1f | %.1f | %.1f | %.1f | %.0f |\n", m, n, a_tmem ? "TMEM" : "smem", issuers, is, dn,
                 tensor, smem, double(m) * n * 16 / dn);
        }
      }
  printf("\n");

  printf("## M1 on all SMs at once (one CTA per SM; the slowest SM counts)\n\n");
  printf("| M | N | A from | done clk/MMA | MAC/clk/SM | TFLOP/s at max clock |\n|---|---|---|---|---|---|\n");
  for (int n : {16, 64, 256}) {
    double is = 0, dn = 0;
    if (!run_tc<0, false>(128, n, count, 1, g_sms, &is, &dn)) return 1;
    printf("| 128 | %d | smem | %.1f | %.0f | %.0f |\n", n, dn, 128.0 * n * 16 / dn, tflops(128.0 * n * 16 / dn));
    if (!run_tc<0, true>(128, n, count, 1, g_sms, &is, &dn)) return 1;
    printf("| 128 | %d | TMEM | %.1f | %.0f | %.0f |\n", n, dn, 128.0 * n * 16 / dn, tflops(128.0 * n * 16 / dn));
  }

  printf("\n## M1p: tcgen05.mma cta_group::2 kind::f16 (M = 256 over a CTA pair, K = 16), one pair\n\n");
  printf("| N | A from | issuers | issue clk/MMA | done clk/MMA | tensor clk | smem clk per CTA | MAC/clk/SM |\n|---|---|---|---|---|---|---|---|\n");
  for (int a_tmem = 0; a_tmem < 2; ++a_tmem)
    for (int n : {16, 32, 64, 128, 256})
      for (int issuers = 1; issuers <= 8; issuers *= 2) {
        if (issuers * n > 256) continue;
        double is = 0, dn = 0;
        const bool ok = a_tmem ? run_pair<true>(n, count, issuers, 2, &is, &dn) : run_pair<false>(n, count, issuers, 2, &is, &dn);
        if (!ok) return 1;
        printf("| %d | %s | %d | %.1f | %.1f | %.1f | %.1f | %.0f |\n", n, a_tmem ? "TMEM" : "smem", issuers, is, dn, 128.0 * n * 16 / 4096.0,
               ((a_tmem ? 0.0 : 128 * 32.0) + n / 2 * 32.0) / 128.0, 128.0 * n * 16 / dn);
      }

  printf("\n## M6: tcgen05.cp 128x256b, shared memory (128-byte swizzle) -> tensor memory\n\n");
  {
    const size_t smem = 1024 + kARegion + kBRegion + sizeof(Barriers) + 64;
    cudaFuncSetAttribute(tc_cp_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    const int tiles = 64;
    long long h[4] = {0, 0, 0, 0};
    for (int rep = 0; rep < 2; ++rep) {
      cudaMemset(d_out, 0, 32);
      tc_cp_kernel<<<1, 128, smem>>>(d_out, tiles, d_err);
      if (!sync_ok("tc_cp")) return 1;
    }
    cudaMemcpy(h, d_out, 32, cudaMemcpyDeviceToHost);
    printf("read-back of a copied 128 x 64 bf16 tile: %lld of 4096 words differ from the logical tile\n\n", h[0]);
    printf("MMA with the copied tile as A (TMEM) vs the same tile as A (shared memory) vs the definition: %lld mismatching "
           "accumulator words of 16384 compared (%lld of 8192 accumulators non-zero)\n\n", h[1], h[3]);
    printf("chain of %d tile copies (16 KB each, 4 instructions): %.1f clocks per tile = %.0f B/clk\n", tiles, double(h[2]) / tiles,
           16384.0 * tiles / double(h[2]));
  }

  printf("\n## M7: shared-memory bandwidth shared by MMA operand reads, tcgen05.cp reads and bulk-copy writes (one CTA)\n\n");
  printf("| MMA warps (N=16, A in TMEM) | cp warps | bulk copies | clk/MMA | MMA B read B/clk | cp clk/tile | cp B/clk | bulk clk/16KB | bulk B/clk | total B/clk |\n|---|---|---|---|---|---|---|---|---|---|\n");
  {
    unsigned char* gsrc = nullptr;
    cudaMalloc(&gsrc, 64 * 16384);
    cudaMemset(gsrc, 0x3c, 64 * 16384);
    const size_t smem = 1024 + kARegion + kBRegion + 64 * 1024 + sizeof(Barriers) + 16 * 8 + 64;
    cudaFuncSetAttribute(smem_share_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    const int combos[][3] = {{8, 0, 0}, {0, 1, 0}, {0, 2, 0}, {0, 4, 0}, {0, 0, 1}, {8, 0, 1}, {0, 4, 1}, {8, 1, 0}, {8, 4, 0}, {8, 4, 1}, {4, 4, 1}, {8, 2, 1}};
    for (const auto& cb : combos) {
      const int mma_count = 512, cp_tiles = cb[1] ? 128 / cb[1] : 0, bulk = cb[2] ? 128 : 0;
      long long h[3] = {0, 0, 0};
      for (int rep = 0; rep < 2; ++rep) {
        cudaMemset(d_out, 0, 32);
        smem_share_kernel<<<1, 448, smem>>>(d_out, cb[0], mma_count, cb[1], cp_tiles, bulk, gsrc, d_err);
        if (!sync_ok("smem_share")) return 1;
      }
      cudaMemcpy(h, d_out, 24, cudaMemcpyDeviceToHost);
      const double mma_clk = cb[0] ? double(h[0]) / (mma_count * cb[0]) : 0.0, mma_bw = cb[0] ? 512.0 / mma_clk : 0.0;
      const double cp_clk = cb[1] ? double(h[1]) / (cp_tiles * cb[1]) : 0.0, cp_bw = cb[1] ? 16384.0 / cp_clk : 0.0;
      const double bk_clk = cb[2] ? double(h[2]) / bulk : 0.0, bk_bw = cb[2] ? 16384.0 / bk_clk : 0.0;
      printf("| %d | %d | %s | %.1f | %.0f | %.1f | %.0f | %.1f | %.0f | %.0f |\n", cb[0], cb[1], cb[2] ? "yes" : "no", mma_clk, mma_bw, cp_clk,
             cp_bw, bk_clk, bk_bw, mma_bw + cp_bw + bk_bw);
    }
    cudaFree(gsrc);
  }

  printf("\n## M8: tensor-memory stores and loads next to 8 warps issuing N = 16 MMAs (A in TMEM), one CTA\n\n");
  printf("| B layout | st warps | ld warps | clk/MMA | st clk per 4 KB (one warp) | TMEM write B/clk (all st warps) | ld clk per 4 KB |\n|---|---|---|---|---|---|---|\n");
  {
    const size_t smem = 1024 + kARegion + kBRegion + sizeof(Barriers) + 64;
    cudaFuncSetAttribute(tmem_share_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    const int combos[][4] = {{0, 0, 0, 1}, {1, 0, 0, 1}, {1, 4, 0, 0}, {1, 4, 0, 1}, {0, 4, 0, 1}, {1, 0, 4, 1}, {1, 4, 4, 1}};
    for (const auto& cb : combos) {
      const int mma_count = cb[3] ? 512 : 0, st_iters = cb[1] ? 256 : 0, ld_iters = cb[2] ? 256 : 0;
      long long h[3] = {0, 0, 0};
      for (int rep = 0; rep < 2; ++rep) {
        cudaMemset(d_out, 0, 32);
        tmem_share_kernel<<<1, 512, smem>>>(d_out, mma_count, cb[0], cb[1], st_iters, cb[2], ld_iters, d_sink, d_err);
        if (!sync_ok("tmem_share")) return 1;
      }
      cudaMemcpy(h, d_out, 24, cudaMemcpyDeviceToHost);
      printf("| %s | %d | %d | %.1f | %.1f | %.0f | %.1f |\n", cb[0] ? "no swizzle" : "128-byte swizzle", cb[1], cb[2],
             mma_count ? double(h[0]) / (mma_count * 8.0) : 0.0, st_iters ? double(h[1]) / st_iters : 0.0,
             st_iters ? 4096.0 * cb[1] * st_iters / double(h[1]) : 0.0, ld_iters ? double(h[2]) / ld_iters : 0.0);
    }
  }

  printf("\n## M9: issue loop in K steps (8 warps, N = 16 MMAs with A in TMEM, per-step fence / commit / ring wait)\n\n");
  printf("| MMAs per warp and step | N | fence | commit | ring wait | A stages cycled | D column stride per warp | clk/step | clk/MMA |\n|---|---|---|---|---|---|---|---|---|\n");
  {
    const size_t smem = 1024 + kARegion + kBRegion + sizeof(Barriers) + 64;
    cudaFuncSetAttribute(stepped_issue_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    const int combos[][7] = {{4, 0, 0, 0, 1, 16, 16}, {4, 0, 0, 0, 1, 32, 16}, {4, 0, 0, 0, 8, 16, 16}, {4, 0, 0, 0, 8, 32, 16}, {4, 0, 0, 0, 2, 32, 16},
                             {4, 1, 1, 1, 8, 32, 16}, {2, 1, 1, 1, 8, 32, 16}, {1, 1, 1, 1, 8, 32, 16}, {1, 1, 1, 1, 1, 32, 16},
                             {4, 1, 1, 1, 8, 32, 32}, {2, 1, 1, 1, 8, 32, 32}, {1, 1, 1, 1, 8, 32, 32}};
    for (const auto& cb : combos) {
      const int steps = 256;
      long long h[1] = {0};
      for (int rep = 0; rep < 2; ++rep) {
        cudaMemset(d_out, 0, 32);
        stepped_issue_kernel<<<1, 256, smem>>>(d_out, steps, cb[0], cb[1], cb[2], cb[3], cb[4], cb[5], cb[6], d_err);
        if (!sync_ok("stepped_issue")) return 1;
      }
      cudaMemcpy(h, d_out, 8, cudaMemcpyDeviceToHost);
      printf("| %d | %d | %s | %s | %s | %d | %d | %.1f | %.1f |\n", cb[0], cb[6], cb[1] ? "yes" : "no", cb[2] ? "yes" : "no", cb[3] ? "yes" : "no",
             cb[4], cb[5], double(h[0]) / steps, double(h[0]) / steps / (cb[0] * 8.0));
    }
  }

  printf("\n## M10: several lanes of a warp issuing N = 16 MMAs (A in TMEM), each lane its own accumulator\n\n");
  printf("| warps | lanes per warp | A slices cycled | clk per MMA (all chains) | clk per MMA of one lane |\n|---|---|---|---|---|\n");
  {
    const size_t smem = 1024 + kARegion + kBRegion + sizeof(Barriers) + 64;
    cudaFuncSetAttribute(lane_issue_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    const int combos[][3] = {{1, 1, 4}, {1, 2, 4}, {1, 4, 4}, {1, 16, 4}, {4, 4, 4}, {8, 2, 4}, {8, 1, 4}, {16, 1, 4}, {8, 1, 1}, {8, 1, 8}, {8, 1, 32}, {16, 1, 32}, {1, 1, 32}};
    for (const auto& cb : combos) {
      const int cnt = 256;
      long long h[1] = {0};
      for (int rep = 0; rep < 2; ++rep) {
        cudaMemset(d_out, 0, 32);
        lane_issue_kernel<<<1, 512, smem>>>(d_out, cnt, cb[0], cb[1], cb[2], d_err);
        if (!sync_ok("lane_issue")) return 1;
      }
      cudaMemcpy(h, d_out, 8, cudaMemcpyDeviceToHost);
      printf("| %d | %d | %d | %.1f | %.1f |\n", cb[0], cb[1], cb[2], double(h[0]) / (double(cnt) * cb[0] * cb[1]), double(h[0]) / cnt);
    }
  }

  printf("\n## M11: two issuing warps with different shapes (warp 0: N = 144, A in shared memory; warp 1: N = 64, A in TMEM)\n\n");
  printf("| MMAs of warp 0 | MMAs of warp 1 | clocks warp 0 | clocks warp 1 | tensor clocks of all MMAs |\n|---|---|---|---|---|\n");
  {
    const size_t smem = 1024 + kARegion + kBRegion + sizeof(Barriers) + 64;
    cudaFuncSetAttribute(mixed_issue_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    const int combos[][2] = {{360, 0}, {0, 270}, {360, 270}, {360, 540}};
    for (const auto& cb : combos) {
      long long h[2] = {0, 0};
      for (int rep = 0; rep < 2; ++rep) {
        cudaMemset(d_out, 0, 32);
        mixed_issue_kernel<<<1, 128, smem>>>(d_out, 144, cb[0], 64, cb[1], d_err);
        if (!sync_ok("mixed_issue")) return 1;
      }
      cudaMemcpy(h, d_out, 16, cudaMemcpyDeviceToHost);
      printf("| %d | %d | %lld | %lld | %.0f |\n", cb[0], cb[1], h[0], h[1], cb[0] * 72.0 + cb[1] * 32.0);
    }
  }

  printf("\n## M12: the small-C_in kernel's A operand: no-swizzle windows of a staged image (M = 128, N = 64, K = 16), one CTA\n\n");
  printf("| row pitch (SBO) | K halves apart (LBO) | shift between MMAs | issuers | done clk/MMA |\n|---|---|---|---|---|\n");
  {
    const size_t smem = 1024 + kARegion + kBRegion + sizeof(Barriers) + 64;
    cudaFuncSetAttribute(ns_window_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem));
    const uint32_t cases[][3] = {{128, 2048, 128}, {128, 16, 16}, {160, 16, 16}, {160, 160, 16}, {160, 2720, 16}, {160, 16, 0},
                                 {256, 16, 16}, {256, 256, 32}, {176, 16, 16}};
    for (const auto& c : cases)
      for (int issuers = 1; issuers <= 3; ++issuers) {
        long long h[6] = {0, 0, 0, 0, 0, 0};
        const int cnt = 240;
        for (int rep = 0; rep < 2; ++rep) {
          ns_window_kernel<<<1, 128, smem>>>(d_out, cnt, issuers, c[0], c[1], c[2], d_err);
          if (!sync_ok("ns_window")) return 1;
        }
        cudaMemcpy(h, d_out, 48, cudaMemcpyDeviceToHost);
        long long md = 0;
        for (int w = 0; w < issuers; ++w) md = h[2 * w + 1] > md ? h[2 * w + 1] : md;
        printf("| %u | %u | %u | %d | %.1f |\n", c[0], c[1], c[2], issuers, double(md) / cnt);
      }
  }

  printf("\n## M2: tcgen05.mma cta_group::1 kind::tf32 (K = 8)\n\n");
  printf("| M | N | A from | issue clk/MMA | done clk/MMA | MAC/clk/SM |\n|---|---|---|---|---|---|\n");
  for (int m : {128, 64})
    for (int a_tmem = 0; a_tmem < 2; ++a_tmem)
      for (int n : ns) {
        if (m == 128 && n < 16) continue;
        if (quick && n != 8 && n != 16 && n != 256) continue;
        double is = 0, dn = 0;
        const bool ok = a_tmem ? run_tc<1, true>(m, n, count, 1, 1, &is, &dn) : run_tc<1, false>(m, n, count, 1, 1, &is, &dn);
        if (!ok) return 1;
        printf("| %d | %d | %s | %.1f | %.1f | %.0f |\n", m, n, a_tmem ? "TMEM" : "smem", is, dn, double(m) * n * 8 / dn);
      }

  printf("\n## M3: mma.sync, operands in registers, 8 independent accumulator tiles per warp, all SMs\n\n");
  printf("| shape | warps/SM | MAC/clk/SM | TFLOP/s at max clock |\n|---|---|---|---|\n");
  const char* names[4] = {"m16n8k16 bf16", "m16n8k8 bf16", "m16n8k8 tf32", "m16n8k4 tf32"};
  for (int shape = 0; shape < 4; ++shape)
    for (int warps : {4, 8, 16}) {
      double r = 0;
      const int iters = 2000;
      bool ok = false;
      if (shape == 0) ok = run_sync<0>(warps, g_sms, iters, &r);
      if (shape == 1) ok = run_sync<1>(warps, g_sms, iters, &r);
      if (shape == 2) ok = run_sync<2>(warps, g_sms, iters, &r);
      if (shape == 3) ok = run_sync<3>(warps, g_sms, iters, &r);
      if (!ok) return 1;
      printf("| %s | %d | %.0f | %.0f |\n", names[shape], warps, r, tflops(r));
    }

  printf("\n## M3g: exact-skip inner loop (ldmatrix A fragments + one B fragment per kept group + m16n8k8 bf16), all SMs\n\n");
  printf("| voxels/warp | kept rows per column | warps/SM | MAC/clk/SM | smem B/clk/SM | TFLOP/s at max clock |\n|---|---|---|---|---|---|\n");
  for (int warps : {8, 16}) {
    double r = 0, sb = 0;
    const int iters = 2000;
    if (!run_gather<64, 1>(warps, g_sms, iters, &r, &sb)) return 1;
    printf("| 64 | 1 | %d | %.0f | %.0f | %.0f |\n", warps, r, sb, tflops(r));
    if (!run_gather<64, 2>(warps, g_sms, iters, &r, &sb)) return 1;
    printf("| 64 | 2 | %d | %.0f | %.0f | %.0f |\n", warps, r, sb, tflops(r));
    if (!run_gather<32, 2>(warps, g_sms, iters, &r, &sb)) return 1;
    printf("| 32 | 2 | %d | %.0f | %.0f | %.0f |\n", warps, r, sb, tflops(r));
    if (!run_gather<32, 4>(warps, g_sms, iters, &r, &sb)) return 1;
    printf("| 32 | 4 | %d | %.0f | %.0f | %.0f |\n", warps, r, sb, tflops(r));
    if (!run_gather<128, 1>(warps, g_sms, iters, &r, &sb)) return 1;
    printf("| 128 | 1 | %d | %.0f | %.0f | %.0f |\n", warps, r, sb, tflops(r));
  }
  printf("\n");
  return 0;
}
