// Device-side building blocks shared by the tcgen05 kernels: mbarrier / TMA / tcgen05 PTX wrappers,
// bounded waits and the shared-memory barrier block.  Included by .cu files only.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cstdint>

namespace rt3d {
namespace {

constexpr int kThreadsUmma = 192;
constexpr int kMaxStages = 8;
constexpr int kABytes = 128 * 128;                  // 128 voxel rows x 64 bf16
constexpr long long kWaitCycles = 1ll << 31;        // about one second of SM clocks
constexpr size_t kSmemBudget = 200 * 1024;

struct __align__(8) Barriers {
  unsigned long long full[kMaxStages];
  unsigned long long empty[kMaxStages];
  unsigned long long tmem_full[2];
  unsigned long long tmem_empty[2];
  unsigned int tmem_base;
  volatile int abort_flag;
  long long wait_limit;      // SM clocks after which a wait gives up: kWaitCycles unless a test shortens it
};

// Bias staging area of a kernel, rounded up to 16 bytes so that the epilogue reads it as float4.
__device__ __forceinline__ float* align16_f32(void* p) {
  return reinterpret_cast<float*>((reinterpret_cast<uintptr_t>(p) + 15) & ~uintptr_t(15));
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}

// Bounded wait.  Returns false (and raises the CTA's abort flag + the global error word) when the
// phase did not complete within bars->wait_limit clocks, or when another role already aborted.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, Barriers* bars, int32_t* err, int code) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long start = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 128; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (bars->abort_flag) return false;
    if (clock64() - start > bars->wait_limit) {
      bars->abort_flag = 1;
      atomicCAS(err, 0, code);
      return false;
    }
  }
}

// Walk over a 4-digit mixed-radix index (digits i0 fastest .. i3 slowest, radices r0, r1, r2) that advances by a
// constant step per iteration: the step is decomposed once, after that every advance is four adds with carries
// instead of the three divisions a fresh decode costs.  i3 is unbounded.
struct Walk4 {
  int i0, i1, i2, i3;
  int d0, d1, d2, d3;
  int r0, r1, r2;
};
__device__ __forceinline__ void walk4_init(Walk4& k, int first, int step, int r0, int r1, int r2) {
  k.r0 = r0; k.r1 = r1; k.r2 = r2;
  int m = first;
  k.i0 = m % r0; m /= r0; k.i1 = m % r1; m /= r1; k.i2 = m % r2; k.i3 = m / r2;
  m = step;
  k.d0 = m % r0; m /= r0; k.d1 = m % r1; m /= r1; k.d2 = m % r2; k.d3 = m / r2;
}
__device__ __forceinline__ void walk4_next(Walk4& k) {
  k.i0 += k.d0; int c = k.i0 >= k.r0; k.i0 -= c * k.r0;
  k.i1 += k.d1 + c; c = k.i1 >= k.r1; k.i1 -= c * k.r1;
  k.i2 += k.d2 + c; c = k.i2 >= k.r2; k.i2 -= c * k.r2;
  k.i3 += k.d3 + c;
}

// Pulls a tensor map (a kernel parameter) into the descriptor cache ahead of its first use.
__device__ __forceinline__ void tma_prefetch_map(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2,
                                            int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2,
                                            int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}

// Shared-memory matrix descriptor: K-major tile of 128-byte rows, 128-byte swizzle, 8-row groups
// 1024 bytes apart; descriptor version 1 (sm_100).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
  uint64_t d = 0;
  d |= uint64_t((addr & 0x3FFFFu) >> 4);
  d |= uint64_t(1) << 16;                 // leading byte offset (unused for swizzled K-major)
  d |= uint64_t(1024 >> 4) << 32;         // stride byte offset between 8-row groups
  d |= uint64_t(1) << 46;                 // version
  d |= uint64_t(2) << 61;                 // SWIZZLE_128B
  return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t instr_desc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(n >> 3) << 17) | (uint32_t(128 >> 4) << 24);
}

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// 16 columns into the low half of a 32-entry register array (upper half zero), without taking the array's
// address in a way that would push it out of registers.
__device__ __forceinline__ void tmem_ld16_into32(uint32_t taddr, uint32_t (&r)[32]) {
  uint32_t t[16];
  tmem_ld16(taddr, t);
#pragma unroll
  for (int q = 0; q < 16; ++q) { r[q] = t[q]; r[q + 16] = 0u; }
}
// 32 (or 16) accumulator columns of this thread's row; `acc2_off` != 0: the tile was accumulated in two halves by
// two issuing threads, the second one `acc2_off` columns further on, and the two are added here (warp-uniform).
__device__ __forceinline__ void tmem_ld_acc(uint32_t taddr, bool wide, uint32_t acc2_off, uint32_t (&v)[32]) {
  if (wide) tmem_ld32(taddr, v);
  else tmem_ld16_into32(taddr, v);
  if (acc2_off) {
    uint32_t v2[32];
    if (wide) tmem_ld32(taddr + acc2_off, v2);
    else tmem_ld16_into32(taddr + acc2_off, v2);
#pragma unroll
    for (int q = 0; q < 32; ++q) v[q] = __float_as_uint(__uint_as_float(v[q]) + __uint_as_float(v2[q]));
  }
}

// Epilogue of NC (16 or 32) accumulator columns of one output voxel: + bias (from shared memory),
// optional ReLU, round to bf16, store.  `valid` = number of real output channels among the NC
// (>= NC: 16-byte vector stores; fewer: scalar tail, channels beyond are left untouched).
// `res`: this voxel's residual channels starting at the same channel as v[0] (nullptr: none), of which
// `res_avail` may be read (the channel pitch bounds the vector loads).
// max(x, 0) and max(y, 0) rounded to nearest-even bf16, x in the low half (as __floats2bfloat162_rn packs them).
__device__ __forceinline__ uint32_t cvt_relu_bf16x2(float x, float y) {
  uint32_t d;
  asm("cvt.rn.relu.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(y), "f"(x));
  return d;
}

template <int NC>
__device__ __forceinline__ void epilogue_cols(const uint32_t* v, const float* bias_s, int relu,
                                              __nv_bfloat16* dst, int valid, const __nv_bfloat16* res, int res_avail) {
  float f[NC];
  if (bias_s != nullptr) {                                            // nullptr: the bias is in the accumulator already
    const float4* b4 = reinterpret_cast<const float4*>(bias_s);      // 16-byte aligned by construction
#pragma unroll
    for (int k = 0; k < NC / 4; ++k) {
      const float4 b = b4[k];
      f[4 * k] = __uint_as_float(v[4 * k]) + b.x; f[4 * k + 1] = __uint_as_float(v[4 * k + 1]) + b.y;
      f[4 * k + 2] = __uint_as_float(v[4 * k + 2]) + b.z; f[4 * k + 3] = __uint_as_float(v[4 * k + 3]) + b.w;
    }
  } else {
#pragma unroll
    for (int q = 0; q < NC; ++q) f[q] = __uint_as_float(v[q]);
  }
  if (res != nullptr) {
#pragma unroll
    for (int k = 0; k < NC / 8; ++k) {
      if (8 * k < res_avail) {
        const uint4 rv = *reinterpret_cast<const uint4*>(res + 8 * k);
        const __nv_bfloat162* pr = reinterpret_cast<const __nv_bfloat162*>(&rv);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 t = __bfloat1622float2(pr[e]);
          f[8 * k + 2 * e] += t.x; f[8 * k + 2 * e + 1] += t.y;
        }
      }
    }
  }
  if (valid >= NC) {
#pragma unroll
    for (int q = 0; q < NC / 8; ++q) {
      uint4 o;
      if (relu) {                                  // activation and rounding in one instruction per pair
        o.x = cvt_relu_bf16x2(f[8 * q], f[8 * q + 1]); o.y = cvt_relu_bf16x2(f[8 * q + 2], f[8 * q + 3]);
        o.z = cvt_relu_bf16x2(f[8 * q + 4], f[8 * q + 5]); o.w = cvt_relu_bf16x2(f[8 * q + 6], f[8 * q + 7]);
      } else {
        __nv_bfloat162* po = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
        for (int e = 0; e < 4; ++e) po[e] = __floats2bfloat162_rn(f[8 * q + 2 * e], f[8 * q + 2 * e + 1]);
      }
      reinterpret_cast<uint4*>(dst)[q] = o;
    }
  } else {
#pragma unroll
    for (int q = 0; q < NC; ++q)                 // static indices: f stays in registers
      if (q < valid) dst[q] = __float2bfloat16_rn(relu ? fmaxf(f[q], 0.f) : f[q]);
  }
}

// Partial sums of the same tile left in scratch by other CTAs (layout of store_partial_row, pointers at this
// thread's row), added to the 32 (or 16) accumulator columns from `col` on in a fixed order: extra_first,
// then extra + p * extra_stride.  Two partial tiles' loads are in flight at a time.
constexpr int kPartRow = 4;   // floats between consecutive rows of a partial tile (see store_partial_row)
__device__ __forceinline__ void add_partials(uint32_t (&v)[32], bool wide, int col, const float* extra_first,
                                             const float* extra, size_t extra_stride, int n_extra) {
  const float* e0 = extra_first + size_t(col) * 128;
  for (int p = -1; p < n_extra; p += 2) {
    const float* ea = p < 0 ? e0 : extra + size_t(p) * extra_stride + size_t(col) * 128;
    const bool two = p + 1 < n_extra;
    const float* eb = two ? extra + size_t(p + 1) * extra_stride + size_t(col) * 128 : ea;
    float4 t0[8], t1[8];
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const bool live = wide || q < 4;
      t0[q] = live ? __ldcg(reinterpret_cast<const float4*>(ea + size_t(q) * 512)) : zero;
      t1[q] = (live && two) ? __ldcg(reinterpret_cast<const float4*>(eb + size_t(q) * 512)) : zero;
    }
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      v[4 * q] = __float_as_uint((__uint_as_float(v[4 * q]) + t0[q].x) + t1[q].x);
      v[4 * q + 1] = __float_as_uint((__uint_as_float(v[4 * q + 1]) + t0[q].y) + t1[q].y);
      v[4 * q + 2] = __float_as_uint((__uint_as_float(v[4 * q + 2]) + t0[q].z) + t1[q].z);
      v[4 * q + 3] = __float_as_uint((__uint_as_float(v[4 * q + 3]) + t0[q].w) + t1[q].w);
    }
  }
}

// One voxel row of a finished accumulator tile: columns [0, n_cols) of the TMEM buffer at `taddr`
// hold output channels m_base.. ; channels >= M are dropped.  Warp-uniform control flow around the
// TMEM loads (.sync.aligned); `in_range` may differ per lane.
// `res_row`: the voxel's residual row at channel m_base (nullptr: none); `res_pitch_left` = channels from
// m_base to the end of the residual tensor's channel pitch.
__device__ __forceinline__ void epilogue_row(uint32_t taddr, int n_cols, bool has_acc, bool in_range,
                                             const float* bias_s, int relu, __nv_bfloat16* dst, int m_base, int M,
                                             const __nv_bfloat16* res_row = nullptr, int res_pitch_left = 0,
                                             int col0 = 0, int col_step = 32, const float* extra_first = nullptr,
                                             const float* extra = nullptr, size_t extra_stride = 0, int n_extra = 0,
                                             uint32_t acc2_off = 0) {
  for (int col = col0; col < n_cols; col += col_step) {
    const int m0 = m_base + col;
    if (m0 >= M) break;
    uint32_t v[32];
    const bool wide = col + 32 <= n_cols;
    if (has_acc) {
      tmem_ld_acc(taddr + col, wide, acc2_off, v);
    } else {
#pragma unroll
      for (int q = 0; q < 32; ++q) v[q] = 0u;
    }
    if (!in_range) continue;
    if (extra_first != nullptr) add_partials(v, wide, col, extra_first, extra, extra_stride, n_extra);
    const __nv_bfloat16* res = res_row ? res_row + col : nullptr;
    const float* bs = bias_s ? bias_s + m0 : nullptr;
    if (wide) epilogue_cols<32>(v, bs, relu, dst + col, M - m0, res, res_pitch_left - col);
    else epilogue_cols<16>(v, bs, relu, dst + col, M - m0, res, res_pitch_left - col);
  }
}

// ------------------------------------------------------------------------------ TMA-store epilogue
// Each epilogue warp owns 32 rows of a tile; when those rows are a rectangular block of output voxels
// the warp writes 32-channel pieces (32 rows x 64 bytes of bf16) into its own two staging buffers in
// shared memory, in the 64-byte swizzle pattern, and one lane hands each piece to the TMA engine as a
// 5-D box store.  The stores drain asynchronously (full 64-byte rows, clipped at the tensor's edges and
// at the channel count), so the threads never wait on global stores.  Only warp-level synchronisation
// is used.
constexpr uint32_t kStoreStageBytes = 32 * 64;          // one piece
constexpr uint32_t kStoreBufs = 2;                      // staging buffers per warp = bulk stores in flight per warp
constexpr uint32_t kStoreWarpBytes = kStoreBufs * kStoreStageBytes;

struct TmaStore {
  const CUtensorMap* map;
  uint32_t smem;              // this warp's two staging buffers (1024-byte aligned)
  int c1, c2, c3, c4;         // output coordinates (w, h, t, n) of the warp's first row
  uint32_t piece;             // pieces issued so far by this warp
  uint32_t bufs = kStoreBufs; // staging buffers this warp cycles through (1 when two warps share a quadrant's pair)
};

// Fused max-pool (window = stride = 1 or 2 per axis) over the 32 voxels of an epilogue warp, which form a
// block of sbw x sbh x sbt(...) voxels whose extents are multiples of the window: lane -> (w, h, t) inside
// the block, partner lanes differ by 1, sbw and sbw*sbh.  Everything that depends only on the lane is worked
// out once per thread (make_pool_lanes), not once per 32-channel piece: it takes a dozen integer divisions.
struct PoolLanes {
  int pw, ph, pt;             // window
  int src_w, src_h, src_t;    // partner lane along each axis
  int out_row;                // row of the pooled block this lane's window leader writes
  bool writer;                // this lane is the leader of its window
};
__device__ __forceinline__ PoolLanes make_pool_lanes(int pw, int ph, int pt, int sbw, int sbh, int lane) {
  PoolLanes p;
  p.pw = pw; p.ph = ph; p.pt = pt;
  const int w = lane % sbw, h = (lane / sbw) % sbh, t = lane / (sbw * sbh);
  p.src_w = lane ^ 1;
  p.src_h = (h & 1) ? lane - sbw : lane + sbw;
  p.src_t = (t & 1) ? lane - sbw * sbh : lane + sbw * sbh;
  p.writer = (w % pw == 0) && (h % ph == 0) && (t % pt == 0);
  p.out_row = ((t / pt) * (sbh / ph) + h / ph) * (sbw / pw) + w / pw;
  return p;
}

__device__ __forceinline__ void tma_store_5d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2, int c3, int c4) {
  asm volatile("cp.async.bulk.tensor.5d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5, %6}], [%1];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
               : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// The store issued kStoreBufs pieces ago has finished reading its staging buffer.
__device__ __forceinline__ void tma_store_wait_read_1() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(kStoreBufs - 1) : "memory");
}
// The warp's previous store has finished reading its (single) staging buffer.
__device__ __forceinline__ void tma_store_wait_read_0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// Before the warp leaves the kernel: all its bulk stores have read their staging buffers (shared memory may go
// away).  Their global writes are part of the grid's memory operations, complete before the grid does.
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// Barrier among the epilogue warps only (named barrier 1): the bias staged after the dependent-launch wait is
// needed by nobody else, so the producer and MMA warps do not stop for it.
__device__ __forceinline__ void epilogue_bar_sync(int n_threads) {
  asm volatile("bar.sync 1, %0;" ::"r"(n_threads) : "memory");
}

// 32 accumulator columns of this thread's row -> bias, ReLU, bf16 -> staging buffer -> TMA box store of
// channels [m0, m0+32) x the warp's 32 voxels.
__device__ __forceinline__ void epilogue_piece_tma(const uint32_t* v, const float* bias_s, int relu, int m0, int lane,
                                                   TmaStore& ts, const __nv_bfloat16* res, int res_avail,
                                                   const PoolLanes* pool) {
  float f[32];
  if (bias_s != nullptr) {                                            // nullptr: the bias is in the accumulator already
    const float4* b4 = reinterpret_cast<const float4*>(bias_s);      // 16-byte aligned by construction
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const float4 b = b4[k];
      f[4 * k] = __uint_as_float(v[4 * k]) + b.x; f[4 * k + 1] = __uint_as_float(v[4 * k + 1]) + b.y;
      f[4 * k + 2] = __uint_as_float(v[4 * k + 2]) + b.z; f[4 * k + 3] = __uint_as_float(v[4 * k + 3]) + b.w;
    }
  } else {
#pragma unroll
    for (int q = 0; q < 32; ++q) f[q] = __uint_as_float(v[q]);
  }
  if (res != nullptr) {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (8 * k < res_avail) {
        const uint4 rv = *reinterpret_cast<const uint4*>(res + 8 * k);
        const __nv_bfloat162* pr = reinterpret_cast<const __nv_bfloat162*>(&rv);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 t = __bfloat1622float2(pr[e]);
          f[8 * k + 2 * e] += t.x; f[8 * k + 2 * e + 1] += t.y;
        }
      }
    }
  }
  uint4 o[4];
  __nv_bfloat162* po = reinterpret_cast<__nv_bfloat162*>(o);
  // ReLU and the rounding to bf16 in one instruction per pair of values (the epilogue warps of the layers with few
  // input channels are bound by their instruction count)
  if (relu) {
    uint32_t* uo = reinterpret_cast<uint32_t*>(o);
#pragma unroll
    for (int q = 0; q < 16; ++q) uo[q] = cvt_relu_bf16x2(f[2 * q], f[2 * q + 1]);
  } else {
#pragma unroll
    for (int q = 0; q < 16; ++q) po[q] = __floats2bfloat162_rn(f[2 * q], f[2 * q + 1]);
  }
  // optional max-pool: after the (monotonic) activation and bf16 rounding, so it equals pooling the stored tensor
  int out_row = lane;
  bool writer = true;
  if (pool != nullptr) {
    uint32_t* u = reinterpret_cast<uint32_t*>(o);
    if (pool->pw == 2) {
#pragma unroll
      for (int q = 0; q < 16; ++q) {
        const uint32_t other = __shfl_sync(0xffffffffu, u[q], pool->src_w);
        po[q] = __hmax2(po[q], *reinterpret_cast<const __nv_bfloat162*>(&other));
      }
    }
    if (pool->ph == 2) {
#pragma unroll
      for (int q = 0; q < 16; ++q) {
        const uint32_t other = __shfl_sync(0xffffffffu, u[q], pool->src_h);
        po[q] = __hmax2(po[q], *reinterpret_cast<const __nv_bfloat162*>(&other));
      }
    }
    if (pool->pt == 2) {
#pragma unroll
      for (int q = 0; q < 16; ++q) {
        const uint32_t other = __shfl_sync(0xffffffffu, u[q], pool->src_t);
        po[q] = __hmax2(po[q], *reinterpret_cast<const __nv_bfloat162*>(&other));
      }
    }
    writer = pool->writer;
    out_row = pool->out_row;
  }
  const uint32_t buf = ts.smem + (ts.piece % ts.bufs) * kStoreStageBytes;
  if (lane == 0) {                                 // the store issued ts.bufs pieces ago has read this buffer
    if (ts.bufs == 1) tma_store_wait_read_0();
    else tma_store_wait_read_1();
  }
  __syncwarp();
  const uint32_t row = buf + uint32_t(out_row) * 64u;
  const uint32_t sw = (uint32_t(out_row) >> 1) & 3u;  // 64-byte swizzle: 16-byte chunk index ^= address bits 7..8
  if (writer) {
#pragma unroll
    for (uint32_t k = 0; k < 4; ++k)
      asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(row + ((k ^ sw) << 4)), "r"(o[k].x), "r"(o[k].y),
                   "r"(o[k].z), "r"(o[k].w) : "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncwarp();
  if (lane == 0) tma_store_5d(ts.map, buf, m0, ts.c1, ts.c2, ts.c3, ts.c4);
  ++ts.piece;
}

// One voxel row of a finished accumulator tile through the TMA-store path: full 32-column pieces go
// through the staging buffers, a 16-column tail (bundle widths that are not multiples of 32) is stored
// directly.  `warp_rows_valid`: this warp's 32 rows belong to the tile (warp-uniform).
__device__ __forceinline__ void epilogue_row_tma(uint32_t taddr, int n_cols, bool has_acc, bool warp_rows_valid,
                                                 bool in_range, const float* bias_s, int relu, __nv_bfloat16* dst,
                                                 int m_base, int M, int lane, TmaStore& ts,
                                                 const __nv_bfloat16* res_row = nullptr, int res_pitch_left = 0,
                                                 const PoolLanes* pool = nullptr, const float* extra_first = nullptr,
                                                 const float* extra = nullptr, size_t extra_stride = 0,
                                                 int n_extra = 0, int col0 = 0, int col_step = 32,
                                                 uint32_t acc2_off = 0) {
  // col0 / col_step: a second warp on the same TMEM lane quadrant takes every other 32-column piece
  for (int col = col0; col < n_cols; col += col_step) {
    const int m0 = m_base + col;
    if (m0 >= M) break;
    uint32_t v[32];
    const bool wide = col + 32 <= n_cols;
    if (has_acc) {
      tmem_ld_acc(taddr + col, wide, acc2_off, v);
    } else {
#pragma unroll
      for (int q = 0; q < 32; ++q) v[q] = 0u;
    }
    if (extra_first != nullptr) add_partials(v, wide, col, extra_first, extra, extra_stride, n_extra);
    const __nv_bfloat16* res = (res_row && in_range) ? res_row + col : nullptr;
    if (wide) {
      if (warp_rows_valid) epilogue_piece_tma(v, bias_s ? bias_s + m0 : nullptr, relu, m0, lane, ts, res, res_pitch_left - col, pool);
    } else if (in_range) {
      epilogue_cols<16>(v, bias_s ? bias_s + m0 : nullptr, relu, dst + col, M - m0, res, res_pitch_left - col);
    }
  }
}

// Split-K partial tiles are stored as [column / 4][128 rows][4 columns] floats: a thread moves four columns of
// its row with one 16-byte access, and the 32 lanes of a warp (32 consecutive rows) touch 512 contiguous bytes
// (a quarter of the memory instructions of a [column][row] layout with 4-byte accesses; a row-major tile with
// 16-byte accesses touches 32 lines per instruction and was far slower).  kPartRow floats from row to row.
// Raw fp32 accumulator row -> scratch; `dst` already points at this thread's row (row * kPartRow) of column 0;
// column c of that row is at dst[(c / 4) * 512 + c % 4], so a piece starting at column `col` begins at col * 128.
__device__ __forceinline__ void store_partial_row(uint32_t taddr, int n_cols, bool has_acc, float* dst, int col0 = 0,
                                                  int col_step = 32, uint32_t acc2_off = 0) {
  for (int col = col0; col < n_cols; col += col_step) {
    uint32_t v[32];
    const bool wide = col + 32 <= n_cols;
    if (has_acc) {
      tmem_ld_acc(taddr + col, wide, acc2_off, v);
    } else {
#pragma unroll
      for (int q = 0; q < 32; ++q) v[q] = 0u;
    }
    float4* d4 = reinterpret_cast<float4*>(dst + size_t(col) * 128);
#pragma unroll
    for (int q = 0; q < 8; ++q)
      if (wide || q < 4)
        d4[q * 128] = make_float4(__uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]), __uint_as_float(v[4 * q + 2]),
                                  __uint_as_float(v[4 * q + 3]));
  }
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }


// Shared-memory matrix descriptor without swizzle: core matrices of 8 rows x 16 bytes stored
// contiguously (rows 16 bytes apart); `lbo` = byte distance between the two core matrices along K,
// `sbo` = byte distance between 8-row groups along M/N.
__device__ __forceinline__ uint64_t smem_desc_noswizzle(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= uint64_t((addr & 0x3FFFFu) >> 4);
  d |= uint64_t((lbo >> 4) & 0x3FFFu) << 16;
  d |= uint64_t((sbo >> 4) & 0x3FFFu) << 32;
  d |= uint64_t(1) << 46;                 // version
  return d;
}

}  // namespace
}  // namespace rt3d
