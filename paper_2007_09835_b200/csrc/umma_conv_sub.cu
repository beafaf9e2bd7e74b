// Tensor-core KGS convolution that skips pruned kernel locations at the grain of one small MMA.
//
// The step-list kernels (umma_conv.cu, umma_conv_pair.cu) drop a K step (kernel location x 64 input
// channels) only when NO kernel group of a whole bundle of up to 256 output channels keeps it.  With the
// paper's group sizes (Section 3: g_m x g_n of 4 x 4, 8 x 4, 8 x 8) that never happens, and pruned tiles are
// multiplied as zeros.  This kernel cuts the step into blocks of 16 output channels x 16 input channels
// (one tcgen05.mma of N = 16, K = 16) and issues only the blocks in which some group keeps the location;
// the weights of the other blocks are neither stored nor loaded.
//
// Two measured facts make that pay (microbench_mma.cu): (1) an N = 16 MMA whose A operand comes from shared
// memory re-reads 4 KB of it and takes 41 clocks, but 8-11 clocks with A in TENSOR MEMORY; (2) one thread
// issues an MMA every 56 clocks, but the limit is per issuing warp: eight warps together issue one N = 16
// MMA every 10.6 clocks (tensor time 8).  So:
//   * the input tile of a step (a 5-D TMA box of the input shifted by the kernel location, out-of-range
//     fill = zero padding) lands in a small ring in shared memory, from where eight "converter" warps move
//     it, one voxel row per thread, into a ring of A stages in tensor memory (tcgen05.st; lane = voxel,
//     32 columns = 64 bf16).  (Loading the rows straight from global memory, one row per thread, was tried
//     first: 32 cache lines per load instruction made a step cost 1800 clocks whatever the mask.)
//   * eight warps issue MMAs, warp w owning the accumulator columns [32w, 32w+32) = ranges 2w and 2w+1.  What
//     it has to issue in a step is precomputed at pack time: a command byte per (range, K slice) in the step's
//     64-byte header (a thread that derives block offsets from bit masks spends several hundred clocks per
//     step on dependent integer instructions, far more than the MMAs take);
//   * one producer warp streams the step's header and blocks (one contiguous run) into a ring in shared
//     memory with one bulk copy per step.
// The accumulator (128 voxels x up to 256 channels, fp32) fills TMEM columns 0..255, the A ring columns
// 256..511.  After a tile's last step the eight issuing warps are its epilogue warps (two per TMEM lane
// quadrant, 128 columns each) while converters and producer already fill the rings for the next tile.
//
// Every wait is bounded: on expiry the CTA records an error word, all roles fall through and TMEM is freed.
#include "kernels.h"
#include "umma_common.cuh"
#include "pdl.cuh"

namespace rt3d {
namespace {

constexpr int kSubMmaWarps = 8;
constexpr int kSubCvtWarps = 8;
constexpr int kThreadsSub = (kSubMmaWarps + kSubCvtWarps + 2) * 32;   // + block producer + input-tile producer
constexpr int kSubMaxStages = 8;
constexpr int kSubAStages = 4;              // input tiles in flight in shared memory (16 KB each)
constexpr uint32_t kSubACol = 256;          // first TMEM column of the A ring (32 columns per stage)

struct __align__(8) SubBars {
  unsigned long long full[kSubMaxStages];       // header + blocks of the step have landed (producer + bulk copy bytes)
                                                // and its four converter warps have written the A stage
  unsigned long long consumed[kSubMaxStages];   // the eight issuing warps' MMAs of the step are complete
  unsigned long long as_full[kSubAStages];      // the step's input tile has landed in shared memory
  unsigned long long as_empty[kSubAStages];     // its four converter warps have read it
  unsigned long long acc_full;                  // all MMAs of the tile are complete
  unsigned long long acc_empty;                 // all eight epilogue warps have read the accumulator
  unsigned int tmem_base;
  volatile int abort_flag;
};

__device__ __forceinline__ bool sub_wait(uint32_t bar, uint32_t parity, SubBars* bars, int32_t* err, int code) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long start = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 128; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (bars->abort_flag) return false;
    if (clock64() - start > kWaitCycles) {
      bars->abort_flag = 1;
      atomicCAS(err, 0, code);
      return false;
    }
  }
}

struct SubItem {
  int bundle, s_begin, nsteps;
  int n0, t0, h0, w0;
};
__device__ __forceinline__ SubItem sub_decode(const SubArgs& a, int item, int n_mtiles) {
  SubItem c;
  c.bundle = item / n_mtiles;
  int mt = item - c.bundle * n_mtiles;
  const int iw = mt % a.tiles_w; mt /= a.tiles_w;
  const int ih = mt % a.tiles_h; mt /= a.tiles_h;
  const int it = mt % a.tiles_t; mt /= a.tiles_t;
  c.w0 = iw * a.box.bw; c.h0 = ih * a.box.bh; c.t0 = it * a.box.bt; c.n0 = mt * a.box.bn;
  c.s_begin = __ldg(a.step_ptr + c.bundle);
  c.nsteps = __ldg(a.step_ptr + c.bundle + 1) - c.s_begin;
  return c;
}

__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint4 (&v)[8]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(v[0].x), "r"(v[0].y), "r"(v[0].z), "r"(v[0].w), "r"(v[1].x), "r"(v[1].y), "r"(v[1].z), "r"(v[1].w),
        "r"(v[2].x), "r"(v[2].y), "r"(v[2].z), "r"(v[2].w), "r"(v[3].x), "r"(v[3].y), "r"(v[3].z), "r"(v[3].w),
        "r"(v[4].x), "r"(v[4].y), "r"(v[4].z), "r"(v[4].w), "r"(v[5].x), "r"(v[5].y), "r"(v[5].z), "r"(v[5].w),
        "r"(v[6].x), "r"(v[6].y), "r"(v[6].z), "r"(v[6].w), "r"(v[7].x), "r"(v[7].y), "r"(v[7].z), "r"(v[7].w)
      : "memory");
}

// D[tmem] (+)= A[tmem] * B[smem]^T, M = 128: A = this CTA's 128 lanes x 8 columns (16 bf16 per lane).
__device__ __forceinline__ void umma_bf16_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n"
      "}\n"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}

__global__ void __launch_bounds__(kThreadsSub, 1)
conv3d_umma_sub_kernel(const __grid_constant__ CUtensorMap xmap, const __grid_constant__ CUtensorMap ymap, const SubArgs a) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t a_ring = (raw + 1023u) & ~1023u;                                         // input tiles, 128-byte swizzle
  const uint32_t b_ring = a_ring + kSubAStages * kABytes;
  const uint32_t store_smem = b_ring + uint32_t(a.stages) * a.slot_bytes;                 // 8 warps x 2 staging buffers
  unsigned char* after = smem_raw + (a_ring - raw) + kSubAStages * kABytes + size_t(a.stages) * a.slot_bytes +
                         kSubMmaWarps * kStoreWarpBytes;
  SubBars* bars = reinterpret_cast<SubBars*>(after);
  float* bias_s = align16_f32(bars + 1);
  int32_t* err = a.sched + 2;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_mtiles = a.tiles_n * a.tiles_t * a.tiles_h * a.tiles_w;
  const int n_items = n_mtiles * a.n_bundles;
  const int box_rows = a.box.bn * a.box.bt * a.box.bh * a.box.bw;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kSubMaxStages; ++s) {
      mbar_init(smem_u32(&bars->full[s]), 5);
      mbar_init(smem_u32(&bars->consumed[s]), kSubMmaWarps);
    }
    for (int s = 0; s < kSubAStages; ++s) {
      mbar_init(smem_u32(&bars->as_full[s]), 1);
      mbar_init(smem_u32(&bars->as_empty[s]), 4);
    }
    mbar_init(smem_u32(&bars->acc_full), kSubMmaWarps);
    mbar_init(smem_u32(&bars->acc_empty), kSubMmaWarps);
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (threadIdx.x == 32) {
    tma_prefetch_map(&xmap);
    if (a.store_tma) tma_prefetch_map(&ymap);
  }
  if (warp == kSubMmaWarps + kSubCvtWarps) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&bars->tmem_base)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;

  pdl_launch();                // the successor may be scheduled: this CTA holds its TMEM
  pdl_wait();                  // predecessor complete: activations, bias, residual are visible
  if (warp < kSubMmaWarps) {   // the epilogue warps stage the bias; the other roles start at once
    for (int i = threadIdx.x; i < a.n_bundles * a.n_tile; i += kSubMmaWarps * 32)
      bias_s[i] = (a.bias != nullptr && i < a.g.M) ? __ldg(a.bias + i) : 0.f;
    epilogue_bar_sync(kSubMmaWarps * 32);
  }

  if (warp < kSubMmaWarps) {
    // ------------------------------------------------------------- MMA issue, then epilogue (warps 0..7)
    const int quad = warp & 3, half = warp >> 2;
    const int row = quad * 32 + lane;
    int r = row;
    const int bw_i = r % a.box.bw; r /= a.box.bw;
    const int bh_i = r % a.box.bh; r /= a.box.bh;
    const int bt_i = r % a.box.bt; r /= a.box.bt;
    const int bn_i = r;
    int r0 = quad * 32;
    const int bw_0 = r0 % a.box.bw; r0 /= a.box.bw;
    const int bh_0 = r0 % a.box.bh; r0 /= a.box.bh;
    const int bt_0 = r0 % a.box.bt; r0 /= a.box.bt;
    const int bn_0 = r0;
    __nv_bfloat16* yb = static_cast<__nv_bfloat16*>(a.y);
    const __nv_bfloat16* rb = static_cast<const __nv_bfloat16*>(a.residual);
    TmaStore ts{&ymap, store_smem + uint32_t(warp) * kStoreWarpBytes, 0, 0, 0, 0, 0u};
    const uint32_t idesc16 = instr_desc_bf16(16);
    const uint32_t d_col = tmem_base + uint32_t(warp) * 32u;      // this warp's accumulator columns
    int stage = 0;
    uint32_t use = 0, it = 0;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++it) {
      const SubItem c = sub_decode(a, item, n_mtiles);
      int ok = 1;
      if (lane == 0) {
        // the previous tile's accumulator has been read by all epilogue warps
        if (it > 0 && !sub_wait(smem_u32(&bars->acc_empty), (it - 1) & 1u, bars, err, 41)) ok = 0;
        tc_fence_after();
        int st = stage;
        uint32_t us = use;
        for (int i = 0; i < c.nsteps && ok; ++i) {
          if (!sub_wait(smem_u32(&bars->full[st]), us & 1u, bars, err, 42)) { ok = 0; break; }
          tc_fence_after();
          const uint32_t slot = b_ring + uint32_t(st) * a.slot_bytes;
          uint32_t cmd0, cmd1;                         // command bytes of this warp's two ranges, K slices 0..3
          asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(cmd0), "=r"(cmd1) : "r"(slot + uint32_t(warp) * 8u));
          const uint64_t bdesc0 = smem_desc_noswizzle(slot + uint32_t(kSubHeaderBytes), 128u, 256u);
          const uint32_t a_t = tmem_base + kSubACol + uint32_t(st) * 32u;
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) {
            const uint32_t c0 = (cmd0 >> (8 * ks)) & 0xFFu, c1 = (cmd1 >> (8 * ks)) & 0xFFu;
            const uint32_t acc = (i | ks) ? 1u : 0u;
            if (c0 & 0x80u) umma_bf16_ta(d_col, a_t + uint32_t(ks) * 8u, bdesc0 + uint64_t((c0 & 0x3Fu) * 32u), idesc16, acc);
            if (c1 & 0x80u) umma_bf16_ta(d_col + 16u, a_t + uint32_t(ks) * 8u, bdesc0 + uint64_t((c1 & 0x3Fu) * 32u), idesc16, acc);
          }
          umma_commit(smem_u32(&bars->consumed[st]));
          if (++st == a.stages) { st = 0; ++us; }
        }
        if (ok) umma_commit(smem_u32(&bars->acc_full));      // with no MMAs pending this arrives at once
      }
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      {                                                       // all lanes: the ring position after this item
        const int adv = stage + c.nsteps;
        use += uint32_t(adv / a.stages);
        stage = adv % a.stages;
      }
      if (!sub_wait(smem_u32(&bars->acc_full), it & 1u, bars, err, 44)) break;
      tc_fence_after();
      // epilogue: this warp takes columns [128 half, 128 half + 128) of its 32 voxels
      const int col0 = half * 128;
      const int n_cols = a.n_tile - col0 < 128 ? a.n_tile - col0 : 128;
      if (n_cols > 0) {
        const int nn = c.n0 + bn_i, to = c.t0 + bt_i, ho = c.h0 + bh_i, wo = c.w0 + bw_i;
        const bool in_range = row < box_rows && nn < a.g.n && to < a.g.To && ho < a.g.Ho && wo < a.g.Wo;
        const long long vox = (((long long)nn * a.g.To + to) * a.g.Ho + ho) * a.g.Wo + wo;
        const int m_base = c.bundle * a.n_tile + col0;
        const uint32_t taddr = tmem_base + (uint32_t(quad * 32) << 16) + uint32_t(col0);
        __nv_bfloat16* dst = yb + vox * a.g.ycs + m_base;
        const __nv_bfloat16* res = (rb != nullptr && in_range) ? rb + vox * a.rcs + m_base : nullptr;
        const int res_left = a.rcs - m_base;
        if (a.store_tma) {
          ts.c1 = c.w0 + bw_0; ts.c2 = c.h0 + bh_0; ts.c3 = c.t0 + bt_0; ts.c4 = c.n0 + bn_0;
          epilogue_row_tma(taddr, n_cols, c.nsteps > 0, quad * 32 < box_rows, in_range, bias_s, a.g.relu, dst, m_base,
                           a.g.M, lane, ts, res, res_left, nullptr);
        } else {
          epilogue_row(taddr, n_cols, c.nsteps > 0, in_range, bias_s, a.g.relu, dst, m_base, a.g.M, res, res_left);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->acc_empty));
    }
    if (lane == 0) tma_store_wait_all();         // all bulk stores done before shared memory goes away
  } else if (warp < kSubMmaWarps + kSubCvtWarps) {
    // ------------------------------------------------------------- converters (warps 8..15)
    // Warp 8 + 4 p + q moves rows [32 q, 32 q + 32) of the input tiles of the steps whose sequence number is
    // p mod 2 from shared memory into the A stage in tensor memory: one voxel row (64 channels = 8 x 16 bytes,
    // un-swizzled on the way) per thread.
    const int quad = warp & 3, par = (warp - kSubMmaWarps) >> 2;
    const int row = quad * 32 + lane;
    const uint32_t row_off = uint32_t(row) * 128u, sw = uint32_t(row & 7);
    uint32_t g = 0;                               // sequence number of the step among all steps of this CTA
    int ok = 1;
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
      const int bundle = item / n_mtiles;
      const int nsteps = __ldg(a.step_ptr + bundle + 1) - __ldg(a.step_ptr + bundle);
      for (int i = 0; i < nsteps; ++i, ++g) {
        if (int(g & 1u) != par) continue;
        const uint32_t sa = g % kSubAStages, ua = g / kSubAStages;
        const uint32_t st = g % uint32_t(a.stages), us = g / uint32_t(a.stages);
        if (lane == 0) ok = sub_wait(smem_u32(&bars->as_full[sa]), ua & 1u, bars, err, 45) ? 1 : 0;
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        uint4 v[8];
        const uint32_t src = a_ring + sa * uint32_t(kABytes) + row_off;
#pragma unroll
        for (uint32_t c = 0; c < 8; ++c)
          asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                       : "=r"(v[c].x), "=r"(v[c].y), "=r"(v[c].z), "=r"(v[c].w) : "r"(src + ((c ^ sw) << 4)));
        if (lane == 0) ok = sub_wait(smem_u32(&bars->consumed[st]), (us & 1u) ^ 1u, bars, err, 47) ? 1 : 0;
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        tc_fence_after();
        tmem_st32(tmem_base + (uint32_t(quad * 32) << 16) + kSubACol + st * 32u, v);
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars->as_empty[sa]));    // the rows are in registers: the tile may be overwritten
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars->full[st]));
      }
    }
  } else if (warp == kSubMmaWarps + kSubCvtWarps) {
    // ------------------------------------------------------------- block producer (warp 16)
    // The whole warp walks the steps: every 32 steps each lane fetches one 32-byte step record, lane 0 gets
    // them by shuffle, waits for the stage and issues the bulk copy of the step's blocks.
    int stage = 0;
    uint32_t use = 0;
    int ok = 1;
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
      const SubItem c = sub_decode(a, item, n_mtiles);
      for (int i0 = 0; i0 < c.nsteps && ok; i0 += 32) {
        uint4 rec = make_uint4(0u, 0u, 0u, 0u);
        if (i0 + lane < c.nsteps) rec = __ldg(reinterpret_cast<const uint4*>(a.steps + c.s_begin + i0 + lane));
        const int n_here = c.nsteps - i0 < 32 ? c.nsteps - i0 : 32;
        for (int q = 0; q < n_here; ++q) {
          const uint32_t off64 = __shfl_sync(0xffffffffu, rec.y, q), nblk = __shfl_sync(0xffffffffu, rec.z, q);
          if (lane == 0) {
            if (!sub_wait(smem_u32(&bars->consumed[stage]), (use & 1u) ^ 1u, bars, err, 46)) ok = 0;
            if (ok) {
              const uint32_t bytes = uint32_t(kSubHeaderBytes) + nblk * uint32_t(kSubBlockBytes);
              const uint32_t full = smem_u32(&bars->full[stage]);
              mbar_expect_tx(full, bytes);
              asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                           ::"r"(b_ring + uint32_t(stage) * a.slot_bytes),
                             "l"(reinterpret_cast<const unsigned char*>(a.blocks) + size_t(off64) * 64), "r"(bytes), "r"(full)
                           : "memory");
            }
          }
          ok = __shfl_sync(0xffffffffu, ok, 0);
          if (!ok) break;
          if (++stage == a.stages) { stage = 0; ++use; }
        }
      }
    }
  } else {
    // ------------------------------------------------------------- input-tile producer (warp 17)
    // Same walk; lane 0 issues one 5-D TMA box per step: the tile's voxels shifted by the kernel location.
    int ok = 1;
    uint32_t g = 0;
    const uint32_t tx_bytes = uint32_t(box_rows) * 128u;
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
      const SubItem c = sub_decode(a, item, n_mtiles);
      const int wq = c.w0 * a.g.sw - a.g.pw, hq = c.h0 * a.g.sh - a.g.ph, tq = c.t0 * a.g.st - a.g.pt;
      for (int i0 = 0; i0 < c.nsteps && ok; i0 += 32) {
        int enc_l = 0;
        if (i0 + lane < c.nsteps) enc_l = __ldg(&a.steps[c.s_begin + i0 + lane].enc);
        const int n_here = c.nsteps - i0 < 32 ? c.nsteps - i0 : 32;
        for (int q = 0; q < n_here; ++q, ++g) {
          const int enc = __shfl_sync(0xffffffffu, enc_l, q);
          if (lane == 0) {
            const uint32_t sa = g % kSubAStages, ua = g / kSubAStages;
            if (!sub_wait(smem_u32(&bars->as_empty[sa]), (ua & 1u) ^ 1u, bars, err, 48)) ok = 0;
            if (ok) {
              const uint32_t full = smem_u32(&bars->as_full[sa]);
              mbar_expect_tx(full, tx_bytes);
              tma_load_5d(a_ring + sa * uint32_t(kABytes), &xmap, full, (enc & 4095) * 64, wq + ((enc >> 12) & 63),
                          hq + ((enc >> 18) & 63), tq + ((enc >> 24) & 63), c.n0);
            }
          }
          ok = __shfl_sync(0xffffffffu, ok, 0);
          if (!ok) break;
        }
      }
    }
  }

  // ---------------------------------------------------------------------- teardown
  if (bars->abort_flag) {
    // error path: give asynchronous copies / MMAs still in flight time to land before TMEM goes away
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000ll) { }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kSubMmaWarps + kSubCvtWarps) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

size_t sub_smem_bytes_impl(int stages, uint32_t slot_bytes, int n_tile, int n_bundles) {
  return 1024 + size_t(kSubAStages) * kABytes + size_t(stages) * slot_bytes + kSubMmaWarps * kStoreWarpBytes + sizeof(SubBars) + 16 +
         size_t(n_tile) * n_bundles * 4;
}

}  // namespace

// Ring geometry for a layout whose largest step has `max_blocks` blocks: slot size and number of stages
// (at most 8: the A ring in tensor memory has 8 stages of 32 columns).  false: does not fit.
bool umma_sub_plan(SubArgs* a, int max_blocks) {
  uint32_t slot = uint32_t(kSubHeaderBytes) + uint32_t(max_blocks < 1 ? 1 : max_blocks) * uint32_t(kSubBlockBytes);
  slot = (slot + 1023u) & ~1023u;
  int stages = int((112u * 1024u) / slot);
  if (stages > kSubMaxStages) stages = kSubMaxStages;
  if (stages < 2) return false;
  a->slot_bytes = slot;
  a->stages = stages;
  return sub_smem_bytes_impl(stages, slot, a->n_tile, a->n_bundles) <= 227 * 1024;
}

cudaError_t launch_conv_umma_sub(const SubArgs& a, const void* xmap, const void* ymap, int sm_count, cudaStream_t stream) {
  if (a.stages < 2 || a.stages > kSubMaxStages || a.n_tile % 16 || a.n_tile > 256) return cudaErrorInvalidValue;
  if (xmap == nullptr || (a.store_tma && ymap == nullptr)) return cudaErrorInvalidValue;
  const size_t smem = sub_smem_bytes_impl(a.stages, a.slot_bytes, a.n_tile, a.n_bundles);
  if (smem > 227 * 1024) return cudaErrorInvalidValue;
  const long long n_items = (long long)a.tiles_n * a.tiles_t * a.tiles_h * a.tiles_w * a.n_bundles;
  if (n_items <= 0) return cudaSuccess;
  static bool attr_done[kMaxDevices] = {};             // the attribute is per device
  const int device = current_device_index();
  if (device < 0) return cudaErrorInvalidDevice;
  if (!attr_done[device]) {
    cudaError_t e = cudaFuncSetAttribute(conv3d_umma_sub_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    attr_done[device] = true;
  }
  const int grid = int(n_items < sm_count ? n_items : sm_count);
  CUtensorMap xm, ym;
  memcpy(&xm, xmap, sizeof(CUtensorMap));
  memcpy(&ym, ymap ? ymap : xmap, sizeof(CUtensorMap));                            // not used when store_tma == 0
  LaunchSetup ls(dim3(grid), dim3(kThreadsSub), smem, stream);
  return cudaLaunchKernelEx(&ls.cfg, conv3d_umma_sub_kernel, xm, ym, a);
}

}  // namespace rt3d
