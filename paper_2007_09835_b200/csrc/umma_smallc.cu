// Tensor-core convolution for layers with very few input channels (C_in <= 8 stored at a channel
// pitch of 8, e.g. the RGB first layers of the C3D- and R(2+1)D-shaped networks), any temporal
// stride, spatial strides up to 4.
//
// With 16 bytes per voxel the input halo of an output tile of 1 x 16 x 8 voxels can be staged in
// shared memory exactly as it lies in global memory, [t][h][w][8 channels], by one TMA box whose
// out-of-range part is zero-filled (= the zero padding; channels >= C_in are zero-filled too).
// In the no-swizzle operand layout a core matrix is 8 rows of 16 bytes, i.e. 8 consecutive voxels
// along w with their 8 channels: every shifted window of the halo is a valid A operand whose
// 8-row groups are one halo row apart, and the two K halves of a K=16 MMA can be two different
// kernel locations (leading byte offset = distance between the two shifted windows).  So each pair
// of kept kernel locations is one MMA, the input is read from L2 once per tile, and the layer is
// bound by writing its output.  Kernel locations that no group keeps are not in the pair list.
// The bias is one more MMA (a ones column times the bias as two bf16 terms): the kernel is bound by the
// instruction count of its epilogue warps, and that removes a third of it.
// With a spatial stride the input is staged as one image per stride phase (strided TMA boxes), so
// that consecutive outputs are again consecutive voxels and every location a window of one image.
//
// Roles as in the main kernel: warp 0 TMA producer, warp 1 MMA issuer / TMEM owner, warps 2..5
// epilogue; bounded mbarrier waits.
#include "kernels.h"
#include "umma_common.cuh"
#include "pdl.cuh"

namespace rt3d {
namespace {

constexpr int kSmallCStages = 3;

template <int kDummy>
__global__ void __launch_bounds__(kThreadsUmma, 3)
conv3d_umma_smallc_kernel(const __grid_constant__ CUtensorMap xmap, const __grid_constant__ CUtensorMap ymap,
                          const SmallCArgs a) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t store_smem = (raw + 1023u) & ~1023u;                   // 4 warps x 2 staging buffers (TMA stores)
  const uint32_t base = store_smem + 4 * kStoreWarpBytes;
  const uint32_t w_bytes = uint32_t(a.n_pairs) * 2u * uint32_t(a.n_pad) * 16u;
  const uint32_t w_smem = base;                                         // weight image, whole layer
  // The bias enters the accumulator through one more MMA instead of 32 additions per 32-channel piece in the
  // epilogue (which is what bounds this kernel): B = one extra "pair" of the weight image whose k = 0 rows hold
  // the bias split into two bf16 terms (high part + remainder: fp32 accuracy to about 2^-17), A = a single core
  // matrix with ones in its k = 0 column that every 8-row group and both K halves read (strides 0).
  const uint32_t bias_b_smem = w_smem + w_bytes;                        // [2 K halves][n_pad][8] bf16
  const uint32_t ones_smem = bias_b_smem + 2u * uint32_t(a.n_pad) * 16u; // [8 rows][8] bf16
  const uint32_t halo_smem = base + ((w_bytes + 2u * uint32_t(a.n_pad) * 16u + 128u + 127u) & ~127u);   // ring of staged halos
  const uint32_t halo_stride = (uint32_t(a.n_phases * a.phase_stride) + 127u) & ~127u;
  unsigned char* gen = smem_raw + (base - raw);
  int32_t* pair_smem = reinterpret_cast<int32_t*>(gen + (halo_smem - base) + kSmallCStages * halo_stride);
  Barriers* bars = reinterpret_cast<Barriers*>(reinterpret_cast<unsigned char*>(pair_smem) +
                                               ((size_t(a.n_pairs) * 8 + 15) & ~size_t(15)));
  float* bias_s = align16_f32(bars + 1);
  int32_t* err = a.sched + 2;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tiles_per_frame = a.tiles_h * a.tiles_w;
  const int n_items = a.g.n * a.g.To * tiles_per_frame;

  if (threadIdx.x == 32) {                     // descriptor fetches overlap the rest of the set-up
    tma_prefetch_map(&xmap);
    tma_prefetch_map(&ymap);
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < kSmallCStages; ++s) {
      mbar_init(smem_u32(&bars->full[s]), 1);
      mbar_init(smem_u32(&bars->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bars->tmem_full[b]), 1);
      mbar_init(smem_u32(&bars->tmem_empty[b]), 4);
    }
    bars->abort_flag = 0;
    bars->wait_limit = kWaitCycles;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&bars->tmem_base)), "r"(uint32_t(a.tmem_cols)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;

  // Everything above touched only shared memory, barriers and TMEM.  The successor may be scheduled now that
  // this CTA holds its TMEM columns (a successor CTA that shared the SM and allocated first could otherwise
  // starve this one while waiting for it); global memory from here on.
  pdl_launch();
  pdl_wait();
  for (int i = threadIdx.x; i < a.n_pad; i += blockDim.x)
    bias_s[i] = (a.bias != nullptr && i < a.g.M) ? __ldg(a.bias + i) : 0.f;
  // weight image and pair offsets: plain cooperative copy, once per CTA
  {
    const uint4* src = reinterpret_cast<const uint4*>(a.wimg);
    uint4* dst = reinterpret_cast<uint4*>(gen);
    for (uint32_t i = threadIdx.x; i < w_bytes / 16; i += blockDim.x) dst[i] = __ldg(src + i);
    for (int i = threadIdx.x; i < a.n_pairs * 2; i += blockDim.x) pair_smem[i] = __ldg(a.pair_off + i);
    // bias operand and ones tile
    __nv_bfloat16* bb = reinterpret_cast<__nv_bfloat16*>(gen + (bias_b_smem - base));
    const int n8 = a.n_pad * 8;
    for (int i = threadIdx.x; i < 2 * n8 + 64; i += blockDim.x) {
      float val = 0.f;
      if (i >= 2 * n8) {
        val = ((i - 2 * n8) & 7) == 0 ? 1.f : 0.f;                    // ones tile: k = 0 column
      } else if ((i & 7) == 0) {                                      // k = 0 of output channel m, K half i / n8
        const int m = (i % n8) >> 3;
        const float b = (a.bias != nullptr && m < a.g.M) ? __ldg(a.bias + m) : 0.f;
        const float hi = __bfloat162float(__float2bfloat16_rn(b));
        val = i < n8 ? hi : b - hi;
      }
      bb[i] = __float2bfloat16_rn(val);
    }
  }
  // generic-proxy writes of the weight image must be visible to the tensor core (async proxy)
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();

  if (warp == 0) {
    if (lane == 0 && a.n_pairs > 0) {
      int stage = 0;
      uint32_t phase = 0;
      Walk4 k;
      walk4_init(k, blockIdx.x, gridDim.x, a.tiles_w, a.tiles_h, a.g.To);
      for (int item = blockIdx.x; item < n_items; item += gridDim.x, walk4_next(k)) {
        const int iw = k.i0, ih = k.i1, to = k.i2, nn = k.i3;
        if (!mbar_wait(smem_u32(&bars->empty[stage]), phase ^ 1u, bars, err, 11)) break;
        const uint32_t full = smem_u32(&bars->full[stage]);
        mbar_expect_tx(full, uint32_t(a.n_phases * a.phase_bytes));
        const int w0 = iw * kSmallCTileW * a.g.sw - a.g.pw, h0 = ih * kSmallCTileH * a.g.sh - a.g.ph;
        if (a.merged_cw) {                           // unit column stride: a whole image row is one contiguous run
          for (int ph = 0; ph < a.n_phases; ++ph)
            tma_load_5d(halo_smem + stage * halo_stride + ph * a.phase_stride, &xmap, full, w0 * 8, 0, h0 + ph,
                        to * a.g.st - a.g.pt, nn);
        } else {
          for (int ph = 0; ph < a.n_phases; ++ph)    // one strided box per (row, column) stride phase
            tma_load_5d(halo_smem + stage * halo_stride + ph * a.phase_stride, &xmap, full, 0, w0 + ph % a.g.sw,
                        h0 + ph / a.g.sw, to * a.g.st - a.g.pt, nn);
        }
        if (++stage == kSmallCStages) { stage = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = instr_desc_bf16(a.n_pad);
      const uint32_t sbo_a = uint32_t(a.img_w) * 16u;             // next 8-voxel group = next image row
      const uint32_t lbo_b = uint32_t(a.n_pad) * 16u;             // second K half of the weight image
      int stage = 0;
      uint32_t phase = 0, j = 0;
      for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++j) {
        const uint32_t buf = j & 1u;
        if (!mbar_wait(smem_u32(&bars->tmem_empty[buf]), ((j >> 1) & 1u) ^ 1u, bars, err, 12)) break;
        if (a.n_pairs == 0) { mbar_arrive(smem_u32(&bars->tmem_full[buf])); continue; }
        if (!mbar_wait(smem_u32(&bars->full[stage]), phase, bars, err, 13)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * uint32_t(a.n_pad);
        const uint32_t halo = halo_smem + stage * halo_stride;
        for (int p = 0; p < a.n_pairs; ++p) {
          const uint32_t o0 = uint32_t(pair_smem[2 * p]), o1 = uint32_t(pair_smem[2 * p + 1]);
          const uint64_t adesc = smem_desc_noswizzle(halo + o0, o1 - o0, sbo_a);
          const uint64_t bdesc = smem_desc_noswizzle(w_smem + uint32_t(p) * 2u * lbo_b, lbo_b, 128u);
          umma_bf16(d_tmem, adesc, bdesc, idesc, p ? 1u : 0u);
        }
        umma_bf16(d_tmem, smem_desc_noswizzle(ones_smem, 0u, 0u), smem_desc_noswizzle(bias_b_smem, lbo_b, 128u), idesc, 1u);
        umma_commit(smem_u32(&bars->empty[stage]));
        umma_commit(smem_u32(&bars->tmem_full[buf]));
        if (++stage == kSmallCStages) { stage = 0; phase ^= 1u; }
      }
    }
  } else {
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    const int bh_i = row / kSmallCTileW, bw_i = row % kSmallCTileW;
    __nv_bfloat16* yb = static_cast<__nv_bfloat16*>(a.y);
    TmaStore ts{&ymap, store_smem + uint32_t(quad) * kStoreWarpBytes, 0, 0, 0, 0, 0u};   // warp = 4 rows x 8 voxels
    const PoolLanes pool_lanes = make_pool_lanes(a.pool_w, a.pool_h, 1, kSmallCTileW, 4, lane);
    const float* bias_e = a.n_pairs > 0 ? nullptr : bias_s;   // with MMAs the bias is in the accumulator already
    const PoolLanes* pool = (a.pool_h * a.pool_w > 1) ? &pool_lanes : nullptr;
    uint32_t j = 0;
    Walk4 k;
    walk4_init(k, blockIdx.x, gridDim.x, a.tiles_w, a.tiles_h, a.g.To);
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++j, walk4_next(k)) {
      const int iw = k.i0, ih = k.i1, to = k.i2, nn = k.i3;
      const uint32_t buf = j & 1u;
      if (!mbar_wait(smem_u32(&bars->tmem_full[buf]), (j >> 1) & 1u, bars, err, 14)) break;
      tc_fence_after();
      const int ho = ih * kSmallCTileH + bh_i, wo = iw * kSmallCTileW + bw_i;
      const bool in_range = ho < a.g.Ho && wo < a.g.Wo;
      // the voxel's linear index is needed only by the direct-store paths and the residual (uniform condition)
      const bool need_vox = a.residual != nullptr || !a.store_tma || (a.n_pad & 31);
      const long long vox = need_vox ? (((long long)nn * a.g.To + to) * a.g.Ho + ho) * a.g.Wo + wo : 0;
      const uint32_t taddr = tmem_base + (uint32_t(quad * 32) << 16) + buf * uint32_t(a.n_pad);
      const __nv_bfloat16* res = (a.residual != nullptr && in_range)
                                     ? static_cast<const __nv_bfloat16*>(a.residual) + vox * a.rcs : nullptr;
      if (a.store_tma) {
        // pooling windows are 1 or 2 wide: the division is a shift
        ts.c1 = (iw * kSmallCTileW) >> (a.pool_w - 1); ts.c2 = (ih * kSmallCTileH + quad * 4) >> (a.pool_h - 1); ts.c3 = to; ts.c4 = nn;
        epilogue_row_tma(taddr, a.n_pad, a.n_pairs > 0, true, in_range, bias_e, a.g.relu, yb + vox * a.g.ycs, 0, a.g.M,
                         lane, ts, res, a.rcs, pool);
      } else {
        epilogue_row(taddr, a.n_pad, a.n_pairs > 0, in_range, bias_e, a.g.relu, yb + vox * a.g.ycs, 0, a.g.M, res, a.rcs);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->tmem_empty[buf]));
    }
    if (lane == 0) tma_store_wait_all();         // all bulk stores done before shared memory goes away
  }

  if (bars->abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000ll) { }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(uint32_t(a.tmem_cols)) : "memory");
  }
}

}  // namespace

size_t smallc_smem_bytes(int n_pairs, int n_pad, int stage_bytes) {
  const size_t w = (size_t(n_pairs + 1) * 2 * n_pad * 16 + 128 + 127) & ~size_t(127);   // + bias operand and ones tile
  const size_t halo = (size_t(stage_bytes) + 127) & ~size_t(127);
  return 1024 + 4 * kStoreWarpBytes + w + kSmallCStages * halo + ((size_t(n_pairs) * 8 + 15) & ~size_t(15)) + sizeof(Barriers) + 16 + size_t(n_pad) * 4;
}

cudaError_t launch_conv_umma_smallc(const SmallCArgs& a_in, const void* xmap, const void* ymap, int sm_count,
                                    cudaStream_t stream) {
  SmallCArgs a = a_in;
  int cols = 32;
  while (cols < 2 * a.n_pad) cols *= 2;
  if (cols > 512) return cudaErrorInvalidValue;
  a.tmem_cols = cols;
  const size_t smem = smallc_smem_bytes(a.n_pairs, a.n_pad, a.n_phases * a.phase_stride);
  if (smem > 227 * 1024) return cudaErrorInvalidValue;
  const long long n_items = (long long)a.g.n * a.g.To * a.tiles_h * a.tiles_w;
  if (n_items <= 0) return cudaSuccess;
  if (a.store_tma && ymap == nullptr) return cudaErrorInvalidValue;
  CUtensorMap xm, ym;
  memcpy(&xm, xmap, sizeof(CUtensorMap));
  memcpy(&ym, ymap ? ymap : xmap, sizeof(CUtensorMap));
  static bool attr_done[kMaxDevices] = {};             // the attributes are per device
  const int dev_idx = current_device_index();
  if (dev_idx < 0) return cudaErrorInvalidDevice;
  if (!attr_done[dev_idx]) {
    cudaError_t e = cudaFuncSetAttribute(conv3d_umma_smallc_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    // ask for the largest shared-memory carve-out: with the default one fewer CTAs fit an SM than the sizes allow
    e = cudaFuncSetAttribute(conv3d_umma_smallc_kernel<0>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    attr_done[dev_idx] = true;
  }
  // Several CTAs per SM (the layer is bound by the latencies of its epilogue): as many as are really resident
  // at once, counted here from the register file, the shared memory (228 KB per SM, 1 KB reserved per CTA)
  // and the 512 TMEM columns of an SM (a CTA that cannot allocate its columns would spin inside
  // tcgen05.alloc), at most four.  (cudaOccupancyMaxActiveBlocksPerMultiprocessor answers 1 for this kernel
  // whatever the sizes, while two and three CTAs per SM measurably run side by side.)  The grid is exactly
  // that many persistent CTAs: surplus CTAs would run as a ragged second wave.
  static int regs_per_thread = 0;
  if (regs_per_thread == 0) {
    cudaFuncAttributes fa;
    regs_per_thread = cudaFuncGetAttributes(&fa, conv3d_umma_smallc_kernel<0>) == cudaSuccess ? fa.numRegs : 128;
  }
  int per_sm = 65536 / (((regs_per_thread + 7) & ~7) * kThreadsUmma);
  const int by_smem = int((228 * 1024) / (smem + 1024));
  if (per_sm > by_smem) per_sm = by_smem;
  if (per_sm > 512 / cols) per_sm = 512 / cols;
  if (per_sm > 4) per_sm = 4;
  if (per_sm < 1) per_sm = 1;
  const long long want = (long long)sm_count * per_sm;
  const int grid = int(n_items < want ? n_items : want);
  LaunchSetup ls(dim3(grid), dim3(kThreadsUmma), smem, stream);
  return cudaLaunchKernelEx(&ls.cfg, conv3d_umma_smallc_kernel<0>, xm, ym, a);
}

}  // namespace rt3d
