// Tensor-core KGS convolution for thin layers: resident weights, one halo tile per output tile.
//
// Layers with few input channels per kernel location and a small weight tensor (the factorised
// 1x3x3 / 3x1x1 convolutions of the early R(2+1)D stages) are bound, in the step-per-location kernels,
// by the per-step barrier hand-shake and by re-reading the same input voxels once per location.
// Here a CTA pair (tcgen05 cta_group::2, as in conv3d_umma_pair_kernel)
//   - loads the whole packed weight tensor of the layer (every kept (location, 64-channel chunk) step,
//     half of the output channels per CTA) into shared memory ONCE, and
//   - stages, per output tile, the input voxels under the tile plus its halo with one TMA box per
//     64-channel chunk (128-byte swizzle); every kernel location is then a shifted window of that
//     staged block: the A descriptor of a step starts (dt*Hh + dh)*Wh + dw rows into the block and walks
//     8-row groups Wh rows apart.  (The swizzle is a function of the shared-memory address, so a start
//     that is not a multiple of 8 rows and a group stride that is not a multiple of 1024 bytes read
//     back exactly what the TMA wrote.)
// One barrier hand-shake per TILE instead of per step, and each input voxel crosses L2 -> SM about
// (halo volume / tile volume) times instead of once per kernel location.
//
// Issue rate.  With so little work per MMA (N <= 144 columns) the issuing thread is the limit, and what
// it costs depends on where the descriptor words come from and on the size of the loop.  Measured on B200
// for a chain of cta_group::2 MMAs (N = 64): 46 clocks per MMA (the hardware floor) when the whole MMA warp
// runs the loop convergently, the words come from kernel parameters (so they live in uniform registers) and
// one elected lane issues; 77..140 clocks when a single lane of a divergent branch builds them from tables in
// registers or shared memory.  Inside this kernel a fully unrolled issue loop is SLOWER than a rolled one:
// the straight-line code of one tile is fetched once per tile while eight epilogue warps run other code, and
// the instruction fetches miss.  Hence: per-tile MMA table in the kernel parameters, convergent MMA warp,
// loop unrolled by two only (about 85 clocks per MMA here).
//
// Epilogue.  A thin layer writes as many bytes as it reads, and one warp needs about 600 clocks per
// 32-column piece; eight epilogue warps (two per TMEM lane quadrant, alternating pieces) keep up with
// the tensor pipe where four do not.
//
// Tile: 8 voxels along w, times 16 (t, h) lines.  The 8-row groups must be evenly spaced in the staged
// block, which holds when the tile is one frame thick (bt = 1) or the kernel is 1 high (Kh = 1).
// Stride 1 only; one bundle (all output channels in one accumulator tile, M <= 256).
#include "kernels.h"
#include "umma_common.cuh"
#include "umma_pair.cuh"
#include "pdl.cuh"

namespace rt3d {
namespace {




constexpr int kThreadsHalo = 320;       // producer warp, MMA warp, 8 epilogue warps

struct HaloBars {
  Barriers b;
  unsigned long long w_full;      // leader: resident weights of both CTAs have landed
};

// Tile walk without divisions: this CTA's tile index advances by a constant number of tiles per item.
struct TileWalk {
  int iw, ih, it, in;             // tile coordinates
  int dw, dh, dt, dn;             // the constant advance, decomposed once
};
__device__ __forceinline__ void walk_init(TileWalk& k, const UmmaArgs& a, int first, int step) {
  int m = first;
  k.iw = m % a.tiles_w; m /= a.tiles_w; k.ih = m % a.tiles_h; m /= a.tiles_h; k.it = m % a.tiles_t; k.in = m / a.tiles_t;
  m = step;
  k.dw = m % a.tiles_w; m /= a.tiles_w; k.dh = m % a.tiles_h; m /= a.tiles_h; k.dt = m % a.tiles_t; k.dn = m / a.tiles_t;
}
__device__ __forceinline__ void walk_next(TileWalk& k, const UmmaArgs& a) {
  k.iw += k.dw; int c = k.iw >= a.tiles_w; k.iw -= c * a.tiles_w;
  k.ih += k.dh + c; c = k.ih >= a.tiles_h; k.ih -= c * a.tiles_h;
  k.it += k.dt + c; c = k.it >= a.tiles_t; k.it -= c * a.tiles_t;
  k.in += k.dn + c;               // beyond tiles_n: the dummy second tile of an odd count (all voxels out of range)
}

template <bool kDense>
__global__ void __launch_bounds__(kThreadsHalo, 1)
conv3d_umma_halo_kernel(const __grid_constant__ CUtensorMap xmap, const __grid_constant__ CUtensorMap wmap_half,
                        const __grid_constant__ CUtensorMap ymap, const HaloArgs h, const int tmem_cols) {
  const UmmaArgs& a = h.u;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  const int n_half = a.n_tile / 2;
  const uint32_t b_bytes = uint32_t(n_half) * 128u;                       // one step's half tile
  const uint32_t w_smem = base;                                            // resident weights
  const uint32_t a_smem = base + uint32_t(h.n_steps) * b_bytes;            // stages of n_chunks planes
  const uint32_t stage_bytes = uint32_t(a.n_chunks) * uint32_t(h.plane_bytes);
  const uint32_t store_smem = a_smem + uint32_t(h.stages) * stage_bytes;   // 8 warps x staging buffers
  unsigned char* tail = smem_raw + (store_smem - raw) + 8 * kStoreWarpBytes;
  HaloBars* hb = reinterpret_cast<HaloBars*>(tail);
  Barriers* bars = &hb->b;
  float* bias_s = align16_f32(hb + 1);
  int32_t* err = a.sched + 2;

  // warp index and CTA rank in forms the compiler can prove uniform (the MMA warp must stay convergent)
  const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;
  const uint32_t rank = blockIdx.x & 1u;          // clusters are pairs of consecutive CTAs of a 1-D grid
  const bool leader = rank == 0;
  const int n_mtiles = a.tiles_n * a.tiles_t * a.tiles_h * a.tiles_w;
  const int n_items = (n_mtiles + 1) / 2;
  const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
  const int box_rows = a.box.bn * a.box.bt * a.box.bh * a.box.bw;

  if (threadIdx.x == 32) {                     // descriptor fetches overlap the rest of the set-up
    tma_prefetch_map(&xmap);
    tma_prefetch_map(&wmap_half);
    tma_prefetch_map(&ymap);
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < h.stages; ++s) {
      mbar_init(smem_u32(&bars->full[s]), 1);
      mbar_init(smem_u32(&bars->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bars->tmem_full[b]), 1);
      mbar_init(smem_u32(&bars->tmem_empty[b]), 16);    // leader: 8 epilogue warps of each CTA
    }
    mbar_init(smem_u32(&hb->w_full), 1);
    bars->abort_flag = 0;
    bars->wait_limit = kWaitCycles;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&bars->tmem_base)), "r"(uint32_t(tmem_cols)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;

  // Everything above touched only shared memory, barriers and TMEM.  The successor may be scheduled now that
  // this CTA holds its TMEM columns (a successor CTA that shared the SM and allocated first could otherwise
  // starve this one while waiting for it); global memory from here on.
  pdl_launch();
  pdl_wait();
  if (warp >= 2) {                               // epilogue warps stage the bias; the other roles start at once
    for (int i = threadIdx.x - 64; i < a.n_tile; i += 256) bias_s[i] = (a.bias != nullptr && i < a.g.M) ? __ldg(a.bias + i) : 0.f;
    epilogue_bar_sync(256);
  }

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      // resident weights: this CTA's half of every step's tile; completion is counted on the leader's barrier
      const uint32_t w_full_local = smem_u32(&hb->w_full);
      const uint32_t w_full_leader = mapa_shared(w_full_local, 0);
      if (leader && h.n_steps > 0) mbar_expect_tx(w_full_local, 2u * uint32_t(h.n_steps) * b_bytes);
      for (int s = 0; s < h.n_steps; ++s)
        tma_load_2d_pair(w_smem + uint32_t(s) * b_bytes, &wmap_half, w_full_leader, 0, s * a.n_tile + int(rank) * n_half);
      int stage = 0;
      uint32_t phase = 0;
      const uint32_t tx_both = 2u * uint32_t(a.n_chunks) * uint32_t(h.halo_rows) * 128u;
      TileWalk k;
      walk_init(k, a, 2 * cluster_id + int(rank), 2 * n_clusters);
      for (int item = cluster_id; item < n_items; item += n_clusters, walk_next(k, a)) {
        const int wq = k.iw * a.box.bw - a.g.pw, hq = k.ih * a.box.bh - a.g.ph, tq = k.it * a.box.bt - a.g.pt;
        const uint32_t full_local = smem_u32(&bars->full[stage]);
        const uint32_t full_leader = mapa_shared(full_local, 0);
        const uint32_t dst = a_smem + uint32_t(stage) * stage_bytes;
        if (!mbar_wait(smem_u32(&bars->empty[stage]), phase ^ 1u, bars, err, 31)) break;
        if (leader) mbar_expect_tx(full_local, tx_both);
        for (int ch = 0; ch < a.n_chunks; ++ch)       // a dummy tile (in >= n) loads only zero fill
          tma_load_5d_pair(dst + uint32_t(ch) * uint32_t(h.plane_bytes), &xmap, full_leader, ch * 64, wq, hq, tq, k.in);
        if (++stage == h.stages) { stage = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA only)
    if (leader) {
      // the whole warp walks the loop (uniform control flow and operands); one elected lane issues
      uint32_t elected;
      asm volatile("{\n.reg .pred p;\nelect.sync _|p, 0xffffffff;\nselp.u32 %0, 1, 0, p;\n}\n" : "=r"(elected));
      const uint32_t idesc = instr_desc_bf16_pair(a.n_tile);
      // high words: stride between 8-row groups (16-byte units), descriptor version 1, 128-byte swizzle
      const uint64_t a_hi = uint64_t(((uint32_t(h.hw) * 128u) >> 4) | (1u << 14) | (2u << 29)) << 32;
      const uint64_t b_hi = uint64_t((1024u >> 4) | (1u << 14) | (2u << 29)) << 32;
      const uint32_t b16 = w_smem >> 4;
      uint32_t j = 0, phase = 0;
      int stage = 0;
      bool ok = h.n_steps == 0 || mbar_wait(smem_u32(&hb->w_full), 0, bars, err, 32);
      for (int item = cluster_id; item < n_items && ok; item += n_clusters, ++j) {
        const uint32_t buf = j & 1u;
        if (!mbar_wait(smem_u32(&bars->tmem_empty[buf]), ((j >> 1) & 1u) ^ 1u, bars, err, 33)) break;
        if (!mbar_wait(smem_u32(&bars->full[stage]), phase, bars, err, 34)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * uint32_t(a.n_tile);
        const uint32_t a16 = (a_smem + uint32_t(stage) * stage_bytes) >> 4;
#pragma unroll 2
        for (int m = 0; m < h.n_mma; ++m) {
          const uint64_t adesc = a_hi | uint64_t(a16 + h.tab[2 * m]);
          const uint64_t bdesc = b_hi | uint64_t(b16 + h.tab[2 * m + 1]);
          if (elected) umma_bf16_pair(d_tmem, adesc, bdesc, idesc, m ? 1u : 0u);
        }
        if (elected) {
          umma_commit_pair(smem_u32(&bars->empty[stage]));
          umma_commit_pair(smem_u32(&bars->tmem_full[buf]));
        }
        if (++stage == h.stages) { stage = 0; phase ^= 1u; }
      }
      __syncwarp();
    }
  } else {
    // ------------------------------------------------------------------ epilogue (both CTAs, 8 warps)
    const int quad = warp & 3;                  // TMEM lane quadrant this warp may read
    const int half = (warp - 2) >> 2;           // 0: even 32-column pieces, 1: odd ones
    const int row = quad * 32 + lane;
    int r = row;
    const int bw_i = r % a.box.bw; r /= a.box.bw;
    const int bh_i = r % a.box.bh; r /= a.box.bh;
    const int bt_i = r % a.box.bt;
    __nv_bfloat16* yb = static_cast<__nv_bfloat16*>(a.y);
    const __nv_bfloat16* rb = static_cast<const __nv_bfloat16*>(a.residual);
    TmaStore ts{&ymap, store_smem + uint32_t(warp - 2) * kStoreWarpBytes, 0, 0, 0, 0, 0u};
    int r0 = quad * 32;
    const int bw_0 = r0 % a.box.bw; r0 /= a.box.bw;
    const int bh_0 = r0 % a.box.bh; r0 /= a.box.bh;
    const int bt_0 = r0 % a.box.bt;
    TileWalk k;
    walk_init(k, a, 2 * cluster_id + int(rank), 2 * n_clusters);
    uint32_t j = 0;
    for (int item = cluster_id; item < n_items; item += n_clusters, ++j, walk_next(k, a)) {
      const uint32_t buf = j & 1u;
      if (!mbar_wait(smem_u32(&bars->tmem_full[buf]), (j >> 1) & 1u, bars, err, 35)) break;
      tc_fence_after();
      const int w0 = k.iw * a.box.bw, h0 = k.ih * a.box.bh, t0 = k.it * a.box.bt;
      const int to = t0 + bt_i, ho = h0 + bh_i, wo = w0 + bw_i;
      const bool in_range = row < box_rows && k.in < a.g.n && to < a.g.To && ho < a.g.Ho && wo < a.g.Wo;
      const long long vox = (((long long)k.in * a.g.To + to) * a.g.Ho + ho) * a.g.Wo + wo;
      const uint32_t taddr = tmem_base + (uint32_t(quad * 32) << 16) + buf * uint32_t(a.n_tile);
      const __nv_bfloat16* res_row = (rb != nullptr && in_range) ? rb + vox * a.rcs : nullptr;
      __nv_bfloat16* dst = yb + vox * a.g.ycs;
      ts.c1 = w0 + bw_0; ts.c2 = h0 + bh_0; ts.c3 = t0 + bt_0; ts.c4 = k.in;
      for (int col = half * 32; col < a.n_tile && col < a.g.M; col += 64) {
        uint32_t v[32];
        const bool wide = col + 32 <= a.n_tile;
        if (h.n_steps > 0) {
          if (wide) tmem_ld32(taddr + col, v);
          else tmem_ld16_into32(taddr + col, v);
        } else {
#pragma unroll
          for (int q = 0; q < 32; ++q) v[q] = 0u;
        }
        const __nv_bfloat16* res = res_row ? res_row + col : nullptr;
        if (wide && a.store_tma) {
          if (quad * 32 < box_rows) epilogue_piece_tma(v, bias_s + col, a.g.relu, col, lane, ts, res, a.rcs - col, nullptr);
        } else if (in_range) {
          if (wide) epilogue_cols<32>(v, bias_s + col, a.g.relu, dst + col, a.g.M - col, res, a.rcs - col);
          else epilogue_cols<16>(v, bias_s + col, a.g.relu, dst + col, a.g.M - col, res, a.rcs - col);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(mapa_shared(smem_u32(&bars->tmem_empty[buf]), 0));
    }
    if (lane == 0) tma_store_wait_all();
  }

  // ---------------------------------------------------------------------- teardown
  if (bars->abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000ll) { }
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(uint32_t(tmem_cols)) : "memory");
  }
}

size_t halo_smem_bytes(const HaloArgs& h) {
  return 1024 + size_t(h.n_steps) * (h.u.n_tile / 2) * 128 + size_t(h.stages) * h.u.n_chunks * h.plane_bytes +
         8 * kStoreWarpBytes + sizeof(HaloBars) + size_t(h.u.n_tile) * 4 + 16;
}

template <bool kDense>
cudaError_t launch_halo_t(const HaloArgs& h, const CUtensorMap& xm, const CUtensorMap& wm, const CUtensorMap& ym,
                          int sm_count, int cols, size_t smem, long long n_items, cudaStream_t stream) {
  static bool attr_done[kMaxDevices] = {};             // the attributes are per device
  const int dev_idx = current_device_index();
  if (dev_idx < 0) return cudaErrorInvalidDevice;
  if (!attr_done[dev_idx]) {
    cudaError_t e = cudaFuncSetAttribute(conv3d_umma_halo_kernel<kDense>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    attr_done[dev_idx] = true;
  }
  long long clusters = sm_count / 2;
  if (clusters > n_items) clusters = n_items;
  LaunchSetup ls(dim3(unsigned(2 * clusters)), dim3(kThreadsHalo), smem, stream, 2);
  return cudaLaunchKernelEx(&ls.cfg, conv3d_umma_halo_kernel<kDense>, xm, wm, ym, h, cols);
}

}  // namespace

// Fills the staging geometry and the MMA table of `h` (h->u.g, box, n_tile, n_chunks, n_steps already set);
// false if the layer does not qualify (weights + two staged blocks beyond shared memory, strides, tile shape,
// more MMAs per tile than the table holds).
bool umma_halo_plan(HaloArgs* h, const int32_t* steps_host) {
  const ConvGeom& g = h->u.g;
  const TileBox& b = h->u.box;
  if (g.st != 1 || g.sh != 1 || g.sw != 1) return false;
  if (b.bn != 1 || b.bw != 8 || b.bt * b.bh != 16) return false;
  if (b.bt > 1 && g.Kh > 1) return false;                 // 8-row groups would not be evenly spaced
  if (h->u.n_bundles != 1 || h->u.n_tile % 16 || h->u.n_tile > 256) return false;
  h->hw = b.bw + g.Kw - 1; h->hh = b.bh + g.Kh - 1; h->ht = b.bt + g.Kt - 1;
  if (h->hw > 256 || h->hh > 256 || h->ht > 256) return false;
  h->halo_rows = h->hw * h->hh * h->ht;
  h->plane_bytes = (h->halo_rows * 128 + 1023) & ~1023;
  const size_t b_bytes = size_t(h->u.n_tile / 2) * 128;
  if (2 * size_t(h->n_steps) * b_bytes > 1000000) return false;        // one barrier counts both CTAs' weight bytes
  // MMA list of one tile: step s contributes 4 K=16 slices, fewer where it is the last, partial chunk
  const int n_chunks = h->u.n_chunks;
  const int last_k16 = (g.c - (n_chunks - 1) * 64 + 15) / 16;
  int m = 0;
  for (int s = 0; s < h->n_steps; ++s) {
    int kt, kh, kw, ch;
    if (steps_host == nullptr) {
      ch = s % n_chunks;
      const int pos = s / n_chunks;
      kw = pos % g.Kw; kh = (pos / g.Kw) % g.Kh; kt = pos / (g.Kw * g.Kh);
    } else {
      const int32_t enc = steps_host[s];
      kt = (enc >> 24) & 63; kh = (enc >> 18) & 63; kw = (enc >> 12) & 63; ch = enc & 4095;
    }
    const int kc = ch == n_chunks - 1 ? last_k16 : 4;
    if (m + kc > kHaloMaxMma) return false;
    const uint32_t a_off = (uint32_t(ch) * uint32_t(h->plane_bytes) + uint32_t((kt * h->hh + kh) * h->hw + kw) * 128u) >> 4;
    const uint32_t b_off = uint32_t(size_t(s) * b_bytes >> 4);
    for (int kk = 0; kk < kc; ++kk, ++m) {
      h->tab[2 * m] = (a_off + 2u * uint32_t(kk)) | (1u << 16);
      h->tab[2 * m + 1] = (b_off + 2u * uint32_t(kk)) | (1u << 16);
    }
  }
  h->n_mma = m;
  for (int q = 2 * m; q < 2 * kHaloMaxMma; ++q) h->tab[q] = 0u;
  for (h->stages = 4; h->stages >= 2; --h->stages)
    if (halo_smem_bytes(*h) <= 227 * 1024) return true;
  return false;
}


cudaError_t launch_conv_umma_halo(const HaloArgs& h, const void* xmap, const void* wmap_half, const void* ymap,
                                  int sm_count, cudaStream_t stream) {
  const UmmaArgs& a = h.u;
  if (h.stages < 2 || a.n_splits != 1 || a.tail_workers != 0 || h.n_mma > kHaloMaxMma) return cudaErrorInvalidValue;
  const size_t smem = halo_smem_bytes(h);
  if (smem > 227 * 1024) return cudaErrorInvalidValue;
  int cols = 32;
  while (cols < 2 * a.n_tile) cols *= 2;
  if (cols > 512) return cudaErrorInvalidValue;
  const long long n_mtiles = (long long)a.tiles_n * a.tiles_t * a.tiles_h * a.tiles_w;
  const long long n_items = (n_mtiles + 1) / 2;
  if (n_items <= 0) return cudaSuccess;
  if (a.store_tma && ymap == nullptr) return cudaErrorInvalidValue;
  CUtensorMap xm, wm, ym;
  memcpy(&xm, xmap, sizeof(CUtensorMap));
  memcpy(&wm, wmap_half, sizeof(CUtensorMap));
  memcpy(&ym, ymap ? ymap : xmap, sizeof(CUtensorMap));
  return a.dense ? launch_halo_t<true>(h, xm, wm, ym, sm_count, cols, smem, n_items, stream)
                 : launch_halo_t<false>(h, xm, wm, ym, sm_count, cols, smem, n_items, stream);
}

}  // namespace rt3d
