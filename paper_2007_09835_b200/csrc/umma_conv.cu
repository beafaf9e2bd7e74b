// Tensor-core KGS convolution for sm_100a: implicit GEMM on tcgen05 with TMA-staged operands
// and fp32 accumulators in tensor memory.
//
// Mapping of the paper's group-matrix view (Section 3) onto the hardware:
//   D[128 output voxels x n_tile output channels] += A[128 x 64] * B[n_tile x 64]^T
// once per K step, where a K step is one kernel location (kt,kh,kw) and one chunk of 64 input
// channels.  A is the input tile shifted by the kernel location (a 5-D TMA box over NDHWC whose
// out-of-range part is zero-filled = the convolution's zero padding); B is the bundle's weight
// tile for that step, pre-arranged at pack time.  For a KGS-pruned layer the producer walks the
// bundle's packed step list, so a (location, chunk) that no kernel group of the bundle keeps
// costs no loads and no MMAs; the dense kernel computes the steps arithmetically.
//
// One persistent CTA per SM, 6 warps: warp 0 = TMA producer, warp 1 = MMA issuer (and TMEM
// owner), warps 2..5 = epilogue (TMEM -> registers -> +bias, ReLU, bf16 -> NDHWC stores).  Two
// accumulator buffers in TMEM let the epilogue of one tile overlap the MMAs of the next.
//
// Layers with few output tiles are split along K: each of `n_splits` CTAs accumulates a slice of
// the step list and writes its fp32 partial tile to a scratch buffer; the CTA that arrives last
// (a counter per output tile and warp) adds the partials in split order, so the result does not depend
// on which CTA that is, applies the epilogue and resets the counter for the next launch.
//
// Every wait on an mbarrier is bounded: on expiry the CTA records an error word in global
// memory, all roles fall through, TMEM is released and the kernel returns.
#include "kernels.h"
#include "umma_common.cuh"
#include "pdl.cuh"

namespace rt3d {
namespace {

struct ItemCoord {
  int bundle, split, tile_id;     // tile_id = bundle * n_mtiles + m-tile
  int n0, t0, h0, w0;             // first output voxel of the box
};

__device__ __forceinline__ ItemCoord decode_item(const UmmaArgs& a, int item, int n_mtiles) {
  ItemCoord c;
  c.split = item % a.n_splits;
  c.tile_id = item / a.n_splits;
  c.bundle = c.tile_id / n_mtiles;
  int mt = c.tile_id - c.bundle * n_mtiles;
  const int iw = mt % a.tiles_w; mt /= a.tiles_w;
  const int ih = mt % a.tiles_h; mt /= a.tiles_h;
  const int it = mt % a.tiles_t; mt /= a.tiles_t;
  c.w0 = iw * a.box.bw; c.h0 = ih * a.box.bh; c.t0 = it * a.box.bt; c.n0 = mt * a.box.bn;
  return c;
}

// Slice of the bundle's step list owned by this item: global index of its first step, number of
// steps, and the index of the first step inside the bundle's list.
template <bool kDense>
__device__ __forceinline__ void item_steps(const UmmaArgs& a, const ItemCoord& c, int& s_begin, int& nsteps, int& local0) {
  const int base = kDense ? c.bundle * a.steps_dense : a.step_ptr[c.bundle];
  const int total = kDense ? a.steps_dense : a.step_ptr[c.bundle + 1] - base;
  local0 = int((long long)total * c.split / a.n_splits);
  const int hi = int((long long)total * (c.split + 1) / a.n_splits);
  s_begin = base + local0;
  nsteps = hi - local0;
}

// Sum of the partials of all splits (in split order, two splits' loads in flight at a time) + epilogue
// for one output voxel; `part0` points at this thread's row of column 0 of split 0.
template <int NC>
__device__ __forceinline__ void reduce_partial_cols(const float* part0, size_t split_stride, int n_splits,
                                                    const float* bias_s, int relu, __nv_bfloat16* dst, int valid,
                                                    const __nv_bfloat16* res, int res_avail) {
  float acc[NC];
#pragma unroll
  for (int q = 0; q < NC; ++q) acc[q] = 0.f;
  int s = 0;
  for (; s + 1 < n_splits; s += 2) {
    float4 t0[NC / 4], t1[NC / 4];
    const float* p0 = part0 + size_t(s) * split_stride;
    const float* p1 = p0 + split_stride;
#pragma unroll
    for (int q = 0; q < NC / 4; ++q) {
      t0[q] = __ldcg(reinterpret_cast<const float4*>(p0 + size_t(q) * 512));
      t1[q] = __ldcg(reinterpret_cast<const float4*>(p1 + size_t(q) * 512));
    }
#pragma unroll
    for (int q = 0; q < NC / 4; ++q) {
      acc[4 * q] = (acc[4 * q] + t0[q].x) + t1[q].x;
      acc[4 * q + 1] = (acc[4 * q + 1] + t0[q].y) + t1[q].y;
      acc[4 * q + 2] = (acc[4 * q + 2] + t0[q].z) + t1[q].z;
      acc[4 * q + 3] = (acc[4 * q + 3] + t0[q].w) + t1[q].w;
    }
  }
  if (s < n_splits) {
    const float* p0 = part0 + size_t(s) * split_stride;
#pragma unroll
    for (int q = 0; q < NC / 4; ++q) {
      const float4 t = __ldcg(reinterpret_cast<const float4*>(p0 + size_t(q) * 512));
      acc[4 * q] += t.x; acc[4 * q + 1] += t.y; acc[4 * q + 2] += t.z; acc[4 * q + 3] += t.w;
    }
  }
  uint32_t v[NC];
#pragma unroll
  for (int q = 0; q < NC; ++q) v[q] = __float_as_uint(acc[q]);
  epilogue_cols<NC>(v, bias_s, relu, dst, valid, res, res_avail);
}

__device__ __forceinline__ void reduce_partial_row(const float* part0, size_t split_stride, int n_splits, int n_cols,
                                                   bool in_range, const float* bias_s, int relu, __nv_bfloat16* dst,
                                                   int m_base, int M, const __nv_bfloat16* res_row, int res_left,
                                                   int col0 = 0, int col_step = 32) {
  if (!in_range) return;
  for (int col = col0; col < n_cols; col += col_step) {
    const int m0 = m_base + col;
    if (m0 >= M) break;
    const float* p = part0 + size_t(col) * 128;
    const __nv_bfloat16* res = res_row ? res_row + col : nullptr;
    if (col + 32 <= n_cols) reduce_partial_cols<32>(p, split_stride, n_splits, bias_s + m0, relu, dst + col, M - m0, res, res_left - col);
    else reduce_partial_cols<16>(p, split_stride, n_splits, bias_s + m0, relu, dst + col, M - m0, res, res_left - col);
  }
}

// kCps: K steps per pipeline stage (and per barrier hand-shake): 1, or 2 for narrow bundles, where the
// issuing thread's hand-shake, not the tensor pipe, bounds a step.
// Threads of the single-CTA kernel: producer warp, MMA warp, two sets of four epilogue warps.  The second set
// works only on plain (unsplit, unpooled) calls, where it takes the odd 32-column pieces of a tile and stores
// them directly: most layers that run here give a CTA a single tile, so the epilogue is a pure latency chain
// of up to eight pieces per warp, and sharing it between two warps per lane quadrant halves the tail of the
// layer.
constexpr int kThreadsSingle = 320;

template <bool kDense, int kCps>
__global__ void __launch_bounds__(kThreadsSingle, 1)
conv3d_umma_kernel(const __grid_constant__ CUtensorMap xmap, const __grid_constant__ CUtensorMap wmap,
                   const __grid_constant__ CUtensorMap ymap, const UmmaArgs a, const int stages, const int tmem_cols) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles_base = (raw + 1023u) & ~1023u;            // operand tiles need 1024-byte alignment
  const uint32_t b_bytes = uint32_t(a.n_tile) * 128u;
  const uint32_t chunk_bytes = kABytes + b_bytes;
  const uint32_t stage_bytes = kCps * chunk_bytes;
  const uint32_t store_smem = tiles_base + uint32_t(stages) * stage_bytes;     // 4 warps x 2 staging buffers
  Barriers* bars = reinterpret_cast<Barriers*>(smem_raw + (tiles_base - raw) + size_t(stages) * stage_bytes +
                                               4 * kStoreWarpBytes);
  float* bias_s = align16_f32(bars + 1);                            // bias of all bundles (zeros if none), padded
  int32_t* err = a.sched + 2;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_mtiles = a.tiles_n * a.tiles_t * a.tiles_h * a.tiles_w;
  const int n_items = n_mtiles * a.n_bundles * a.n_splits;
  const int box_rows = a.box.bn * a.box.bt * a.box.bh * a.box.bw;
  const bool two_sets = a.n_splits == 1 && a.pool_t * a.pool_h * a.pool_w == 1;   // both epilogue warp sets work on a plain tile
  const bool split_sets = a.n_splits > 1;      // and on a K split: each takes every other 32-column piece of the share and of the sum

  if (threadIdx.x == 32) {                     // descriptor fetches overlap the rest of the set-up
    tma_prefetch_map(&xmap);
    tma_prefetch_map(&wmap);
    tma_prefetch_map(&ymap);
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(smem_u32(&bars->full[s]), 1);
      mbar_init(smem_u32(&bars->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bars->tmem_full[b]), 1);
      mbar_init(smem_u32(&bars->tmem_empty[b]), (two_sets || split_sets) ? 8 : 4);
    }
    bars->abort_flag = 0;
    bars->wait_limit = a.wait_cycles > 0 ? a.wait_cycles : kWaitCycles;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&bars->tmem_base)), "r"(uint32_t(tmem_cols)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;

  // Everything above touched only shared memory, barriers and TMEM.  The successor may be scheduled now that
  // this CTA holds its TMEM columns (a successor CTA that shared the SM and allocated first could otherwise
  // starve this one while waiting for it).
  pdl_launch();
  // Work that needs none of the predecessor's results is done while the CTA still waits for it: every thread
  // decodes the CTA's first item (a chain of integer divisions: half a microsecond in the single producer
  // thread) and reads that item's bounds in the step list, the producer also its first encoded steps.  The
  // step lists belong to the packed handle, which no kernel writes; after the wait these reads are two
  // dependent trips to L2 in front of the first TMA request of a layer that takes 4 to 10 us in all.
  // (Only registers survive the wait: a plain prefetch into L1 did not help.)
  constexpr int kPreSteps = 4;
  ItemCoord pre_c = {};
  int pre_sbegin = 0, pre_nsteps = 0, pre_local0 = 0, pre_enc[kPreSteps] = {0, 0, 0, 0};
  if (int(blockIdx.x) < n_items) {
    pre_c = decode_item(a, blockIdx.x, n_mtiles);
    item_steps<kDense>(a, pre_c, pre_sbegin, pre_nsteps, pre_local0);
    if (!kDense && threadIdx.x == 0) {
#pragma unroll
      for (int q = 0; q < kPreSteps; ++q)
        if (q < pre_nsteps) pre_enc[q] = __ldg(a.steps + pre_sbegin + q);
    }
  }
  pdl_wait();                                    // predecessor complete: activations, bias, residual are visible
  if (warp >= 2) {                               // epilogue warps stage the bias; the other roles start at once
    for (int i = threadIdx.x - 64; i < a.n_bundles * a.n_tile; i += 256)
      bias_s[i] = (a.bias != nullptr && i < a.g.M) ? __ldg(a.bias + i) : 0.f;
    epilogue_bar_sync(256);
  }

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      const uint32_t tx_bytes = uint32_t(box_rows) * 128u + b_bytes;
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
        const bool first_item = item == int(blockIdx.x);                // decoded before the dependency wait
        const ItemCoord c = first_item ? pre_c : decode_item(a, item, n_mtiles);
        int s_begin = pre_sbegin, nsteps = pre_nsteps, local0 = pre_local0;
        if (!first_item) item_steps<kDense>(a, c, s_begin, nsteps, local0);
        const int wq = c.w0 * a.g.sw - a.g.pw, hq = c.h0 * a.g.sh - a.g.ph, tq = c.t0 * a.g.st - a.g.pt;
        // Everything a step needs is computed (dense) or fetched one step ahead (indexed) before the
        // wait on the stage, so a freed stage is re-armed without further latency.
        int kt = 0, kh = 0, kw = 0, ch = 0;
        if (kDense) {
          ch = local0 % a.n_chunks;
          const int pos = local0 / a.n_chunks;
          kw = pos % a.g.Kw; kh = (pos / a.g.Kw) % a.g.Kh; kt = pos / (a.g.Kw * a.g.Kh);
        }
        int wrow = s_begin * a.n_tile;
        for (int i = 0; i < nsteps; i += kCps) {
          const int nload = nsteps - i < kCps ? nsteps - i : kCps;
          int c_ch[kCps], c_w[kCps], c_h[kCps], c_t[kCps];
#pragma unroll
          for (int q = 0; q < kCps; ++q) {
            if (q >= nload) break;
            if (kDense) {
              c_ch[q] = ch * 64; c_w[q] = wq + kw; c_h[q] = hq + kh; c_t[q] = tq + kt;
              if (++ch == a.n_chunks) { ch = 0; if (++kw == a.g.Kw) { kw = 0; if (++kh == a.g.Kh) { kh = 0; ++kt; } } }
            } else {
              int enc;
              if (first_item && i + q < kPreSteps) {             // kDense is false here
                enc = pre_enc[0];
#pragma unroll
                for (int e = 1; e < kPreSteps; ++e) enc = (i + q == e) ? pre_enc[e] : enc;
              } else {
                enc = __ldg(a.steps + s_begin + i + q);
              }
              c_t[q] = tq + ((enc >> 24) & 63); c_h[q] = hq + ((enc >> 18) & 63); c_w[q] = wq + ((enc >> 12) & 63);
              c_ch[q] = (enc & 4095) * 64;
            }
          }
          const uint32_t full = smem_u32(&bars->full[stage]);
          const uint32_t s_dst = tiles_base + stage * stage_bytes;
          if (!mbar_wait(smem_u32(&bars->empty[stage]), phase ^ 1u, bars, err, 1)) { ok = false; break; }
          mbar_expect_tx(full, tx_bytes * uint32_t(nload));
          // test hook: the loads of this CTA's very last stage are never issued, so that the MMA warp's wait on
          // them runs into the (shortened) limit and the error path can be exercised without any fault
          if (a.debug_drop_last_load && i + kCps >= nsteps && item + int(gridDim.x) >= n_items) continue;
#pragma unroll
          for (int q = 0; q < kCps; ++q) {
            if (q >= nload) break;
            const uint32_t a_dst = s_dst + q * chunk_bytes;
            tma_load_5d(a_dst, &xmap, full, c_ch[q], c_w[q], c_h[q], c_t[q], c.n0);
            tma_load_2d(a_dst + kABytes, &wmap, full, 0, wrow);
            wrow += a.n_tile;
          }
          if (++stage == stages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = instr_desc_bf16(a.n_tile);
      uint32_t j = 0, phase = 0;
      int stage = 0;
      bool ok = true, ready = false;
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++j) {
        const bool first_item = item == int(blockIdx.x);
        const ItemCoord c = first_item ? pre_c : decode_item(a, item, n_mtiles);
        int s_begin = pre_sbegin, nsteps = pre_nsteps, local0 = pre_local0;
        if (!first_item) item_steps<kDense>(a, c, s_begin, nsteps, local0);
        const uint32_t buf = j & 1u;
        if (!mbar_wait(smem_u32(&bars->tmem_empty[buf]), ((j >> 1) & 1u) ^ 1u, bars, err, 2)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * uint32_t(a.n_tile);
        for (int i = 0; i < nsteps; i += kCps) {
          const int nload = nsteps - i < kCps ? nsteps - i : kCps;
          if (!ready && !mbar_wait(smem_u32(&bars->full[stage]), phase, bars, err, 3)) { ok = false; break; }
          // poll the next stage's barrier now: its answer arrives while this stage's MMAs are issued
          const int stage_n = stage + 1 == stages ? 0 : stage + 1;
          const uint32_t phase_n = stage + 1 == stages ? phase ^ 1u : phase;
          ready = mbar_try_wait(smem_u32(&bars->full[stage_n]), phase_n);
          tc_fence_after();
#pragma unroll
          for (int q = 0; q < kCps; ++q) {
            if (q >= nload) break;
            const uint32_t a_addr = tiles_base + stage * stage_bytes + q * chunk_bytes;
            const uint64_t adesc = smem_desc_sw128(a_addr);
            const uint64_t bdesc = smem_desc_sw128(a_addr + kABytes);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)    // 4 x K=16 per 64-channel chunk: +32 bytes = +2 in descriptor units
              umma_bf16(d_tmem, adesc + 2 * kk, bdesc + 2 * kk, idesc, (i | q | kk) ? 1u : 0u);
          }
          umma_commit(smem_u32(&bars->empty[stage]));
          stage = stage_n; phase = phase_n;
        }
        if (!ok) break;
        if (nsteps > 0) umma_commit(smem_u32(&bars->tmem_full[buf]));
        else mbar_arrive(smem_u32(&bars->tmem_full[buf]));
      }
    }
  } else if (warp < 6 || two_sets || split_sets) {
    // ------------------------------------------------------------------ epilogue (warps 2..5, and 6..9 on plain calls)
    const int quad = warp & 3;                 // TMEM lane quadrant this warp may read
    const int half = (warp - 2) >> 2;          // second set: odd pieces, direct stores
    const int row = quad * 32 + lane;          // voxel row inside the box
    int r = row;
    const int bw_i = r % a.box.bw; r /= a.box.bw;
    const int bh_i = r % a.box.bh; r /= a.box.bh;
    const int bt_i = r % a.box.bt; r /= a.box.bt;
    const int bn_i = r;
    __nv_bfloat16* yb = static_cast<__nv_bfloat16*>(a.y);
    const __nv_bfloat16* rb = static_cast<const __nv_bfloat16*>(a.residual);
    TmaStore ts{&ymap, store_smem + uint32_t(quad) * kStoreWarpBytes, 0, 0, 0, 0, 0u};
    const PoolLanes pool_lanes = make_pool_lanes(a.pool_w, a.pool_h, a.pool_t, a.sbw, a.sbh, lane);
    const PoolLanes* pool = (a.pool_t * a.pool_h * a.pool_w > 1) ? &pool_lanes : nullptr;
    int r0 = quad * 32;                        // coordinates of the warp's first row inside the box
    const int bw_0 = r0 % a.box.bw; r0 /= a.box.bw;
    const int bh_0 = r0 % a.box.bh; r0 /= a.box.bh;
    const int bt_0 = r0 % a.box.bt; r0 /= a.box.bt;
    const int bn_0 = r0;
    const size_t part_tile = size_t(128) * a.n_tile;       // floats per partial tile
    uint32_t j = 0;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++j) {
      const bool first_item = item == int(blockIdx.x);
      const ItemCoord c = first_item ? pre_c : decode_item(a, item, n_mtiles);
      int s_begin = pre_sbegin, nsteps = pre_nsteps, local0 = pre_local0;
      if (!first_item) item_steps<kDense>(a, c, s_begin, nsteps, local0);
      const uint32_t buf = j & 1u;
      if (!mbar_wait(smem_u32(&bars->tmem_full[buf]), (j >> 1) & 1u, bars, err, 4)) break;
      tc_fence_after();
      const int nn = c.n0 + bn_i, to = c.t0 + bt_i, ho = c.h0 + bh_i, wo = c.w0 + bw_i;
      const bool in_range = row < box_rows && nn < a.g.n && to < a.g.To && ho < a.g.Ho && wo < a.g.Wo;
      const long long vox = (((long long)nn * a.g.To + to) * a.g.Ho + ho) * a.g.Wo + wo;
      const int m_base = c.bundle * a.n_tile;
      const uint32_t taddr = tmem_base + (uint32_t(quad * 32) << 16) + buf * uint32_t(a.n_tile);
      __nv_bfloat16* dst = yb + vox * a.g.ycs + m_base;
      const __nv_bfloat16* res = (rb != nullptr && in_range) ? rb + vox * a.rcs + m_base : nullptr;
      const int res_left = a.rcs - m_base;
      if (two_sets) {
        ts.c1 = c.w0 + bw_0; ts.c2 = c.h0 + bh_0; ts.c3 = c.t0 + bt_0; ts.c4 = c.n0 + bn_0;
        for (int col = half * 32; col < a.n_tile; col += 64) {
          const int m0 = m_base + col;
          if (m0 >= a.g.M) break;
          uint32_t v[32];
          const bool wide = col + 32 <= a.n_tile;
          if (nsteps > 0) {
            if (wide) tmem_ld32(taddr + col, v);
            else tmem_ld16_into32(taddr + col, v);
          } else {
#pragma unroll
            for (int q = 0; q < 32; ++q) v[q] = 0u;
          }
          const __nv_bfloat16* rp = res ? res + col : nullptr;
          if (half == 0 && wide && a.store_tma) {
            if (quad * 32 < box_rows) epilogue_piece_tma(v, bias_s + m0, a.g.relu, m0, lane, ts, rp, res_left - col, nullptr);
          } else if (in_range) {
            if (wide) epilogue_cols<32>(v, bias_s + m0, a.g.relu, dst + col, a.g.M - m0, rp, res_left - col);
            else epilogue_cols<16>(v, bias_s + m0, a.g.relu, dst + col, a.g.M - m0, rp, res_left - col);
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars->tmem_empty[buf]));
      } else if (a.n_splits == 1) {
        if (a.store_tma) {
          ts.c1 = (c.w0 + bw_0) / a.pool_w; ts.c2 = (c.h0 + bh_0) / a.pool_h; ts.c3 = (c.t0 + bt_0) / a.pool_t; ts.c4 = c.n0 + bn_0;
          epilogue_row_tma(taddr, a.n_tile, nsteps > 0, quad * 32 < box_rows, in_range, bias_s, a.g.relu, dst, m_base,
                           a.g.M, lane, ts, res, res_left, pool);
        } else {
          epilogue_row(taddr, a.n_tile, nsteps > 0, in_range, bias_s, a.g.relu, dst, m_base, a.g.M, res, res_left);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars->tmem_empty[buf]));
      } else {
        float* tile_part = a.scratch + size_t(c.tile_id) * a.n_splits * part_tile;
        store_partial_row(taddr, a.n_tile, nsteps > 0, tile_part + size_t(c.split) * part_tile + row * kPartRow, half * 32, 64);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars->tmem_empty[buf]));    // accumulator consumed: MMAs may go on
        // Each warp owns 32 rows of the tile in every split, so the hand-over is per warp: fence the
        // partial, count this warp in, and the warp that counts last reduces those 32 rows.
        __threadfence();
        __syncwarp();
        int last = 0;
        if (lane == 0) last = atomicAdd(a.counters + c.tile_id * 8 + half * 4 + quad, 1) == a.n_splits - 1;
        last = __shfl_sync(0xffffffffu, last, 0);
        if (last) {
          __threadfence();
          reduce_partial_row(tile_part + row * kPartRow, part_tile, a.n_splits, a.n_tile, in_range, bias_s,
                             a.g.relu, dst, m_base, a.g.M, res, res_left, half * 32, 64);
          __syncwarp();
          if (lane == 0) a.counters[c.tile_id * 8 + half * 4 + quad] = 0;   // ready for the next launch
        }
      }
    }
    if (lane == 0) tma_store_wait_all();         // all bulk stores done before shared memory goes away
  }

  // ---------------------------------------------------------------------- teardown
  if (bars->abort_flag) {
    // error path: give asynchronous copies / MMAs still in flight time to land before TMEM goes away
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000ll) { }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(uint32_t(tmem_cols)) : "memory");
  }
}

int pick_cps_single(int n_tile) { return n_tile <= 128 ? 2 : 1; }

int pick_stages(int n_tile) {
  const size_t stage = pick_cps_single(n_tile) * (kABytes + size_t(n_tile) * 128);
  const int s = int(kSmemBudget / stage);
  return s > kMaxStages ? kMaxStages : s;
}

template <bool kDense, int kCps>
cudaError_t launch_single_t(const UmmaArgs& a, const CUtensorMap& xm, const CUtensorMap& wm, const CUtensorMap& ym, int grid,
                            size_t smem, int stages, int cols, cudaStream_t stream) {
  static bool attr_done[kMaxDevices] = {};             // the attribute is per device
  const int dev = current_device_index();
  if (dev < 0) return cudaErrorInvalidDevice;
  if (!attr_done[dev]) {
    cudaError_t e = cudaFuncSetAttribute(conv3d_umma_kernel<kDense, kCps>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    attr_done[dev] = true;
  }
  LaunchSetup ls(dim3(grid), dim3(kThreadsSingle), smem, stream);
  return cudaLaunchKernelEx(&ls.cfg, conv3d_umma_kernel<kDense, kCps>, xm, wm, ym, a, stages, cols);
}

}  // namespace

size_t umma_smem_bytes(int n_tile, int n_bundles) {
  return size_t(pick_stages(n_tile)) * pick_cps_single(n_tile) * (kABytes + size_t(n_tile) * 128) + 1024 + 4 * kStoreWarpBytes + sizeof(Barriers) + 16 +
         size_t(n_tile) * n_bundles * 4;
}

cudaError_t launch_conv_umma(const UmmaArgs& a, const void* xmap, const void* wmap, const void* ymap, int sm_count,
                             cudaStream_t stream) {
  const int stages = pick_stages(a.n_tile);
  if (stages < 2) return cudaErrorInvalidValue;
  const size_t smem = umma_smem_bytes(a.n_tile, a.n_bundles);
  if (smem > 227 * 1024) return cudaErrorInvalidValue;
  int cols = 32;
  while (cols < 2 * a.n_tile) cols *= 2;
  if (cols > 512) return cudaErrorInvalidValue;
  if (a.n_splits < 1 || (a.n_splits > 1 && (a.scratch == nullptr || a.counters == nullptr))) return cudaErrorInvalidValue;
  const long long n_items = (long long)a.tiles_n * a.tiles_t * a.tiles_h * a.tiles_w * a.n_bundles * a.n_splits;
  if (n_items <= 0) return cudaSuccess;
  const int grid = int(n_items < sm_count ? n_items : sm_count);
  if (a.store_tma && ymap == nullptr) return cudaErrorInvalidValue;
  CUtensorMap xm, wm, ym;
  memcpy(&xm, xmap, sizeof(CUtensorMap));
  memcpy(&wm, wmap, sizeof(CUtensorMap));
  memcpy(&ym, ymap ? ymap : xmap, sizeof(CUtensorMap));
  const bool two = pick_cps_single(a.n_tile) == 2;
  if (a.dense) return two ? launch_single_t<true, 2>(a, xm, wm, ym, grid, smem, stages, cols, stream)
                          : launch_single_t<true, 1>(a, xm, wm, ym, grid, smem, stages, cols, stream);
  return two ? launch_single_t<false, 2>(a, xm, wm, ym, grid, smem, stages, cols, stream)
             : launch_single_t<false, 1>(a, xm, wm, ym, grid, smem, stages, cols, stream);
}

}  // namespace rt3d
