// Tensor-core KGS convolution on CTA pairs (tcgen05 cta_group::2).
//
// Same implicit GEMM as conv3d_umma_kernel, but two CTAs on neighbouring SMs form a cluster and
// work on two output tiles of the same bundle at once: one MMA instruction, issued by a single
// thread of the leader CTA, multiplies a 256-row A operand (128 voxels from each CTA's shared
// memory) by the bundle's B tile, of which each CTA stages only half (n_tile/2 rows).  Per SM this
// halves the weight bytes pulled from L2 per step and the per-step cost of the issuing thread,
// which bound the single-CTA kernel.  Accumulators stay per CTA (128 TMEM lanes each), so the
// epilogue is unchanged.
//
// Synchronisation: both producers wait on their own `empty[s]` (released for both CTAs by one
// multicast commit), both send their loads' completion bytes to the leader's `full[s]`; the
// leader's MMA thread waits there, issues, and commits to `empty[s]` / `tmem_full[b]` of both CTAs
// (bundles up to 128 wide: two MMA threads, which take the stages by parity and accumulate into
// two accumulators that the epilogue adds); the epilogue warps of both CTAs release the
// accumulator on the leader's `tmem_empty[b]`.  All waits are bounded as in the single-CTA kernel.
#include "kernels.h"
#include "umma_common.cuh"
#include "umma_pair.cuh"
#include "pdl.cuh"

namespace rt3d {
namespace {

// Work of one CTA pair: whole items dealt round-robin.  With the tail split, the items that would not
// fill a last round are instead laid end to end as one line of K-step groups, cut into `tail_workers`
// equal ranges and done FIRST: an item is then computed by up to a few pairs, each leaving its fp32
// partial tile in global scratch.  The pair that holds the item's first steps owns it: its own share
// stays in tensor memory, and while its tensor pipe is already busy with the first whole item, its
// epilogue warps add the other pairs' partial tiles to it in a fixed order and write the output.
struct TailSeg { int item, g0, g1, part, nparts; };
constexpr int kMaxTailSeg = 6;
constexpr int kMaxBundles = 64;
constexpr int kMaxTail = 128;  // left-over items are fewer than the pairs of the grid (at most 74)
struct TailWork {
  int n_full;                 // whole items of this pair: item = cluster_id + k * n_clusters
  int n_seg;
  int t_first;                // first left-over item this pair has a share of
  TailSeg seg[kMaxTailSeg];
  int g[kMaxTail];            // step groups of each left-over item
  int sp[kMaxBundles + 1];    // the layout's per-bundle step offsets (and group offsets, t-grouped variant): the three
  int gp[kMaxBundles + 1];    // roles read them once per item, and two dependent global loads per item showed on short items
};
struct Work { int item, g0, g1, part, nparts; };

// Order of a pair's work: its tail segments first (the first one is a share of a tile another pair owns and is
// wanted early by that pair), then its whole items.
__device__ __forceinline__ Work get_work(const TailWork* tw, int wi, int cluster_id, int n_clusters) {
  if (wi >= tw->n_seg) return Work{cluster_id + (wi - tw->n_seg) * n_clusters, 0, 1 << 28, 0, 1};
  const TailSeg& g = tw->seg[wi];
  return Work{g.item, g.g0, g.g1, g.part, g.nparts};
}

// Threads of a CTA: producer warp, MMA warp, two sets of four epilogue warps, and a second MMA warp (warp 10) that
// only narrow bundles use.  The second epilogue set (warps 6..9) takes the
// odd 32-column pieces of every tile, so that a tile with few K steps (a heavily pruned layer with tall kernel
// groups, a 1x1x1 or 1x3x3 layer) is not bound by its epilogue: four warps need about 15 k clocks for a 128 x 256
// tile, as long as 30 K steps.  Shares and fix-ups of split tiles are divided between the sets the same way.
constexpr int kThreadsPair = 352;

// t-grouped variant: step and group tables (all bundles together) live in shared memory, up to this many steps.
constexpr int kTsTable = 2048;

// kCps: K steps per pipeline stage (and per barrier hand-shake): 1, or 2 for narrow bundles.
// kTS: t-grouped layout.  A pipeline stage then holds ONE input tile that is Kt - 1 frames deeper and the weight
// tiles of the up to Kt steps (kt = 0 .. Kt-1 at one (kh, kw, chunk)) that read it, each through a descriptor that
// starts kt frames into the tile: a third as many input bytes per step cross from L2, so more steps are in flight
// in the same shared memory (a 64 -> 128 channel 3x3x3 layer was bound by that, at 387 clocks per step against 256).
template <bool kDense, int kCps, bool kTS, bool kDual>
__global__ void __launch_bounds__(kThreadsPair, 1)
conv3d_umma_pair_kernel(const __grid_constant__ CUtensorMap xmap, const __grid_constant__ CUtensorMap wmap_half,
                        const __grid_constant__ CUtensorMap ymap, const UmmaArgs a, const int stages, const int tmem_cols) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles_base = (raw + 1023u) & ~1023u;
  const int n_half = a.n_tile / 2;
  const uint32_t b_bytes = uint32_t(n_half) * 128u;             // this CTA's half of the B tile
  const uint32_t chunk_bytes = kABytes + b_bytes;
  const uint32_t ts_a_slot = (uint32_t(a.ts_a_bytes) + 1023u) & ~1023u;
  const uint32_t ts_a_all = ts_a_slot * uint32_t(a.ts_phases);       // one deeper tile per phase of the temporal stride
  const uint32_t stage_bytes = kTS ? ts_a_all + uint32_t(a.g.Kt) * b_bytes : kCps * chunk_bytes;
  const uint32_t store_smem = tiles_base + uint32_t(stages) * stage_bytes;     // 4 warps x 2 staging buffers
  Barriers* bars = reinterpret_cast<Barriers*>(smem_raw + (tiles_base - raw) + size_t(stages) * stage_bytes +
                                               4 * kStoreWarpBytes);
  TailWork* tw = reinterpret_cast<TailWork*>(bars + 1);
  float* bias_s = align16_f32(tw + 1);
  int32_t* steps_s = reinterpret_cast<int32_t*>(bias_s + a.n_bundles * a.n_tile);   // kTS only: steps, then group starts
  int32_t* grp_s = steps_s + a.ts_table;
  uint32_t* aoff_s = reinterpret_cast<uint32_t*>(grp_s + a.ts_table + 8);   // per step: where its A operand starts in the stage
  const int ts_groups_dense = a.g.Kh * a.g.Kw * a.n_chunks;
  int32_t* err = a.sched + 2;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  const int n_mtiles = a.tiles_n * a.tiles_t * a.tiles_h * a.tiles_w;
  const int pairs_per_bundle = (n_mtiles + 1) / 2;
  const int n_items = pairs_per_bundle * a.n_bundles;
  const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
  const int box_rows = a.box.bn * a.box.bt * a.box.bh * a.box.bw;
  constexpr int epi_sets = 2;
  // Narrow bundles (kDual, N <= 128): one thread cannot issue MMAs and run the barrier hand-shakes as fast as
  // the tensor pipe executes them, so two threads issue alternate step groups, each into its own accumulator
  // (2 buffers x 2 x N <= 512 columns); the epilogue adds the two.  Fixed order, so results stay repeatable.
  constexpr int kIss = kDual ? 2 : 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(smem_u32(&bars->full[s]), 1);     // leader: its producer's arrive + both CTAs' bytes
      mbar_init(smem_u32(&bars->empty[s]), 1);    // multicast commit
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bars->tmem_full[b]), kIss);  // multicast commit of every issuing thread
      mbar_init(smem_u32(&bars->tmem_empty[b]), uint32_t(8 * epi_sets));   // leader: the working epilogue warps of both CTAs
    }
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
  cluster_sync_all();              // barriers of both CTAs are initialised before anyone signals them
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;

  // Everything above touched only shared memory, barriers and TMEM.  The successor may be scheduled now that
  // this CTA holds its TMEM columns (a successor CTA that shared the SM and allocated first could otherwise
  // starve this one while waiting for it); global memory from here on.
  pdl_launch();
  if (!kDense)
    for (int i = threadIdx.x; i <= a.n_bundles; i += blockDim.x) {
      tw->sp[i] = __ldg(a.step_ptr + i);
      if (kTS) tw->gp[i] = __ldg(a.grp_ptr + i);
    }
  // The step counts belong to the packed layout, which only host uploads write, never a kernel: the work list
  // is built before the wait on the predecessor grid (the caller's tensors, bias included, are read after it).
  // This pair's work list.  The tail split's segment table is built by one thread per left-over item (a lone
  // thread walking the items, two dependent global loads each, took longer than the split saved).
  if (threadIdx.x == 0) {
    tw->n_seg = 0;
    tw->t_first = 1 << 30;
    const int rounds = n_items / n_clusters;
    tw->n_full = a.tail_workers == 0 ? (cluster_id < n_items ? (n_items - cluster_id + n_clusters - 1) / n_clusters : 0)
                                     : rounds;
  }
  if (a.tail_workers > 0) {                                 // uniform over the grid
    const int first_tail = (n_items / n_clusters) * n_clusters, n_tail = n_items - first_tail;   // n_tail < kMaxTail
    const int t = threadIdx.x;
    if (t < n_tail) {
      const int b = (first_tail + t) / pairs_per_bundle;
      if (kTS) {
        tw->g[t] = kDense ? ts_groups_dense : __ldg(a.grp_ptr + b + 1) - __ldg(a.grp_ptr + b);
      } else {
        const int ns = kDense ? a.steps_dense : __ldg(a.step_ptr + b + 1) - __ldg(a.step_ptr + b);
        tw->g[t] = (ns + kCps - 1) / kCps;
      }
    }
    __syncthreads();
    bool mine = false;
    long long pre = 0, lo = 0, hi = 0, total = 0;
    int G = 0;
    if (t < n_tail && cluster_id < a.tail_workers) {
      for (int u = 0; u < n_tail; ++u) {
        const int gu = tw->g[u];
        if (u < t) pre += gu;
        total += gu;
      }
      G = tw->g[t];
      const long long W = a.tail_workers;
      lo = cluster_id * total / W; hi = (cluster_id + 1) * total / W;
      mine = pre + G > lo && pre < hi;
      if (mine) atomicMin(&tw->t_first, t);
    }
    __syncthreads();
    if (mine && t - tw->t_first < kMaxTailSeg) {
      const long long W = a.tail_workers;
      TailSeg& sg = tw->seg[t - tw->t_first];
      sg.item = first_tail + t;
      sg.g0 = int((lo > pre ? lo : pre) - pre);
      sg.g1 = int((hi < pre + G ? hi : pre + G) - pre);
      const int first = int(((pre + 1) * W - 1) / total), last = int(((pre + G) * W - 1) / total);
      sg.part = cluster_id - first;
      sg.nparts = last - first + 1;
      atomicAdd(&tw->n_seg, 1);
    }
  }
  if (kTS && !kDense) {                    // the layout's tables (host uploads only, as above)
    const int total_steps = __ldg(a.step_ptr + a.n_bundles), total_groups = __ldg(a.grp_ptr + a.n_bundles);
    for (int i = threadIdx.x; i < total_steps; i += blockDim.x) {
      const int enc = __ldg(a.steps + i);
      const uint32_t kt = uint32_t(enc >> 24) & 63u;
      steps_s[i] = enc;
      // tap kt = q * st + r reads phase tile r from frame q on
      aoff_s[i] = (kt % uint32_t(a.ts_phases)) * ts_a_slot + (kt / uint32_t(a.ts_phases)) * uint32_t(a.ts_frame_bytes);
    }
    for (int i = threadIdx.x; i <= total_groups; i += blockDim.x) grp_s[i] = __ldg(a.grp_first + i);
  }

  pdl_wait();
  for (int i = threadIdx.x; i < a.n_bundles * a.n_tile; i += blockDim.x)
    bias_s[i] = (a.bias != nullptr && i < a.g.M) ? __ldg(a.bias + i) : 0.f;
  __syncthreads();

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      const uint32_t tx_chunk_both = 2u * (uint32_t(box_rows) * 128u + b_bytes);
      const int n_work = tw->n_full + tw->n_seg;
      for (int wi = 0; kTS && wi < n_work && ok; ++wi) {
        const Work wk = get_work(tw, wi, cluster_id, n_clusters);
        const PairItem c = decode_pair_item(a, wk.item, pairs_per_bundle, n_mtiles, rank);
        const int gbase = kDense ? 0 : tw->gp[c.bundle];
        const int ngrp = kDense ? ts_groups_dense : tw->gp[c.bundle + 1] - gbase;
        const int g1 = wk.g1 < ngrp ? wk.g1 : ngrp;
        const int wq = c.w0 * a.g.sw - a.g.pw, hq = c.h0 * a.g.sh - a.g.ph, tq = c.t0 * a.g.st - a.g.pt;
        // computed steps: (kh, kw, chunk) of the share's first group by division once, then carried (three divisions
        // per group made this lone thread the limit of the dense path on 128-wide layers)
        int d_ch = 0, d_kw = 0, d_kh = 0;
        if (kDense) {
          d_ch = wk.g0 % a.n_chunks;
          const int hw = wk.g0 / a.n_chunks;
          d_kw = hw % a.g.Kw; d_kh = hw / a.g.Kw;
        }
        for (int g = wk.g0; g < g1; ++g) {
          int s0, ns, kh, kw, ch;
          if (kDense) {
            s0 = c.bundle * a.steps_dense + g * a.g.Kt; ns = a.g.Kt;
            ch = d_ch; kw = d_kw; kh = d_kh;
            if (++d_ch == a.n_chunks) { d_ch = 0; if (++d_kw == a.g.Kw) { d_kw = 0; ++d_kh; } }
          } else {
            s0 = grp_s[gbase + g]; ns = grp_s[gbase + g + 1] - s0;
            const int enc = steps_s[s0];
            kh = (enc >> 18) & 63; kw = (enc >> 12) & 63; ch = enc & 4095;
          }
          const uint32_t full_local = smem_u32(&bars->full[stage]);
          const uint32_t full_leader = mapa_shared(full_local, 0);
          const uint32_t s_dst = tiles_base + stage * stage_bytes;
          if (!mbar_wait(smem_u32(&bars->empty[stage]), phase ^ 1u, bars, err, 21)) { ok = false; break; }
          if (leader) mbar_expect_tx(full_local, 2u * (uint32_t(a.ts_phases * a.ts_a_bytes) + uint32_t(ns) * b_bytes));
          // tile r: the frames t * st + r (traversal stride st along t), so that tap kt = q * st + r is its rows from frame q on
          for (int r = 0; r < a.ts_phases; ++r)
            tma_load_5d_pair(s_dst + uint32_t(r) * ts_a_slot, &xmap, full_leader, ch * 64, wq + kw, hq + kh, tq + r, c.n0);
          const int wrow = s0 * a.n_tile + int(rank) * n_half;
          for (int q = 0; q < ns; ++q)
            tma_load_2d_pair(s_dst + ts_a_all + uint32_t(q) * b_bytes, &wmap_half, full_leader, 0, wrow + q * a.n_tile);
          if (++stage == stages) { stage = 0; phase ^= 1u; }
        }
      }
      for (int wi = 0; !kTS && wi < n_work && ok; ++wi) {
        const Work wk = get_work(tw, wi, cluster_id, n_clusters);
        const PairItem c = decode_pair_item(a, wk.item, pairs_per_bundle, n_mtiles, rank);
        const int s_begin = kDense ? c.bundle * a.steps_dense : tw->sp[c.bundle];
        const int nsteps = kDense ? a.steps_dense : tw->sp[c.bundle + 1] - s_begin;
        const int i0 = wk.g0 * kCps, i1 = wk.g1 * kCps < nsteps ? wk.g1 * kCps : nsteps;
        const int wq = c.w0 * a.g.sw - a.g.pw, hq = c.h0 * a.g.sh - a.g.ph, tq = c.t0 * a.g.st - a.g.pt;
        int kt = 0, kh = 0, kw = 0, ch = 0;
        if (kDense && i0 > 0) {
          ch = i0 % a.n_chunks;
          const int pos = i0 / a.n_chunks;
          kw = pos % a.g.Kw; kh = (pos / a.g.Kw) % a.g.Kh; kt = pos / (a.g.Kw * a.g.Kh);
        }
        int wrow = (s_begin + i0) * a.n_tile + int(rank) * n_half;
        for (int i = i0; i < i1; i += kCps) {
          const int nload = i1 - i < kCps ? i1 - i : kCps;
          int c_ch[kCps], c_w[kCps], c_h[kCps], c_t[kCps];
#pragma unroll
          for (int q = 0; q < kCps; ++q) {
            if (q >= nload) break;
            if (kDense) {
              c_ch[q] = ch * 64; c_w[q] = wq + kw; c_h[q] = hq + kh; c_t[q] = tq + kt;
              if (++ch == a.n_chunks) { ch = 0; if (++kw == a.g.Kw) { kw = 0; if (++kh == a.g.Kh) { kh = 0; ++kt; } } }
            } else {
              const int enc = __ldg(a.steps + s_begin + i + q);
              c_t[q] = tq + ((enc >> 24) & 63); c_h[q] = hq + ((enc >> 18) & 63); c_w[q] = wq + ((enc >> 12) & 63);
              c_ch[q] = (enc & 4095) * 64;
            }
          }
          const uint32_t full_local = smem_u32(&bars->full[stage]);
          const uint32_t full_leader = mapa_shared(full_local, 0);
          const uint32_t s_dst = tiles_base + stage * stage_bytes;
          if (!mbar_wait(smem_u32(&bars->empty[stage]), phase ^ 1u, bars, err, 21)) { ok = false; break; }
          if (leader) mbar_expect_tx(full_local, tx_chunk_both * uint32_t(nload));
#pragma unroll
          for (int q = 0; q < kCps; ++q) {
            if (q >= nload) break;
            const uint32_t a_dst = s_dst + q * chunk_bytes;
            tma_load_5d_pair(a_dst, &xmap, full_leader, c_ch[q], c_w[q], c_h[q], c_t[q], c.n0);
            tma_load_2d_pair(a_dst + kABytes, &wmap_half, full_leader, 0, wrow);
            wrow += a.n_tile;
          }
          if (++stage == stages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1 || (kDual && warp == 10)) {
    // ------------------------------------------------------------------ MMA issuer(s) (leader CTA only)
    if (lane == 0 && leader) {
      const int me = warp == 1 ? 0 : 1;                      // which step groups of an item: even / odd
      const uint32_t idesc = instr_desc_bf16_pair(a.n_tile);
      uint32_t j = 0, phase = 0;
      int stage = 0;
      bool ok = true, ready = false;
      // Two issuing threads share the groups by the parity of the RUNNING group number, i.e. by stage parity (the
      // ring has an even number of stages then): a thread that skipped one fill of a stage and came back for the
      // next could take the older completion of that stage's barrier for the one it waits for.
      uint32_t gg = 0;
      const int n_work = tw->n_full + tw->n_seg;
      for (int wi = 0; kTS && wi < n_work && ok; ++wi, ++j) {
        const Work wk = get_work(tw, wi, cluster_id, n_clusters);
        const int bundle = wk.item / pairs_per_bundle;
        const int gbase = kDense ? 0 : tw->gp[bundle];
        const int ngrp = kDense ? ts_groups_dense : tw->gp[bundle + 1] - gbase;
        const int g1 = wk.g1 < ngrp ? wk.g1 : ngrp;
        const uint32_t buf = j & 1u;
        if (!mbar_wait(smem_u32(&bars->tmem_empty[buf]), ((j >> 1) & 1u) ^ 1u, bars, err, 22)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (buf * uint32_t(kIss) + uint32_t(me)) * uint32_t(a.n_tile);
        bool fresh = true;                                   // this thread's accumulator has nothing of this item yet
        for (int g = wk.g0; g < g1; ++g, ++gg) {
          if (!kDual || int(gg & 1u) == me) {
            int s0 = 0, ns = a.g.Kt;
            if (!kDense) { s0 = grp_s[gbase + g]; ns = grp_s[gbase + g + 1] - s0; }
            if (!mbar_wait(smem_u32(&bars->full[stage]), phase, bars, err, 23)) { ok = false; break; }
            tc_fence_after();
            const uint32_t s_base = tiles_base + stage * stage_bytes;
            for (int q = 0; q < ns; ++q) {
              // computed steps (temporal stride 1 only): kt = q.  Every instruction in this loop shows in the time of
              // a 128-wide layer (four more ALU operations per step cost 6 %).
              const uint64_t adesc = smem_desc_sw128(s_base + (kDense ? uint32_t(q) * uint32_t(a.ts_frame_bytes) : aoff_s[s0 + q]));
              const uint64_t bdesc = smem_desc_sw128(s_base + ts_a_all + uint32_t(q) * b_bytes);
#pragma unroll
              for (int kk = 0; kk < 4; ++kk)
                umma_bf16_pair(d_tmem, adesc + 2 * kk, bdesc + 2 * kk, idesc, (!fresh | q | kk) ? 1u : 0u);
            }
            fresh = false;
            umma_commit_pair(smem_u32(&bars->empty[stage]));
          }
          if (++stage == stages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit_pair(smem_u32(&bars->tmem_full[buf]));
      }
      for (int wi = 0; !kTS && wi < n_work && ok; ++wi, ++j) {
        const Work wk = get_work(tw, wi, cluster_id, n_clusters);
        const int bundle = wk.item / pairs_per_bundle;
        const int nsteps = kDense ? a.steps_dense : tw->sp[bundle + 1] - tw->sp[bundle];
        const int i0 = wk.g0 * kCps, i1 = wk.g1 * kCps < nsteps ? wk.g1 * kCps : nsteps;
        const uint32_t buf = j & 1u;
        if (!mbar_wait(smem_u32(&bars->tmem_empty[buf]), ((j >> 1) & 1u) ^ 1u, bars, err, 22)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (buf * uint32_t(kIss) + uint32_t(me)) * uint32_t(a.n_tile);
        bool fresh = true;
        for (int i = i0; i < i1; i += kCps, ++gg) {
          const int nload = i1 - i < kCps ? i1 - i : kCps;
          const int stage_n = stage + 1 == stages ? 0 : stage + 1;
          const uint32_t phase_n = stage + 1 == stages ? phase ^ 1u : phase;
          if (!kDual || int(gg & 1u) == me) {
            if (!ready && !mbar_wait(smem_u32(&bars->full[stage]), phase, bars, err, 23)) { ok = false; break; }
            // one issuer: poll the next stage's barrier now, its answer arrives while this stage's MMAs are issued
            ready = kDual ? false : mbar_try_wait(smem_u32(&bars->full[stage_n]), phase_n);
            tc_fence_after();
#pragma unroll
            for (int q = 0; q < kCps; ++q) {
              if (q >= nload) break;
              const uint32_t a_addr = tiles_base + stage * stage_bytes + q * chunk_bytes;
              const uint64_t adesc = smem_desc_sw128(a_addr);
              const uint64_t bdesc = smem_desc_sw128(a_addr + kABytes);
#pragma unroll
              for (int kk = 0; kk < 4; ++kk)
                umma_bf16_pair(d_tmem, adesc + 2 * kk, bdesc + 2 * kk, idesc, (!fresh | q | kk) ? 1u : 0u);
            }
            fresh = false;
            umma_commit_pair(smem_u32(&bars->empty[stage]));
          }
          stage = stage_n; phase = phase_n;
        }
        if (!ok) break;
        umma_commit_pair(smem_u32(&bars->tmem_full[buf]));     // with no MMAs pending this arrives at once
      }
    }
  } else if (warp < 10) {
    // ------------------------------------------------------------------ epilogue (both CTAs)
    const int quad = warp & 3;
    const int set = (warp - 2) >> 2;                       // 0: warps 2..5, 1: warps 6..9
    const int col0 = set * 32, col_step = 32 * epi_sets;   // which 32-column pieces this warp takes
    const int row = quad * 32 + lane;
    int r = row;
    const int bw_i = r % a.box.bw; r /= a.box.bw;
    const int bh_i = r % a.box.bh; r /= a.box.bh;
    const int bt_i = r % a.box.bt; r /= a.box.bt;
    const int bn_i = r;
    __nv_bfloat16* yb = static_cast<__nv_bfloat16*>(a.y);
    const __nv_bfloat16* rb = static_cast<const __nv_bfloat16*>(a.residual);
    // two sets: each warp of a quadrant uses one of the quadrant's two staging buffers
    TmaStore ts{&ymap, store_smem + uint32_t(quad) * kStoreWarpBytes + uint32_t(set) * kStoreStageBytes, 0, 0, 0, 0, 0u,
                1u};
    const PoolLanes pool_lanes = make_pool_lanes(a.pool_w, a.pool_h, a.pool_t, a.sbw, a.sbh, lane);
    const PoolLanes* pool = (a.pool_t * a.pool_h * a.pool_w > 1) ? &pool_lanes : nullptr;
    int r0 = quad * 32;                        // coordinates of the warp's first row inside the box
    const int bw_0 = r0 % a.box.bw; r0 /= a.box.bw;
    const int bh_0 = r0 % a.box.bh; r0 /= a.box.bh;
    const int bt_0 = r0 % a.box.bt; r0 /= a.box.bt;
    const int bn_0 = r0;
    uint32_t j = 0;
    uint32_t gg = 0;                                       // running group number, as the issuing threads count it
    const size_t part_tile = size_t(128) * a.n_tile;       // floats per partial tile
    const int n_work = tw->n_full + tw->n_seg;
    for (int wi = 0; wi < n_work; ++wi, ++j) {
      const Work wk = get_work(tw, wi, cluster_id, n_clusters);
      const PairItem c = decode_pair_item(a, wk.item, pairs_per_bundle, n_mtiles, rank);
      const int nsteps = kDense ? a.steps_dense : tw->sp[c.bundle + 1] - tw->sp[c.bundle];
      const uint32_t buf = j & 1u;
      if (!mbar_wait(smem_u32(&bars->tmem_full[buf]), (j >> 1) & 1u, bars, err, 24)) break;
      tc_fence_after();
      const int nn = c.n0 + bn_i, to = c.t0 + bt_i, ho = c.h0 + bh_i, wo = c.w0 + bw_i;
      const bool in_range = row < box_rows && nn < a.g.n && to < a.g.To && ho < a.g.Ho && wo < a.g.Wo;
      const long long vox = (((long long)nn * a.g.To + to) * a.g.Ho + ho) * a.g.Wo + wo;
      const int m_base = c.bundle * a.n_tile;
      uint32_t taddr = tmem_base + (uint32_t(quad * 32) << 16) + buf * uint32_t(kIss * a.n_tile);
      // the second issuer's accumulator holds something once the item (or share) has two step groups
      int units_here;                                      // step groups (of kCps steps, or t-groups) of this item or share
      if (kTS) {
        const int ngrp = kDense ? ts_groups_dense : tw->gp[c.bundle + 1] - tw->gp[c.bundle];
        units_here = (wk.g1 < ngrp ? wk.g1 : ngrp) - wk.g0;
      } else {
        units_here = ((wk.g1 * kCps < nsteps ? wk.g1 * kCps : nsteps) - wk.g0 * kCps + kCps - 1) / kCps;
      }
      // two issuing threads: groups with an even running number went into the first accumulator, odd ones into the
      // second; an item (or share) of a single group is in one of them only
      const uint32_t acc2 = (kDual && units_here >= 2) ? uint32_t(a.n_tile) : 0u;
      if (kDual && units_here == 1 && (gg & 1u)) taddr += uint32_t(a.n_tile);
      gg += uint32_t(units_here > 0 ? units_here : 0);
      const __nv_bfloat16* res = (rb != nullptr && in_range) ? rb + vox * a.rcs + m_base : nullptr;
      const int res_left = a.rcs - m_base;
      if (wk.nparts > 1 && wk.part != 0) {
        // A share of a tile another pair owns: leave the raw partial sums in scratch and raise this warp's flag.
        // It is the first segment of this pair's range.
        const int slot = cluster_id * 2 + int(rank);
        store_partial_row(taddr, a.n_tile, true, a.tail_scratch + size_t(slot) * part_tile + row * kPartRow, col0, col_step, acc2);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(mapa_shared(smem_u32(&bars->tmem_empty[buf]), 0));
        __threadfence();
        __syncwarp();
        if (lane == 0) *reinterpret_cast<volatile int32_t*>(a.tail_flags + slot * 8 + set * 4 + quad) = 1;
        continue;
      }
      if (wk.nparts > 1) {
        // The share of the tile this pair owns (the last segment of its range; its accumulator is still in tensor
        // memory).  The other shares were computed at the same time by the next pairs, each as the first segment of
        // its range: wait for their flags, then add their partial tiles to the accumulator in the epilogue.
        int ok = 1;
        if (lane == 0) {
          const long long start = clock64();
          for (int p = 1; p < wk.nparts && ok; ++p) {
            const volatile int32_t* f = a.tail_flags + ((cluster_id + p) * 2 + int(rank)) * 8 + set * 4 + quad;
            while (*f == 0) {
              if (bars->abort_flag || clock64() - start > kWaitCycles) {
                bars->abort_flag = 1;
                atomicCAS(err, 0, 25);
                ok = 0;
                break;
              }
            }
          }
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        __threadfence();
        const float* e_first = a.tail_scratch + size_t((cluster_id + 1) * 2 + int(rank)) * part_tile + row * kPartRow;
        const float* e_more = a.tail_scratch + size_t((cluster_id + 2) * 2 + int(rank)) * part_tile + row * kPartRow;
        if (a.store_tma) {
          ts.c1 = (c.w0 + bw_0) / a.pool_w; ts.c2 = (c.h0 + bh_0) / a.pool_h; ts.c3 = (c.t0 + bt_0) / a.pool_t; ts.c4 = c.n0 + bn_0;
          epilogue_row_tma(taddr, a.n_tile, true, quad * 32 < box_rows, in_range, bias_s, a.g.relu,
                           yb + vox * a.g.ycs + m_base, m_base, a.g.M, lane, ts, res, res_left, pool,
                           e_first, e_more, 2 * part_tile, wk.nparts - 2, col0, col_step, acc2);
        } else {
          epilogue_row(taddr, a.n_tile, true, in_range, bias_s, a.g.relu, yb + vox * a.g.ycs + m_base, m_base, a.g.M,
                       res, res_left, col0, col_step, e_first, e_more, 2 * part_tile, wk.nparts - 2, acc2);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive_cluster(mapa_shared(smem_u32(&bars->tmem_empty[buf]), 0));
          for (int p = 1; p < wk.nparts; ++p)                        // ready for the next launch
            a.tail_flags[((cluster_id + p) * 2 + int(rank)) * 8 + set * 4 + quad] = 0;
        }
        continue;
      }
      if (a.store_tma) {
        ts.c1 = (c.w0 + bw_0) / a.pool_w; ts.c2 = (c.h0 + bh_0) / a.pool_h; ts.c3 = (c.t0 + bt_0) / a.pool_t; ts.c4 = c.n0 + bn_0;
        epilogue_row_tma(taddr, a.n_tile, nsteps > 0, quad * 32 < box_rows, in_range, bias_s, a.g.relu,
                         yb + vox * a.g.ycs + m_base, m_base, a.g.M, lane, ts, res, res_left, pool, nullptr, nullptr, 0, 0,
                         col0, col_step, acc2);
      } else {
        epilogue_row(taddr, a.n_tile, nsteps > 0, in_range, bias_s, a.g.relu, yb + vox * a.g.ycs + m_base, m_base, a.g.M,
                     res, res_left, col0, col_step, nullptr, nullptr, 0, 0, acc2);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(mapa_shared(smem_u32(&bars->tmem_empty[buf]), 0));
    }
    if (lane == 0) tma_store_wait_all();         // all bulk stores done before shared memory goes away
  }

  // ---------------------------------------------------------------------- teardown
  if (bars->abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000ll) { }
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();              // the peer may still be signalling barriers in this CTA's shared memory
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(uint32_t(tmem_cols)) : "memory");
  }
}

// Two K steps share one barrier hand-shake when a step is short (narrow bundles: the issuing thread, not
// the tensor pipe, is the limit there); wide bundles keep one step per stage (deeper pipeline).
int pick_cps(int n_tile) { return n_tile <= 160 ? 2 : 1; }
// Two issuing threads (two accumulators per buffer: 2 x 2 x N <= 512 TMEM columns).
bool pick_dual(int n_tile) { return n_tile <= 128; }

int pick_stages_pair(int n_tile) {
  const size_t stage = pick_cps(n_tile) * (kABytes + size_t(n_tile / 2) * 128);
  int s = int(kSmemBudget / stage);
  if (s > kMaxStages) s = kMaxStages;
  if (pick_dual(n_tile)) s &= ~1;               // two issuing threads take the stages by parity
  return s;
}

size_t pair_smem_bytes(int n_tile, int n_bundles) {
  return size_t(pick_stages_pair(n_tile)) * pick_cps(n_tile) * (kABytes + size_t(n_tile / 2) * 128) + 1024 + 4 * kStoreWarpBytes +
         sizeof(Barriers) + sizeof(TailWork) + 16 +
         size_t(n_tile) * n_bundles * 4;
}

// t-grouped variant: a stage = one deeper input tile + Kt weight half-tiles; the tables come after the bias.
size_t ts_stage_bytes(const UmmaArgs& a) {
  return size_t(a.ts_phases) * ((size_t(a.ts_a_bytes) + 1023) & ~size_t(1023)) + size_t(a.g.Kt) * size_t(a.n_tile / 2) * 128;
}
int pick_stages_pair_ts(const UmmaArgs& a) {
  const size_t fixed = 1024 + 4 * kStoreWarpBytes + sizeof(Barriers) + sizeof(TailWork) + 16 +
                       size_t(a.n_tile) * a.n_bundles * 4 + (3 * size_t(a.ts_table) + 16) * 4;
  int s = int((size_t(227) * 1024 - fixed) / ts_stage_bytes(a));
  if (s > kMaxStages) s = kMaxStages;
  if (pick_dual(a.n_tile)) s &= ~1;             // two issuing threads take the stages by parity
  return s;
}
size_t pair_smem_bytes_ts(const UmmaArgs& a) {
  return size_t(pick_stages_pair_ts(a)) * ts_stage_bytes(a) + 1024 + 4 * kStoreWarpBytes + sizeof(Barriers) + sizeof(TailWork) +
         16 + size_t(a.n_tile) * a.n_bundles * 4 + (3 * size_t(a.ts_table) + 16) * 4;
}

template <bool kDense, int kCps, bool kTS, bool kDual>
cudaError_t prepare_pair_t() {
  static bool attr_done[kMaxDevices] = {};             // the attribute is per device
  const int dev = current_device_index();
  if (dev < 0) return cudaErrorInvalidDevice;
  if (!attr_done[dev]) {
    cudaError_t e = cudaFuncSetAttribute(conv3d_umma_pair_kernel<kDense, kCps, kTS, kDual>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    attr_done[dev] = true;
  }
  return cudaSuccess;
}

void pair_launch_config(cudaLaunchConfig_t& cfg, cudaLaunchAttribute* attr, unsigned grid, size_t smem, cudaStream_t stream) {
  cfg = cudaLaunchConfig_t{};
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kThreadsPair);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
}

// CTA pairs that can be resident at once (the persistent grid), never more than SMs / 2.
template <bool kDense, int kCps, bool kTS, bool kDual>
int pair_max_clusters_t(int sm_count, size_t smem) {
  static int max_clusters_dev[kMaxDevices] = {};       // the occupancy answer is per device
  const int dev = current_device_index();
  if (dev < 0) return sm_count / 2;
  int& max_clusters = max_clusters_dev[dev];
  if (max_clusters == 0) {
    if (prepare_pair_t<kDense, kCps, kTS, kDual>() != cudaSuccess) return sm_count / 2;
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    pair_launch_config(cfg, attr, unsigned(sm_count & ~1), smem, nullptr);
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, conv3d_umma_pair_kernel<kDense, kCps, kTS, kDual>, &cfg) != cudaSuccess || n <= 0) n = sm_count / 2;
    max_clusters = n;
  }
  return max_clusters < sm_count / 2 ? max_clusters : sm_count / 2;
}

// The instantiation for a bundle width: <dense path, K steps per stage, t-grouped, two issuing threads>.
// t-grouped: a stage is a group whatever kCps says; two issuing threads up to 128 columns.  Otherwise two steps per
// stage up to 192 columns (one issuing thread needs about 550 clocks per hand-shake and four MMAs, more than the
// 288-384 clocks of MMAs of a 144- to 192-wide step), with two issuing threads up to 128.
#define RT3D_PAIR_VARIANT(DENSE, TS, N_TILE, CALL)                                             \
  do {                                                                                         \
    if (TS) {                                                                                  \
      if (pick_dual(N_TILE)) { if (DENSE) return CALL(true, 2, true, true); return CALL(false, 2, true, true); }       \
      if (DENSE) return CALL(true, 1, true, false); return CALL(false, 1, true, false);         \
    }                                                                                          \
    if (pick_dual(N_TILE)) { if (DENSE) return CALL(true, 2, false, true); return CALL(false, 2, false, true); }       \
    if (pick_cps(N_TILE) == 2) { if (DENSE) return CALL(true, 2, false, false); return CALL(false, 2, false, false); } \
    if (DENSE) return CALL(true, 1, false, false); return CALL(false, 1, false, false);         \
  } while (0)

int pair_max_clusters(int n_tile, int n_bundles, bool dense, int sm_count) {
  const size_t smem = pair_smem_bytes(n_tile, n_bundles);
#define RT3D_CALL(D, C, T, U) pair_max_clusters_t<D, C, T, U>(sm_count, smem)
  RT3D_PAIR_VARIANT(dense, false, n_tile, RT3D_CALL);
#undef RT3D_CALL
}
int pair_max_clusters_ts(const UmmaArgs& a, int sm_count) {
  const size_t smem = pair_smem_bytes_ts(a);
#define RT3D_CALL(D, C, T, U) pair_max_clusters_t<D, C, T, U>(sm_count, smem)
  RT3D_PAIR_VARIANT(a.dense != 0, true, a.n_tile, RT3D_CALL);
#undef RT3D_CALL
}

template <bool kDense, int kCps, bool kTS, bool kDual>
cudaError_t launch_pair_t(const UmmaArgs& a, const CUtensorMap& xm, const CUtensorMap& wm, const CUtensorMap& ym,
                          int sm_count, int stages,
                          int cols, size_t smem, long long n_items, cudaStream_t stream) {
  cudaError_t e = prepare_pair_t<kDense, kCps, kTS, kDual>();
  if (e != cudaSuccess) return e;
  long long clusters = pair_max_clusters_t<kDense, kCps, kTS, kDual>(sm_count, smem);
  const long long want = n_items > a.tail_workers ? n_items : a.tail_workers;
  if (clusters > want) clusters = want;
  LaunchSetup ls(dim3(unsigned(2 * clusters)), dim3(kThreadsPair), smem, stream, 2);
  return cudaLaunchKernelEx(&ls.cfg, conv3d_umma_pair_kernel<kDense, kCps, kTS, kDual>, xm, wm, ym, a, stages, cols);
}

}  // namespace

bool umma_pair_supported(int n_tile, int n_bundles) {
  return n_tile % 16 == 0 && n_tile <= 256 && n_bundles <= kMaxBundles && pick_stages_pair(n_tile) >= 2 &&
         pair_smem_bytes(n_tile, n_bundles) <= 227 * 1024;
}

// Tail split: decides how many CTA pairs share the items that do not fill a last round (0 = no split)
// and how much scratch that needs.  `step_ptr_host`: the layout's per-bundle step offsets (sparse path).
bool umma_pair_ts_supported(UmmaArgs* a, int total_steps) {
  if (a->n_tile > 256 || a->n_tile % 16 || a->g.st < 1 || a->g.st > 2 || a->box.bn != 1 || a->box.bt < 2) return false;
  if (a->g.Kt < 2 || a->g.Kt > 8 || a->g.Kt <= a->g.st) return false;
  if (a->dense && a->g.st != 1) return false;               // the computed-step path has no phase tiles
  UmmaArgs t = *a;
  t.ts_phases = a->g.st;
  const int frames = a->box.bt + (a->g.Kt - 1) / a->g.st;          // per phase tile (the deepest phase; the others load as many)
  if (frames * a->g.st > 256 || total_steps > kTsTable) return false;
  t.ts_frame_bytes = a->box.bh * a->box.bw * 128;
  t.ts_a_bytes = frames * t.ts_frame_bytes;
  t.ts_table = a->dense ? 0 : (total_steps + 3) & ~3;
  // it has to fit with at least as many steps in flight as the step-per-location form has
  const int stages = pick_stages_pair_ts(t);
  if (stages < 2 || stages * a->g.Kt < 8 || pair_smem_bytes_ts(t) > 227 * 1024) return false;
  // and to stage fewer input bytes than one tile per step does
  if (size_t(t.ts_phases) * t.ts_a_bytes * 4 > size_t(a->g.Kt) * a->box.bt * t.ts_frame_bytes * 3) return false;
  a->ts_frame_bytes = t.ts_frame_bytes; a->ts_a_bytes = t.ts_a_bytes; a->ts_table = t.ts_table; a->ts_phases = t.ts_phases;
  return true;
}

void umma_pair_tail_plan(UmmaArgs* a, const int32_t* step_ptr_host, int sm_count, size_t* scratch_bytes,
                         size_t* flag_bytes, const int32_t* grp_ptr_host) {
  a->tail_workers = 0;
  *scratch_bytes = 0; *flag_bytes = 0;
  if (!umma_pair_supported(a->n_tile, a->n_bundles)) return;
  const long long n_mtiles = (long long)a->tiles_n * a->tiles_t * a->tiles_h * a->tiles_w;
  const long long pairs_per_bundle = (n_mtiles + 1) / 2;
  const long long n_items = pairs_per_bundle * a->n_bundles;
  const int clusters = a->ts ? pair_max_clusters_ts(*a, sm_count)
                             : pair_max_clusters(a->n_tile, a->n_bundles, a->dense != 0, sm_count);
  if (clusters <= 0) return;
  // fewer items than pairs: every item is a left-over item, the grid is `tail_workers` pairs
  const long long rounds = n_items / clusters;
  const int n_tail = int(n_items - rounds * clusters);
  if (n_tail == 0 || n_tail > kMaxTail) return;
  const int cps = a->ts ? a->g.Kt : pick_cps(a->n_tile);   // steps per unit of the split, about
  long long total = 0, g_min = 1 << 30, g_max = 0;
  for (int t = 0; t < n_tail; ++t) {
    const int b = int((rounds * clusters + t) / pairs_per_bundle);
    const int ns = a->dense ? a->steps_dense : step_ptr_host[b + 1] - step_ptr_host[b];
    if (ns < 8) return;                                   // nothing worth cutting
    long long g = (ns + cps - 1) / cps;
    if (a->ts) g = a->dense ? (long long)a->g.Kh * a->g.Kw * a->n_chunks : grp_ptr_host[b + 1] - grp_ptr_host[b];
    total += g;
    g_min = g < g_min ? g : g_min; g_max = g > g_max ? g : g_max;
  }
  long long workers = clusters;
  const long long max_parts = rounds == 0 ? 8 : 4;        // parts per item, about
  if (workers > max_parts * n_tail) workers = max_parts * n_tail;
  if (workers > total / 4) workers = total / 4;           // at least four step groups per part
  if (workers <= n_tail) return;
  const long long range = (total + workers - 1) / workers;
  if (range / g_min + 2 > kMaxTailSeg) return;
  // Storing the shares and the owner's fix-up (four warps pulling the other shares through registers)
  // cost about as much as this many K steps (measured on 256-wide bundles: the split pays for itself
  // from about 100 steps per item).
  const long long fixup_groups = (12 + cps - 1) / cps;
  if (range + fixup_groups >= g_max) return;
  a->tail_workers = int(workers);
  // per pair: one share (the first segment of its range) x two CTAs; one flag per epilogue warp
  *scratch_bytes = size_t(workers) * 2 * 128 * a->n_tile * sizeof(float);
  *flag_bytes = size_t(workers) * 2 * 8 * sizeof(int32_t);
}

cudaError_t launch_conv_umma_pair(const UmmaArgs& a, const void* xmap, const void* wmap_half, const void* ymap,
                                  int sm_count, cudaStream_t stream) {
  if (!umma_pair_supported(a.n_tile, a.n_bundles) || a.n_splits != 1) return cudaErrorInvalidValue;
  if (a.tail_workers > 0 && (a.tail_scratch == nullptr || a.tail_flags == nullptr)) return cudaErrorInvalidValue;
  const int stages = a.ts ? pick_stages_pair_ts(a) : pick_stages_pair(a.n_tile);
  const size_t smem = a.ts ? pair_smem_bytes_ts(a) : pair_smem_bytes(a.n_tile, a.n_bundles);
  if (a.ts && (smem > 227 * 1024 || stages < 2)) return cudaErrorInvalidValue;
  int cols = 32;
  while (cols < 2 * a.n_tile * (pick_dual(a.n_tile) ? 2 : 1)) cols *= 2;     // two issuing threads: two accumulators
  if (cols > 512) return cudaErrorInvalidValue;
  const long long n_mtiles = (long long)a.tiles_n * a.tiles_t * a.tiles_h * a.tiles_w;
  const long long n_items = ((n_mtiles + 1) / 2) * a.n_bundles;
  if (n_items <= 0) return cudaSuccess;
  if (a.store_tma && ymap == nullptr) return cudaErrorInvalidValue;
  CUtensorMap xm, wm, ym;
  memcpy(&xm, xmap, sizeof(CUtensorMap));
  memcpy(&wm, wmap_half, sizeof(CUtensorMap));
  memcpy(&ym, ymap ? ymap : xmap, sizeof(CUtensorMap));
#define RT3D_CALL(D, C, T, U) launch_pair_t<D, C, T, U>(a, xm, wm, ym, sm_count, stages, cols, smem, n_items, stream)
  RT3D_PAIR_VARIANT(a.dense != 0, a.ts != 0, a.n_tile, RT3D_CALL);
#undef RT3D_CALL
}

}  // namespace rt3d
