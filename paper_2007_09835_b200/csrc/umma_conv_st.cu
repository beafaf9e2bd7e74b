// Fused factorised (2+1)D convolution: spatial 1 x Kh x Kw conv (+bias, ReLU, bf16 rounding) followed by the
// temporal 3 x 1 x 1 conv (+bias, residual, ReLU) in ONE kernel; the wide intermediate tensor between the
// two never reaches global memory.
//
// The temporal conv is pointwise in space, so a CTA that owns a spatial patch of 16 x 8 voxels can slide
// along t: for every frame p it
//   S(p)  contracts the staged input frame (patch + spatial halo, one TMA box) with the resident spatial
//         weights into a TMEM accumulator D1 (double buffered),
//   E1(p) eight epilogue warps turn D1 into the intermediate frame IN PLACE: + bias, ReLU, round to bf16, and
//         the packed bf16 values go back into the first half of the same TMEM columns (tcgen05.st), where
//         they are the A operand of the second contraction (tcgen05.mma with A in tensor memory): the
//         intermediate tensor never touches shared memory either,
//   T(p)  adds that frame's contribution to the THREE output frames it touches, out(p-1) += mid(p) Wt[2],
//         out(p) += mid(p) Wt[1], out(p+1) += mid(p) Wt[0]: three output accumulators live in TMEM, so only
//         one intermediate frame is ever held and nothing is recomputed along t,
//   E2    eight more epilogue warps (two per lane quadrant, alternating 32-channel pieces) drain each output
//         frame once its last contribution has landed (+ bias, residual, ReLU, bf16, 16-byte global stores).
// CTA pairs (tcgen05 cta_group::2): two patches per MMA, each CTA holds half of both weight tensors.
// S and T are issued by two warps (the narrow temporal MMAs are bound by the issue rate of a thread, and two issuing
// warps overlap on the pipe); S(p+1) is issued before T(p) can start, so E1(p) overlaps S(p+1) on the tensor pipe.
//
// Work split: the sequence of (patch pair, output frame) steps is cut into equal contiguous ranges, one per
// CTA pair.  A range that begins inside a clip first computes the intermediate frame before its first
// output frame, and one that ends inside a clip the frame after its last (two extra S per cut): perfectly
// balanced at a few per cent of extra work, where whole patches per pair would leave half the SMs idle in
// the second round (112 patch pairs over 74 CTA pairs for the R(2+1)D stage-2 shapes).
//
// Tried and not kept: the three taps of T as ONE MMA of N = 3 x C_out per 16 channels over the three adjacent
// accumulators (taps stacked in shared memory as the cyclic sequence Wt2 Wt1 Wt0 Wt2 Wt1, of which a rotation
// picks three blocks; E2 clearing each accumulator after use since a wide MMA cannot start one frame from zero):
// correct, 9 instead of 27 temporal MMAs per frame, and the same 90-92 us, with narrower limits
// (3 x C_out <= 256, two input stages).  The kernel is not bound by the temporal MMAs' issue rate alone.
//
// Limits (else the caller runs the two layers separately): bf16; C_in <= 64; intermediate and output
// channels <= 256 with 2 * n1 + 3 * n2 <= 512 TMEM columns; all strides 1; temporal kernel 3 with padding 1;
// both weight tensors and two staged input frames within 227 KB of shared memory.
// Every wait is bounded (error word + abort flag, as in the other tensor-core kernels).
#include "kernels.h"
#include "umma_common.cuh"
#include "umma_pair.cuh"
#include "pdl.cuh"

namespace rt3d {
namespace {

constexpr int kThreadsSt = 608;         // producer, MMA (spatial), 8 x E1, 8 x E2 warps, MMA (temporal)
constexpr int kStOuts = 3;              // output accumulators in flight = temporal kernel extent

struct StBars {
  Barriers b;                           // full/empty: staged input frames; tmem_full/empty: D1 buffers
  unsigned long long w_full;            // leader: both weight tensors of both CTAs have landed
  unsigned long long mid_full;          // leader: 16 E1 warps wrote the intermediate frame back into D1
  unsigned long long out_full[kStOuts]; // both: last contribution to an output accumulator is done
  unsigned long long out_empty[kStOuts];// leader: 16 E2 warps drained it
  unsigned long long t_done[2];         // leader: the temporal MMAs that read D1 buffer b are done (it may be overwritten)
};

// Walk over this CTA pair's frame jobs.  g counts (patch pair, output frame) steps; a segment is the part of
// the pair's range inside one patch pair: output frames [ta, tb), intermediate frames p = max(ta-1,0) ..
// min(tb, T-1).
struct StWalk {
  int T;
  int g0, g, g_end;                     // the launcher keeps the step count below 2^31
  int item, ta, tb, p, pb;
  bool live;
};
__device__ __forceinline__ void st_segment(StWalk& k) {
  k.item = k.g / k.T;
  k.ta = k.g - k.item * k.T;
  const int left = k.g_end - k.g;
  k.tb = (left < k.T - k.ta) ? k.ta + left : k.T;
  k.p = k.ta > 0 ? k.ta - 1 : 0;
  k.pb = k.tb < k.T ? k.tb : k.T - 1;
}
__device__ __forceinline__ void st_init(StWalk& k, int T, long long total, int cluster, int n_clusters) {
  k.T = T;
  k.g0 = k.g = int(total * cluster / n_clusters);
  k.g_end = int(total * (cluster + 1) / n_clusters);
  k.live = k.g < k.g_end;
  if (k.live) st_segment(k);
}
__device__ __forceinline__ void st_next(StWalk& k) {
  if (++k.p > k.pb) {
    k.g += k.tb - k.ta;
    k.live = k.g < k.g_end;
    if (k.live) st_segment(k);
  }
}

// D[tmem] (+)= A[tmem] * B[smem]: the A operand (this CTA's 128 rows, K-major, two bf16 per 32-bit column) is
// read from tensor memory.
__device__ __forceinline__ void umma_bf16_pair_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n"
      "}\n"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
// 16 (8) consecutive 32-bit columns of this thread's TMEM lane <- 4 (2) uint4 of packed bf16 pairs.
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint4 (&o)[4]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(o[0].x), "r"(o[0].y), "r"(o[0].z), "r"(o[0].w), "r"(o[1].x), "r"(o[1].y), "r"(o[1].z), "r"(o[1].w),
        "r"(o[2].x), "r"(o[2].y), "r"(o[2].z), "r"(o[2].w), "r"(o[3].x), "r"(o[3].y), "r"(o[3].z), "r"(o[3].w)
      : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint4 (&o)[4]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"r"(taddr), "r"(o[0].x), "r"(o[0].y), "r"(o[0].z), "r"(o[0].w), "r"(o[1].x), "r"(o[1].y), "r"(o[1].z), "r"(o[1].w)
               : "memory");
}

__global__ void __launch_bounds__(kThreadsSt, 1)
conv3d_umma_st_kernel(const __grid_constant__ CUtensorMap xmap, const __grid_constant__ CUtensorMap w1map,
                      const __grid_constant__ CUtensorMap w2map, const StArgs a, const int tmem_cols) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  const uint32_t b1_bytes = uint32_t(a.n1 / 2) * 128u, b2_bytes = uint32_t(a.n2 / 2) * 128u;
  const uint32_t w1_smem = base;
  const uint32_t w2_smem = w1_smem + uint32_t(a.n_steps1) * b1_bytes;
  const uint32_t in_smem = w2_smem + uint32_t(a.n_steps2) * b2_bytes;
  unsigned char* tail = smem_raw + (in_smem - raw) + size_t(a.stages) * a.plane_bytes;
  StBars* sb = reinterpret_cast<StBars*>(tail);
  Barriers* bars = &sb->b;
  float* bias1_s = align16_f32(sb + 1);
  float* bias2_s = bias1_s + a.n1;
  int32_t* err = a.sched + 2;

  const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;
  const uint32_t rank = blockIdx.x & 1u;
  const bool leader = rank == 0;
  const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
  const int T = a.g.To;
  const int n_patches = a.g.n * a.tiles_h * a.tiles_w;
  const long long total = (long long)((n_patches + 1) / 2) * T;

  if (threadIdx.x == 32) {
    tma_prefetch_map(&xmap);
    tma_prefetch_map(&w1map);
    tma_prefetch_map(&w2map);
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < a.stages; ++s) {
      mbar_init(smem_u32(&bars->full[s]), 1);
      mbar_init(smem_u32(&bars->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) mbar_init(smem_u32(&bars->tmem_full[b]), 1);
    mbar_init(smem_u32(&sb->w_full), 1);
    mbar_init(smem_u32(&sb->mid_full), 16);              // leader: 8 E1 warps of each CTA
    for (int b = 0; b < 2; ++b) mbar_init(smem_u32(&sb->t_done[b]), 1);
    for (int s = 0; s < kStOuts; ++s) {
      mbar_init(smem_u32(&sb->out_full[s]), 1);
      mbar_init(smem_u32(&sb->out_empty[s]), 16);        // leader: 8 E2 warps of each CTA
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
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;
  const uint32_t out_tmem = tmem_base + 2u * uint32_t(a.n1);

  // Shared memory, barriers and TMEM only so far; the successor may be scheduled now that this CTA holds its
  // TMEM columns.  Global memory from here on.
  pdl_launch();
  pdl_wait();
  if (warp >= 2) {
    for (int i = threadIdx.x - 64; i < a.n1; i += kThreadsSt - 64)
      bias1_s[i] = (a.bias1 != nullptr && i < a.g.M) ? __ldg(a.bias1 + i) : 0.f;
    for (int i = threadIdx.x - 64; i < a.n2; i += kThreadsSt - 64)
      bias2_s[i] = (a.bias2 != nullptr && i < a.M2) ? __ldg(a.bias2 + i) : 0.f;
    epilogue_bar_sync(kThreadsSt - 64);
  }

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      const uint32_t w_full_local = smem_u32(&sb->w_full);
      const uint32_t w_full_leader = mapa_shared(w_full_local, 0);
      if (leader) mbar_expect_tx(w_full_local, 2u * (uint32_t(a.n_steps1) * b1_bytes + uint32_t(a.n_steps2) * b2_bytes));
      for (int s = 0; s < a.n_steps1; ++s)
        tma_load_2d_pair(w1_smem + uint32_t(s) * b1_bytes, &w1map, w_full_leader, 0, s * a.n1 + int(rank) * (a.n1 / 2));
      for (int s = 0; s < a.n_steps2; ++s)
        tma_load_2d_pair(w2_smem + uint32_t(s) * b2_bytes, &w2map, w_full_leader, 0, s * a.n2 + int(rank) * (a.n2 / 2));
      int stage = 0;
      uint32_t phase = 0;
      const uint32_t tx_both = 2u * uint32_t(a.halo_rows) * 128u;
      const int per_clip = a.tiles_h * a.tiles_w;
      StWalk k;
      int item = -1, nn = 0, wq = 0, hq = 0;
      for (st_init(k, T, total, cluster_id, n_clusters); k.live; st_next(k)) {
        if (k.item != item) {                       // new patch: decode once
          item = k.item;
          const int patch = 2 * item + int(rank);
          nn = patch / per_clip;                    // == a.g.n for the dummy second patch of an odd count: zero fill
          const int r = patch - nn * per_clip;
          const int ih = r / a.tiles_w;
          hq = ih * 16 - a.g.ph; wq = (r - ih * a.tiles_w) * 8 - a.g.pw;
        }
        const uint32_t full_local = smem_u32(&bars->full[stage]);
        const uint32_t full_leader = mapa_shared(full_local, 0);
        if (!mbar_wait(smem_u32(&bars->empty[stage]), phase ^ 1u, bars, err, 41)) break;
        if (leader) mbar_expect_tx(full_local, tx_both);
        tma_load_5d_pair(in_smem + uint32_t(stage) * uint32_t(a.plane_bytes), &xmap, full_leader, 0, wq, hq, k.p, nn);
        if (++stage == a.stages) { stage = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA only)
    if (leader) {
      uint32_t elected;
      asm volatile("{\n.reg .pred p;\nelect.sync _|p, 0xffffffff;\nselp.u32 %0, 1, 0, p;\n}\n" : "=r"(elected));
      const uint32_t idesc1 = instr_desc_bf16_pair(a.n1);
      // high descriptor words.  Staged input: 128-byte swizzle, 8-row groups one halo row apart.  Weights:
      // 128-byte swizzle, groups 1024 bytes apart.  (The intermediate frame is read from tensor memory.)
      const uint64_t a1_hi = uint64_t(((uint32_t(a.hw) * 128u) >> 4) | (1u << 14) | (2u << 29)) << 32;
      const uint64_t b_hi = uint64_t((1024u >> 4) | (1u << 14) | (2u << 29)) << 32;
      const uint32_t w1_16 = w1_smem >> 4;
      int stage = 0;
      uint32_t phase = 0;
      bool ok = mbar_wait(smem_u32(&sb->w_full), 0, bars, err, 42);
      StWalk cur, nxt;
      st_init(cur, T, total, cluster_id, n_clusters);
      nxt = cur;
      if (nxt.live) st_next(nxt);
      uint32_t j = 0;
      // S of job jj into D1 buffer jj & 1.  The buffer's previous contents (the intermediate frame of job jj - 2)
      // were last read by T(jj - 2), issued earlier from this same thread: the tensor pipe keeps that order, so
      // no barrier guards the reuse.
      auto issue_s = [&](uint32_t jj) -> bool {
        const uint32_t buf = jj & 1u;
        if (!mbar_wait(smem_u32(&bars->full[stage]), phase, bars, err, 44)) return false;
        tc_fence_after();
        const uint32_t d = tmem_base + buf * uint32_t(a.n1);
        const uint32_t a16 = (in_smem + uint32_t(stage) * uint32_t(a.plane_bytes)) >> 4;
#pragma unroll 2
        for (int m = 0; m < a.n_mma1; ++m) {
          const uint64_t adesc = a1_hi | uint64_t(a16 + a.tab1[2 * m]);
          const uint64_t bdesc = b_hi | uint64_t(w1_16 + a.tab1[2 * m + 1]);
          if (elected) umma_bf16_pair(d, adesc, bdesc, idesc1, m ? 1u : 0u);
        }
        if (elected) {
          umma_commit_pair(smem_u32(&bars->empty[stage]));
          umma_commit_pair(smem_u32(&bars->tmem_full[buf]));
        }
        if (++stage == a.stages) { stage = 0; phase ^= 1u; }
        return true;
      };
      // The spatial MMAs S(j) come from this warp and the temporal ones T(j) from warp 18: one thread issuing both
      // needed about 4350 clocks per frame for 36 + 27 MMAs whose tensor time is 3460 (the 27 narrow ones are bound
      // by the issue rate of a single thread), while two issuing warps overlap on the pipe.  S(j + 1) overwrites the
      // D1 buffer that T(j - 1) read its A operand from, so it waits for that T to be done.
      if (ok && cur.live) ok = issue_s(0);
      while (ok && cur.live) {
        if (nxt.live) {
          if (j >= 1 && !mbar_wait(smem_u32(&sb->t_done[(j + 1) & 1u]), ((j - 1) >> 1) & 1u, bars, err, 48)) break;
          if (!issue_s(j + 1)) break;
        }
        cur = nxt;
        if (nxt.live) st_next(nxt);
        ++j;
      }
      __syncwarp();
    }
  } else if (warp < 10) {
    // ------------------------------------------------------------------ E1: D1 -> intermediate frame (both CTAs, 8 warps)
    const int quad = warp & 3;
    const int half = (warp - 2) >> 2;           // 0: columns [0, c_split), 1: [c_split, n1)
    const uint32_t mid_full_leader = mapa_shared(smem_u32(&sb->mid_full), 0);
    StWalk k;
    uint32_t j = 0;
    for (st_init(k, T, total, cluster_id, n_clusters); k.live; st_next(k), ++j) {
      const uint32_t buf = j & 1u;
      if (!mbar_wait(smem_u32(&bars->tmem_full[buf]), (j >> 1) & 1u, bars, err, 47)) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + (uint32_t(quad * 32) << 16) + buf * uint32_t(a.n1);
      // The two warps of a lane quadrant split the columns at c_split (a multiple of 16).  Each walks its range in
      // pieces of 32 columns and writes the packed values of piece k back over columns [16k, 16k + 16) of ITS OWN
      // range: those belong to piece k / 2, which it has read already, and never to the other warp's range.
      const int r0 = half ? a.c_split : 0, r1 = half ? a.n1 : a.c_split;
      for (int col = r0, dst_col = r0; col < r1; col += 32, dst_col += 16) {
        uint32_t v[32];
        const bool wide = col + 32 <= r1;
        if (wide) tmem_ld32(taddr + col, v);
        else tmem_ld16_into32(taddr + col, v);
        uint4 o[4];
        __nv_bfloat162* po = reinterpret_cast<__nv_bfloat162*>(o);
        const float4* b4 = reinterpret_cast<const float4*>(bias1_s + col);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          const float4 b = (wide || q < 4) ? b4[q] : make_float4(0.f, 0.f, 0.f, 0.f);
          float f0 = __uint_as_float(v[4 * q]) + b.x, f1 = __uint_as_float(v[4 * q + 1]) + b.y;
          float f2 = __uint_as_float(v[4 * q + 2]) + b.z, f3 = __uint_as_float(v[4 * q + 3]) + b.w;
          if (a.g.relu) {                         // activation and rounding in one instruction per pair
            reinterpret_cast<uint32_t*>(po)[2 * q] = cvt_relu_bf16x2(f0, f1);
            reinterpret_cast<uint32_t*>(po)[2 * q + 1] = cvt_relu_bf16x2(f2, f3);
          } else {
            po[2 * q] = __floats2bfloat162_rn(f0, f1);
            po[2 * q + 1] = __floats2bfloat162_rn(f2, f3);
          }
        }
        if (wide) tmem_st16(taddr + uint32_t(dst_col), o);
        else tmem_st8(taddr + uint32_t(dst_col), o);
      }
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(mid_full_leader);
    }
  } else if (warp == 18) {
    // ------------------------------------------------------------------ MMA issuer of the temporal conv (leader CTA only)
    if (leader) {
      uint32_t elected;
      asm volatile("{\n.reg .pred p;\nelect.sync _|p, 0xffffffff;\nselp.u32 %0, 1, 0, p;\n}\n" : "=r"(elected));
      const uint32_t idesc2 = instr_desc_bf16_pair(a.n2);
      const uint64_t b_hi = uint64_t((1024u >> 4) | (1u << 14) | (2u << 29)) << 32;
      const uint32_t w2_16 = w2_smem >> 4;
      bool ok = mbar_wait(smem_u32(&sb->w_full), 0, bars, err, 42);
      StWalk cur;
      st_init(cur, T, total, cluster_id, n_clusters);
      uint32_t j = 0;
      while (ok && cur.live) {
        if (!mbar_wait(smem_u32(&sb->mid_full), j & 1u, bars, err, 45)) break;
        tc_fence_after();
        const int qb = cur.g - cur.g0 - cur.ta;            // running number of output frame o is qb + o
        const uint32_t mid_tmem = tmem_base + (j & 1u) * uint32_t(a.n1);
        // The taps this job issues, oldest output frame first.  The last one, out(p + 1) += mid(p) Wt[0], starts a
        // frame and needs its accumulator drained of out(p - 2), which the tap before this job completed: the wait
        // for that comes just before the tap, so that the output warps have the time of the other two taps (this
        // warp issues nothing else, so waiting in the middle holds up no other MMA).
#pragma unroll
        for (int dt = 2; dt >= 0; --dt) {
          const int o = cur.p + 1 - dt;
          if (!(o >= cur.ta && o < cur.tb)) continue;
          const uint32_t q = uint32_t(qb + o), slot = q % kStOuts;
          const bool first = cur.p == (o > 0 ? o - 1 : 0);
          if (first) {
            if (!mbar_wait(smem_u32(&sb->out_empty[slot]), ((q / kStOuts) & 1u) ^ 1u, bars, err, 46)) { ok = false; break; }
            tc_fence_after();
          }
          const int m0 = a.mma2_ptr[dt], m1 = a.mma2_ptr[dt + 1];
          const uint32_t d = out_tmem + slot * uint32_t(a.n2);
          uint32_t acc = first ? 0u : 1u;
#pragma unroll 2
          for (int m = m0; m < m1; ++m) {
            const uint64_t bdesc = b_hi | uint64_t(w2_16 + a.tab2[2 * m + 1]);
            if (elected) umma_bf16_pair_ta(d, mid_tmem + a.tab2[2 * m], bdesc, idesc2, acc);
            acc = 1u;
          }
          // a frame is complete with the tap of the frame after it (the last frame of a clip with its own centre tap):
          // its output warps are told at once, not after the remaining taps of this job
          if (elected && (dt == 2 || (dt == 1 && cur.p == T - 1))) umma_commit_pair(smem_u32(&sb->out_full[slot]));
        }
        if (!ok) break;
        if (elected) umma_commit_pair(smem_u32(&sb->t_done[j & 1u]));
        st_next(cur);
        ++j;
      }
      __syncwarp();
    }
  } else {
    // ------------------------------------------------------------------ E2: output accumulators -> y (both CTAs, 8 warps)
    const int quad = warp & 3;
    const int half2 = (warp - 10) >> 2;        // two warps per lane quadrant: even / odd 32-column pieces
    const int row = quad * 32 + lane;
    const int bh_i = row >> 3, bw_i = row & 7;
    __nv_bfloat16* yb = static_cast<__nv_bfloat16*>(a.y);
    const __nv_bfloat16* rb = static_cast<const __nv_bfloat16*>(a.residual);
    const int per_clip = a.tiles_h * a.tiles_w;
    StWalk k;
    bool ok = true;
    for (st_init(k, T, total, cluster_id, n_clusters); k.live && ok; st_next(k)) {
      const int qb = k.g - k.g0 - k.ta;
      for (int which = 0; which < 2 && ok; ++which) {
        const int o = which == 0 ? k.p - 1 : k.p;
        if (o < k.ta || o >= k.tb || (which == 1 && k.p != T - 1)) continue;
        const uint32_t q = uint32_t(qb + o), slot = q % kStOuts;
        const int patch = 2 * k.item + int(rank);
        const int nn = patch / per_clip;
        const int r = patch - nn * per_clip;
        const int ih = r / a.tiles_w;
        const int ho = ih * 16 + bh_i, wo = (r - ih * a.tiles_w) * 8 + bw_i;
        const bool in_range = nn < a.g.n && ho < a.g.Ho && wo < a.g.Wo;
        const long long vox = (((long long)nn * T + o) * a.g.Ho + ho) * a.g.Wo + wo;
        const __nv_bfloat16* res_row = (rb != nullptr && in_range) ? rb + vox * a.rcs : nullptr;
        __nv_bfloat16* dst_row = yb + vox * a.ycs;
        // the residual of the first piece is fetched before the accumulator is waited for, that of every
        // further piece while the one before it is converted
        uint4 rv[4];
#pragma unroll
        for (int e = 0; e < 4; ++e)
          rv[e] = (res_row != nullptr && half2 * 32 + 8 * e < a.rcs)
                      ? __ldg(reinterpret_cast<const uint4*>(res_row + half2 * 32) + e) : make_uint4(0u, 0u, 0u, 0u);
        if (!mbar_wait(smem_u32(&sb->out_full[slot]), (q / kStOuts) & 1u, bars, err, 49)) { ok = false; break; }
        tc_fence_after();
        const uint32_t taddr = out_tmem + (uint32_t(quad * 32) << 16) + slot * uint32_t(a.n2);
        for (int col = half2 * 32; col < a.n2 && col < a.M2; col += 64) {
          uint32_t v[32];
          const bool wide = col + 32 <= a.n2;
          if (wide) tmem_ld32(taddr + col, v);
          else tmem_ld16_into32(taddr + col, v);
          uint4 rc[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) rc[e] = rv[e];
          if (col + 64 < a.n2) {
#pragma unroll
            for (int e = 0; e < 4; ++e)
              rv[e] = (res_row != nullptr && col + 64 + 8 * e < a.rcs)
                          ? __ldg(reinterpret_cast<const uint4*>(res_row + col + 64) + e) : make_uint4(0u, 0u, 0u, 0u);
          }
          const float4* b4 = reinterpret_cast<const float4*>(bias2_s + col);
          uint4 ov[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float4 b0 = (wide || e < 2) ? b4[2 * e] : make_float4(0.f, 0.f, 0.f, 0.f);
            const float4 b1 = (wide || e < 2) ? b4[2 * e + 1] : make_float4(0.f, 0.f, 0.f, 0.f);
            const __nv_bfloat162* pr = reinterpret_cast<const __nv_bfloat162*>(&rc[e]);
            const float2 r0 = __bfloat1622float2(pr[0]), r1 = __bfloat1622float2(pr[1]);
            const float2 r2 = __bfloat1622float2(pr[2]), r3 = __bfloat1622float2(pr[3]);
            float f0 = __uint_as_float(v[8 * e]) + b0.x + r0.x, f1 = __uint_as_float(v[8 * e + 1]) + b0.y + r0.y;
            float f2 = __uint_as_float(v[8 * e + 2]) + b0.z + r1.x, f3 = __uint_as_float(v[8 * e + 3]) + b0.w + r1.y;
            float f4 = __uint_as_float(v[8 * e + 4]) + b1.x + r2.x, f5 = __uint_as_float(v[8 * e + 5]) + b1.y + r2.y;
            float f6 = __uint_as_float(v[8 * e + 6]) + b1.z + r3.x, f7 = __uint_as_float(v[8 * e + 7]) + b1.w + r3.y;
            if (a.relu2) {
              ov[e].x = cvt_relu_bf16x2(f0, f1); ov[e].y = cvt_relu_bf16x2(f2, f3);
              ov[e].z = cvt_relu_bf16x2(f4, f5); ov[e].w = cvt_relu_bf16x2(f6, f7);
            } else {
              __nv_bfloat162* po = reinterpret_cast<__nv_bfloat162*>(&ov[e]);
              po[0] = __floats2bfloat162_rn(f0, f1); po[1] = __floats2bfloat162_rn(f2, f3);
              po[2] = __floats2bfloat162_rn(f4, f5); po[3] = __floats2bfloat162_rn(f6, f7);
            }
          }
          if (in_range) {
            const int valid = a.M2 - col;              // real output channels from here on
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              if (valid >= 8 * e + 8) {
                reinterpret_cast<uint4*>(dst_row + col)[e] = ov[e];
              } else {
                const __nv_bfloat16* pe = reinterpret_cast<const __nv_bfloat16*>(&ov[e]);
#pragma unroll
                for (int c = 0; c < 8; ++c)
                  if (8 * e + c < valid) dst_row[col + 8 * e + c] = pe[c];
              }
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(mapa_shared(smem_u32(&sb->out_empty[slot]), 0));
      }
    }
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


size_t st_smem_bytes(const StArgs& a) {
  return 1024 + size_t(a.n_steps1) * (a.n1 / 2) * 128 + size_t(a.n_steps2) * (a.n2 / 2) * 128 +
         size_t(a.stages) * a.plane_bytes + sizeof(StBars) + size_t(a.n1 + a.n2) * 4 + 16;
}

}  // namespace

// Completes the staging geometry and the two MMA tables of `a` (g, n1, n2, c_mid, n_steps1/2 already set;
// steps*_host = encoded step lists, nullptr = every location and chunk in order); false if the pair of layers
// does not qualify.
bool umma_st_plan(StArgs* a, const int32_t* steps1_host, const int32_t* steps2_host) {
  const ConvGeom& g = a->g;
  if (g.st != 1 || g.sh != 1 || g.sw != 1 || g.Kt != 1 || g.pt != 0 || g.c > 64) return false;
  if (a->n1 % 16 || a->n2 % 16 || a->n1 < 16 || a->n2 < 16 || a->n1 > 256 || a->n2 > 256) return false;
  if (2 * a->n1 + kStOuts * a->n2 > 512) return false;
  if (a->n_steps1 < 1 || a->n_steps2 < 1) return false;
  a->hw = 8 + g.Kw - 1; a->hh = 16 + g.Kh - 1;
  if (a->hw > 256 || a->hh > 256) return false;
  a->halo_rows = a->hw * a->hh;
  a->plane_bytes = (a->halo_rows * 128 + 1023) & ~1023;
  a->tiles_h = (g.Ho + 15) / 16; a->tiles_w = (g.Wo + 7) / 8;
  const size_t b1 = size_t(a->n1 / 2) * 128, b2 = size_t(a->n2 / 2) * 128;
  if (2 * (a->n_steps1 * b1 + a->n_steps2 * b2) > 1000000) return false;     // one barrier counts all weight bytes
  // spatial MMAs: step s = (kh, kw) on the single chunk, one MMA per 16 input channels
  const int k16_in = (g.c + 15) / 16;
  int m = 0;
  for (int s = 0; s < a->n_steps1; ++s) {
    int kh, kw;
    if (steps1_host == nullptr) { kw = s % g.Kw; kh = s / g.Kw; }
    else { const int32_t enc = steps1_host[s]; kh = (enc >> 18) & 63; kw = (enc >> 12) & 63; }
    if (m + k16_in > kStMaxMma1) return false;
    const uint32_t a_off = uint32_t((kh * a->hw + kw) * 128) >> 4;
    const uint32_t b_off = uint32_t(size_t(s) * b1 >> 4);
    for (int kk = 0; kk < k16_in; ++kk, ++m) {
      a->tab1[2 * m] = (a_off + 2u * uint32_t(kk)) | (1u << 16);
      a->tab1[2 * m + 1] = (b_off + 2u * uint32_t(kk)) | (1u << 16);
    }
  }
  a->n_mma1 = m;
  for (int q = 2 * m; q < 2 * kStMaxMma1; ++q) a->tab1[q] = 0u;
  a->c_split = 16 * ((a->n1 / 16 + 1) / 2);
  // temporal MMAs, grouped by dt: step = (dt, 64-channel chunk of the intermediate frame)
  const int chunks2 = (a->c_mid + 63) / 64;
  const int last_k16 = (a->c_mid - (chunks2 - 1) * 64 + 15) / 16;
  m = 0;
  int s = 0;
  for (int dt = 0; dt < 3; ++dt) {
    a->mma2_ptr[dt] = m;
    for (; s < a->n_steps2; ++s) {
      int kt, ch;
      if (steps2_host == nullptr) { ch = s % chunks2; kt = s / chunks2; }
      else { const int32_t enc = steps2_host[s]; kt = (enc >> 24) & 63; ch = enc & 4095; }
      if (kt < dt) return false;                       // list not sorted by dt
      if (kt > dt) break;
      const int kc = ch == chunks2 - 1 ? last_k16 : 4;
      if (m + kc > kStMaxMma2) return false;
      const uint32_t b_off = uint32_t(size_t(s) * b2 >> 4);
      for (int kk = 0; kk < kc; ++kk, ++m) {
        // 16 channels of the intermediate frame = 8 TMEM columns of packed bf16 pairs; the slices of the second
        // half of the channels start at column c_split (see E1 in the kernel)
        const int s16 = ch * 4 + kk, s_half = a->c_split / 16;
        a->tab2[2 * m] = uint32_t(s16 < s_half ? s16 * 8 : a->c_split + (s16 - s_half) * 8);
        a->tab2[2 * m + 1] = (b_off + 2u * uint32_t(kk)) | (1u << 16);
      }
    }
    if (m == a->mma2_ptr[dt]) return false;            // a temporal tap with no kept weights: not handled here
  }
  if (s != a->n_steps2) return false;
  a->mma2_ptr[3] = m;
  for (int q = 2 * m; q < 2 * kStMaxMma2; ++q) a->tab2[q] = 0u;
  for (a->stages = 4; a->stages >= 2; --a->stages)
    if (st_smem_bytes(*a) <= 227 * 1024) return true;
  return false;
}

cudaError_t launch_conv_umma_st(const StArgs& a, const void* xmap, const void* w1map_half, const void* w2map_half,
                                int sm_count, cudaStream_t stream) {
  if (a.stages < 2 || a.n_mma1 < 1 || a.n_mma1 > kStMaxMma1 || a.mma2_ptr[3] > kStMaxMma2) return cudaErrorInvalidValue;
  const size_t smem = st_smem_bytes(a);
  if (smem > 227 * 1024) return cudaErrorInvalidValue;
  int cols = 32;
  while (cols < 2 * a.n1 + kStOuts * a.n2) cols *= 2;
  if (cols > 512) return cudaErrorInvalidValue;
  const long long n_patches = (long long)a.g.n * a.tiles_h * a.tiles_w;
  const long long total = ((n_patches + 1) / 2) * a.g.To;
  if (total <= 0) return cudaSuccess;
  if (total >= (1ll << 31)) return cudaErrorInvalidValue;
  CUtensorMap xm, w1m, w2m;
  memcpy(&xm, xmap, sizeof(CUtensorMap));
  memcpy(&w1m, w1map_half, sizeof(CUtensorMap));
  memcpy(&w2m, w2map_half, sizeof(CUtensorMap));
  static bool attr_done[kMaxDevices] = {};             // the attributes are per device
  const int dev_idx = current_device_index();
  if (dev_idx < 0) return cudaErrorInvalidDevice;
  if (!attr_done[dev_idx]) {
    cudaError_t e = cudaFuncSetAttribute(conv3d_umma_st_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    attr_done[dev_idx] = true;
  }
  long long clusters = sm_count / 2;
  if (clusters > total) clusters = total;
  LaunchSetup ls(dim3(unsigned(2 * clusters)), dim3(kThreadsSt), smem, stream, 2);
  return cudaLaunchKernelEx(&ls.cfg, conv3d_umma_st_kernel, xm, w1m, w2m, a, cols);
}

}  // namespace rt3d
