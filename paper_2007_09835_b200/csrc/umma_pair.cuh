// Device-side helpers of the CTA-pair (tcgen05 cta_group::2) kernels: cluster addressing, pair TMA loads
// that signal the leader's barrier, the pair MMA / commit wrappers and the tile-pair work decoding.
// Included by .cu files only, after umma_common.cuh.
#pragma once

#include "kernels.h"
#include "umma_common.cuh"

namespace rt3d {
namespace {

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t mapa_shared(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  // default semantics (release at CTA scope): the cluster-scope release costs about 1500 clocks per arrive
  // when global stores are in flight, and nothing but the TMEM reads (fenced separately) needs ordering here
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void tma_load_5d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster, int c0, int c1,
                                                 int c2, int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
      : "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
// Arrive on the barrier at this shared-memory offset in both CTAs once all prior MMAs are done.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask) : "memory");
}
// bf16 x bf16 -> fp32, K-major operands, M = 256 (128 rows per CTA), N = n.
__device__ __forceinline__ uint32_t instr_desc_bf16_pair(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(n >> 3) << 17) | (uint32_t(256 >> 4) << 24);
}

struct PairItem {
  int bundle;
  int n0, t0, h0, w0;     // first output voxel of this CTA's box (beyond the tensor for a dummy tile)
};

__device__ __forceinline__ PairItem decode_pair_item(const UmmaArgs& a, int item, int pairs_per_bundle, int n_mtiles,
                                                     uint32_t rank) {
  PairItem c;
  c.bundle = item / pairs_per_bundle;
  int mt = (item - c.bundle * pairs_per_bundle) * 2 + int(rank);
  if (mt >= n_mtiles) {            // odd tile count: the last pair's second tile does not exist
    c.n0 = a.g.n; c.t0 = 0; c.h0 = 0; c.w0 = 0;
    return c;
  }
  const int iw = mt % a.tiles_w; mt /= a.tiles_w;
  const int ih = mt % a.tiles_h; mt /= a.tiles_h;
  const int it = mt % a.tiles_t; mt /= a.tiles_t;
  c.w0 = iw * a.box.bw; c.h0 = ih * a.box.bh; c.t0 = it * a.box.bt; c.n0 = mt * a.box.bn;
  return c;
}

}  // namespace
}  // namespace rt3d
