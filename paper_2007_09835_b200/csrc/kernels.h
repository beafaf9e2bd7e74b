// Launch interfaces of the CUDA kernels (device work), called from api.cu.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

#include "tile_consts.h"

namespace rt3d {

// Geometry of one convolution call (all extents already validated on the host).
struct ConvGeom {
  int n, t, h, w, c, xcs;          // input extents and channel pitch
  int To, Ho, Wo, M, ycs;          // output extents and channel pitch
  int Kt, Kh, Kw;
  int st, sh, sw, pt, ph, pw;
  int relu;
};

// CUDA-core kernel driven by the canonical packed arrays.  dtype: 0 fp32, 1 bf16.
// residual: tensor of the output's extents and dtype (pitch rcs) added before the ReLU, or nullptr.
cudaError_t launch_conv_simt(int dtype, const ConvGeom& g, const void* x, void* y,
                             const int32_t* group_ptr, const uint16_t* pos_idx, const void* tiles,
                             const float* bias, int g_m, int g_n, int P, int Q, bool dense,
                             const void* residual, int rcs, cudaStream_t stream);

cudaError_t launch_maxpool3d(int dtype, const void* x, int n, int t, int h, int w, int c, int xcs,
                             int kt, int kh, int kw, int st, int sh, int sw, int pt, int ph, int pw,
                             void* y, int To, int Ho, int Wo, int ycs, cudaStream_t stream);

cudaError_t launch_add_relu(int dtype, const void* a, int acs, const void* b, int bcs, void* y, int ycs,
                            int64_t voxels, int c, int relu, cudaStream_t stream);

// Output-voxel box of one tensor-core tile: bn*bt*bh*bw <= 128 voxels.
struct TileBox { int bn, bt, bh, bw; };

// Everything the tcgen05 kernel needs besides the two tensor maps.
struct UmmaArgs {
  ConvGeom g;
  TileBox box;
  int n_tile, n_bundles, n_chunks;
  int tiles_n, tiles_t, tiles_h, tiles_w;   // number of boxes along each axis
  int dense;                                // 1: steps are computed, not read
  int steps_dense;                          // Ks * n_chunks (dense only)
  const int32_t* step_ptr;                  // device, [n_bundles + 1]   (sparse)
  const int32_t* steps;                     // device                     (sparse)
  const float* bias;                        // device or nullptr
  void* y;
  int32_t* sched;                           // device [8]: [2] = error word set by a bounded wait that gave up
  int store_tma;                            // 1: epilogue stores go through shared memory + TMA (needs ymap)
  const void* residual;                     // device bf16 tensor of the output's extents added before the ReLU, or nullptr
  int rcs;                                  // its channel pitch
  int pool_t, pool_h, pool_w;               // fused max-pool window (1,1,1 = none); needs store_tma, ymap over the pooled tensor
  int sbw, sbh;                             // extents along w, h of the block of 32 voxels an epilogue warp owns
  int n_splits;                             // K splits per output tile (1 = none)
  float* scratch;                           // device, split-K partial tiles [tile][split][128][n_tile] (n_splits > 1)
  int32_t* counters;                        // device, [tiles * 8] arrival counters (one per epilogue warp), zero between launches
  int tail_workers;                         // CTA-pair kernel: pairs sharing the left-over items of the last round (0 = off)
  float* tail_scratch;                      // device, [tail_workers][2 shares][2 CTAs][n_tile][128] fp32 partial tiles
  int32_t* tail_flags;                      // device, [tail_workers][2][2][4 warps] "partial written" flags, zero between launches
  // CTA-pair kernel, t-grouped layout (ts != 0): steps that differ only in kt share one staged input tile that is
  // Kt - 1 frames deeper (the xmap's box); needs temporal stride 1, one clip per box and bundles up to 128 wide.
  int ts;
  const int32_t* grp_ptr;                   // device, [n_bundles + 1]
  const int32_t* grp_first;                 // device, first step of each group + sentinel
  int ts_a_bytes;                           // bytes of one deeper input tile
  int ts_phases;                            // deeper tiles per group = temporal stride: tile r holds the frames t*st + r
  int ts_frame_bytes;                       // bytes of one frame of it (bh * bw rows of 128 bytes)
  int ts_table;                             // entries reserved in shared memory for the step list (the group list follows)
  long long wait_cycles;                    // single-CTA kernel: SM clocks after which a wait gives up (0 = the default, about 1 s)
  int debug_drop_last_load;                 // single-CTA kernel, tests only: never issue the loads of each CTA's last stage
};

// xmap / wmap point to 128-byte CUtensorMap objects in host memory.
// ymap: tensor map of the output for the TMA-store epilogue (box = 32 channels x one warp's 32 voxels,
// 64-byte swizzle); used when a.store_tma != 0, may be nullptr otherwise.
cudaError_t launch_conv_umma(const UmmaArgs& a, const void* xmap, const void* wmap, const void* ymap, int sm_count,
                             cudaStream_t stream);

// CTA-pair variant (cta_group::2): wmap_half is a tensor map over the same weight tiles whose box is
// half a tile high (n_tile/2 rows).  Needs n_tile % 16 == 0 and a.n_splits == 1.
bool umma_pair_supported(int n_tile, int n_bundles);
// Fills a->tail_workers (0 = whole items only) and the scratch the tail split needs; the caller provides
// a->tail_scratch / a->tail_flags of at least those sizes (flags zero-initialised).
// With a->ts the unit of the split is a group: `grp_ptr_host` = the layout's per-bundle group offsets.
void umma_pair_tail_plan(UmmaArgs* a, const int32_t* step_ptr_host, int sm_count, size_t* scratch_bytes,
                         size_t* flag_bytes, const int32_t* grp_ptr_host = nullptr);
// Whether the t-grouped variant can run this shape (and is expected to pay); `total_steps`: all bundles' lists.
// Fills a->ts_a_bytes, ts_frame_bytes and ts_table when it can.
bool umma_pair_ts_supported(UmmaArgs* a, int total_steps);
cudaError_t launch_conv_umma_pair(const UmmaArgs& a, const void* xmap, const void* wmap_half, const void* ymap,
                                  int sm_count, cudaStream_t stream);

constexpr int kHaloMaxMma = 112;      // MMAs per tile the resident-weight kernel can issue (table in the kernel parameters)

// Resident-weight kernel for thin stride-1 layers (CTA pairs): u.box = {1, bt, bh, 8} with bt*bh = 16.
struct HaloArgs {
  UmmaArgs u;
  int n_steps;                        // kept (location, chunk) steps of the single bundle (dense: Ks * n_chunks)
  int n_mma;                          // K=16 MMAs per tile: 4 per step, fewer where the step is the last, partial chunk
  uint32_t tab[2 * kHaloMaxMma];      // per MMA: low descriptor words of A (relative to the staged block) and of B
                                      // (relative to the resident weights), both with the fixed LBO field set
  int hw, hh, ht;                     // staged input block under one tile: box + kernel extent - 1 per axis
  int halo_rows;                      // hw * hh * ht voxels
  int plane_bytes;                    // halo_rows * 128 rounded up to 1024: one 64-channel chunk of the block
  int stages;                         // staged blocks in flight (filled in by umma_halo_plan)
};
// Completes the staging geometry and the MMA table; false if the layer does not qualify (see
// umma_conv_halo.cu).  steps_host: the bundle's encoded step list (nullptr for the dense path).
bool umma_halo_plan(HaloArgs* h, const int32_t* steps_host);
// xmap: input tensor map whose box is the staged block {64, hw, hh, ht, 1}; wmap_half as for the pair kernel.
cudaError_t launch_conv_umma_halo(const HaloArgs& h, const void* xmap, const void* wmap_half, const void* ymap,
                                  int sm_count, cudaStream_t stream);

constexpr int kStMaxMma1 = 64;        // spatial / temporal MMAs per frame the fused (2+1)D kernel can issue
constexpr int kStMaxMma2 = 48;

// Fused spatial (1 x Kh x Kw) -> temporal (3 x 1 x 1) convolution pair (umma_conv_st.cu).
struct StArgs {
  ConvGeom g;                         // the spatial conv: input -> intermediate tensor (To, Ho, Wo; relu = its ReLU)
  int c_mid;                          // intermediate channels = g.M
  int n1, n2;                         // accumulator widths: intermediate / output channels rounded up to 16
  int c_split;                        // intermediate channels [0, c_split) / [c_split, n1) are converted by different warps
  int M2, ycs, relu2;                 // output channels, output channel pitch, final ReLU
  int n_steps1, n_steps2;             // kept (location, chunk) steps of each layer's single bundle
  int n_mma1;                         // K=16 MMAs of S per frame
  int mma2_ptr[4];                    // temporal MMAs of tap dt: [mma2_ptr[dt], mma2_ptr[dt+1])
  uint32_t tab1[2 * kStMaxMma1];      // per MMA: low descriptor words of A (staged frame) and B (resident weights)
  uint32_t tab2[2 * kStMaxMma2];      // T: TMEM column offset of the A slice (intermediate frame), low descriptor word of B
  int hw, hh, halo_rows, plane_bytes; // staged input frame under a 16 x 8 patch (patch + kernel extent - 1)
  int stages;                         // staged frames in flight
  int tiles_h, tiles_w;               // patches per frame
  const float* bias1;                 // device or nullptr
  const float* bias2;
  void* y;
  const void* residual;               // device bf16 tensor of the output's extents added before the final ReLU, or nullptr
  int rcs;
  int32_t* sched;                     // [2] = error word
};
bool umma_st_plan(StArgs* a, const int32_t* steps1_host, const int32_t* steps2_host);
// xmap: input tensor map with box {64, hw, hh, 1, 1}; w?map_half: half-tile weight maps of the two layers.
cudaError_t launch_conv_umma_st(const StArgs& a, const void* xmap, const void* w1map_half, const void* w2map_half,
                                int sm_count, cudaStream_t stream);

// Sub-tile kernel (umma_conv_sub.cu): skips pruned kernel locations per block of 16 output x 16 input channels.
struct SubArgs {
  ConvGeom g;
  TileBox box;
  int n_tile, n_bundles;
  int tiles_n, tiles_t, tiles_h, tiles_w;
  const SubStep* steps;               // device: the bundles' step records
  const int32_t* step_ptr;            // device, [n_bundles + 1]
  const void* blocks;                 // device: 512-byte weight blocks
  const float* bias;                  // device or nullptr
  void* y;
  int32_t* sched;                     // [2] = error word
  int store_tma;                      // 1: TMA-store epilogue (needs ymap)
  const void* residual;               // device bf16 tensor of the output's extents added before the ReLU, or nullptr
  int rcs;
  int stages;                         // ring depth (filled in by umma_sub_plan)
  uint32_t slot_bytes;                // bytes of one stage of the block ring
};
bool umma_sub_plan(SubArgs* a, int max_blocks);
// xmap: input tensor map whose box is the tile box (as for the step-list kernels).
cudaError_t launch_conv_umma_sub(const SubArgs& a, const void* xmap, const void* ymap, int sm_count, cudaStream_t stream);

// Arguments of the small-C_in tensor-core kernel (C_in <= 8 at channel pitch 8).
struct SmallCArgs {
  ConvGeom g;
  int n_pad, n_pairs;                 // padded output channels; pairs of kept kernel locations
  int n_phases, phase_stride;         // sh*sw phase images per tile, bytes between them in shared memory
  int img_w, phase_bytes;             // voxels per image row; bytes one phase load delivers
  int merged_cw;                      // 1: the tensor map's first axis is (w, channel) merged: one request per image row
  int tiles_h, tiles_w;               // 16 x 8 output tiles per frame
  int tmem_cols;                      // filled in by the launcher
  int store_tma;                      // 1: TMA-store epilogue (needs ymap)
  const void* residual;               // device bf16 tensor added before the ReLU, or nullptr
  int rcs;                            // its channel pitch
  int pool_t, pool_h, pool_w;         // fused max-pool window (1,1,1 = none; pool_t must be 1); needs store_tma
  const void* wimg;                   // device: [n_pairs][2][n_pad/8][8][8] bf16
  const int32_t* pair_off;            // device: [n_pairs][2] byte offsets inside the staged images
  const float* bias;
  void* y;
  int32_t* sched;
};
cudaError_t launch_conv_umma_smallc(const SmallCArgs& a, const void* xmap, const void* ymap, int sm_count,
                                    cudaStream_t stream);
size_t smallc_smem_bytes(int n_pairs, int n_pad, int stage_bytes);

// Test hook (debug_poison.cu): every SM's shared memory and tensor memory filled with `pattern`; `sink`: a device int.
cudaError_t launch_debug_poison(uint32_t pattern, int sm_count, int* sink, cudaStream_t stream);

// Shared memory the tcgen05 kernel needs for a bundle width (for the host-side eligibility check).
size_t umma_smem_bytes(int n_tile, int n_bundles);

}  // namespace rt3d
