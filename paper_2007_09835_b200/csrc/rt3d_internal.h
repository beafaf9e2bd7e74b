// Internal declarations shared by the translation units of librt3d (host side).
#pragma once

#include <cstdint>
#include <cstddef>
#include <map>
#include <mutex>
#include <vector>

#include "rt3d.h"
#include "tile_consts.h"

namespace rt3d {

constexpr int kMaxGroup = 256;      // g_m, g_n <= 256 (pack, tensor-core kernels)
constexpr int kMaxGroupSimt = 8;    // the CUDA-core kernel keeps one group row in registers: g_m, g_n <= 8
constexpr int kChunk = 64;          // input channels per tensor-core K step (one 128-byte swizzle row of bf16)
constexpr int kTileM = 128;         // output voxels per tensor-core tile (TMEM lanes)

inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
inline int64_t ceil_div64(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline int round_up(int a, int b) { return ceil_div(a, b) * b; }

// Round-to-nearest-even float -> bfloat16 bits (NaN kept quiet), and back.
uint16_t f32_to_bf16_bits(float f);
float bf16_bits_to_f32(uint16_t b);

// Encoded K step of the tensor-core path: which kernel location and which 64-channel chunk.
inline int32_t encode_step(int kt, int kh, int kw, int chunk) {
  return (kt << 24) | (kh << 18) | (kw << 12) | chunk;
}
inline void decode_step(int32_t s, int& kt, int& kh, int& kw, int& chunk) {
  kt = (s >> 24) & 63; kh = (s >> 18) & 63; kw = (s >> 12) & 63; chunk = s & 4095;
}

// Weight layout consumed by the tcgen05 kernel, derived from the canonical arrays for one
// bundle width n_tile (output channels per accumulator tile).
struct UmmaLayout {
  int n_tile = 0;                    // multiple of 16, <= 256
  int n_bundles = 0;                 // ceil(M / n_tile)
  int n_chunks = 0;                  // ceil(N / 64)
  std::vector<int32_t> step_ptr;     // [n_bundles + 1] offsets into steps / weight tiles
  std::vector<int32_t> steps;        // encoded (kt,kh,kw,chunk), only non-empty steps of each bundle
  std::vector<uint16_t> wtiles;      // [steps.size()][n_tile][64] bf16 bits, zero where pruned / absent
  int max_steps = 0;                 // longest bundle list
  bool t_groups = false;             // steps ordered (kh, kw), chunk, kt; groups = runs that differ only in kt
  std::vector<int32_t> grp_ptr;      // [n_bundles + 1] offsets into grp_first            (t_groups only)
  std::vector<int32_t> grp_first;    // first step of each group, + one sentinel           (t_groups only)
};

// Layout for the small-C_in tensor-core kernel (C_in <= 8, channel pitch 8) at spatial strides
// (sh, sw): the input under a 1x16x8 output tile is staged as sh*sw phase images (every sh-th row and
// sw-th column), so that consecutive outputs are consecutive voxels of an image and every kernel
// location is a shifted window of one image.  K is walked in pairs of kernel locations (8 padded
// channels each), one K=16 MMA per pair.
struct SmallCLayout {
  int sh = 1, sw = 1;
  int n_pad = 0;                     // output channels rounded up to 16 (<= 256)
  int n_pairs = 0;
  int n_phases = 1;                  // sh * sw
  int img_w = 0, img_h = 0, img_t = 0;   // voxels of one phase image
  int phase_stride = 0;              // bytes between phase images in shared memory
  std::vector<int32_t> pair_off;     // [n_pairs][2] byte offset of each location's window inside the staged images
  std::vector<uint16_t> wimg;        // [n_pairs][2][n_pad/8][8][8] bf16 bits, zero where pruned / absent
};

// Layout consumed by the sub-tile kernel: per bundle of n_tile output channels the list of non-empty K steps in
// chunk-major order (all kernel locations of a 64-channel chunk, then the next chunk: the input block under a
// tile is then re-read from the L1 cache), each with its block mask, and the blocks themselves.  A block holds
// W[16 output channels][16 input channels] of one kernel location as four 8 x 8 core matrices
// [row group][K half][8 rows][8 channels] (no-swizzle K-major operand: 128 bytes between K halves, 256 between
// row groups).
struct SubLayout {
  int n_tile = 0, n_bundles = 0, n_chunks = 0;
  std::vector<int32_t> step_ptr;     // [n_bundles + 1]
  std::vector<SubStep> steps;
  std::vector<unsigned char> payload; // per step: 64-byte header + its blocks ([nblk][256] bf16 bits)
  int max_blocks = 0;                // most blocks in one step
  int max_steps = 0;                 // longest bundle list
};

// Per-device copies of a handle's arrays.
struct DeviceBlob {
  int device = -1;
  int32_t* group_ptr = nullptr;      // canonical arrays (CUDA-core kernel)
  uint16_t* pos_idx = nullptr;
  void* tiles = nullptr;
  struct Umma {
    void* wtiles = nullptr;
    int32_t* step_ptr = nullptr;
    int32_t* steps = nullptr;
    alignas(64) unsigned char wmap[128];   // CUtensorMap of wtiles, box = one [n_tile][64] tile
    alignas(64) unsigned char wmap_half[128];   // same tensor, box = half a tile (CTA-pair kernel)
    int32_t* grp_ptr = nullptr;                 // t-grouped layouts only
    int32_t* grp_first = nullptr;
    bool ready = false;
  };
  std::map<int, Umma> umma;          // keyed like the handle's layouts
  struct Sub { void* steps = nullptr; int32_t* step_ptr = nullptr; void* blocks = nullptr; bool ready = false; };
  std::map<int, Sub> sub;            // sub-tile kernel, keyed by n_tile
  struct SmallC { void* wimg = nullptr; int32_t* pairs = nullptr; };
  std::map<int, SmallC> smallc;      // small-C_in kernel: weight image and pair offsets, keyed by sh*16+sw
  float* splitk = nullptr; size_t splitk_bytes = 0;            // split-K partial tiles (grown on demand)
  int32_t* splitk_cnt = nullptr; size_t splitk_cnt_bytes = 0;  // split-K arrival counters, zero between launches
  void* stage_x = nullptr; size_t stage_x_bytes = 0;   // staging for rt3d_conv3d_host
  void* stage_y = nullptr; size_t stage_y_bytes = 0;
  float* stage_bias = nullptr;
  // rt3d_conv3d_host pipelines a large batch in chunks: copy-in and copy-out streams and events
  // (cudaStream_t / cudaEvent_t, created on first use)
  void* host_streams[2] = {nullptr, nullptr};
  void* host_events[18] = {};
};

}  // namespace rt3d

struct rt3d_packed {
  int M = 0, N = 0, Kt = 0, Kh = 0, Kw = 0, g_m = 0, g_n = 0, P = 0, Q = 0, Ks = 0;
  int dtype = 0, is_vanilla = 0, is_dense = 0;
  int64_t nnz = 0;
  std::vector<int32_t> group_ptr;
  std::vector<uint16_t> pos_idx;
  std::vector<unsigned char> tiles;  // nnz * g_m * g_n elements of float or bf16 bits
  std::mutex mu;                     // guards the lazily built members below
  std::map<int, rt3d::UmmaLayout> umma_layouts;   // keyed by n_tile (+ 4096: the t-grouped order)
  std::map<int, rt3d::SubLayout> sub_layouts;     // keyed by n_tile
  std::map<int, rt3d::SmallCLayout> smallc_layouts;   // keyed by sh*16+sw, built on first use
  std::vector<rt3d::DeviceBlob*> blobs;
};

namespace rt3d {

// Default bundle width for M output channels: as few bundles as possible with n_tile <= 256.
int default_n_tile(int M);
// Builds (or returns the cached) tensor-core layout; nullptr if the handle cannot use it.
const UmmaLayout* get_umma_layout(rt3d_packed* p, int n_tile, bool t_groups = false);
bool umma_layout_possible(const rt3d_packed* p);
// Builds (or returns the cached) layout of the sub-tile kernel; nullptr if the handle cannot use it.
const SubLayout* get_sub_layout(rt3d_packed* p, int n_tile);

// Small-C_in layout (nullptr if the handle does not qualify: needs bf16, N <= 8, M <= 256).
const SmallCLayout* get_smallc_layout(rt3d_packed* p, int sh, int sw);

}  // namespace rt3d
