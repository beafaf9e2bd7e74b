// Tile constants shared by the host-side packer and the kernels.
#pragma once
namespace rt3d {
constexpr int kSmallCTileH = 16, kSmallCTileW = 8;   // output tile of the small-C_in kernel: 1 x 16 x 8 voxels

// Sub-tile kernel (umma_conv_sub.cu): a bundle's output channels are cut into ranges of 16, a 64-channel chunk
// into four K slices of 16; a (range, slice) block of a K step exists only where a kernel group keeps the
// step's kernel location inside it.
constexpr int kSubRange = 16;            // output channels per range = N of the smallest MMA
constexpr int kSubBlockElems = 256;      // one block: 16 output channels x 16 input channels, bf16
constexpr int kSubBlockBytes = 512;
constexpr int kSubHeaderBytes = 64;      // per step: one command byte per (range, K slice)
// One K step (kernel location x 64-channel chunk) of a bundle.  Its payload in the block array starts at byte
// 64 * off64 and consists of a 64-byte header followed by `nblk` blocks of 512 bytes.  Header byte 4 r + ks
// belongs to range r and K slice ks: bit 7 = the block exists, bits 0..5 = its index among the step's blocks.
// In the first step of a bundle every range has a block in K slice 0 (a zero block if no kernel group feeds
// it), so the MMA of (first step, slice 0) overwrites the accumulator and every other one adds to it.
struct SubStep {
  int enc;                               // encode_step(kt, kh, kw, chunk)
  unsigned off64;
  int nblk;
  int pad;
};
}  // namespace rt3d
