// Tile constants shared by the host-side packer and the kernels.
#pragma once
namespace rt3d {
constexpr int kSmallCTileH = 16, kSmallCTileW = 8;   // output tile of the small-C_in kernel: 1 x 16 x 8 voxels
}  // namespace rt3d
