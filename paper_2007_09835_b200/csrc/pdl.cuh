// Programmatic dependent launch for the kernels of a layer sequence.
//
// A forward pass is dozens of short kernels on one stream; between two of them the GPU idles for the launch
// latency of the second.  Every kernel of the network path is therefore launched with the programmatic
// stream-serialisation attribute and begins with pdl_entry(): it lets ITS successor be scheduled at once
// (launch_dependents) and then waits until its predecessor has completed and flushed its memory
// (griddepcontrol.wait) before touching any global memory; the tensor-core kernels first initialise their
// barriers and allocate TMEM, which overlaps the predecessor's tail.  The successor's CTAs thus sit ready on SMs as
// these free up; nothing is read or written earlier than it would be without the attribute, so results are
// unchanged.  A successor is scheduled only once all CTAs of its predecessor have started, and our grids
// are at most one resident wave (or short-lived CTAs), so waiting CTAs cannot starve the kernel they wait for.
// RT3D_PDL=0 in the environment turns the launch attribute off (the device instructions are then no-ops).
#pragma once

#include <cstdlib>
#include <cuda_runtime.h>

namespace rt3d {

// The successor may be scheduled.  The tensor-core kernels call this only after their TMEM allocation: a
// successor's CTA that became resident on the same SM and allocated TMEM first could otherwise block a CTA of
// the kernel it is waiting for.
__device__ __forceinline__ void pdl_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
// Before the first access to global memory: the predecessor has completed and its writes are visible.
// Set-up that touches only shared memory, barriers and TMEM may run before it.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_entry() { pdl_launch(); pdl_wait(); }

// One-time set-up that CUDA keeps per device (function attributes, occupancy answers): index of the current
// device, or -1.  The launchers keep their "done" flags and cached values in arrays of kMaxDevices entries.
constexpr int kMaxDevices = 64;
inline int current_device_index() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
  return dev;
}

inline bool pdl_enabled() {
  static const bool on = [] {
    const char* e = getenv("RT3D_PDL");
    return !(e && e[0] == '0');
  }();
  return on;
}

// cudaLaunchConfig_t with the optional cluster dimension and the programmatic-serialisation attribute.
struct LaunchSetup {
  cudaLaunchConfig_t cfg;
  cudaLaunchAttribute attr[2];
  LaunchSetup(dim3 grid, dim3 block, size_t smem, cudaStream_t stream, unsigned cluster_x = 1) {
    cfg = cudaLaunchConfig_t{};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    unsigned n = 0;
    if (cluster_x > 1) {
      attr[n].id = cudaLaunchAttributeClusterDimension;
      attr[n].val.clusterDim.x = cluster_x; attr[n].val.clusterDim.y = 1; attr[n].val.clusterDim.z = 1;
      ++n;
    }
    if (pdl_enabled()) {
      attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr[n].val.programmaticStreamSerializationAllowed = 1;
      ++n;
    }
    cfg.attrs = attr; cfg.numAttrs = n;
  }
};

}  // namespace rt3d
