// Data-free part of the paper's pruning step, run where the weights already are (Section 4):
// the group-lasso norm of every (kernel group, kernel location), the reweighted penalty
// 1 / (norm^2 + eps) of the update rule below Eq. 3, the keep / prune decision norm > threshold,
// and the expansion of that group-level decision to the per-weight mask rt3d_pack_kgs takes.
// Bandwidth-bound kernels: the weight tensor is read once.
#include <cuda_runtime.h>

#include <atomic>

#include "rt3d.h"

namespace {

// One thread per (group, location): consecutive threads walk consecutive kernel locations, so the
// reads of a warp are contiguous runs of the [M][N][Ks] weight tensor.  GM x GN > 0: compile-time group
// size (all loads of a thread independent and in flight together); 0: run-time size.
template <int G, int GM, int GN>
__global__ void group_norms_kernel(const float* __restrict__ w, int M, int N, int Ks, int g_m_rt, int g_n_rt, int Q,
                                   float* __restrict__ norms, long long total) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int g_m = GM ? GM : g_m_rt, g_n = GN ? GN : g_n_rt;
  const int k = int(idx % Ks);
  const long long pq = idx / Ks;
  const int q = int(pq % Q), p = int(pq / Q);
  float s = 0.f;
  if (GM && GN && (p + 1) * GM <= M && (q + 1) * GN <= N) {
    float v[(GM ? GM : 1) * (GN ? GN : 1)];
#pragma unroll
    for (int i = 0; i < GM; ++i)
#pragma unroll
      for (int j = 0; j < GN; ++j)
        v[i * GN + j] = fabsf(__ldg(w + ((long long)(p * GM + i) * N + (q * GN + j)) * Ks + k));
#pragma unroll
    for (int e = 0; e < GM * GN; ++e) s += (G == 1) ? v[e] : v[e] * v[e];
  } else {
    for (int i = 0; i < g_m; ++i) {
      const int m = p * g_m + i;
      if (m >= M) break;
      for (int j = 0; j < g_n; ++j) {
        const int c = q * g_n + j;
        if (c >= N) break;
        const float v = fabsf(__ldg(w + ((long long)m * N + c) * Ks + k));
        s += (G == 1) ? v : v * v;
      }
    }
  }
  norms[idx] = (G == 1) ? s : sqrtf(s);
}

template <int G>
void launch_group_norms(const float* w, int M, int N, int Ks, int g_m, int g_n, int Q, float* norms, long long total,
                        cudaStream_t st) {
  const int threads = 256;
  const unsigned blocks = unsigned((total + threads - 1) / threads);
  if (g_m == 4 && g_n == 4) group_norms_kernel<G, 4, 4><<<blocks, threads, 0, st>>>(w, M, N, Ks, g_m, g_n, Q, norms, total);
  else if (g_m == 8 && g_n == 4) group_norms_kernel<G, 8, 4><<<blocks, threads, 0, st>>>(w, M, N, Ks, g_m, g_n, Q, norms, total);
  else if (g_m == 8 && g_n == 8) group_norms_kernel<G, 8, 8><<<blocks, threads, 0, st>>>(w, M, N, Ks, g_m, g_n, Q, norms, total);
  else group_norms_kernel<G, 0, 0><<<blocks, threads, 0, st>>>(w, M, N, Ks, g_m, g_n, Q, norms, total);
}

__global__ void reweight_kernel(const float* __restrict__ norms, long long count, float eps, float threshold,
                                float* __restrict__ penalty, uint8_t* __restrict__ keep) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= count) return;
  const float n = norms[idx];
  if (penalty) penalty[idx] = 1.f / (n * n + eps);
  if (keep) keep[idx] = n > threshold ? 1 : 0;
}

__global__ void expand_mask_kernel(const uint8_t* __restrict__ gmask, int M, int N, int Ks, int g_m, int g_n, int Q,
                                   uint8_t* __restrict__ mask, long long total) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int k = int(idx % Ks);
  const long long mc = idx / Ks;
  const int c = int(mc % N), m = int(mc / N);
  mask[idx] = gmask[((long long)(m / g_m) * Q + c / g_n) * Ks + k];
}

}  // namespace

extern "C" {

rt3d_status rt3d_kgs_group_norms(const float* w, int M, int N, int Kt, int Kh, int Kw, int g_m, int g_n, int norm,
                                 float* norms, void* stream) {
  if (!w || !norms || M <= 0 || N <= 0 || Kt <= 0 || Kh <= 0 || Kw <= 0 || g_m <= 0 || g_n <= 0) return RT3D_ERR_INVALID_ARG;
  if (norm != 1 && norm != 2) return RT3D_ERR_INVALID_ARG;
  const int Ks = Kt * Kh * Kw;
  const int P = (M + g_m - 1) / g_m, Q = (N + g_n - 1) / g_n;
  const long long total = (long long)P * Q * Ks;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (norm == 1) launch_group_norms<1>(w, M, N, Ks, g_m, g_n, Q, norms, total, st);
  else launch_group_norms<2>(w, M, N, Ks, g_m, g_n, Q, norms, total, st);
  return cudaGetLastError() == cudaSuccess ? RT3D_OK : RT3D_ERR_CUDA;
}

rt3d_status rt3d_kgs_reweight(const float* norms, int64_t count, float eps, float threshold, float* penalty,
                              uint8_t* keep, void* stream) {
  if (!norms || count <= 0 || (!penalty && !keep) || !(eps > 0.f)) return RT3D_ERR_INVALID_ARG;
  const int threads = 256;
  reweight_kernel<<<unsigned((count + threads - 1) / threads), threads, 0, static_cast<cudaStream_t>(stream)>>>(
      norms, count, eps, threshold, penalty, keep);
  return cudaGetLastError() == cudaSuccess ? RT3D_OK : RT3D_ERR_CUDA;
}

rt3d_status rt3d_kgs_expand_mask(const uint8_t* group_mask, int M, int N, int Kt, int Kh, int Kw, int g_m, int g_n,
                                 uint8_t* mask, void* stream) {
  if (!group_mask || !mask || M <= 0 || N <= 0 || Kt <= 0 || Kh <= 0 || Kw <= 0 || g_m <= 0 || g_n <= 0) return RT3D_ERR_INVALID_ARG;
  const int Ks = Kt * Kh * Kw;
  const int Q = (N + g_n - 1) / g_n;
  const long long total = (long long)M * N * Ks;
  const int threads = 256;
  expand_mask_kernel<<<unsigned((total + threads - 1) / threads), threads, 0, static_cast<cudaStream_t>(stream)>>>(
      group_mask, M, N, Ks, g_m, g_n, Q, mask, total);
  return cudaGetLastError() == cudaSuccess ? RT3D_OK : RT3D_ERR_CUDA;
}

}  // extern "C"
