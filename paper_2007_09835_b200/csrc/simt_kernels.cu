// CUDA-core kernels: the index-driven KGS convolution (any shape, fp32 or bf16 storage, fp32
// accumulation), 3-D max-pool and add(+ReLU) over NDHWC tensors.
//
// The convolution follows the group view of Section 3 of the paper directly: one thread owns
// one output voxel and one row of kernel groups (g_m output channels); for every kernel
// group of that row it walks the kept kernel locations of the packed index and applies the
// group's g_m x g_n weight tile to the g_n input channels at the shifted voxel.  Pruned
// locations are never visited.  It is the cross-check for the tensor-core kernel and the
// production path for shapes that kernel does not take.
#include <cuda_bf16.h>

#include "kernels.h"
#include "pdl.cuh"

namespace rt3d {
namespace {

constexpr int kThreads = 128;

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// GM/GN > 0: compile-time group size; 0: run-time size (<= 8).
// All threads of a block work on the same row p of kernel groups, so the row's packed index and weight tiles are
// staged once per block in shared memory (in pieces of kStageEntries kept entries across the row's Q groups, which
// are contiguous in the packed arrays), with each kept location
// decoded to its (kt, kh, kw) there: the inner loop then has no integer division and no dependent global load
// besides the input voxel itself, which is fetched with one 16-byte load when the group is four channels wide.
constexpr int kStageEntries = 64;

template <typename T, int GM, int GN, bool DENSE>
__global__ void __launch_bounds__(kThreads)
conv3d_kgs_simt_kernel(ConvGeom g, const T* __restrict__ x, T* __restrict__ y,
                       const int32_t* __restrict__ group_ptr, const uint16_t* __restrict__ pos_idx,
                       const T* __restrict__ tiles, const float* __restrict__ bias,
                       int g_m_rt, int g_n_rt, int Q, long long total_voxels, const T* __restrict__ residual, int rcs) {
  pdl_entry();
  constexpr int MAXM = GM ? GM : 8;
  constexpr int MAXN = GN ? GN : 8;
  __shared__ float w_s[kStageEntries * MAXM * MAXN];
  __shared__ int off_s[kStageEntries];             // (kt << 20) | (kh << 10) | kw
  __shared__ int c0_s[kStageEntries];              // first input channel of the entry's group
  const int g_m = GM ? GM : g_m_rt;
  const int g_n = GN ? GN : g_n_rt;
  const int p = blockIdx.y;
  const long long v = (long long)blockIdx.x * kThreads + threadIdx.x;
  const bool valid = v < total_voxels;
  int wo = 0, ho = 0, to = 0, nn = 0;
  if (valid) {
    long long r = v;
    wo = int(r % g.Wo); r /= g.Wo;
    ho = int(r % g.Ho); r /= g.Ho;
    to = int(r % g.To); nn = int(r / g.To);
  }
  const int t0 = to * g.st - g.pt, h0 = ho * g.sh - g.ph, w0 = wo * g.sw - g.pw;
  float acc[MAXM];
#pragma unroll
  for (int i = 0; i < MAXM; ++i) acc[i] = 0.f;

  const int tile_elems = g_m * g_n;
  const bool vec4 = GN == 4 && sizeof(T) == 4 && (g.xcs & 3) == 0 && (g.c & 3) == 0;
  // the kept entries of all Q groups of row p are one contiguous range of the packed arrays
  const int row0 = group_ptr[p * Q], row1 = group_ptr[p * Q + Q];
  for (int eb = row0; eb < row1; eb += kStageEntries) {
    const int n_e = row1 - eb < kStageEntries ? row1 - eb : kStageEntries;
    __syncthreads();                               // the previous piece has been consumed
    for (int i = threadIdx.x; i < n_e * tile_elems; i += kThreads) {
      const int e = i / tile_elems, k = i - e * tile_elems;
      w_s[e * (MAXM * MAXN) + (k / g_n) * MAXN + k % g_n] = to_f32<T>(tiles[(long long)(eb + e) * tile_elems + k]);
    }
    for (int e = threadIdx.x; e < n_e; e += kThreads) {
      int q = 0;                                     // the group this entry belongs to
      while (q + 1 < Q && group_ptr[p * Q + q + 1] <= eb + e) ++q;
      const int kpos = DENSE ? (eb + e - group_ptr[p * Q + q]) : int(pos_idx[eb + e]);
      off_s[e] = ((kpos / (g.Kw * g.Kh)) << 20) | (((kpos / g.Kw) % g.Kh) << 10) | (kpos % g.Kw);
      c0_s[e] = q * g_n;
    }
    __syncthreads();
#pragma unroll 4
    for (int e = 0; e < n_e; ++e) {
      const int off = off_s[e], c0 = c0_s[e];
      const int ti = t0 + (off >> 20), hi = h0 + ((off >> 10) & 1023), wi = w0 + (off & 1023);
      const bool inb = valid && unsigned(ti) < unsigned(g.t) && unsigned(hi) < unsigned(g.h) && unsigned(wi) < unsigned(g.w);
      const T* xp = x + ((((long long)nn * g.t + (inb ? ti : 0)) * g.h + (inb ? hi : 0)) * g.w + (inb ? wi : 0)) * g.xcs + c0;
      float xv[MAXN];
      if (vec4) {
        const float4 t4 = inb ? __ldg(reinterpret_cast<const float4*>(xp)) : make_float4(0.f, 0.f, 0.f, 0.f);
        xv[0] = t4.x; xv[1] = t4.y; xv[2] = t4.z; xv[3] = t4.w;
#pragma unroll
        for (int j = 4; j < MAXN; ++j) xv[j] = 0.f;
      } else {
#pragma unroll
        for (int j = 0; j < MAXN; ++j) xv[j] = (inb && j < g_n && c0 + j < g.c) ? to_f32<T>(xp[j]) : 0.f;
      }
      const float* tp = w_s + e * (MAXM * MAXN);
#pragma unroll
      for (int i = 0; i < MAXM; ++i) {
        if (i < g_m) {
#pragma unroll
          for (int j = 0; j < MAXN; ++j)
            if (j < g_n) acc[i] = fmaf(xv[j], tp[i * MAXN + j], acc[i]);
        }
      }
    }
  }
  if (!valid) return;
  T* yp = y + v * g.ycs + p * g_m;
#pragma unroll
  for (int i = 0; i < MAXM; ++i) {
    const int m = p * g_m + i;
    if (i < g_m && m < g.M) {
      float r = acc[i] + (bias ? bias[m] : 0.f);
      if (residual) r += to_f32<T>(residual[v * rcs + m]);
      if (g.relu) r = fmaxf(r, 0.f);
      yp[i] = from_f32<T>(r);
    }
  }
}

template <typename T, bool DENSE>
cudaError_t launch_conv_t(const ConvGeom& g, const void* x, void* y, const int32_t* group_ptr,
                          const uint16_t* pos_idx, const void* tiles, const float* bias, int g_m, int g_n,
                          int P, int Q, const void* residual, int rcs, cudaStream_t stream) {
  const long long total = (long long)g.n * g.To * g.Ho * g.Wo;
  if (total == 0) return cudaSuccess;
  dim3 grid((unsigned)((total + kThreads - 1) / kThreads), (unsigned)P);
  const T* xt = static_cast<const T*>(x);
  T* yt = static_cast<T*>(y);
  const T* tt = static_cast<const T*>(tiles);
  LaunchSetup ls(grid, dim3(kThreads), 0, stream);
  const T* rt = static_cast<const T*>(residual);
  cudaError_t le = cudaSuccess;
#define RT3D_LAUNCH(GM_, GN_) \
  le = cudaLaunchKernelEx(&ls.cfg, conv3d_kgs_simt_kernel<T, GM_, GN_, DENSE>, g, xt, yt, group_ptr, pos_idx, tt, bias, g_m, g_n, Q, total, rt, rcs)
  if (g_m == 4 && g_n == 4) RT3D_LAUNCH(4, 4);
  else if (g_m == 8 && g_n == 4) RT3D_LAUNCH(8, 4);
  else if (g_m == 8 && g_n == 8) RT3D_LAUNCH(8, 8);
  else RT3D_LAUNCH(0, 0);
#undef RT3D_LAUNCH
  return le;
}

// ------------------------------------------------------------------------------- max-pool
template <typename T>
__global__ void maxpool3d_kernel(const T* __restrict__ x, int t, int h, int w, int c, int xcs,
                                 int kt, int kh, int kw, int st, int sh, int sw, int pt, int ph, int pw,
                                 T* __restrict__ y, int To, int Ho, int Wo, int ycs, long long total) {
  pdl_entry();
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int cc = int(idx % c);
  long long r = idx / c;
  const int wo = int(r % Wo); r /= Wo;
  const int ho = int(r % Ho); r /= Ho;
  const int to = int(r % To);
  const int nn = int(r / To);
  float best = -INFINITY;
  for (int a = 0; a < kt; ++a) {
    const int ti = to * st - pt + a;
    if (ti < 0 || ti >= t) continue;
    for (int b = 0; b < kh; ++b) {
      const int hi = ho * sh - ph + b;
      if (hi < 0 || hi >= h) continue;
      for (int d = 0; d < kw; ++d) {
        const int wi = wo * sw - pw + d;
        if (wi < 0 || wi >= w) continue;
        best = fmaxf(best, to_f32<T>(x[((((long long)nn * t + ti) * h + hi) * w + wi) * xcs + cc]));
      }
    }
  }
  y[((((long long)nn * To + to) * Ho + ho) * Wo + wo) * ycs + cc] = from_f32<T>(best);
}

// Same for a window known at compile time: all loads of the window are issued together (clamped address,
// result masked to -inf outside the tensor) instead of one after the other behind run-time branches.
template <int KT, int KH, int KW>
__global__ void maxpool3d_bf16x8_win_kernel(const uint4* __restrict__ x, int t, int h, int w, int c8, int xcs8,
                                            int st, int sh, int sw, int pt, int ph, int pw,
                                            uint4* __restrict__ y, int To, int Ho, int Wo, int ycs8, long long total) {
  pdl_entry();
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int cc = int(idx % c8);
  long long r = idx / c8;
  const int wo = int(r % Wo); r /= Wo;
  const int ho = int(r % Ho); r /= Ho;
  const int to = int(r % To);
  const int nn = int(r / To);
  const int t0 = to * st - pt, h0 = ho * sh - ph, w0 = wo * sw - pw;
  uint4 v[KT * KH * KW];
  bool ok[KT * KH * KW];
#pragma unroll
  for (int a = 0; a < KT; ++a)
#pragma unroll
    for (int b = 0; b < KH; ++b)
#pragma unroll
      for (int d = 0; d < KW; ++d) {
        const int ti = t0 + a, hi = h0 + b, wi = w0 + d;
        const bool in = ti >= 0 && ti < t && hi >= 0 && hi < h && wi >= 0 && wi < w;
        const int tc = min(max(ti, 0), t - 1), hc = min(max(hi, 0), h - 1), wc = min(max(wi, 0), w - 1);
        ok[(a * KH + b) * KW + d] = in;
        v[(a * KH + b) * KW + d] = __ldg(x + ((((long long)nn * t + tc) * h + hc) * w + wc) * xcs8 + cc);
      }
  const __nv_bfloat162 ninf = __float2bfloat162_rn(-INFINITY);
  __nv_bfloat162 best[4] = {ninf, ninf, ninf, ninf};
#pragma unroll
  for (int i = 0; i < KT * KH * KW; ++i) {
    const __nv_bfloat162* pv = reinterpret_cast<const __nv_bfloat162*>(&v[i]);
#pragma unroll
    for (int k = 0; k < 4; ++k) best[k] = ok[i] ? __hmax2(best[k], pv[k]) : best[k];
  }
  uint4 out;
  __nv_bfloat162* po = reinterpret_cast<__nv_bfloat162*>(&out);
#pragma unroll
  for (int k = 0; k < 4; ++k) po[k] = best[k];
  y[((((long long)nn * To + to) * Ho + ho) * Wo + wo) * ycs8 + cc] = out;
}

// Unit stride along w: a thread produces WB consecutive outputs of one image row.  The windows of neighbouring
// outputs share KW - 1 columns, so the (t, h) maximum of each of the WB + KW - 1 input columns is formed once and
// every output is the maximum of KW adjacent column maxima: (WB + KW - 1) * KT * KH loads for WB outputs instead
// of WB * KT * KH * KW (a 3x3x3 stride-1 pool is bound by L1 bandwidth: 27 loads of 16 bytes per 16 bytes written).
template <int KT, int KH, int KW, int WB>
__global__ void maxpool3d_bf16x8_row_kernel(const uint4* __restrict__ x, int t, int h, int w, int c8, int xcs8,
                                            int st, int sh, int pt, int ph, int pw,
                                            uint4* __restrict__ y, int To, int Ho, int Wo, int ycs8, int w_blocks, long long total) {
  pdl_entry();
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int cc = int(idx % c8);
  long long r = idx / c8;
  const int wb = int(r % w_blocks); r /= w_blocks;
  const int ho = int(r % Ho); r /= Ho;
  const int to = int(r % To);
  const int nn = int(r / To);
  const int t0 = to * st - pt, h0 = ho * sh - ph, w0 = wb * WB - pw;
  const __nv_bfloat162 ninf = __float2bfloat162_rn(-INFINITY);
  __nv_bfloat162 cm[WB + KW - 1][4];
#pragma unroll
  for (int d = 0; d < WB + KW - 1; ++d) {
    const int wi = w0 + d;
    const bool w_in = wi >= 0 && wi < w;
    const int wc = min(max(wi, 0), w - 1);
    uint4 v[KT * KH];
    bool ok[KT * KH];
#pragma unroll
    for (int a = 0; a < KT; ++a)
#pragma unroll
      for (int b = 0; b < KH; ++b) {
        const int ti = t0 + a, hi = h0 + b;
        ok[a * KH + b] = w_in && ti >= 0 && ti < t && hi >= 0 && hi < h;
        const int tc = min(max(ti, 0), t - 1), hc = min(max(hi, 0), h - 1);
        v[a * KH + b] = __ldg(x + ((((long long)nn * t + tc) * h + hc) * w + wc) * xcs8 + cc);
      }
#pragma unroll
    for (int k = 0; k < 4; ++k) cm[d][k] = ninf;
#pragma unroll
    for (int i = 0; i < KT * KH; ++i) {
      const __nv_bfloat162* pv = reinterpret_cast<const __nv_bfloat162*>(&v[i]);
#pragma unroll
      for (int k = 0; k < 4; ++k) cm[d][k] = ok[i] ? __hmax2(cm[d][k], pv[k]) : cm[d][k];
    }
  }
  uint4* yrow = y + ((((long long)nn * To + to) * Ho + ho) * Wo) * ycs8 + cc;
#pragma unroll
  for (int j = 0; j < WB; ++j) {
    const int wo = wb * WB + j;
    if (wo >= Wo) break;
    uint4 out;
    __nv_bfloat162* po = reinterpret_cast<__nv_bfloat162*>(&out);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      __nv_bfloat162 m = cm[j][k];
#pragma unroll
      for (int d = 1; d < KW; ++d) m = __hmax2(m, cm[j + d][k]);
      po[k] = m;
    }
    yrow[(long long)wo * ycs8] = out;
  }
}

// bf16, 8 channels (16 bytes) per thread; needs c % 8 == 0 and 8-element pitches.
__global__ void maxpool3d_bf16x8_kernel(const uint4* __restrict__ x, int t, int h, int w, int c8, int xcs8,
                                        int kt, int kh, int kw, int st, int sh, int sw, int pt, int ph, int pw,
                                        uint4* __restrict__ y, int To, int Ho, int Wo, int ycs8, long long total) {
  pdl_entry();
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int cc = int(idx % c8);
  long long r = idx / c8;
  const int wo = int(r % Wo); r /= Wo;
  const int ho = int(r % Ho); r /= Ho;
  const int to = int(r % To);
  const int nn = int(r / To);
  const __nv_bfloat162 ninf = __float2bfloat162_rn(-INFINITY);
  __nv_bfloat162 best[4] = {ninf, ninf, ninf, ninf};
  for (int a = 0; a < kt; ++a) {
    const int ti = to * st - pt + a;
    if (ti < 0 || ti >= t) continue;
    for (int b = 0; b < kh; ++b) {
      const int hi = ho * sh - ph + b;
      if (hi < 0 || hi >= h) continue;
      for (int d = 0; d < kw; ++d) {
        const int wi = wo * sw - pw + d;
        if (wi < 0 || wi >= w) continue;
        const uint4 v = __ldg(x + ((((long long)nn * t + ti) * h + hi) * w + wi) * xcs8 + cc);
        const __nv_bfloat162* pv = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
        for (int k = 0; k < 4; ++k) best[k] = __hmax2(best[k], pv[k]);
      }
    }
  }
  uint4 out;
  __nv_bfloat162* po = reinterpret_cast<__nv_bfloat162*>(&out);
#pragma unroll
  for (int k = 0; k < 4; ++k) po[k] = best[k];
  y[((((long long)nn * To + to) * Ho + ho) * Wo + wo) * ycs8 + cc] = out;
}

// ----------------------------------------------------------------------------- add + relu
template <typename T>
__global__ void add_relu_kernel(const T* __restrict__ a, int acs, const T* __restrict__ b, int bcs,
                                T* __restrict__ y, int ycs, int c, int relu, long long total) {
  pdl_entry();
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int cc = int(idx % c);
  const long long v = idx / c;
  float r = to_f32<T>(a[v * acs + cc]) + to_f32<T>(b[v * bcs + cc]);
  if (relu) r = fmaxf(r, 0.f);
  y[v * ycs + cc] = from_f32<T>(r);
}

__global__ void add_relu_bf16x8_kernel(const uint4* __restrict__ a, int acs8, const uint4* __restrict__ b,
                                       int bcs8, uint4* __restrict__ y, int ycs8, int c8, int relu,
                                       long long total) {
  pdl_entry();
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int cc = int(idx % c8);
  const long long v = idx / c8;
  const uint4 va = a[v * acs8 + cc], vb = b[v * bcs8 + cc];
  const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&va);
  const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&vb);
  uint4 out;
  __nv_bfloat162* po = reinterpret_cast<__nv_bfloat162*>(&out);
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    float2 fa = __bfloat1622float2(pa[k]), fb = __bfloat1622float2(pb[k]);
    float2 r = make_float2(fa.x + fb.x, fa.y + fb.y);
    if (relu) { r.x = fmaxf(r.x, 0.f); r.y = fmaxf(r.y, 0.f); }
    po[k] = __float22bfloat162_rn(r);
  }
  y[v * ycs8 + cc] = out;
}

}  // namespace

cudaError_t launch_conv_simt(int dtype, const ConvGeom& g, const void* x, void* y, const int32_t* group_ptr,
                             const uint16_t* pos_idx, const void* tiles, const float* bias, int g_m, int g_n,
                             int P, int Q, bool dense, const void* residual, int rcs, cudaStream_t stream) {
  if (dtype == 0)
    return dense ? launch_conv_t<float, true>(g, x, y, group_ptr, pos_idx, tiles, bias, g_m, g_n, P, Q, residual, rcs, stream)
                 : launch_conv_t<float, false>(g, x, y, group_ptr, pos_idx, tiles, bias, g_m, g_n, P, Q, residual, rcs, stream);
  return dense ? launch_conv_t<__nv_bfloat16, true>(g, x, y, group_ptr, pos_idx, tiles, bias, g_m, g_n, P, Q, residual, rcs, stream)
               : launch_conv_t<__nv_bfloat16, false>(g, x, y, group_ptr, pos_idx, tiles, bias, g_m, g_n, P, Q, residual, rcs, stream);
}

cudaError_t launch_maxpool3d(int dtype, const void* x, int n, int t, int h, int w, int c, int xcs,
                             int kt, int kh, int kw, int st, int sh, int sw, int pt, int ph, int pw,
                             void* y, int To, int Ho, int Wo, int ycs, cudaStream_t stream) {
  const long long vox = (long long)n * To * Ho * Wo;
  if (vox == 0) return cudaSuccess;
  const int threads = 256;
  if (dtype == 1 && c % 8 == 0 && xcs % 8 == 0 && ycs % 8 == 0) {
    const long long total = vox * (c / 8);
    LaunchSetup ls(dim3((unsigned)((total + threads - 1) / threads)), dim3(threads), 0, stream);
    if (sw == 1 && kw == 3 && kh == 3 && (kt == 3 || kt == 1) && Wo >= 4) {       // unit stride along w: shared column maxima
      const int w_blocks = (Wo + 3) / 4;
      const long long total_r = (long long)n * To * Ho * w_blocks * (c / 8);
      LaunchSetup lr(dim3((unsigned)((total_r + threads - 1) / threads)), dim3(threads), 0, stream);
      if (kt == 3)
        return cudaLaunchKernelEx(&lr.cfg, maxpool3d_bf16x8_row_kernel<3, 3, 3, 4>, static_cast<const uint4*>(x), t, h, w, c / 8,
                                  xcs / 8, st, sh, pt, ph, pw, static_cast<uint4*>(y), To, Ho, Wo, ycs / 8, w_blocks, total_r);
      return cudaLaunchKernelEx(&lr.cfg, maxpool3d_bf16x8_row_kernel<1, 3, 3, 4>, static_cast<const uint4*>(x), t, h, w, c / 8,
                                xcs / 8, st, sh, pt, ph, pw, static_cast<uint4*>(y), To, Ho, Wo, ycs / 8, w_blocks, total_r);
    }
#define RT3D_POOL_WIN(KT_, KH_, KW_)                                                                                   \
  if (kt == KT_ && kh == KH_ && kw == KW_)                                                                              \
    return cudaLaunchKernelEx(&ls.cfg, maxpool3d_bf16x8_win_kernel<KT_, KH_, KW_>, static_cast<const uint4*>(x), t, h, w, \
                              c / 8, xcs / 8, st, sh, sw, pt, ph, pw, static_cast<uint4*>(y), To, Ho, Wo, ycs / 8, total)
    RT3D_POOL_WIN(3, 3, 3);
    RT3D_POOL_WIN(1, 3, 3);
    RT3D_POOL_WIN(2, 2, 2);
    RT3D_POOL_WIN(1, 2, 2);
#undef RT3D_POOL_WIN
    return cudaLaunchKernelEx(&ls.cfg, maxpool3d_bf16x8_kernel, static_cast<const uint4*>(x), t, h, w, c / 8, xcs / 8, kt, kh, kw,
                              st, sh, sw, pt, ph, pw, static_cast<uint4*>(y), To, Ho, Wo, ycs / 8, total);
  } else {
    const long long total = vox * c;
    const unsigned blocks = (unsigned)((total + threads - 1) / threads);
    LaunchSetup ls(dim3(blocks), dim3(threads), 0, stream);
    if (dtype == 0)
      return cudaLaunchKernelEx(&ls.cfg, maxpool3d_kernel<float>, static_cast<const float*>(x), t, h, w, c, xcs, kt, kh, kw,
                                st, sh, sw, pt, ph, pw, static_cast<float*>(y), To, Ho, Wo, ycs, total);
    return cudaLaunchKernelEx(&ls.cfg, maxpool3d_kernel<__nv_bfloat16>, static_cast<const __nv_bfloat16*>(x), t, h, w, c, xcs,
                              kt, kh, kw, st, sh, sw, pt, ph, pw, static_cast<__nv_bfloat16*>(y), To, Ho, Wo, ycs, total);
  }
}

cudaError_t launch_add_relu(int dtype, const void* a, int acs, const void* b, int bcs, void* y, int ycs,
                            int64_t voxels, int c, int relu, cudaStream_t stream) {
  if (voxels == 0) return cudaSuccess;
  const int threads = 256;
  if (dtype == 1 && c % 8 == 0 && acs % 8 == 0 && bcs % 8 == 0 && ycs % 8 == 0) {
    const long long total = voxels * (c / 8);
    LaunchSetup ls(dim3((unsigned)((total + threads - 1) / threads)), dim3(threads), 0, stream);
    return cudaLaunchKernelEx(&ls.cfg, add_relu_bf16x8_kernel, static_cast<const uint4*>(a), acs / 8, static_cast<const uint4*>(b),
                              bcs / 8, static_cast<uint4*>(y), ycs / 8, c / 8, relu, total);
  } else {
    const long long total = voxels * c;
    const unsigned blocks = (unsigned)((total + threads - 1) / threads);
    LaunchSetup ls(dim3(blocks), dim3(threads), 0, stream);
    if (dtype == 0)
      return cudaLaunchKernelEx(&ls.cfg, add_relu_kernel<float>, static_cast<const float*>(a), acs, static_cast<const float*>(b),
                                bcs, static_cast<float*>(y), ycs, c, relu, total);
    return cudaLaunchKernelEx(&ls.cfg, add_relu_kernel<__nv_bfloat16>, static_cast<const __nv_bfloat16*>(a), acs,
                              static_cast<const __nv_bfloat16*>(b), bcs, static_cast<__nv_bfloat16*>(y), ycs, c, relu, total);
  }
}

}  // namespace rt3d
