// C ABI of librt3d: argument validation, per-device weight upload, tile planning, TMA tensor
// maps and kernel dispatch.  All numerical work happens in the kernels launched from here.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <vector>

#include "kernels.h"
#include "rt3d_internal.h"

using namespace rt3d;

namespace {

std::atomic<int64_t> g_launches{0};
std::atomic<int64_t> g_allocs{0};            // device allocations made by this library (rt3d_alloc_count)

// Every device allocation of the library goes through here.
cudaError_t dev_malloc(void** p, size_t bytes) {
  g_allocs.fetch_add(1);
  return cudaMalloc(p, bytes);
}
template <typename T>
cudaError_t dev_malloc(T** p, size_t bytes) { return dev_malloc(reinterpret_cast<void**>(p), bytes); }

// Planning mode of the calling thread (rt3d_plan_begin / rt3d_plan_end): compute calls do everything they would do
// before their launch (choose the kernel, build and upload weight layouts, size the workspaces) and return.
thread_local bool t_plan_only = false;

// Test hooks of the single-CTA tensor-core kernel (rt3d_debug_set).
std::atomic<long long> g_debug_wait_cycles{-1};      // -1: not set yet (RT3D_DEBUG_TIMEOUT_POLLS is read on first use)
std::atomic<int> g_debug_drop_last_load{0};
// t-grouped CTA-pair variant: on unless the environment says RT3D_T_GROUPS=0; RT3D_DEBUG_T_GROUPS switches it at run time
std::atomic<int> g_ts_enabled{[] { const char* e = getenv("RT3D_T_GROUPS"); return (e && e[0] == '0') ? 0 : 1; }()};
long long debug_wait_cycles() {
  long long v = g_debug_wait_cycles.load();
  if (v < 0) {
    const char* e = getenv("RT3D_DEBUG_TIMEOUT_POLLS");
    v = e ? atoll(e) : 0;
    if (v < 0) v = 0;
    g_debug_wait_cycles.store(v);
  }
  return v;
}

// All device blobs of live handles: their K-split counters are cleared when a kernel reported a timeout.
std::mutex g_blobs_mu;
std::vector<DeviceBlob*> g_blobs;

struct DeviceState {
  bool init = false;
  int sm_count = 0;
  int cc_major = 0;
  int32_t* sched = nullptr;     // [256] words: [2] = error word written by kernels on a bounded-wait expiry
};
std::mutex g_dev_mu;
DeviceState g_dev[64];

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

rt3d_status get_device_state(DeviceState** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return RT3D_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_dev_mu);
  DeviceState& d = g_dev[dev];
  if (!d.init) {
    if (cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return RT3D_ERR_CUDA;
    if (cudaDeviceGetAttribute(&d.cc_major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return RT3D_ERR_CUDA;
    if (dev_malloc(&d.sched, 256 * sizeof(int32_t)) != cudaSuccess) return RT3D_ERR_ALLOC;
    if (cudaMemset(d.sched, 0, 256 * sizeof(int32_t)) != cudaSuccess) return RT3D_ERR_CUDA;
    if (!g_encode) {
      void* fn = nullptr;
      cudaDriverEntryPointQueryResult qres;
      if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn)
        return RT3D_ERR_CUDA;
      g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    d.init = true;
  }
  *out = &d;
  return RT3D_OK;
}

bool valid_dtype(int d) { return d == RT3D_F32 || d == RT3D_BF16; }
size_t elem_size(int d) { return d == RT3D_BF16 ? 2 : 4; }

rt3d_status check_tensor(const rt3d_tensor* t) {
  if (!t || !t->data) return RT3D_ERR_INVALID_ARG;
  if (t->n <= 0 || t->t <= 0 || t->h <= 0 || t->w <= 0 || t->c <= 0) return RT3D_ERR_INVALID_ARG;
  if (!valid_dtype(t->dtype) || t->c_stride < t->c) return RT3D_ERR_INVALID_ARG;
  return RT3D_OK;
}

int64_t tensor_span_bytes(const rt3d_tensor* t) {
  const int64_t vox = int64_t(t->n) * t->t * t->h * t->w;
  return ((vox - 1) * t->c_stride + t->c) * int64_t(elem_size(t->dtype));
}

rt3d_status make_geom(const rt3d_tensor* x, const rt3d_packed* w, const rt3d_conv_params* p, const rt3d_tensor* y,
                      ConvGeom* g) {
  rt3d_status s = check_tensor(x);
  if (s != RT3D_OK) return s;
  if (!w || !p) return RT3D_ERR_INVALID_ARG;
  if (p->st < 1 || p->sh < 1 || p->sw < 1 || p->pt < 0 || p->ph < 0 || p->pw < 0) return RT3D_ERR_INVALID_ARG;
  if (p->algo < RT3D_ALGO_AUTO || p->algo > RT3D_ALGO_UMMA_SUB) return RT3D_ERR_INVALID_ARG;
  if (x->c != w->N || x->dtype != w->dtype) return RT3D_ERR_SHAPE;
  const int64_t To = (int64_t(x->t) + 2 * p->pt - w->Kt) / p->st + 1;
  const int64_t Ho = (int64_t(x->h) + 2 * p->ph - w->Kh) / p->sh + 1;
  const int64_t Wo = (int64_t(x->w) + 2 * p->pw - w->Kw) / p->sw + 1;
  if (x->t + 2 * p->pt < w->Kt || x->h + 2 * p->ph < w->Kh || x->w + 2 * p->pw < w->Kw) return RT3D_ERR_SHAPE;
  if (int64_t(x->n) * x->t * x->h * x->w >= (int64_t(1) << 31)) return RT3D_ERR_UNSUPPORTED;
  g->n = x->n; g->t = x->t; g->h = x->h; g->w = x->w; g->c = x->c; g->xcs = x->c_stride;
  g->To = int(To); g->Ho = int(Ho); g->Wo = int(Wo); g->M = w->M; g->ycs = 0;
  g->Kt = w->Kt; g->Kh = w->Kh; g->Kw = w->Kw;
  g->st = p->st; g->sh = p->sh; g->sw = p->sw; g->pt = p->pt; g->ph = p->ph; g->pw = p->pw;
  g->relu = p->relu ? 1 : 0;
  if (y) {
    s = check_tensor(y);
    if (s != RT3D_OK) return s;
    if (y->n != x->n || y->t != To || y->h != Ho || y->w != Wo || y->c != w->M || y->dtype != w->dtype)
      return RT3D_ERR_SHAPE;
    g->ycs = y->c_stride;
  }
  return RT3D_OK;
}

// Alignment rules of the device entry points.
rt3d_status check_alignment(const rt3d_tensor* t) {
  const int mult = t->dtype == RT3D_BF16 ? 8 : 4;
  if (t->c_stride % mult) return RT3D_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(t->data) % 16) return RT3D_ERR_INVALID_ARG;
  return RT3D_OK;
}

bool overlaps(const rt3d_tensor* a, const rt3d_tensor* b) {
  const char* a0 = static_cast<const char*>(a->data);
  const char* b0 = static_cast<const char*>(b->data);
  return a0 < b0 + tensor_span_bytes(b) && b0 < a0 + tensor_span_bytes(a);
}

// ------------------------------------------------------------------------- device blobs
DeviceBlob* find_blob(rt3d_packed* h, int dev) {
  for (DeviceBlob* b : h->blobs)
    if (b->device == dev) return b;
  return nullptr;
}

// Returns the blob of the current device, creating and uploading the canonical arrays on first use.
rt3d_status get_blob(rt3d_packed* h, DeviceBlob** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return RT3D_ERR_CUDA;
  std::lock_guard<std::mutex> lock(h->mu);
  DeviceBlob* b = find_blob(h, dev);
  if (!b) {
    b = new (std::nothrow) DeviceBlob;
    if (!b) return RT3D_ERR_ALLOC;
    b->device = dev;
    rt3d_status s = RT3D_OK;
    if (dev_malloc(&b->group_ptr, h->group_ptr.size() * 4) != cudaSuccess ||
        dev_malloc(&b->pos_idx, h->pos_idx.size() * 2 + 16) != cudaSuccess ||
        dev_malloc(&b->tiles, h->tiles.size() + 16) != cudaSuccess)
      s = RT3D_ERR_ALLOC;
    if (s == RT3D_OK &&
        (cudaMemcpy(b->group_ptr, h->group_ptr.data(), h->group_ptr.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess ||
         (h->nnz && cudaMemcpy(b->pos_idx, h->pos_idx.data(), h->pos_idx.size() * 2, cudaMemcpyHostToDevice) != cudaSuccess) ||
         (h->nnz && cudaMemcpy(b->tiles, h->tiles.data(), h->tiles.size(), cudaMemcpyHostToDevice) != cudaSuccess)))
      s = RT3D_ERR_CUDA;
    if (s != RT3D_OK) {
      cudaFree(b->group_ptr); cudaFree(b->pos_idx); cudaFree(b->tiles);
      delete b;
      return s;
    }
    h->blobs.push_back(b);
    std::lock_guard<std::mutex> reg(g_blobs_mu);
    g_blobs.push_back(b);
  }
  *out = b;
  return RT3D_OK;
}

rt3d_status get_umma_blob(rt3d_packed* h, DeviceBlob* blob, const UmmaLayout* L, DeviceBlob::Umma** out) {
  std::lock_guard<std::mutex> lock(h->mu);
  DeviceBlob::Umma& u = blob->umma[L->n_tile + (L->t_groups ? 4096 : 0)];
  if (!u.ready) {
    const size_t wbytes = L->wtiles.size() * 2;
    if (dev_malloc(&u.wtiles, wbytes + 1024) != cudaSuccess ||
        dev_malloc(&u.step_ptr, L->step_ptr.size() * 4) != cudaSuccess ||
        dev_malloc(&u.steps, L->steps.size() * 4 + 16) != cudaSuccess)
      return RT3D_ERR_ALLOC;
    if ((wbytes && cudaMemcpy(u.wtiles, L->wtiles.data(), wbytes, cudaMemcpyHostToDevice) != cudaSuccess) ||
        cudaMemcpy(u.step_ptr, L->step_ptr.data(), L->step_ptr.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess ||
        (!L->steps.empty() &&
         cudaMemcpy(u.steps, L->steps.data(), L->steps.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess))
      return RT3D_ERR_CUDA;
    if (L->t_groups) {
      if (dev_malloc(&u.grp_ptr, L->grp_ptr.size() * 4) != cudaSuccess ||
          dev_malloc(&u.grp_first, L->grp_first.size() * 4) != cudaSuccess)
        return RT3D_ERR_ALLOC;
      if (cudaMemcpy(u.grp_ptr, L->grp_ptr.data(), L->grp_ptr.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess ||
          cudaMemcpy(u.grp_first, L->grp_first.data(), L->grp_first.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess)
        return RT3D_ERR_CUDA;
    }
    // 2-D map over the weight tiles: rows of 64 bf16 (128 bytes), one box = one [n_tile][64] tile
    const cuuint64_t rows = L->steps.empty() ? cuuint64_t(L->n_tile) : cuuint64_t(L->steps.size()) * L->n_tile;
    cuuint64_t dims[2] = {64, rows};
    cuuint64_t strides[1] = {128};
    cuuint32_t box[2] = {64, cuuint32_t(L->n_tile)};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode(reinterpret_cast<CUtensorMap*>(u.wmap), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, u.wtiles, dims,
                          strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return RT3D_ERR_CUDA;
    if (L->n_tile % 16 == 0) {
      cuuint32_t box_half[2] = {64, cuuint32_t(L->n_tile / 2)};
      r = g_encode(reinterpret_cast<CUtensorMap*>(u.wmap_half), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, u.wtiles, dims,
                   strides, box_half, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
      if (r != CUDA_SUCCESS) return RT3D_ERR_CUDA;
    }
    u.ready = true;
  }
  *out = &u;
  return RT3D_OK;
}

// Device copy of the sub-tile kernel's layout (step records, step offsets, weight blocks).
rt3d_status get_sub_blob(rt3d_packed* h, DeviceBlob* blob, const SubLayout* L, DeviceBlob::Sub** out) {
  std::lock_guard<std::mutex> lock(h->mu);
  DeviceBlob::Sub& u = blob->sub[L->n_tile];
  if (!u.ready) {
    const size_t sbytes = L->steps.size() * sizeof(SubStep), bbytes = L->payload.size();
    if (dev_malloc(&u.steps, sbytes + 64) != cudaSuccess ||
        dev_malloc(&u.step_ptr, L->step_ptr.size() * 4) != cudaSuccess ||
        dev_malloc(&u.blocks, bbytes + 512) != cudaSuccess)
      return RT3D_ERR_ALLOC;
    if ((sbytes && cudaMemcpy(u.steps, L->steps.data(), sbytes, cudaMemcpyHostToDevice) != cudaSuccess) ||
        cudaMemcpy(u.step_ptr, L->step_ptr.data(), L->step_ptr.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess ||
        (bbytes && cudaMemcpy(u.blocks, L->payload.data(), bbytes, cudaMemcpyHostToDevice) != cudaSuccess))
      return RT3D_ERR_CUDA;
    u.ready = true;
  }
  *out = &u;
  return RT3D_OK;
}

// ------------------------------------------------------------------------ tile planning
// Box of output voxels (bn x bt x bh x bw <= 128) that covers the output with the fewest tiles;
// ties go to the wider box along w, then h (longer contiguous runs for the TMA engine).
// `prefer_deep`: ties go first to boxes inside one clip, then to the deeper box along t (the t-grouped CTA-pair
// variant shares one staged input tile between the kt steps; the deeper the box, the less the extra frames weigh).
TileBox choose_box_search(const ConvGeom& g, bool prefer_deep);
// The search is a few thousand iterations; repeated calls on the same shape (every eager forward pass) take the
// answer from a small per-thread table.
TileBox choose_box(const ConvGeom& g, bool prefer_deep = false) {
  struct Entry { int n, To, Ho, Wo, st, sh, sw, deep; TileBox box; };
  thread_local Entry cache[16];
  thread_local int used = 0, next = 0;
  for (int i = 0; i < used; ++i) {
    const Entry& e = cache[i];
    if (e.n == g.n && e.To == g.To && e.Ho == g.Ho && e.Wo == g.Wo && e.st == g.st && e.sh == g.sh && e.sw == g.sw &&
        e.deep == int(prefer_deep))
      return e.box;
  }
  const TileBox box = choose_box_search(g, prefer_deep);
  cache[next] = Entry{g.n, g.To, g.Ho, g.Wo, g.st, g.sh, g.sw, int(prefer_deep), box};
  next = (next + 1) % 16;
  if (used < 16) ++used;
  return box;
}
TileBox choose_box_search(const ConvGeom& g, bool prefer_deep) {
  TileBox best{1, 1, 1, 1};
  long long best_tiles = -1;
  for (int bw = 1; bw <= g.Wo && bw <= kTileM; ++bw) {
    if (bw * g.sw > 256) break;
    for (int bh = 1; bh <= g.Ho && bw * bh <= kTileM; ++bh) {
      if (bh * g.sh > 256) break;
      for (int bt = 1; bt <= g.To && bw * bh * bt <= kTileM; ++bt) {
        if (bt * g.st > 256) break;
        int bn = kTileM / (bw * bh * bt);
        if (bn > g.n) bn = g.n;
        const long long tiles = (long long)ceil_div(g.n, bn) * ceil_div(g.To, bt) * ceil_div(g.Ho, bh) * ceil_div(g.Wo, bw);
        bool better = best_tiles < 0 || tiles < best_tiles;
        if (!better && tiles == best_tiles && prefer_deep && ((bn == 1) != (best.bn == 1) || bt != best.bt)) {
          better = (bn == 1) != (best.bn == 1) ? bn == 1 : bt > best.bt;
        } else if (!better && tiles == best_tiles) {
          if (bw > best.bw) better = true;
          else if (bw == best.bw && bh > best.bh) better = true;
        }
        if (better) { best = TileBox{bn, bt, bh, bw}; best_tiles = tiles; }
      }
    }
  }
  return best;
}

// Bundle width and number of K splits for a call.  Model (fitted to timings on B200): a K step costs
// the issuing thread about 175 ns of barrier hand-shake plus 4 MMA issues, or the tensor time of the
// step if that is longer; a layer with few output tiles runs as many serial steps per CTA as its
// step list is long, so it is split along K (at the price of writing and re-reading fp32 partial
// tiles) until the SMs are occupied.  The step count of each candidate bundle width comes from the
// handle's real step lists: with kernel groups as wide as a bundle, pruned (location, chunk) steps
// vanish and a narrower bundle that matches the group height can win.
struct UmmaPlan { int n_tile, n_splits; };

UmmaPlan pick_plan(rt3d_packed* w, long long m_tiles, int sm_count) {
  const int M = w->M;
  const int widest = default_n_tile(M);
  UmmaPlan best{widest, 1};
  double best_ns = -1.0;
  static const int kSplits[] = {1, 2, 3, 4, 6, 8};
  for (int n = widest; n >= 32; n = (n > 128 ? 128 : n / 2)) {
    if (n % 16) break;
    // narrower bundles only pay when they let pruned steps drop out (groups at least 16 rows high)
    // or when the layer has too few tiles; for the paper's 4..8-row groups the lists are full anyway
    const int bundles = ceil_div(M, n);
    const long long items = m_tiles * bundles;
    double steps = double(w->Ks) * ceil_div(w->N, kChunk);      // full lists: true for groups a few rows high
    if (w->g_m >= 16 && !w->is_dense) {
      const UmmaLayout* L = get_umma_layout(w, n);
      if (!L) break;
      steps = items < sm_count ? double(L->max_steps) : double(L->steps.size()) / bundles;
    }
    const double issue = 175.0 + 4.0 * (25.0 + 0.06 * n), tensor = 1.4 * n;
    const double step_ns = issue > tensor ? issue : tensor;
    for (int S : kSplits) {
      if (S > 1 && (steps / S < 8 || items >= 2LL * sm_count)) continue;
      const double waves = double(ceil_div64(items * S, sm_count));
      double ns = waves * (steps / S) * step_ns;
      // partial tile out (every split) and S partial tiles back in (the CTA that arrives last), plus the
      // traffic of all partials (written once, read once) at about 2.5 TB/s
      if (S > 1) ns += 3000.0 + (1.0 + S) * n * 4.0 + double(items) * S * (kTileM * n * 4.0 * 2.0) / 2500.0;
      if (best_ns < 0 || ns < best_ns * 0.97) { best = UmmaPlan{n, S}; best_ns = ns; }
    }
    if (n == 32) break;
  }
  return best;
}

bool umma_eligible(const DeviceState* d, const rt3d_packed* w, const rt3d_tensor* x, const rt3d_tensor* y,
                   const rt3d_conv_params* p) {
  if (d->cc_major != 10) return false;
  if (!umma_layout_possible(w)) return false;
  if (x->c_stride % 8 || y->c_stride % 8) return false;
  if (p->st > 8 || p->sh > 8 || p->sw > 8) return false;
  if (int64_t(x->w) * x->c_stride * 2 >= (int64_t(1) << 40)) return false;
  return true;
}

// `extra_t`: frames added to the box along t (the t-grouped CTA-pair variant stages Kt - 1 more; temporal stride 1).
rt3d_status encode_xmap(const rt3d_tensor* x, const ConvGeom& g, const TileBox& box, CUtensorMap* map, int extra_t = 0) {
  const cuuint64_t cs = cuuint64_t(x->c_stride) * 2;
  cuuint64_t dims[5] = {cuuint64_t(x->c), cuuint64_t(x->w), cuuint64_t(x->h), cuuint64_t(x->t), cuuint64_t(x->n)};
  cuuint64_t strides[4] = {cs, cs * x->w, cs * x->w * x->h, cs * x->w * x->h * x->t};
  // with a traversal stride s the engine loads ceil(box / s) elements, so a box of b outputs spans b*s inputs
  cuuint32_t bx[5] = {64, cuuint32_t(box.bw * g.sw), cuuint32_t(box.bh * g.sh), cuuint32_t(box.bt * g.st + extra_t),
                      cuuint32_t(box.bn)};
  cuuint32_t estr[5] = {1, cuuint32_t(g.sw), cuuint32_t(g.sh), cuuint32_t(g.st), 1};
  CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, x->data, dims, strides, bx, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? RT3D_OK : RT3D_ERR_CUDA;
}

// Block of 32 output voxels (w, h, t, n extents) that one epilogue warp owns in a box of bw x bh x bt x bn
// voxels; false when 32 consecutive box rows are not a rectangular block.
bool warp_block(int bw, int bh, int bt, int bn, int sb[4]) {
  if ((bw * bh * bt * bn) % 32) return false;
  int rem = 32;
  const int dims_box[4] = {bw, bh, bt, bn};
  for (int i = 0; i < 4; ++i) {
    sb[i] = 1;
    if (rem == 1) continue;
    const int d = dims_box[i];
    if (d >= rem) { if (d % rem) return false; sb[i] = rem; rem = 1; }
    else { if (rem % d) return false; sb[i] = d; rem /= d; }
  }
  return rem == 1;
}

// Output tensor map for the TMA-store epilogue: box = 32 channels x the voxels one epilogue warp stores per
// piece (its block of 32 voxels, divided by the fused pooling window), 64-byte swizzle.  The tensor is y,
// i.e. already the pooled one when pooling is fused.
bool encode_ymap(const rt3d_tensor* y, const int sb[4], int pw, int ph, int pt, CUtensorMap* map) {
  if (y->c < 32 || sb[0] % pw || sb[1] % ph || sb[2] % pt) return false;
  const cuuint64_t cs = cuuint64_t(y->c_stride) * 2;
  cuuint64_t dims[5] = {cuuint64_t(y->c), cuuint64_t(y->w), cuuint64_t(y->h), cuuint64_t(y->t), cuuint64_t(y->n)};
  cuuint64_t strides[4] = {cs, cs * y->w, cs * y->w * y->h, cs * y->w * y->h * y->t};
  cuuint32_t bx[5] = {32, cuuint32_t(sb[0] / pw), cuuint32_t(sb[1] / ph), cuuint32_t(sb[2] / pt), cuuint32_t(sb[3])};
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  return g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, y->data, dims, strides, bx, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Box for a call with fused pooling: fewest tiles among the boxes whose extents and whose per-warp block
// are multiples of the pooling window (every window then lies inside one warp's 32 voxels).
bool choose_box_pool_search(const ConvGeom& g, int pw, int ph, int pt, TileBox* out, int sb_out[4], bool prefer_deep);
bool choose_box_pool(const ConvGeom& g, int pw, int ph, int pt, TileBox* out, int sb_out[4], bool prefer_deep = false) {
  struct Entry { int n, To, Ho, Wo, st, sh, sw, pw, ph, pt, deep; bool ok; TileBox box; int sb[4]; };   // as in choose_box
  thread_local Entry cache[16];
  thread_local int used = 0, next = 0;
  for (int i = 0; i < used; ++i) {
    const Entry& e = cache[i];
    if (e.n == g.n && e.To == g.To && e.Ho == g.Ho && e.Wo == g.Wo && e.st == g.st && e.sh == g.sh && e.sw == g.sw &&
        e.pw == pw && e.ph == ph && e.pt == pt && e.deep == int(prefer_deep)) {
      if (e.ok) { *out = e.box; for (int k = 0; k < 4; ++k) sb_out[k] = e.sb[k]; }
      return e.ok;
    }
  }
  Entry e{g.n, g.To, g.Ho, g.Wo, g.st, g.sh, g.sw, pw, ph, pt, int(prefer_deep), false, TileBox{1, 1, 1, 1}, {1, 1, 1, 1}};
  e.ok = choose_box_pool_search(g, pw, ph, pt, &e.box, e.sb, prefer_deep);
  cache[next] = e;
  next = (next + 1) % 16;
  if (used < 16) ++used;
  if (e.ok) { *out = e.box; for (int k = 0; k < 4; ++k) sb_out[k] = e.sb[k]; }
  return e.ok;
}
bool choose_box_pool_search(const ConvGeom& g, int pw, int ph, int pt, TileBox* out, int sb_out[4], bool prefer_deep) {
  long long best_tiles = -1;
  for (int bw = pw; bw <= kTileM && bw <= round_up(g.Wo, pw); bw += pw) {
    if (bw * g.sw > 256) break;
    for (int bh = ph; bw * bh <= kTileM && bh <= round_up(g.Ho, ph); bh += ph) {
      if (bh * g.sh > 256) break;
      for (int bt = pt; bw * bh * bt <= kTileM && bt <= round_up(g.To, pt); bt += pt) {
        if (bt * g.st > 256) break;
        int bn = kTileM / (bw * bh * bt);
        if (bn > g.n) bn = g.n;
        int sb[4];
        if (!warp_block(bw, bh, bt, bn, sb) || sb[0] % pw || sb[1] % ph || sb[2] % pt) continue;
        const long long tiles = (long long)ceil_div(g.n, bn) * ceil_div(g.To, bt) * ceil_div(g.Ho, bh) * ceil_div(g.Wo, bw);
        bool better = best_tiles < 0 || tiles < best_tiles;
        if (!better && tiles == best_tiles) {
          if (prefer_deep && ((bn == 1) != (out->bn == 1) || bt != out->bt)) better = (bn == 1) != (out->bn == 1) ? bn == 1 : bt > out->bt;
          else better = bw > out->bw;
        }
        if (better) {
          best_tiles = tiles;
          *out = TileBox{bn, bt, bh, bw};
          for (int i = 0; i < 4; ++i) sb_out[i] = sb[i];
        }
      }
    }
  }
  return best_tiles > 0;
}

// Small-C_in kernel: bf16, C_in <= 8 stored at pitch 8, spatial strides <= 4, M <= 256.
bool smallc_eligible(const DeviceState* d, rt3d_packed* w, const rt3d_tensor* x, const rt3d_tensor* y,
                     const rt3d_conv_params* p, const SmallCLayout** out) {
  if (d->cc_major != 10 || w->dtype != RT3D_BF16) return false;
  if (x->c > 8 || x->c_stride != 8 || y->c_stride % 8) return false;
  if (p->st > 8 || p->sh > 4 || p->sw > 4) return false;
  if (w->Kt > 16 || w->Kh > 32 || w->Kw > 32) return false;
  const SmallCLayout* L = get_smallc_layout(w, p->sh, p->sw);
  if (!L) return false;
  if (L->img_w * p->sw > 256 || L->img_h * p->sh > 256) return false;
  if (smallc_smem_bytes(L->n_pairs, L->n_pad, L->n_phases * L->phase_stride) > 227 * 1024) return false;
  *out = L;
  return true;
}

rt3d_status launch_smallc(rt3d_packed* w, DeviceBlob* blob, const DeviceState* d, const SmallCLayout* L,
                          const rt3d_tensor* x, const ConvGeom& g, const float* bias, rt3d_tensor* y, cudaStream_t st,
                          const void* residual, int rcs, int pool_h, int pool_w, bool x_pad_zero) {
  // pooled rows leave as whole 32-channel pieces through the bulk-store epilogue; a trailing 16-channel piece is
  // written by plain per-voxel stores, which know nothing of pooling
  if (pool_h * pool_w > 1 && L->n_pad % 32) return RT3D_ERR_UNSUPPORTED;
  DeviceBlob::SmallC* sc = nullptr;
  {
    std::lock_guard<std::mutex> lock(w->mu);
    sc = &blob->smallc[L->sh * 16 + L->sw];
    if (!sc->wimg) {
      void* wi = nullptr;
      int32_t* po = nullptr;
      if (dev_malloc(&wi, L->wimg.size() * 2 + 16) != cudaSuccess ||
          dev_malloc(&po, L->pair_off.size() * 4 + 16) != cudaSuccess)
        return RT3D_ERR_ALLOC;
      if ((!L->wimg.empty() && cudaMemcpy(wi, L->wimg.data(), L->wimg.size() * 2, cudaMemcpyHostToDevice) != cudaSuccess) ||
          (!L->pair_off.empty() &&
           cudaMemcpy(po, L->pair_off.data(), L->pair_off.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess))
        return RT3D_ERR_CUDA;
      sc->pairs = po;
      sc->wimg = wi;
    }
  }
  SmallCArgs a;
  a.g = g;
  a.n_pad = L->n_pad; a.n_pairs = L->n_pairs;
  a.n_phases = L->n_phases; a.phase_stride = L->phase_stride;
  a.img_w = L->img_w; a.phase_bytes = L->img_w * L->img_h * L->img_t * 16;
  a.tiles_h = ceil_div(g.Ho, kSmallCTileH); a.tiles_w = ceil_div(g.Wo, kSmallCTileW);
  a.tmem_cols = 0;
  a.residual = residual; a.rcs = rcs;
  a.pool_t = 1; a.pool_h = pool_h; a.pool_w = pool_w;
  a.wimg = sc->wimg; a.pair_off = sc->pairs;
  a.bias = bias; a.y = y->data; a.sched = d->sched;
  // input as [n][t][h][w][8]: one box = one phase image of a 1 x 16 x 8 output tile (every sh-th row and
  // sw-th column: a traversal stride s loads ceil(box / s) elements), no swizzle
  CUtensorMap xmap;
  const cuuint64_t cs = 16;
  cuuint64_t dims[5] = {cuuint64_t(x->c), cuuint64_t(x->w), cuuint64_t(x->h), cuuint64_t(x->t), cuuint64_t(x->n)};
  cuuint64_t strides[4] = {cs, cs * x->w, cs * x->w * x->h, cs * x->w * x->h * x->t};
  cuuint32_t bx[5] = {8, cuuint32_t(L->img_w * g.sw), cuuint32_t(L->img_h * g.sh), cuuint32_t(L->img_t), 1};
  cuuint32_t estr[5] = {1, cuuint32_t(g.sw), cuuint32_t(g.sh), 1, 1};
  // Unit column stride and all 8 channels real (or the caller vouches for zero padding channels): merge the (w, channel) axes, so that the engine fetches each
  // image row as one contiguous run instead of one 16-byte request per voxel (the tile load was the
  // kernel's bottleneck).  Otherwise the separate channel axis stays: its out-of-range
  // fill is what zeroes the padding channels, whatever the caller's buffer holds there.
  a.merged_cw = (g.sw == 1 && (x->c == 8 || x_pad_zero) && L->img_w * 8 <= 256) ? 1 : 0;
  if (a.merged_cw) {
    dims[0] = cuuint64_t(x->w) * 8; dims[1] = 1;
    strides[0] = cs;                                   // the unit axis never moves
    bx[0] = cuuint32_t(L->img_w * 8); bx[1] = 1;
    estr[1] = 1;
  }
  if (g_encode(&xmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, x->data, dims, strides, bx, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return RT3D_ERR_CUDA;
  CUtensorMap ymap;
  const int sb[4] = {kSmallCTileW, 4, 1, 1};          // a warp owns 4 rows of 8 voxels of the 16 x 8 tile
  a.store_tma = encode_ymap(y, sb, pool_w, pool_h, 1, &ymap) ? 1 : 0;
  if (!a.store_tma && pool_h * pool_w > 1) return RT3D_ERR_UNSUPPORTED;
  if (t_plan_only) return RT3D_OK;
  if (launch_conv_umma_smallc(a, &xmap, a.store_tma ? &ymap : nullptr, d->sm_count, st) != cudaSuccess) return RT3D_ERR_CUDA;
  g_launches.fetch_add(1);
  return RT3D_OK;
}

thread_local rt3d_plan_info t_last_plan = {-1, 0, 0, 0, 0};

// Grows the handle's K-split workspace on this device: `bytes` of partial tiles and `cnt_bytes` of
// counters / flags, which every kernel that uses them leaves zeroed.
rt3d_status ensure_splitk(rt3d_packed* w, DeviceBlob* blob, size_t bytes, size_t cnt_bytes) {
  std::lock_guard<std::mutex> lock(w->mu);
  if (blob->splitk_bytes < bytes) {
    cudaFree(blob->splitk);
    blob->splitk = nullptr; blob->splitk_bytes = 0;
    if (dev_malloc(&blob->splitk, bytes) != cudaSuccess) return RT3D_ERR_ALLOC;
    blob->splitk_bytes = bytes;
  }
  if (blob->splitk_cnt_bytes < cnt_bytes) {
    cudaFree(blob->splitk_cnt);
    blob->splitk_cnt = nullptr; blob->splitk_cnt_bytes = 0;
    if (dev_malloc(&blob->splitk_cnt, cnt_bytes) != cudaSuccess) return RT3D_ERR_ALLOC;
    if (cudaMemset(blob->splitk_cnt, 0, cnt_bytes) != cudaSuccess) return RT3D_ERR_CUDA;
    blob->splitk_cnt_bytes = cnt_bytes;
  }
  return RT3D_OK;
}

// Resident-weight kernel for thin stride-1 layers: used when the layer qualifies and (unless forced) has
// at least one tile per SM.  *launched = false (and RT3D_OK) when the caller should take another kernel.
rt3d_status try_halo(rt3d_packed* w, DeviceBlob* blob, DeviceState* d, const rt3d_tensor* x, const ConvGeom& g,
                     const float* bias, rt3d_tensor* y, const void* res_data, int res_pitch, bool dense_entry,
                     bool forced, cudaStream_t st, bool* launched) {
  *launched = false;
  if (g.st != 1 || g.sh != 1 || g.sw != 1 || w->M > 256) return RT3D_OK;
  const int n_tile = round_up(w->M, 16);
  const int n_chunks = ceil_div(w->N, kChunk);
  // cheap size screen before the layout is built: all locations kept is the upper bound
  if (!dense_entry && w->is_dense == 0 && size_t(w->Ks) * n_chunks * (n_tile / 2) * 128 > size_t(4) * 227 * 1024) return RT3D_OK;
  HaloArgs h;
  UmmaArgs& a = h.u;
  a.g = g;
  // tile: 8 voxels along w times 16 (t, h) lines; one frame thick unless the kernel is 1 high
  int bt = 1, bh = 16;
  if (g.Kh == 1) {
    long long best = -1;
    for (int t = 1; t <= 16; t *= 2) {
      const int hh = 16 / t;
      const long long cost = (long long)ceil_div(g.To, t) * ceil_div(g.Ho, hh) * (t + g.Kt - 1) * hh;
      if (best < 0 || cost < best) { best = cost; bt = t; bh = hh; }
    }
  }
  a.box = TileBox{1, bt, bh, 8};
  a.tiles_n = g.n; a.tiles_t = ceil_div(g.To, bt); a.tiles_h = ceil_div(g.Ho, bh); a.tiles_w = ceil_div(g.Wo, 8);
  const long long m_tiles = (long long)a.tiles_n * a.tiles_t * a.tiles_h * a.tiles_w;
  if (!forced && m_tiles < d->sm_count) return RT3D_OK;
  if (m_tiles > (1ll << 30)) return RT3D_OK;
  const UmmaLayout* L = get_umma_layout(w, n_tile);
  if (!L || L->n_bundles != 1) return RT3D_OK;
  a.n_tile = L->n_tile; a.n_bundles = 1; a.n_chunks = L->n_chunks;
  a.dense = dense_entry ? 1 : 0;
  a.steps_dense = w->Ks * L->n_chunks;
  h.n_steps = dense_entry ? a.steps_dense : L->step_ptr[1];
  if (!umma_halo_plan(&h, dense_entry ? nullptr : L->steps.data())) return RT3D_OK;
  // waste of the fixed 16 x 8 tile against the free-form boxes of the other kernels
  if (!forced && m_tiles * 128 > 3 * ((long long)g.n * g.To * g.Ho * g.Wo) / 2) return RT3D_OK;
  DeviceBlob::Umma* u = nullptr;
  rt3d_status s = get_umma_blob(w, blob, L, &u);
  if (s != RT3D_OK) return s;
  a.step_ptr = u->step_ptr; a.steps = u->steps;
  a.bias = bias; a.y = y->data; a.sched = d->sched;
  a.residual = res_data; a.rcs = res_pitch;
  a.pool_t = a.pool_h = a.pool_w = 1;
  a.n_splits = 1; a.scratch = nullptr; a.counters = nullptr;
  a.tail_workers = 0; a.tail_scratch = nullptr; a.tail_flags = nullptr;
  a.ts = 0; a.grp_ptr = nullptr; a.grp_first = nullptr; a.ts_a_bytes = 0; a.ts_frame_bytes = 0; a.ts_table = 0; a.ts_phases = 1;
  a.wait_cycles = 0; a.debug_drop_last_load = 0;
  ConvGeom unit = g;                       // the staged block is a plain box of input voxels
  CUtensorMap xmap, ymap;
  if ((s = encode_xmap(x, unit, TileBox{1, h.ht, h.hh, h.hw}, &xmap)) != RT3D_OK) return s;
  int sb[4] = {1, 1, 1, 1};
  const bool rect = warp_block(a.box.bw, a.box.bh, a.box.bt, a.box.bn, sb);
  a.sbw = sb[0]; a.sbh = sb[1];
  a.store_tma = (rect && encode_ymap(y, sb, 1, 1, 1, &ymap)) ? 1 : 0;
  t_last_plan = rt3d_plan_info{4, a.n_tile, 1, 0, 0};
  *launched = true;
  if (t_plan_only) return RT3D_OK;
  cudaError_t e = launch_conv_umma_halo(h, &xmap, u->wmap_half, a.store_tma ? &ymap : nullptr, d->sm_count, st);
  if (e != cudaSuccess) return RT3D_ERR_CUDA;
  g_launches.fetch_add(1);
  return RT3D_OK;
}

// Sub-tile kernel: blocks of 16 x 16 channels in which no kernel group keeps the step's location are skipped.
// Runs only when asked for (RT3D_ALGO_UMMA_SUB): measured on B200 it loses to the masked-dense CTA-pair kernel at
// every group size and pruning rate of the sweep, because moving a step's input tile through shared memory into
// tensor memory costs about as much as the dense MMAs of that step.
// *launched = false (and RT3D_OK) when the handle cannot use it.
rt3d_status try_sub(rt3d_packed* w, DeviceBlob* blob, DeviceState* d, const rt3d_tensor* x, const ConvGeom& g,
                    const float* bias, rt3d_tensor* y, const void* res_data, int res_pitch, cudaStream_t st, bool* launched) {
  *launched = false;
  if (w->is_dense) return RT3D_OK;
  SubArgs a;
  a.g = g;
  a.box = choose_box(g);
  a.tiles_n = ceil_div(g.n, a.box.bn); a.tiles_t = ceil_div(g.To, a.box.bt);
  a.tiles_h = ceil_div(g.Ho, a.box.bh); a.tiles_w = ceil_div(g.Wo, a.box.bw);
  const long long m_tiles = (long long)a.tiles_n * a.tiles_t * a.tiles_h * a.tiles_w;
  if (m_tiles > (1ll << 30)) return RT3D_OK;
  const SubLayout* L = get_sub_layout(w, 0);
  if (!L) return RT3D_OK;
  a.n_tile = L->n_tile; a.n_bundles = L->n_bundles;
  if (!umma_sub_plan(&a, L->max_blocks)) return RT3D_OK;
  DeviceBlob::Sub* u = nullptr;
  rt3d_status s = get_sub_blob(w, blob, L, &u);
  if (s != RT3D_OK) return s;
  a.steps = static_cast<const SubStep*>(u->steps); a.step_ptr = u->step_ptr; a.blocks = u->blocks;
  a.bias = bias; a.y = y->data; a.sched = d->sched;
  a.residual = res_data; a.rcs = res_pitch;
  CUtensorMap xmap, ymap;
  if ((s = encode_xmap(x, g, a.box, &xmap)) != RT3D_OK) return s;
  int sb[4] = {1, 1, 1, 1};
  const bool rect = warp_block(a.box.bw, a.box.bh, a.box.bt, a.box.bn, sb);
  a.store_tma = (rect && encode_ymap(y, sb, 1, 1, 1, &ymap)) ? 1 : 0;
  t_last_plan = rt3d_plan_info{6, a.n_tile, 1, 0, 0};
  *launched = true;
  if (t_plan_only) return RT3D_OK;
  if (launch_conv_umma_sub(a, &xmap, a.store_tma ? &ymap : nullptr, d->sm_count, st) != cudaSuccess) return RT3D_ERR_CUDA;
  g_launches.fetch_add(1);
  return RT3D_OK;
}

rt3d_status conv_impl(const rt3d_tensor* x, const rt3d_packed* wc, const float* bias, const rt3d_conv_params* p,
                      rt3d_tensor* y, void* stream, bool dense_entry, const rt3d_fusion* fz = nullptr) {
  ConvGeom g;
  if (!y) return RT3D_ERR_INVALID_ARG;
  const bool pooled = fz && (fz->pool_t != 1 || fz->pool_h != 1 || fz->pool_w != 1);
  if (fz && (fz->pool_t < 1 || fz->pool_t > 2 || fz->pool_h < 1 || fz->pool_h > 2 || fz->pool_w < 1 || fz->pool_w > 2))
    return RT3D_ERR_INVALID_ARG;
  const int pl_t = fz ? fz->pool_t : 1, pl_h = fz ? fz->pool_h : 1, pl_w = fz ? fz->pool_w : 1;
  rt3d_status s = make_geom(x, wc, p, pooled ? nullptr : y, &g);
  if (s != RT3D_OK) return s;
  if (pooled) {                     // y holds the pooled tensor; g keeps the extents of the convolution output
    if ((s = check_tensor(y)) != RT3D_OK) return s;
    if (y->n != g.n || y->t != g.To / pl_t || y->h != g.Ho / pl_h || y->w != g.Wo / pl_w || y->c != wc->M ||
        y->dtype != wc->dtype || y->t < 1 || y->h < 1 || y->w < 1)
      return RT3D_ERR_SHAPE;
    if (fz->residual) return RT3D_ERR_UNSUPPORTED;
    g.ycs = y->c_stride;
  }
  if ((s = check_alignment(x)) != RT3D_OK || (s = check_alignment(y)) != RT3D_OK) return s;
  if (overlaps(x, y)) return RT3D_ERR_INVALID_ARG;
  const rt3d_tensor* res = fz ? fz->residual : nullptr;
  if (res) {
    if ((s = check_tensor(res)) != RT3D_OK || (s = check_alignment(res)) != RT3D_OK) return s;
    if (res->n != g.n || res->t != g.To || res->h != g.Ho || res->w != g.Wo || res->c != g.M || res->dtype != wc->dtype)
      return RT3D_ERR_SHAPE;
    if (overlaps(res, y)) return RT3D_ERR_INVALID_ARG;
  }
  const void* res_data = res ? res->data : nullptr;
  const int res_pitch = res ? res->c_stride : 0;
  if (dense_entry && !wc->is_dense) return RT3D_ERR_INVALID_ARG;
  rt3d_packed* w = const_cast<rt3d_packed*>(wc);
  DeviceState* d = nullptr;
  if ((s = get_device_state(&d)) != RT3D_OK) return s;
  DeviceBlob* blob = nullptr;
  if ((s = get_blob(w, &blob)) != RT3D_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  const bool can_umma = umma_eligible(d, w, x, y, p);
  const bool can_simt = w->g_m <= kMaxGroupSimt && w->g_n <= kMaxGroupSimt;
  if (!can_umma && !can_simt) return RT3D_ERR_UNSUPPORTED;
  if (p->algo == RT3D_ALGO_SIMT && !can_simt) return RT3D_ERR_UNSUPPORTED;
  const bool want_umma = p->algo == RT3D_ALGO_UMMA || p->algo == RT3D_ALGO_UMMA_PAIR || p->algo == RT3D_ALGO_UMMA_HALO ||
                         p->algo == RT3D_ALGO_UMMA_SUB;
  if (want_umma && !can_umma) return RT3D_ERR_UNSUPPORTED;
  const bool use_umma = want_umma || (p->algo == RT3D_ALGO_AUTO && can_umma);
  if (!use_umma) {
    if (pooled) return RT3D_ERR_UNSUPPORTED;
    t_last_plan = rt3d_plan_info{0, 0, 1, 0, 0};
    if (t_plan_only) return RT3D_OK;
    cudaError_t e = launch_conv_simt(w->dtype, g, x->data, y->data, blob->group_ptr, blob->pos_idx, blob->tiles, bias,
                                     w->g_m, w->g_n, w->P, w->Q, dense_entry, res_data, res_pitch, st);
    if (e != cudaSuccess) return RT3D_ERR_CUDA;
    g_launches.fetch_add(1);
    t_last_plan = rt3d_plan_info{0, 0, 1, 0, 0};
    return RT3D_OK;
  }

  const SmallCLayout* SL = nullptr;
  if (p->algo != RT3D_ALGO_UMMA_PAIR && p->algo != RT3D_ALGO_UMMA_HALO && p->algo != RT3D_ALGO_UMMA_SUB && (!pooled || pl_t == 1) &&
      smallc_eligible(d, w, x, y, p, &SL)) {
    s = launch_smallc(w, blob, d, SL, x, g, bias, y, st, res_data, res_pitch, pl_h, pl_w, p->x_pad_zero != 0);
    if (s == RT3D_OK) t_last_plan = rt3d_plan_info{3, SL->n_pad, 1, 0, pooled ? 1 : 0};
    return s;
  }

  if ((p->algo == RT3D_ALGO_AUTO || p->algo == RT3D_ALGO_UMMA_HALO) && !pooled) {
    bool launched = false;
    s = try_halo(w, blob, d, x, g, bias, y, res_data, res_pitch, dense_entry, p->algo == RT3D_ALGO_UMMA_HALO, st, &launched);
    if (s != RT3D_OK || launched) return s;
  }
  if (p->algo == RT3D_ALGO_UMMA_HALO) return RT3D_ERR_UNSUPPORTED;
  if (p->algo == RT3D_ALGO_UMMA_SUB) {
    bool launched = false;
    if (!pooled && !dense_entry) {
      s = try_sub(w, blob, d, x, g, bias, y, res_data, res_pitch, st, &launched);
      if (s != RT3D_OK || launched) return s;
    }
    return RT3D_ERR_UNSUPPORTED;
  }

  UmmaArgs a;
  a.g = g;
  int sb[4] = {1, 1, 1, 1};
  bool rect;
  if (pooled) {
    if (!choose_box_pool(g, pl_w, pl_h, pl_t, &a.box, sb)) return RT3D_ERR_UNSUPPORTED;
    rect = true;
  } else {
    a.box = choose_box(g);
    rect = warp_block(a.box.bw, a.box.bh, a.box.bt, a.box.bn, sb);
  }
  a.pool_t = pl_t; a.pool_h = pl_h; a.pool_w = pl_w; a.sbw = sb[0]; a.sbh = sb[1];
  a.tiles_n = ceil_div(g.n, a.box.bn); a.tiles_t = ceil_div(g.To, a.box.bt);
  a.tiles_h = ceil_div(g.Ho, a.box.bh); a.tiles_w = ceil_div(g.Wo, a.box.bw);
  const long long m_tiles = (long long)a.tiles_n * a.tiles_t * a.tiles_h * a.tiles_w;
  UmmaPlan plan = pick_plan(w, m_tiles, d->sm_count);
  if (pooled) {                     // pooling lives in the TMA-store epilogue, which a K split does not use
    // A layer this small is faster split over K and pooled by a second launch: AUTO declines the fusion.
    if (p->algo == RT3D_ALGO_AUTO && plan.n_splits > 1) return RT3D_ERR_UNSUPPORTED;
    plan.n_splits = 1;
  }
  // CTA pairs: two tiles per MMA.  Worth it when every pair has work; forced by RT3D_ALGO_UMMA_PAIR.
  bool use_pair = false;
  if (p->algo == RT3D_ALGO_UMMA_PAIR) {
    plan = UmmaPlan{default_n_tile(w->M), 1};
    if (!umma_pair_supported(plan.n_tile, ceil_div(w->M, plan.n_tile))) return RT3D_ERR_UNSUPPORTED;
    use_pair = true;
  } else if (p->algo == RT3D_ALGO_AUTO && plan.n_splits == 1 &&
             umma_pair_supported(plan.n_tile, ceil_div(w->M, plan.n_tile)) &&
             m_tiles * ceil_div(w->M, plan.n_tile) >= d->sm_count) {
    use_pair = true;
  }
  if (pooled && plan.n_tile % 32) return RT3D_ERR_UNSUPPORTED;      // pooled rows leave as whole 32-channel pieces
  // CTA pairs on bundles up to 128 wide with a kernel that is 2 or 3 deep: one deeper input tile per (kh, kw, chunk)
  // (its box: among the boxes with as few tiles, one inside a single clip and as deep along t as possible)
  bool use_ts = false;
  UmmaArgs probe = a;
  // (wide bundles: only kernels that are also wide in space; a 3x1x1 layer with 192-wide bundles lost 8 us of 43
  // inside the S3D-shaped forward with it, while 3x3x3 layers gain 1-4 %)
  if (use_pair && g_ts_enabled.load() && g.st <= 2 && g.Kt >= 2 && g.Kt <= 8 && (plan.n_tile <= 128 || g.Kh * g.Kw >= 4)) {
    int sb2[4] = {1, 1, 1, 1};
    TileBox deep = a.box;
    const bool ok2 = pooled ? choose_box_pool(g, pl_w, pl_h, pl_t, &deep, sb2, true)
                            : (deep = choose_box(g, true), warp_block(deep.bw, deep.bh, deep.bt, deep.bn, sb2) == rect);
    const long long tiles2 = (long long)ceil_div(g.n, deep.bn) * ceil_div(g.To, deep.bt) * ceil_div(g.Ho, deep.bh) * ceil_div(g.Wo, deep.bw);
    if (ok2 && tiles2 == m_tiles) {
      probe.box = deep;
      probe.sbw = sb2[0]; probe.sbh = sb2[1];
      probe.tiles_n = ceil_div(g.n, deep.bn); probe.tiles_t = ceil_div(g.To, deep.bt);
      probe.tiles_h = ceil_div(g.Ho, deep.bh); probe.tiles_w = ceil_div(g.Wo, deep.bw);
    }
    probe.n_tile = plan.n_tile; probe.n_bundles = ceil_div(w->M, plan.n_tile); probe.dense = dense_entry ? 1 : 0;
    use_ts = umma_pair_ts_supported(&probe, w->Ks * ceil_div(w->N, kChunk) * probe.n_bundles);
    if (use_ts) {
      a.box = probe.box; a.sbw = probe.sbw; a.sbh = probe.sbh;
      a.tiles_n = probe.tiles_n; a.tiles_t = probe.tiles_t; a.tiles_h = probe.tiles_h; a.tiles_w = probe.tiles_w;
      for (int i = 0; i < 4; ++i) sb[i] = sb2[i];
    }
  }
  const UmmaLayout* L = get_umma_layout(w, plan.n_tile, use_ts);
  if (!L) return RT3D_ERR_UNSUPPORTED;
  DeviceBlob::Umma* u = nullptr;
  if ((s = get_umma_blob(w, blob, L, &u)) != RT3D_OK) return s;
  a.n_tile = L->n_tile; a.n_bundles = L->n_bundles; a.n_chunks = L->n_chunks;
  a.dense = dense_entry ? 1 : 0;
  a.steps_dense = w->Ks * L->n_chunks;
  a.step_ptr = u->step_ptr; a.steps = u->steps;
  a.bias = bias; a.y = y->data; a.sched = d->sched;
  a.residual = res_data; a.rcs = res_pitch;
  a.n_splits = plan.n_splits; a.scratch = nullptr; a.counters = nullptr;
  a.tail_workers = 0; a.tail_scratch = nullptr; a.tail_flags = nullptr;
  a.ts = 0; a.grp_ptr = nullptr; a.grp_first = nullptr; a.ts_a_bytes = 0; a.ts_frame_bytes = 0; a.ts_table = 0; a.ts_phases = 1;
  a.wait_cycles = debug_wait_cycles(); a.debug_drop_last_load = g_debug_drop_last_load.load();
  if (a.n_splits > 1) {
    // split-K workspace of this handle on this device: partial tiles + per-warp arrival counters
    const long long tiles = m_tiles * L->n_bundles;
    if ((s = ensure_splitk(w, blob, size_t(tiles) * a.n_splits * kTileM * L->n_tile * sizeof(float),
                           size_t(tiles) * 8 * sizeof(int32_t))) != RT3D_OK) return s;
    a.scratch = blob->splitk; a.counters = blob->splitk_cnt;
  }
  if (use_ts) {
    a.ts = 1; a.grp_ptr = u->grp_ptr; a.grp_first = u->grp_first;
    a.ts_a_bytes = probe.ts_a_bytes; a.ts_frame_bytes = probe.ts_frame_bytes; a.ts_table = probe.ts_table;
    a.ts_phases = probe.ts_phases;
  }
  CUtensorMap xmap;
  if ((s = encode_xmap(x, g, a.box, &xmap, use_ts ? ((g.Kt - 1) / g.st) * g.st : 0)) != RT3D_OK) return s;
  CUtensorMap ymap;
  a.store_tma = (a.n_splits == 1 && rect && encode_ymap(y, sb, pl_w, pl_h, pl_t, &ymap)) ? 1 : 0;
  if (pooled && !a.store_tma) return RT3D_ERR_UNSUPPORTED;
  if (use_pair) {
    // items that do not fill a last round of CTA pairs are cut along K and shared (same workspace as split-K)
    // (its CTA pairs wait for one another, which needs the whole grid resident at once: not used when the caller
    // says that other kernels may run beside this call)
    size_t tail_bytes = 0, flag_bytes = 0;
    if (!p->concurrent)
      umma_pair_tail_plan(&a, L->step_ptr.data(), d->sm_count, &tail_bytes, &flag_bytes, use_ts ? L->grp_ptr.data() : nullptr);
    if (a.tail_workers > 0) {
      if ((s = ensure_splitk(w, blob, tail_bytes, flag_bytes)) != RT3D_OK) return s;
      a.tail_scratch = blob->splitk; a.tail_flags = blob->splitk_cnt;
    }
  }
  const void* ym = a.store_tma ? &ymap : nullptr;
  t_last_plan = rt3d_plan_info{use_pair ? (use_ts ? 7 : 2) : 1, a.n_tile, a.n_splits, a.tail_workers, pooled ? 1 : 0};
  if (t_plan_only) return RT3D_OK;
  cudaError_t e = use_pair ? launch_conv_umma_pair(a, &xmap, u->wmap_half, ym, d->sm_count, st)
                           : launch_conv_umma(a, &xmap, u->wmap, ym, d->sm_count, st);
  if (e != cudaSuccess) return RT3D_ERR_CUDA;
  g_launches.fetch_add(1);
  return RT3D_OK;
}


// Fused spatial -> temporal pair.  Argument errors first (as the two separate calls would report them), then
// the eligibility screen of the one-kernel path.
rt3d_status conv2plus1d_impl(const rt3d_tensor* x, const rt3d_packed* wsc, const float* bias_s, const rt3d_conv_params* ps,
                             const rt3d_packed* wtc, const float* bias_t, const rt3d_conv_params* pt,
                             const rt3d_tensor* res, rt3d_tensor* y, void* stream) {
  if (!wsc || !wtc || !ps || !pt || !y) return RT3D_ERR_INVALID_ARG;
  ConvGeom g;
  rt3d_status s = make_geom(x, wsc, ps, nullptr, &g);
  if (s != RT3D_OK) return s;
  if (pt->st < 1 || pt->sh < 1 || pt->sw < 1 || pt->pt < 0 || pt->ph < 0 || pt->pw < 0) return RT3D_ERR_INVALID_ARG;
  if ((s = check_tensor(y)) != RT3D_OK) return s;
  if (wtc->N != wsc->M || wtc->dtype != wsc->dtype) return RT3D_ERR_SHAPE;
  if (g.To + 2 * pt->pt < wtc->Kt || g.Ho + 2 * pt->ph < wtc->Kh || g.Wo + 2 * pt->pw < wtc->Kw) return RT3D_ERR_SHAPE;
  const int64_t To2 = (int64_t(g.To) + 2 * pt->pt - wtc->Kt) / pt->st + 1;
  const int64_t Ho2 = (int64_t(g.Ho) + 2 * pt->ph - wtc->Kh) / pt->sh + 1;
  const int64_t Wo2 = (int64_t(g.Wo) + 2 * pt->pw - wtc->Kw) / pt->sw + 1;
  if (y->n != g.n || y->t != To2 || y->h != Ho2 || y->w != Wo2 || y->c != wtc->M || y->dtype != wtc->dtype)
    return RT3D_ERR_SHAPE;
  if ((s = check_alignment(x)) != RT3D_OK || (s = check_alignment(y)) != RT3D_OK) return s;
  if (overlaps(x, y)) return RT3D_ERR_INVALID_ARG;
  if (res) {
    if ((s = check_tensor(res)) != RT3D_OK || (s = check_alignment(res)) != RT3D_OK) return s;
    if (res->n != y->n || res->t != y->t || res->h != y->h || res->w != y->w || res->c != y->c || res->dtype != y->dtype)
      return RT3D_ERR_SHAPE;
    if (overlaps(res, y)) return RT3D_ERR_INVALID_ARG;
  }
  // what the one-kernel path takes
  if (wsc->dtype != RT3D_BF16) return RT3D_ERR_UNSUPPORTED;
  if (wsc->Kt != 1 || g.st != 1 || g.sh != 1 || g.sw != 1 || g.pt != 0 || wsc->N > kChunk || wsc->M > 256) return RT3D_ERR_UNSUPPORTED;
  if (wtc->Kt != 3 || wtc->Kh != 1 || wtc->Kw != 1 || pt->st != 1 || pt->sh != 1 || pt->sw != 1 || pt->pt != 1 ||
      pt->ph != 0 || pt->pw != 0 || wtc->M > 256)
    return RT3D_ERR_UNSUPPORTED;
  rt3d_packed* ws = const_cast<rt3d_packed*>(wsc);
  rt3d_packed* wt = const_cast<rt3d_packed*>(wtc);
  DeviceState* d = nullptr;
  if ((s = get_device_state(&d)) != RT3D_OK) return s;
  if (!umma_eligible(d, ws, x, y, ps) || !umma_layout_possible(wt)) return RT3D_ERR_UNSUPPORTED;
  if (res && res->c_stride % 8) return RT3D_ERR_UNSUPPORTED;
  StArgs a;
  a.g = g;
  a.c_mid = ws->M;
  a.n1 = round_up(ws->M, 16); a.n2 = round_up(wt->M, 16);
  if (2 * a.n1 + 3 * a.n2 > 512) return RT3D_ERR_UNSUPPORTED;
  const UmmaLayout* L1 = get_umma_layout(ws, a.n1);
  const UmmaLayout* L2 = get_umma_layout(wt, a.n2);
  if (!L1 || !L2 || L1->n_bundles != 1 || L2->n_bundles != 1 || L1->n_chunks != 1) return RT3D_ERR_UNSUPPORTED;
  a.n_steps1 = L1->step_ptr[1]; a.n_steps2 = L2->step_ptr[1];
  if (!umma_st_plan(&a, L1->steps.data(), L2->steps.data())) return RT3D_ERR_UNSUPPORTED;
  DeviceBlob *blob1 = nullptr, *blob2 = nullptr;
  if ((s = get_blob(ws, &blob1)) != RT3D_OK || (s = get_blob(wt, &blob2)) != RT3D_OK) return s;
  DeviceBlob::Umma *u1 = nullptr, *u2 = nullptr;
  if ((s = get_umma_blob(ws, blob1, L1, &u1)) != RT3D_OK || (s = get_umma_blob(wt, blob2, L2, &u2)) != RT3D_OK) return s;
  a.M2 = wt->M; a.ycs = y->c_stride; a.relu2 = pt->relu ? 1 : 0;
  a.bias1 = bias_s; a.bias2 = bias_t; a.y = y->data;
  a.residual = res ? res->data : nullptr; a.rcs = res ? res->c_stride : 0;
  a.sched = d->sched;
  CUtensorMap xmap;
  ConvGeom unit = g;
  if ((s = encode_xmap(x, unit, TileBox{1, 1, a.hh, a.hw}, &xmap)) != RT3D_OK) return s;
  t_last_plan = rt3d_plan_info{5, a.n1, 1, 0, 0};
  if (t_plan_only) return RT3D_OK;
  cudaError_t e = launch_conv_umma_st(a, &xmap, u1->wmap_half, u2->wmap_half, d->sm_count, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return RT3D_ERR_CUDA;
  g_launches.fetch_add(1);
  return RT3D_OK;
}

}  // namespace

// ------------------------------------------------------------------ entry point without allocation
// Fixed workspace for rt3d_conv3d_sparse_noalloc: split-K partial tiles followed by the per-warp
// arrival counters.  It lives in every GPU context that loads this library, for the life of the
// process.  In host code `g_noalloc_ws` is only a handle for the runtime, never a device address:
// the address is looked up per device with cudaGetSymbolAddress below.
#define RT3D_NOALLOC_PARTIAL_TILES 128                                   /* 128 x 256 fp32 each */
#define RT3D_NOALLOC_PARTIAL_BYTES (RT3D_NOALLOC_PARTIAL_TILES * 128 * 256 * 4)   /* 16 MiB */
#define RT3D_NOALLOC_COUNTER_BYTES (RT3D_NOALLOC_PARTIAL_TILES * 8 * 4)  /* 8 counters (epilogue warps) per output tile */
static __device__ __align__(256) unsigned char g_noalloc_ws[RT3D_NOALLOC_PARTIAL_BYTES + RT3D_NOALLOC_COUNTER_BYTES];

namespace {
struct NoAllocState { bool ready = false; unsigned char* ws = nullptr; };
NoAllocState g_noalloc[64];
std::mutex g_noalloc_mu;

// Once per device, with that device current: resolve the device address of the workspace.  Called from
// rt3d_packed_prepare, the documented set-up point: the first look-up may make the CUDA runtime load this
// module on the device, which is when the driver sets the array's memory aside.
rt3d_status noalloc_workspace_setup(int dev) {
  std::lock_guard<std::mutex> lock(g_noalloc_mu);
  NoAllocState& st = g_noalloc[dev];
  if (!st.ready) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_ws) != cudaSuccess || p == nullptr) return RT3D_ERR_CUDA;
    st.ws = static_cast<unsigned char*>(p);
    st.ready = true;
  }
  return RT3D_OK;
}
// The cached address, or nullptr if no handle has been prepared on this device yet.
unsigned char* noalloc_workspace(int dev) {
  std::lock_guard<std::mutex> lock(g_noalloc_mu);
  return g_noalloc[dev].ready ? g_noalloc[dev].ws : nullptr;
}
}  // namespace

extern "C" {

rt3d_status rt3d_conv2plus1d_fused(const rt3d_tensor* x, const rt3d_packed* w_s, const float* bias_s,
                                   const rt3d_conv_params* p_s, const rt3d_packed* w_t, const float* bias_t,
                                   const rt3d_conv_params* p_t, const rt3d_tensor* residual, rt3d_tensor* y,
                                   void* stream) {
  return conv2plus1d_impl(x, w_s, bias_s, p_s, w_t, bias_t, p_t, residual, y, stream);
}

rt3d_status rt3d_conv3d_sparse(const rt3d_tensor* x, const rt3d_packed* w, const float* bias,
                               const rt3d_conv_params* p, rt3d_tensor* y, void* stream) {
  return conv_impl(x, w, bias, p, y, stream, false);
}

rt3d_status rt3d_conv3d_dense(const rt3d_tensor* x, const rt3d_packed* w, const float* bias,
                              const rt3d_conv_params* p, rt3d_tensor* y, void* stream) {
  return conv_impl(x, w, bias, p, y, stream, true);
}

rt3d_status rt3d_conv3d_sparse_fused(const rt3d_tensor* x, const rt3d_packed* w, const float* bias,
                                     const rt3d_conv_params* p, const rt3d_fusion* fusion, rt3d_tensor* y,
                                     void* stream) {
  if (!fusion || !w) return RT3D_ERR_INVALID_ARG;
  return conv_impl(x, w, bias, p, y, stream, w->is_dense != 0, fusion);
}

rt3d_status rt3d_conv3d_host(const rt3d_tensor* x, rt3d_packed* w, const float* bias, const rt3d_conv_params* p,
                             rt3d_tensor* y, void* stream) {
  ConvGeom g;
  if (!y) return RT3D_ERR_INVALID_ARG;
  rt3d_status s = make_geom(x, w, p, y, &g);
  if (s != RT3D_OK) return s;
  DeviceBlob* blob = nullptr;
  if ((s = get_blob(w, &blob)) != RT3D_OK) return s;
  const size_t xb = size_t(tensor_span_bytes(x)), yb = size_t(tensor_span_bytes(y));
  {
    std::lock_guard<std::mutex> lock(w->mu);
    if (blob->stage_x_bytes < xb) {
      cudaFree(blob->stage_x);
      blob->stage_x = nullptr; blob->stage_x_bytes = 0;
      if (dev_malloc(&blob->stage_x, xb + 256) != cudaSuccess) return RT3D_ERR_ALLOC;
      blob->stage_x_bytes = xb;
    }
    if (blob->stage_y_bytes < yb) {
      cudaFree(blob->stage_y);
      blob->stage_y = nullptr; blob->stage_y_bytes = 0;
      if (dev_malloc(&blob->stage_y, yb + 256) != cudaSuccess) return RT3D_ERR_ALLOC;
      blob->stage_y_bytes = yb;
    }
    if (!blob->stage_bias && dev_malloc(&blob->stage_bias, size_t(w->M) * 4) != cudaSuccess)
      return RT3D_ERR_ALLOC;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (bias && cudaMemcpyAsync(blob->stage_bias, bias, size_t(w->M) * 4, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return RT3D_ERR_CUDA;
  const float* bias_d = bias ? blob->stage_bias : nullptr;
  // Clips are independent, so a large batch goes through in up to eight chunks of whole clips: chunk k+1 is
  // copied in on one stream while chunk k is convolved on the caller's stream and chunk k-1 is copied out on a
  // third (PCIe is full duplex; the call is bound by the larger of the two copies instead of their sum).
  constexpr int kHostChunks = 8;
  const int n_chunks = (x->n >= 2 && xb + yb >= (size_t(8) << 20)) ? (x->n < kHostChunks ? x->n : kHostChunks) : 1;
  if (n_chunks == 1) {
    if (cudaMemcpyAsync(blob->stage_x, x->data, xb, cudaMemcpyHostToDevice, st) != cudaSuccess) return RT3D_ERR_CUDA;
    rt3d_tensor xd = *x, yd = *y;
    xd.data = blob->stage_x;
    yd.data = blob->stage_y;
    s = conv_impl(&xd, w, bias_d, p, &yd, stream, w->is_dense != 0);
    if (s != RT3D_OK) return s;
    if (cudaMemcpyAsync(y->data, blob->stage_y, yb, cudaMemcpyDeviceToHost, st) != cudaSuccess) return RT3D_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return RT3D_ERR_CUDA;
    return RT3D_OK;
  }
  {
    std::lock_guard<std::mutex> lock(w->mu);
    for (void*& hs : blob->host_streams)
      if (!hs) {
        cudaStream_t ns;
        if (cudaStreamCreateWithFlags(&ns, cudaStreamNonBlocking) != cudaSuccess) return RT3D_ERR_CUDA;
        hs = ns;
      }
    for (void*& he : blob->host_events)
      if (!he) {
        cudaEvent_t ne;
        if (cudaEventCreateWithFlags(&ne, cudaEventDisableTiming) != cudaSuccess) return RT3D_ERR_CUDA;
        he = ne;
      }
  }
  cudaStream_t s_in = static_cast<cudaStream_t>(blob->host_streams[0]);
  cudaStream_t s_out = static_cast<cudaStream_t>(blob->host_streams[1]);
  auto ev = [&](int i) { return static_cast<cudaEvent_t>(blob->host_events[i]); };
  const size_t es = elem_size(x->dtype);
  const size_t x_clip = size_t(x->t) * x->h * x->w * x->c_stride * es, y_clip = size_t(y->t) * y->h * y->w * y->c_stride * es;
  bool cuda_ok = cudaEventRecord(ev(0), st) == cudaSuccess && cudaStreamWaitEvent(s_in, ev(0), 0) == cudaSuccess &&
                 cudaStreamWaitEvent(s_out, ev(0), 0) == cudaSuccess;
  rt3d_status cs = RT3D_OK;
  int n0 = 0;
  for (int k = 0; k < n_chunks && cuda_ok && cs == RT3D_OK; ++k) {
    const int n1 = int((long long)x->n * (k + 1) / n_chunks), nc = n1 - n0;
    const size_t xo = size_t(n0) * x_clip, yo = size_t(n0) * y_clip;
    const size_t xn = n1 == x->n ? xb - xo : size_t(nc) * x_clip, yn = n1 == x->n ? yb - yo : size_t(nc) * y_clip;
    cuda_ok = cudaMemcpyAsync(static_cast<char*>(blob->stage_x) + xo, static_cast<const char*>(x->data) + xo, xn,
                              cudaMemcpyHostToDevice, s_in) == cudaSuccess &&
              cudaEventRecord(ev(1 + k), s_in) == cudaSuccess && cudaStreamWaitEvent(st, ev(1 + k), 0) == cudaSuccess;
    if (!cuda_ok) break;
    rt3d_tensor xd = *x, yd = *y;
    xd.n = nc; yd.n = nc;
    xd.data = static_cast<char*>(blob->stage_x) + xo;
    yd.data = static_cast<char*>(blob->stage_y) + yo;
    cs = conv_impl(&xd, w, bias_d, p, &yd, stream, w->is_dense != 0);
    if (cs != RT3D_OK) break;
    cuda_ok = cudaEventRecord(ev(1 + kHostChunks + k), st) == cudaSuccess &&
              cudaStreamWaitEvent(s_out, ev(1 + kHostChunks + k), 0) == cudaSuccess &&
              cudaMemcpyAsync(static_cast<char*>(y->data) + yo, static_cast<char*>(blob->stage_y) + yo, yn,
                              cudaMemcpyDeviceToHost, s_out) == cudaSuccess;
    n0 = n1;
  }
  // the caller's stream ends up behind everything this call enqueued, whatever happened
  const bool joined = cudaEventRecord(ev(17), s_out) == cudaSuccess && cudaStreamWaitEvent(st, ev(17), 0) == cudaSuccess &&
                      cudaEventRecord(ev(0), s_in) == cudaSuccess && cudaStreamWaitEvent(st, ev(0), 0) == cudaSuccess;
  const bool synced = cudaStreamSynchronize(st) == cudaSuccess;
  if (cs != RT3D_OK) return cs;
  return (cuda_ok && joined && synced) ? RT3D_OK : RT3D_ERR_CUDA;
}

rt3d_status rt3d_packed_prepare(rt3d_packed* p) {
  if (!p) return RT3D_ERR_INVALID_ARG;
  DeviceState* d = nullptr;
  rt3d_status s = get_device_state(&d);
  if (s != RT3D_OK) return s;
  DeviceBlob* blob = nullptr;
  if ((s = get_blob(p, &blob)) != RT3D_OK) return s;
  if (d->cc_major == 10 && umma_layout_possible(p)) {
    const UmmaLayout* L = get_umma_layout(p, 0);
    DeviceBlob::Umma* u = nullptr;
    if (L && (s = get_umma_blob(p, blob, L, &u)) != RT3D_OK) return s;
  }
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return RT3D_ERR_CUDA;
  if ((s = noalloc_workspace_setup(dev)) != RT3D_OK) return s;
  return cudaDeviceSynchronize() == cudaSuccess ? RT3D_OK : RT3D_ERR_CUDA;
}

void rt3d_packed_free(rt3d_packed* p) {
  if (!p) return;
  int cur = -1;
  const bool have_dev = !p->blobs.empty() && cudaGetDevice(&cur) == cudaSuccess;
  {
    std::lock_guard<std::mutex> reg(g_blobs_mu);
    for (DeviceBlob* b : p->blobs)
      g_blobs.erase(std::remove(g_blobs.begin(), g_blobs.end(), b), g_blobs.end());
  }
  for (DeviceBlob* b : p->blobs) {
    if (have_dev) cudaSetDevice(b->device);
    cudaFree(b->group_ptr); cudaFree(b->pos_idx); cudaFree(b->tiles);
    for (auto& kv : b->umma) {
      cudaFree(kv.second.wtiles); cudaFree(kv.second.step_ptr); cudaFree(kv.second.steps);
      cudaFree(kv.second.grp_ptr); cudaFree(kv.second.grp_first);
    }
    cudaFree(b->stage_x); cudaFree(b->stage_y); cudaFree(b->stage_bias);
    for (void* hs : b->host_streams) if (hs) cudaStreamDestroy(static_cast<cudaStream_t>(hs));
    for (void* he : b->host_events) if (he) cudaEventDestroy(static_cast<cudaEvent_t>(he));
    for (auto& kv : b->smallc) { cudaFree(kv.second.wimg); cudaFree(kv.second.pairs); }
    for (auto& kv : b->sub) { cudaFree(kv.second.steps); cudaFree(kv.second.step_ptr); cudaFree(kv.second.blocks); }
    cudaFree(b->splitk); cudaFree(b->splitk_cnt);
    delete b;
  }
  if (have_dev && cur >= 0) cudaSetDevice(cur);
  delete p;
}

rt3d_status rt3d_maxpool3d(const rt3d_tensor* x, int kt, int kh, int kw, int st, int sh, int sw, int pt, int ph,
                           int pw, rt3d_tensor* y, void* stream) {
  rt3d_status s;
  if ((s = check_tensor(x)) != RT3D_OK || (s = check_tensor(y)) != RT3D_OK) return s;
  if (kt < 1 || kh < 1 || kw < 1 || st < 1 || sh < 1 || sw < 1 || pt < 0 || ph < 0 || pw < 0) return RT3D_ERR_INVALID_ARG;
  if (pt >= kt || ph >= kh || pw >= kw) return RT3D_ERR_INVALID_ARG;   // every window must see an input
  if (x->t + 2 * pt < kt || x->h + 2 * ph < kh || x->w + 2 * pw < kw) return RT3D_ERR_SHAPE;
  const int To = (x->t + 2 * pt - kt) / st + 1, Ho = (x->h + 2 * ph - kh) / sh + 1, Wo = (x->w + 2 * pw - kw) / sw + 1;
  if (y->n != x->n || y->t != To || y->h != Ho || y->w != Wo || y->c != x->c || y->dtype != x->dtype) return RT3D_ERR_SHAPE;
  // windows that start inside the padding but end before the tensor would see nothing
  if ((To - 1) * st - pt >= x->t || (Ho - 1) * sh - ph >= x->h || (Wo - 1) * sw - pw >= x->w) return RT3D_ERR_SHAPE;
  if ((s = check_alignment(x)) != RT3D_OK || (s = check_alignment(y)) != RT3D_OK) return s;
  if (overlaps(x, y)) return RT3D_ERR_INVALID_ARG;
  if (t_plan_only) return RT3D_OK;
  cudaError_t e = launch_maxpool3d(x->dtype, x->data, x->n, x->t, x->h, x->w, x->c, x->c_stride, kt, kh, kw, st, sh, sw,
                                   pt, ph, pw, y->data, To, Ho, Wo, y->c_stride, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return RT3D_ERR_CUDA;
  g_launches.fetch_add(1);
  return RT3D_OK;
}

rt3d_status rt3d_add_relu(const rt3d_tensor* a, const rt3d_tensor* b, int relu, rt3d_tensor* y, void* stream) {
  rt3d_status s;
  if ((s = check_tensor(a)) != RT3D_OK || (s = check_tensor(b)) != RT3D_OK || (s = check_tensor(y)) != RT3D_OK) return s;
  if (a->n != b->n || a->t != b->t || a->h != b->h || a->w != b->w || a->c != b->c || a->dtype != b->dtype) return RT3D_ERR_SHAPE;
  if (a->n != y->n || a->t != y->t || a->h != y->h || a->w != y->w || a->c != y->c || a->dtype != y->dtype) return RT3D_ERR_SHAPE;
  if ((s = check_alignment(a)) != RT3D_OK || (s = check_alignment(b)) != RT3D_OK || (s = check_alignment(y)) != RT3D_OK) return s;
  const int64_t vox = int64_t(a->n) * a->t * a->h * a->w;
  if (t_plan_only) return RT3D_OK;
  cudaError_t e = launch_add_relu(a->dtype, a->data, a->c_stride, b->data, b->c_stride, y->data, y->c_stride, vox, a->c,
                                  relu ? 1 : 0, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return RT3D_ERR_CUDA;
  g_launches.fetch_add(1);
  return RT3D_OK;
}

rt3d_status rt3d_conv3d_cost(const rt3d_tensor* x, const rt3d_packed* w, const rt3d_conv_params* p,
                             int64_t* kept_macs, int64_t* dense_macs, int64_t* alg_bytes) {
  ConvGeom g;
  rt3d_status s = make_geom(x, w, p, nullptr, &g);
  if (s != RT3D_OK) return s;
  const int64_t vox_out = int64_t(g.n) * g.To * g.Ho * g.Wo;
  // kept weights that exist (ragged groups hold fewer than g_m*g_n kernels)
  int64_t kept_w = 0;
  for (int pr = 0; pr < w->P; ++pr) {
    const int rows = std::min(w->g_m, w->M - pr * w->g_m);
    for (int q = 0; q < w->Q; ++q) {
      const int cols = std::min(w->g_n, w->N - q * w->g_n);
      kept_w += int64_t(w->group_ptr[size_t(pr) * w->Q + q + 1] - w->group_ptr[size_t(pr) * w->Q + q]) * rows * cols;
    }
  }
  if (kept_macs) *kept_macs = vox_out * kept_w;
  if (dense_macs) *dense_macs = vox_out * int64_t(w->M) * w->N * w->Ks;
  if (alg_bytes) {
    const int64_t e = int64_t(elem_size(w->dtype));
    const int64_t vox_in = int64_t(g.n) * g.t * g.h * g.w;
    *alg_bytes = vox_in * g.c * e + vox_out * g.M * e + w->nnz * w->g_m * w->g_n * e + w->nnz * 2 +
                 int64_t(w->P) * w->Q * 4 + 4 + int64_t(w->M) * 4;
  }
  return RT3D_OK;
}

rt3d_status rt3d_conv3d_query_algo(const rt3d_tensor* x, const rt3d_packed* w, const rt3d_conv_params* p,
                                   const rt3d_tensor* y, int* algo) {
  ConvGeom g;
  if (!algo || !y) return RT3D_ERR_INVALID_ARG;
  rt3d_status s = make_geom(x, w, p, y, &g);
  if (s != RT3D_OK) return s;
  DeviceState* d = nullptr;
  if ((s = get_device_state(&d)) != RT3D_OK) return s;
  const bool can = umma_eligible(d, w, x, y, p);
  if (p->algo == RT3D_ALGO_UMMA && !can) return RT3D_ERR_UNSUPPORTED;
  *algo = (p->algo == RT3D_ALGO_SIMT || !can) ? RT3D_ALGO_SIMT : RT3D_ALGO_UMMA;
  return RT3D_OK;
}

rt3d_status rt3d_last_plan(rt3d_plan_info* info) {
  if (!info || t_last_plan.kernel < 0) return RT3D_ERR_INVALID_ARG;
  *info = t_last_plan;
  return RT3D_OK;
}

long long rt3d_debug_get(int what) {
  if (what != RT3D_DEBUG_WAIT_SITE) return -1;
  DeviceState* d = nullptr;
  if (get_device_state(&d) != RT3D_OK) return -1;
  if (cudaDeviceSynchronize() != cudaSuccess) return -1;
  int32_t word = 0;
  if (cudaMemcpy(&word, d->sched + 2, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return -1;
  return word;
}

rt3d_status rt3d_last_device_status(void* stream) {
  DeviceState* d = nullptr;
  rt3d_status s = get_device_state(&d);
  if (s != RT3D_OK) return s;
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return RT3D_ERR_CUDA;
  int32_t word = 0;
  if (cudaMemcpy(&word, d->sched + 2, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return RT3D_ERR_CUDA;
  if (word != 0) {
    cudaMemset(d->sched + 2, 0, 4);
    // A kernel that gave up may have left K-split arrival counters and tail-split flags non-zero (they are
    // cleared by the CTA that finishes a tile): clear them for every handle on this device, so that later
    // calls do not take a stale count for "all other splits have arrived".
    int dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) {
      cudaDeviceSynchronize();
      std::lock_guard<std::mutex> reg(g_blobs_mu);
      for (DeviceBlob* b : g_blobs)
        if (b->device == dev && b->splitk_cnt) cudaMemset(b->splitk_cnt, 0, b->splitk_cnt_bytes);
    }
    return RT3D_ERR_TIMEOUT;
  }
  return RT3D_OK;
}

rt3d_status rt3d_conv3d_sparse_noalloc(const rt3d_tensor* x, const rt3d_packed* wc, const float* bias,
                                       const rt3d_conv_params* p, rt3d_tensor* y, void* stream) {
  ConvGeom g;
  if (!y) return RT3D_ERR_INVALID_ARG;
  rt3d_status s = make_geom(x, wc, p, y, &g);
  if (s != RT3D_OK) return s;
  if ((s = check_alignment(x)) != RT3D_OK || (s = check_alignment(y)) != RT3D_OK) return s;
  if (overlaps(x, y)) return RT3D_ERR_INVALID_ARG;
  if (p->algo == RT3D_ALGO_SIMT) return RT3D_ERR_UNSUPPORTED;
  rt3d_packed* w = const_cast<rt3d_packed*>(wc);
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return RT3D_ERR_CUDA;
  // everything that needs an allocation must already exist: device state, weight blobs (rt3d_packed_prepare)
  DeviceState* d = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_dev_mu);
    if (g_dev[dev].init) d = &g_dev[dev];
  }
  if (!d) return RT3D_ERR_NOT_PREPARED;
  if (!umma_eligible(d, w, x, y, p)) return RT3D_ERR_UNSUPPORTED;
  const int n_tile = default_n_tile(w->M);
  DeviceBlob* blob = nullptr;
  DeviceBlob::Umma* u = nullptr;
  const UmmaLayout* L = nullptr;
  {
    std::lock_guard<std::mutex> lock(w->mu);
    blob = find_blob(w, dev);
    if (blob) {
      auto it = blob->umma.find(n_tile);
      if (it != blob->umma.end() && it->second.ready) u = &it->second;
    }
    auto li = w->umma_layouts.find(n_tile);
    if (li != w->umma_layouts.end()) L = &li->second;
  }
  if (!blob || !u || !L) return RT3D_ERR_NOT_PREPARED;
  unsigned char* ws = noalloc_workspace(dev);
  if (!ws) return RT3D_ERR_NOT_PREPARED;

  UmmaArgs a;
  a.g = g;
  a.box = choose_box(g);
  a.tiles_n = ceil_div(g.n, a.box.bn); a.tiles_t = ceil_div(g.To, a.box.bt);
  a.tiles_h = ceil_div(g.Ho, a.box.bh); a.tiles_w = ceil_div(g.Wo, a.box.bw);
  a.n_tile = L->n_tile; a.n_bundles = L->n_bundles; a.n_chunks = L->n_chunks;
  a.dense = 0;
  a.steps_dense = w->Ks * L->n_chunks;
  a.step_ptr = u->step_ptr; a.steps = u->steps;
  a.bias = bias; a.y = y->data; a.sched = d->sched;
  // Split rule of this entry point: as many K splits (at most 8) as keep every SM busy, each with at
  // least 8 of the K steps of the layer's longest step list.
  const long long tiles = (long long)a.tiles_n * a.tiles_t * a.tiles_h * a.tiles_w * L->n_bundles;
  long long splits = tiles > 0 ? d->sm_count / tiles : 1;
  if (splits > 8) splits = 8;
  if (splits > L->max_steps / 8) splits = L->max_steps / 8;
  if (splits < 1) splits = 1;
  a.n_splits = int(splits);
  a.residual = nullptr; a.rcs = 0;
  a.scratch = nullptr; a.counters = nullptr;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (a.n_splits > 1) {
    const long long partial_bytes = tiles * a.n_splits * kTileM * L->n_tile * 4LL;
    if (partial_bytes > RT3D_NOALLOC_PARTIAL_BYTES || tiles * 32 > RT3D_NOALLOC_COUNTER_BYTES)
      return RT3D_ERR_WORKSPACE;
    a.scratch = reinterpret_cast<float*>(ws);
    a.counters = reinterpret_cast<int32_t*>(ws + RT3D_NOALLOC_PARTIAL_BYTES);
    // the counters must start at zero; the workspace keeps whatever the last call left behind
    if (cudaMemsetAsync(a.counters, 0, size_t(tiles) * 32, st) != cudaSuccess) return RT3D_ERR_CUDA;
  }
  CUtensorMap xmap;
  if ((s = encode_xmap(x, g, a.box, &xmap)) != RT3D_OK) return s;
  CUtensorMap ymap;
  int sb[4];
  a.pool_t = a.pool_h = a.pool_w = 1; a.sbw = a.sbh = 1;
  a.tail_workers = 0; a.tail_scratch = nullptr; a.tail_flags = nullptr;
  a.ts = 0; a.grp_ptr = nullptr; a.grp_first = nullptr; a.ts_a_bytes = 0; a.ts_frame_bytes = 0; a.ts_table = 0; a.ts_phases = 1;
  a.wait_cycles = 0; a.debug_drop_last_load = 0;
  a.store_tma = (a.n_splits == 1 && warp_block(a.box.bw, a.box.bh, a.box.bt, a.box.bn, sb) &&
                 encode_ymap(y, sb, 1, 1, 1, &ymap)) ? 1 : 0;
  if (launch_conv_umma(a, &xmap, u->wmap, a.store_tma ? &ymap : nullptr, d->sm_count, st) != cudaSuccess) return RT3D_ERR_CUDA;
  g_launches.fetch_add(1);
  t_last_plan = rt3d_plan_info{1, a.n_tile, a.n_splits, 0, 0};
  return RT3D_OK;
}

int64_t rt3d_launch_count(void) { return g_launches.load(); }

int64_t rt3d_alloc_count(void) { return g_allocs.load(); }

void rt3d_plan_begin(void) { t_plan_only = true; }
void rt3d_plan_end(void) { t_plan_only = false; }

rt3d_status rt3d_debug_set(int what, long long value) {
  if (what == RT3D_DEBUG_WAIT_CYCLES) { if (value < 0) return RT3D_ERR_INVALID_ARG; g_debug_wait_cycles.store(value); return RT3D_OK; }
  if (what == RT3D_DEBUG_DROP_LAST_LOAD) { g_debug_drop_last_load.store(value != 0); return RT3D_OK; }
  if (what == RT3D_DEBUG_T_GROUPS) { g_ts_enabled.store(value != 0); return RT3D_OK; }
  if (what == RT3D_DEBUG_POISON) {
    DeviceState* d = nullptr;
    rt3d_status s = get_device_state(&d);
    if (s != RT3D_OK) return s;
    if (d->cc_major != 10) return RT3D_ERR_UNSUPPORTED;
    if (launch_debug_poison(uint32_t(value), d->sm_count, d->sched + 8, nullptr) != cudaSuccess) return RT3D_ERR_CUDA;
    if (cudaDeviceSynchronize() != cudaSuccess) return RT3D_ERR_CUDA;
    // the K splits' partial tiles in global memory too (all ones: NaNs as fp32); their counters and flags stay zero
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return RT3D_ERR_CUDA;
    std::lock_guard<std::mutex> reg(g_blobs_mu);
    for (DeviceBlob* b : g_blobs)
      if (b->device == dev && b->splitk && cudaMemset(b->splitk, 0xFF, b->splitk_bytes) != cudaSuccess) return RT3D_ERR_CUDA;
    return RT3D_OK;
  }
  return RT3D_ERR_INVALID_ARG;
}


const char* rt3d_status_string(rt3d_status s) {
  switch (s) {
    case RT3D_OK: return "ok";
    case RT3D_ERR_INVALID_ARG: return "invalid argument";
    case RT3D_ERR_SHAPE: return "shape or dtype mismatch";
    case RT3D_ERR_MASK_NOT_GROUP_UNIFORM: return "mask is not uniform inside a kernel group";
    case RT3D_ERR_UNSUPPORTED: return "unsupported";
    case RT3D_ERR_ALLOC: return "allocation failed";
    case RT3D_ERR_CUDA: return "CUDA error";
    case RT3D_ERR_TIMEOUT: return "device-side wait timed out";
    case RT3D_ERR_WORKSPACE: return "request needs more than the library's fixed workspace";
    case RT3D_ERR_NOT_PREPARED: return "handle not prepared on this device (call rt3d_packed_prepare first)";
  }
  return "unknown status";
}

const char* rt3d_version(void) { return "rt3d-b200 0.1 (sm_100a)"; }

}  // extern "C"
