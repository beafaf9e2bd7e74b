// Host-side weight reorganisation: the KGS pack (Section 3 / Section 5.2 of the paper), its
// inverse, and the derivation of the tensor-core weight layout from the canonical arrays.
// Pure host code: no CUDA calls, usable without a GPU.
#include <algorithm>
#include <cstring>
#include <new>
#include <utility>

#include "rt3d_internal.h"

namespace rt3d {

uint16_t f32_to_bf16_bits(float f) {
  uint32_t u;
  std::memcpy(&u, &f, 4);
  if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu)) return uint16_t((u >> 16) | 0x40u);
  u += 0x7FFFu + ((u >> 16) & 1u);   // ties to even
  return uint16_t(u >> 16);
}

float bf16_bits_to_f32(uint16_t b) {
  uint32_t u = uint32_t(b) << 16;
  float f;
  std::memcpy(&f, &u, 4);
  return f;
}

int default_n_tile(int M) {
  const int bundles = ceil_div(round_up(M, 16), 256);
  return round_up(ceil_div(M, bundles), 16);
}

bool umma_layout_possible(const rt3d_packed* p) {
  return p->dtype == RT3D_BF16 && p->Kt <= 63 && p->Kh <= 63 && p->Kw <= 63 && ceil_div(p->N, kChunk) <= 4095;
}

static float tile_value(const rt3d_packed* p, int64_t e, int i, int j) {
  const int64_t o = (e * p->g_m + i) * p->g_n + j;
  if (p->dtype == RT3D_BF16) return bf16_bits_to_f32(reinterpret_cast<const uint16_t*>(p->tiles.data())[o]);
  return reinterpret_cast<const float*>(p->tiles.data())[o];
}

// For each bundle of n_tile output channels, list the (kernel location, 64-channel chunk)
// steps in which at least one kernel group of the bundle keeps that location, and build the
// matching [n_tile][64] weight tiles (zeros where a group prunes the location).  Steps are
// ordered by location, then chunk.
// `t_groups`: the order is (kh, kw), chunk, kt instead, and the steps that differ only in kt form a
// group (grp_ptr / grp_first): the CTA-pair kernel stages one input tile, Kt - 1 frames deeper, per group.
const UmmaLayout* get_umma_layout(rt3d_packed* p, int n_tile, bool t_groups) {
  if (!umma_layout_possible(p)) return nullptr;
  if (n_tile <= 0) n_tile = default_n_tile(p->M);
  if (n_tile % 16 || n_tile > 256) return nullptr;
  std::lock_guard<std::mutex> lock(p->mu);
  const int key = n_tile + (t_groups ? 4096 : 0);
  auto it = p->umma_layouts.find(key);
  if (it != p->umma_layouts.end()) return &it->second;

  UmmaLayout L;
  L.n_tile = n_tile;
  L.t_groups = t_groups;
  if (t_groups) L.grp_ptr.assign(1, 0);
  L.n_bundles = ceil_div(p->M, n_tile);
  L.n_chunks = ceil_div(p->N, kChunk);
  L.step_ptr.assign(L.n_bundles + 1, 0);
  const int Ks = p->Ks;
  std::vector<int32_t> slot(size_t(Ks) * L.n_chunks);
  for (int b = 0; b < L.n_bundles; ++b) {
    const int m_lo = b * n_tile, m_hi = std::min(p->M, m_lo + n_tile);
    const int p_lo = m_lo / p->g_m, p_hi = ceil_div(m_hi, p->g_m);
    // pass 1: which steps are non-empty
    std::fill(slot.begin(), slot.end(), -1);
    for (int pr = p_lo; pr < p_hi; ++pr)
      for (int q = 0; q < p->Q; ++q) {
        const int c_lo = q * p->g_n, c_hi = std::min(p->N, c_lo + p->g_n);
        for (int32_t e = p->group_ptr[pr * p->Q + q]; e < p->group_ptr[pr * p->Q + q + 1]; ++e)
          for (int ch = c_lo / kChunk; ch <= (c_hi - 1) / kChunk; ++ch)
            slot[size_t(p->pos_idx[e]) * L.n_chunks + ch] = 0;
      }
    const int32_t base = L.step_ptr[b];
    int32_t cnt = 0;
    if (!t_groups) {
      for (int kpos = 0; kpos < Ks; ++kpos)
        for (int ch = 0; ch < L.n_chunks; ++ch)
          if (slot[size_t(kpos) * L.n_chunks + ch] == 0) {
            slot[size_t(kpos) * L.n_chunks + ch] = base + cnt++;
            const int kw = kpos % p->Kw, kh = (kpos / p->Kw) % p->Kh, kt = kpos / (p->Kw * p->Kh);
            L.steps.push_back(encode_step(kt, kh, kw, ch));
          }
    } else {
      for (int hw = 0; hw < p->Kh * p->Kw; ++hw)
        for (int ch = 0; ch < L.n_chunks; ++ch) {
          bool open = false;
          for (int kt = 0; kt < p->Kt; ++kt) {
            const int kpos = kt * p->Kh * p->Kw + hw;
            if (slot[size_t(kpos) * L.n_chunks + ch] != 0) continue;
            if (!open) { L.grp_first.push_back(base + cnt); open = true; }
            slot[size_t(kpos) * L.n_chunks + ch] = base + cnt++;
            L.steps.push_back(encode_step(kt, hw / p->Kw, hw % p->Kw, ch));
          }
        }
      L.grp_ptr.push_back(int32_t(L.grp_first.size()));
    }
    L.step_ptr[b + 1] = base + cnt;
    L.max_steps = std::max(L.max_steps, int(cnt));
    L.wtiles.resize(size_t(base + cnt) * n_tile * kChunk, 0);
    // pass 2: scatter the kept tiles
    for (int pr = p_lo; pr < p_hi; ++pr)
      for (int q = 0; q < p->Q; ++q)
        for (int32_t e = p->group_ptr[pr * p->Q + q]; e < p->group_ptr[pr * p->Q + q + 1]; ++e)
          for (int i = 0; i < p->g_m; ++i) {
            const int m = pr * p->g_m + i;
            if (m < m_lo || m >= m_hi) continue;
            for (int j = 0; j < p->g_n; ++j) {
              const int c = q * p->g_n + j;
              if (c >= p->N) continue;
              const int32_t s = slot[size_t(p->pos_idx[e]) * L.n_chunks + c / kChunk];
              L.wtiles[(size_t(s) * n_tile + (m - m_lo)) * kChunk + c % kChunk] =
                  reinterpret_cast<const uint16_t*>(p->tiles.data())[(int64_t(e) * p->g_m + i) * p->g_n + j];
            }
          }
  }
  if (t_groups) L.grp_first.push_back(int32_t(L.steps.size()));     // sentinel: end of the last group
  auto res = p->umma_layouts.emplace(key, std::move(L));
  return &res.first->second;
}

// Layout of the sub-tile kernel (see SubLayout and SubStep).
const SubLayout* get_sub_layout(rt3d_packed* p, int n_tile) {
  if (!umma_layout_possible(p)) return nullptr;
  if (n_tile <= 0) n_tile = default_n_tile(p->M);
  if (n_tile % 16 || n_tile > 256) return nullptr;
  std::lock_guard<std::mutex> lock(p->mu);
  auto it = p->sub_layouts.find(n_tile);
  if (it != p->sub_layouts.end()) return &it->second;

  SubLayout L;
  L.n_tile = n_tile;
  L.n_bundles = ceil_div(p->M, n_tile);
  L.n_chunks = ceil_div(p->N, kChunk);
  L.step_ptr.assign(L.n_bundles + 1, 0);
  const int Ks = p->Ks;
  const uint16_t* tiles = reinterpret_cast<const uint16_t*>(p->tiles.data());
  std::vector<uint64_t> pres(size_t(Ks) * L.n_chunks);     // bit ks*16 + r: block (range r, K slice ks) exists
  std::vector<int32_t> slot(size_t(Ks) * L.n_chunks);
  for (int b = 0; b < L.n_bundles; ++b) {
    const int m_lo = b * n_tile, m_hi = std::min(p->M, m_lo + n_tile);
    const int n_ranges = ceil_div(m_hi - m_lo, kSubRange);
    const int p_lo = m_lo / p->g_m, p_hi = ceil_div(m_hi, p->g_m);
    // pass 1: which (range, K slice) blocks exist in which (location, chunk) step
    std::fill(pres.begin(), pres.end(), uint64_t(0));
    for (int pr = p_lo; pr < p_hi; ++pr) {
      const int r_lo = (std::max(pr * p->g_m, m_lo) - m_lo) / kSubRange;
      const int r_hi = (std::min(std::min((pr + 1) * p->g_m, p->M), m_hi) - 1 - m_lo) / kSubRange;
      uint64_t rbits = 0;
      for (int r = r_lo; r <= r_hi; ++r) rbits |= uint64_t(1) << r;
      for (int q = 0; q < p->Q; ++q) {
        const int c_lo = q * p->g_n, c_hi = std::min(p->N, c_lo + p->g_n);
        for (int32_t e = p->group_ptr[size_t(pr) * p->Q + q]; e < p->group_ptr[size_t(pr) * p->Q + q + 1]; ++e)
          for (int sl = c_lo / 16; sl <= (c_hi - 1) / 16; ++sl)       // 16-channel slices the group touches
            pres[size_t(p->pos_idx[e]) * L.n_chunks + sl / 4] |= rbits << ((sl % 4) * 16);
      }
    }
    const int32_t first_step = int32_t(L.steps.size());
    for (int ch = 0; ch < L.n_chunks; ++ch)
      for (int kpos = 0; kpos < Ks; ++kpos) {
        uint64_t m = pres[size_t(kpos) * L.n_chunks + ch];
        slot[size_t(kpos) * L.n_chunks + ch] = -1;
        if (!m) continue;
        if (int32_t(L.steps.size()) == first_step) {          // first step: every range starts its accumulator here
          m |= (uint64_t(1) << n_ranges) - 1;
          pres[size_t(kpos) * L.n_chunks + ch] = m;
        }
        slot[size_t(kpos) * L.n_chunks + ch] = int32_t(L.steps.size());
        const int kw = kpos % p->Kw, kh = (kpos / p->Kw) % p->Kh, kt = kpos / (p->Kw * p->Kh);
        SubStep st{};
        st.enc = encode_step(kt, kh, kw, ch);
        st.off64 = unsigned(L.payload.size() / 64);
        st.nblk = __builtin_popcountll(m);
        L.steps.push_back(st);
        L.max_blocks = std::max(L.max_blocks, st.nblk);
        const size_t base = L.payload.size();
        L.payload.resize(base + kSubHeaderBytes + size_t(st.nblk) * kSubBlockBytes, 0);
        int idx = 0;
        for (int bit = 0; bit < 64; ++bit)
          if ((m >> bit) & 1) L.payload[base + size_t(4 * (bit % 16) + bit / 16)] = uint8_t(0x80 | idx++);
      }
    const int32_t end_step = int32_t(L.steps.size());
    L.step_ptr[b + 1] = end_step;
    L.max_steps = std::max(L.max_steps, int(end_step - first_step));
    // pass 2: scatter the kept weights into their blocks
    for (int pr = p_lo; pr < p_hi; ++pr)
      for (int q = 0; q < p->Q; ++q)
        for (int32_t e = p->group_ptr[size_t(pr) * p->Q + q]; e < p->group_ptr[size_t(pr) * p->Q + q + 1]; ++e)
          for (int i = 0; i < p->g_m; ++i) {
            const int m = pr * p->g_m + i;
            if (m < m_lo || m >= m_hi) continue;
            const int r = (m - m_lo) / kSubRange, ri = (m - m_lo) % kSubRange;
            for (int j = 0; j < p->g_n; ++j) {
              const int c = q * p->g_n + j;
              if (c >= p->N) continue;
              const SubStep& st = L.steps[slot[size_t(p->pos_idx[e]) * L.n_chunks + c / kChunk]];
              const size_t base = size_t(st.off64) * 64;
              const int ks = (c % kChunk) / 16, kj = c % 16;
              const size_t blk = L.payload[base + size_t(4 * r + ks)] & 0x3F;
              uint16_t* dst = reinterpret_cast<uint16_t*>(L.payload.data() + base + kSubHeaderBytes + blk * kSubBlockBytes);
              dst[((ri / 8) * 2 + kj / 8) * 64 + (ri % 8) * 8 + kj % 8] = tiles[(int64_t(e) * p->g_m + i) * p->g_n + j];
            }
          }
  }
  auto res = p->sub_layouts.emplace(n_tile, std::move(L));
  return &res.first->second;
}

// Small-C_in layout for spatial strides (sh, sw): kernel locations kept by at least one group are
// sorted by the offset of their window inside the staged phase images and paired; each pair is one
// K=16 MMA whose two K halves are the 8 (padded) channels at the two locations.  Operands use the
// no-swizzle core-matrix layout (8 rows x 16 bytes).
const SmallCLayout* get_smallc_layout(rt3d_packed* p, int sh, int sw) {
  if (p->dtype != RT3D_BF16 || p->N > 8 || p->M > 256 || sh < 1 || sw < 1 || sh > 4 || sw > 4) return nullptr;
  std::lock_guard<std::mutex> lock(p->mu);
  const int key = sh * 16 + sw;
  auto it = p->smallc_layouts.find(key);
  if (it != p->smallc_layouts.end()) return &it->second;
  SmallCLayout L;
  L.sh = sh; L.sw = sw;
  L.n_pad = round_up(p->M, 16);
  L.n_phases = sh * sw;
  L.img_w = kSmallCTileW - 1 + ceil_div(p->Kw, sw);
  L.img_h = kSmallCTileH - 1 + ceil_div(p->Kh, sh);
  L.img_t = p->Kt;
  L.phase_stride = round_up(L.img_w * L.img_h * L.img_t * 16, 128);   // a TMA box must land on a 128-byte boundary
  std::vector<uint8_t> used(size_t(p->Ks), 0);
  for (int64_t e = 0; e < p->nnz; ++e) used[p->pos_idx[size_t(e)]] = 1;
  std::vector<std::pair<int, int>> pos;            // (window offset, kernel location)
  for (int k = 0; k < p->Ks; ++k) {
    if (!used[size_t(k)]) continue;
    const int kw = k % p->Kw, kh = (k / p->Kw) % p->Kh, kt = k / (p->Kw * p->Kh);
    const int phase = (kh % sh) * sw + (kw % sw);
    pos.emplace_back(phase * L.phase_stride + ((kt * L.img_h + kh / sh) * L.img_w + kw / sw) * 16, k);
  }
  std::sort(pos.begin(), pos.end());
  L.n_pairs = ceil_div(int(pos.size()), 2);
  L.pair_off.assign(size_t(L.n_pairs) * 2, 0);
  L.wimg.assign(size_t(L.n_pairs) * 2 * L.n_pad * 8, 0);
  std::vector<int> slot(size_t(p->Ks), -1);       // location -> pair*2 + half
  for (size_t i = 0; i < pos.size(); ++i) {
    L.pair_off[i] = pos[i].first;
    slot[size_t(pos[i].second)] = int(i);
  }
  // An odd count leaves the last pair's second K half without a location: zero weights, read through the SAME window
  // as the first half.  (A window 16 bytes further on runs, for the tile's last voxel, past the end of the staged
  // image into shared memory that no load ever wrote; a NaN or infinity there times zero is a NaN in that voxel's
  // accumulators, which a following max-pool silently drops: rare, run-to-run different outputs.)
  if (pos.size() % 2) L.pair_off[pos.size()] = L.pair_off[pos.size() - 1];
  const uint16_t* tiles = reinterpret_cast<const uint16_t*>(p->tiles.data());
  for (int pr = 0; pr < p->P; ++pr)
    for (int q = 0; q < p->Q; ++q)
      for (int32_t e = p->group_ptr[size_t(pr) * p->Q + q]; e < p->group_ptr[size_t(pr) * p->Q + q + 1]; ++e) {
        const int s = slot[p->pos_idx[size_t(e)]];
        for (int i = 0; i < p->g_m && pr * p->g_m + i < p->M; ++i)
          for (int j = 0; j < p->g_n && q * p->g_n + j < p->N; ++j) {
            const int m = pr * p->g_m + i, c = q * p->g_n + j;
            L.wimg[((size_t(s) * (L.n_pad / 8) + m / 8) * 8 + m % 8) * 8 + c] =
                tiles[(size_t(e) * p->g_m + i) * p->g_n + j];
          }
      }
  auto res = p->smallc_layouts.emplace(key, std::move(L));
  return &res.first->second;
}

static rt3d_status pack_impl(const float* w, const uint8_t* mask, int M, int N, int Kt, int Kh, int Kw,
                             int g_m, int g_n, int dtype, int is_dense, rt3d_packed** out) {
  if (!w || !out) return RT3D_ERR_INVALID_ARG;
  *out = nullptr;
  if (M <= 0 || N <= 0 || Kt <= 0 || Kh <= 0 || Kw <= 0) return RT3D_ERR_INVALID_ARG;
  if (g_m < 1 || g_n < 1 || g_m > kMaxGroup || g_n > kMaxGroup) return RT3D_ERR_INVALID_ARG;
  if (dtype != RT3D_F32 && dtype != RT3D_BF16) return RT3D_ERR_INVALID_ARG;
  const int64_t Ks64 = int64_t(Kt) * Kh * Kw;
  if (Ks64 > 65535) return RT3D_ERR_INVALID_ARG;
  rt3d_packed* h = new (std::nothrow) rt3d_packed;
  if (!h) return RT3D_ERR_ALLOC;
  try {
    h->M = M; h->N = N; h->Kt = Kt; h->Kh = Kh; h->Kw = Kw; h->g_m = g_m; h->g_n = g_n;
    h->P = ceil_div(M, g_m); h->Q = ceil_div(N, g_n); h->Ks = int(Ks64);
    h->dtype = dtype; h->is_dense = is_dense;
    const int Ks = h->Ks;
    const size_t esz = dtype == RT3D_BF16 ? 2 : 4;
    h->group_ptr.resize(size_t(h->P) * h->Q + 1);
    // pass 1: group-level decisions with the uniformity check of the KGS definition
    std::vector<uint8_t> keep(size_t(h->P) * h->Q * Ks);
    int64_t nnz = 0;
    bool vanilla = true;
    for (int pr = 0; pr < h->P; ++pr)
      for (int q = 0; q < h->Q; ++q) {
        int kept_here = 0;
        for (int k = 0; k < Ks; ++k) {
          int decided = -1;
          if (!mask) decided = 1;
          else
            for (int i = 0; i < g_m && pr * g_m + i < M; ++i)
              for (int j = 0; j < g_n && q * g_n + j < N; ++j) {
                const int bit = mask[(int64_t(pr * g_m + i) * N + (q * g_n + j)) * Ks + k] ? 1 : 0;
                if (decided < 0) decided = bit;
                else if (decided != bit) { delete h; return RT3D_ERR_MASK_NOT_GROUP_UNIFORM; }
              }
          keep[(size_t(pr) * h->Q + q) * Ks + k] = uint8_t(decided > 0);
          kept_here += decided > 0;
        }
        if (kept_here != 0 && kept_here != Ks) vanilla = false;
        nnz += kept_here;
      }
    if (nnz > 0x7FFFFFFF) { delete h; return RT3D_ERR_UNSUPPORTED; }
    h->nnz = nnz;
    h->is_vanilla = vanilla;
    h->pos_idx.resize(size_t(nnz));
    h->tiles.assign(size_t(nnz) * g_m * g_n * esz, 0);
    // pass 2: emit index and tiles
    int64_t e = 0;
    for (int pr = 0; pr < h->P; ++pr)
      for (int q = 0; q < h->Q; ++q) {
        h->group_ptr[size_t(pr) * h->Q + q] = int32_t(e);
        for (int k = 0; k < Ks; ++k) {
          if (!keep[(size_t(pr) * h->Q + q) * Ks + k]) continue;
          h->pos_idx[size_t(e)] = uint16_t(k);
          for (int i = 0; i < g_m && pr * g_m + i < M; ++i)
            for (int j = 0; j < g_n && q * g_n + j < N; ++j) {
              const float v = w[(int64_t(pr * g_m + i) * N + (q * g_n + j)) * Ks + k];
              const size_t o = (size_t(e) * g_m + i) * g_n + j;
              if (dtype == RT3D_BF16) reinterpret_cast<uint16_t*>(h->tiles.data())[o] = f32_to_bf16_bits(v);
              else reinterpret_cast<float*>(h->tiles.data())[o] = v;
            }
          ++e;
        }
      }
    h->group_ptr[size_t(h->P) * h->Q] = int32_t(e);
  } catch (const std::bad_alloc&) {
    delete h;
    return RT3D_ERR_ALLOC;
  }
  *out = h;
  return RT3D_OK;
}

}  // namespace rt3d

using namespace rt3d;

extern "C" {

rt3d_status rt3d_pack_kgs(const float* w, const uint8_t* mask, int M, int N, int Kt, int Kh, int Kw,
                          int g_m, int g_n, int compute_dtype, rt3d_packed** out) {
  return pack_impl(w, mask, M, N, Kt, Kh, Kw, g_m, g_n, compute_dtype, 0, out);
}

rt3d_status rt3d_pack_dense(const float* w, int M, int N, int Kt, int Kh, int Kw, int compute_dtype,
                            rt3d_packed** out) {
  return pack_impl(w, nullptr, M, N, Kt, Kh, Kw, 4, 4, compute_dtype, 1, out);
}

rt3d_status rt3d_packed_view_get(const rt3d_packed* p, rt3d_packed_view* v) {
  if (!p || !v) return RT3D_ERR_INVALID_ARG;
  v->M = p->M; v->N = p->N; v->Kt = p->Kt; v->Kh = p->Kh; v->Kw = p->Kw;
  v->g_m = p->g_m; v->g_n = p->g_n; v->P = p->P; v->Q = p->Q; v->Ks = p->Ks;
  v->dtype = p->dtype; v->is_vanilla = p->is_vanilla; v->is_dense = p->is_dense; v->nnz = p->nnz;
  v->group_ptr = p->group_ptr.data();
  v->pos_idx = p->pos_idx.data();
  v->tiles = p->tiles.data();
  return RT3D_OK;
}

rt3d_status rt3d_unpack_to_dense(const rt3d_packed* p, float* w_out) {
  if (!p || !w_out) return RT3D_ERR_INVALID_ARG;
  std::memset(w_out, 0, sizeof(float) * size_t(p->M) * p->N * p->Ks);
  for (int pr = 0; pr < p->P; ++pr)
    for (int q = 0; q < p->Q; ++q)
      for (int32_t e = p->group_ptr[size_t(pr) * p->Q + q]; e < p->group_ptr[size_t(pr) * p->Q + q + 1]; ++e)
        for (int i = 0; i < p->g_m && pr * p->g_m + i < p->M; ++i)
          for (int j = 0; j < p->g_n && q * p->g_n + j < p->N; ++j)
            w_out[(int64_t(pr * p->g_m + i) * p->N + (q * p->g_n + j)) * p->Ks + p->pos_idx[e]] =
                tile_value(p, e, i, j);
  return RT3D_OK;
}

namespace {
rt3d_status unpack_device_layout(const rt3d_packed* p, int n_tile, bool t_groups, float* w_out);
}
rt3d_status rt3d_unpack_device_layout(const rt3d_packed* p, int n_tile, float* w_out) {
  return unpack_device_layout(p, n_tile, false, w_out);
}
rt3d_status rt3d_unpack_device_layout_tgroups(const rt3d_packed* p, int n_tile, float* w_out) {
  return unpack_device_layout(p, n_tile, true, w_out);
}
namespace {
rt3d_status unpack_device_layout(const rt3d_packed* p, int n_tile, bool t_groups, float* w_out) {
  if (!p || !w_out) return RT3D_ERR_INVALID_ARG;
  const UmmaLayout* L = get_umma_layout(const_cast<rt3d_packed*>(p), n_tile, t_groups);
  if (!L) return RT3D_ERR_UNSUPPORTED;
  if (t_groups) {
    // groups tile each bundle's list exactly; inside a group only kt changes, upwards
    if (int(L->grp_ptr.size()) != L->n_bundles + 1 || L->grp_first.size() != size_t(L->grp_ptr.back()) + 1 ||
        L->grp_first.back() != int32_t(L->steps.size()))
      return RT3D_ERR_INVALID_ARG;
    for (int b = 0; b < L->n_bundles; ++b) {
      if (L->grp_ptr[b] > L->grp_ptr[b + 1]) return RT3D_ERR_INVALID_ARG;
      const int32_t first = L->grp_ptr[b] < L->grp_ptr[b + 1] ? L->grp_first[L->grp_ptr[b]] : L->step_ptr[b];
      if (first != L->step_ptr[b]) return RT3D_ERR_INVALID_ARG;
      for (int32_t g = L->grp_ptr[b]; g < L->grp_ptr[b + 1]; ++g) {
        const int32_t s0 = L->grp_first[g], s1 = L->grp_first[g + 1];
        if (s1 <= s0 || s1 - s0 > p->Kt || s1 > L->step_ptr[b + 1]) return RT3D_ERR_INVALID_ARG;
        int kt0, kh0, kw0, ch0;
        decode_step(L->steps[s0], kt0, kh0, kw0, ch0);
        for (int32_t s = s0 + 1; s < s1; ++s) {
          int kt, kh, kw, ch;
          decode_step(L->steps[s], kt, kh, kw, ch);
          if (kh != kh0 || kw != kw0 || ch != ch0 || kt <= kt0) return RT3D_ERR_INVALID_ARG;
          kt0 = kt;
        }
      }
    }
  }
  std::memset(w_out, 0, sizeof(float) * size_t(p->M) * p->N * p->Ks);
  for (int b = 0; b < L->n_bundles; ++b)
    for (int32_t s = L->step_ptr[b]; s < L->step_ptr[b + 1]; ++s) {
      int kt, kh, kw, ch;
      decode_step(L->steps[s], kt, kh, kw, ch);
      const int kpos = (kt * p->Kh + kh) * p->Kw + kw;
      for (int r = 0; r < L->n_tile && b * L->n_tile + r < p->M; ++r)
        for (int j = 0; j < kChunk && ch * kChunk + j < p->N; ++j)
          w_out[(int64_t(b * L->n_tile + r) * p->N + (ch * kChunk + j)) * p->Ks + kpos] =
              bf16_bits_to_f32(L->wtiles[(size_t(s) * L->n_tile + r) * kChunk + j]);
    }
  return RT3D_OK;
}
}  // namespace

rt3d_status rt3d_unpack_sub_layout(const rt3d_packed* p, int n_tile, float* w_out) {
  if (!p || !w_out) return RT3D_ERR_INVALID_ARG;
  const SubLayout* L = get_sub_layout(const_cast<rt3d_packed*>(p), n_tile);
  if (!L) return RT3D_ERR_UNSUPPORTED;
  std::memset(w_out, 0, sizeof(float) * size_t(p->M) * p->N * p->Ks);
  for (int b = 0; b < L->n_bundles; ++b) {
    const int n_ranges = ceil_div(std::min(L->n_tile, p->M - b * L->n_tile), kSubRange);
    for (int32_t s = L->step_ptr[b]; s < L->step_ptr[b + 1]; ++s) {
      const SubStep& st = L->steps[s];
      int kt, kh, kw, ch;
      decode_step(st.enc, kt, kh, kw, ch);
      const int kpos = (kt * p->Kh + kh) * p->Kw + kw;
      const unsigned char* hdr = L->payload.data() + size_t(st.off64) * 64;
      int seen = 0;
      for (int r = 0; r < 16; ++r)
        for (int ks = 0; ks < 4; ++ks) {
          const unsigned char cmd = hdr[4 * r + ks];
          // the first step of a bundle must start every range's accumulator in K slice 0
          if (s == L->step_ptr[b] && ks == 0 && r < n_ranges && !(cmd & 0x80)) return RT3D_ERR_INVALID_ARG;
          if (!(cmd & 0x80)) continue;
          if (r >= n_ranges || (cmd & 0x3F) >= st.nblk) return RT3D_ERR_INVALID_ARG;
          ++seen;
          const uint16_t* blk = reinterpret_cast<const uint16_t*>(hdr + kSubHeaderBytes + size_t(cmd & 0x3F) * kSubBlockBytes);
          for (int i = 0; i < 16; ++i)
            for (int j = 0; j < 16; ++j) {
              const int m = b * L->n_tile + r * 16 + i, c = ch * kChunk + ks * 16 + j;
              const float v = bf16_bits_to_f32(blk[((i / 8) * 2 + j / 8) * 64 + (i % 8) * 8 + j % 8]);
              if (m < p->M && c < p->N) w_out[(int64_t(m) * p->N + c) * p->Ks + kpos] += v;
              else if (v != 0.f) return RT3D_ERR_INVALID_ARG;
            }
        }
      if (seen != st.nblk) return RT3D_ERR_INVALID_ARG;
    }
  }
  return RT3D_OK;
}

}  // extern "C"
