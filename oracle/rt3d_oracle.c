/*
 * CPU oracle for the RT3D conv3d hot path.  TEST INFRASTRUCTURE ONLY: nothing in the
 * product (the CUDA library, its Python binding) may include, link or call this file.
 * It shares no code, header, table or helper with the CUDA path.
 *
 * What it computes.  The KGS / vanilla sparsity schemes (Section 3 of the paper) only
 * remove multiplications by weights that are structurally zero; the sparse execution
 * reaches exactly (up to rounding order) the result of an ordinary 3-D convolution with
 * the masked weights W (.) mask.  So the oracle is that definition written out:
 *
 *   y[n,to,ho,wo,m] = act( b[m] + sum_{c,kt,kh,kw} xhat[n, to*st+kt-pt, ho*sh+kh-ph,
 *                                                     wo*sw+kw-pw, c] * Wm[m,c,kt,kh,kw] )
 *
 * xhat = x inside the tensor and 0 outside (zero padding), no kernel flip
 * (cross-correlation), no dilation, output extent floor((in + 2*pad - K)/stride) + 1.
 * Weight tensor axes follow Section 3: M filters x N input channels x kernel
 * (Kt = the paper's depth K_d, then K_h, K_w).  Accumulation is double precision in the
 * fixed order (c, kt, kh, kw); bias is added in double; the result is cast to float.
 *
 * Pins (tests/test_oracle_pins.py): oracle_conv3d is checked against the structurally
 * different scatter-form oracle_conv3d_scatter on exhaustive tiny shapes, an impulse
 * response, an integer closed form (x = W = 1), the T = 1 reduction to oracle_conv2d
 * (Section 1 footnote: 2-D conv is 3-D conv with temporal size 1), a library
 * convolution in float64, and the masking identities.  The paper prints no numeric
 * input/output example of a convolution, so absolute output values are pinned only by
 * those checks ("parity unpinned by the paper" for absolute values).
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

/* ------------------------------------------------------------------ bf16 helpers ---- */
/* Round-to-nearest-even float -> bfloat16 bit pattern.  NaN stays NaN (quiet). */
uint16_t oracle_bf16_bits(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu) != 0u)
        return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

float oracle_bf16_widen(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

void oracle_bf16_round_array(const float* in, uint16_t* out, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) out[i] = oracle_bf16_bits(in[i]);
}

static float round_through_bf16(float f) { return oracle_bf16_widen(oracle_bf16_bits(f)); }

static int out_extent(int in, int pad, int k, int stride) { return (in + 2 * pad - k) / stride + 1; }

/* ------------------------------------------------------------ conv3d, gather form ---- */
/*
 * x    : [n][t][h][w][c] float, dense (channel pitch = c)
 * w    : [M][N][Kt][Kh][Kw] float;  mask same shape (uint8, nonzero = keep) or NULL
 * bias : [M] or NULL
 * y    : [n][To][Ho][Wo][M] float
 * round_bf16 != 0: x and (W (.) mask) are first rounded to bfloat16 and widened back
 *                  (the storage precision of the bf16 path); sums stay double.
 * Returns 0, or -1 on a bad argument.
 */
int oracle_conv3d(const float* x, int n, int t, int h, int w_, int c,
                  const float* w, const uint8_t* mask, const float* bias,
                  int M, int Kt, int Kh, int Kw,
                  int st, int sh, int sw, int pt, int ph, int pw,
                  int relu, int round_bf16, float* y)
{
    if (!x || !w || !y || n < 0 || c <= 0 || M <= 0 || st <= 0 || sh <= 0 || sw <= 0) return -1;
    const int N = c;
    const int To = out_extent(t, pt, Kt, st), Ho = out_extent(h, ph, Kh, sh), Wo = out_extent(w_, pw, Kw, sw);
    if (To <= 0 || Ho <= 0 || Wo <= 0) return -1;
    const int64_t Ks = (int64_t)Kt * Kh * Kw;

    /* masked weights, transposed once to [c][kt][kh][kw][m] so the m loop is contiguous;
       the per-output summation order is still (c, kt, kh, kw). */
    double* wt = (double*)malloc(sizeof(double) * (size_t)(N * Ks * M));
    if (!wt) return -1;
    for (int m = 0; m < M; ++m)
        for (int cc = 0; cc < N; ++cc)
            for (int64_t k = 0; k < Ks; ++k) {
                int64_t src = ((int64_t)m * N + cc) * Ks + k;
                float v = (mask && !mask[src]) ? 0.0f : w[src];
                if (round_bf16) v = round_through_bf16(v);
                wt[((int64_t)cc * Ks + k) * M + m] = (double)v;
            }

    const int64_t nrows = (int64_t)n * To * Ho;
#pragma omp parallel
    {
        double* acc = (double*)malloc(sizeof(double) * (size_t)M);
#pragma omp for schedule(dynamic, 4)
        for (int64_t row = 0; row < nrows; ++row) {
            const int ho = (int)(row % Ho);
            const int to = (int)((row / Ho) % To);
            const int nn = (int)(row / ((int64_t)Ho * To));
            for (int wo = 0; wo < Wo; ++wo) {
                for (int m = 0; m < M; ++m) acc[m] = 0.0;
                for (int cc = 0; cc < N; ++cc)
                    for (int kt = 0; kt < Kt; ++kt) {
                        const int ti = to * st + kt - pt;
                        if (ti < 0 || ti >= t) continue;
                        for (int kh = 0; kh < Kh; ++kh) {
                            const int hi = ho * sh + kh - ph;
                            if (hi < 0 || hi >= h) continue;
                            for (int kw = 0; kw < Kw; ++kw) {
                                const int wi = wo * sw + kw - pw;
                                if (wi < 0 || wi >= w_) continue;
                                float xv = x[((((int64_t)nn * t + ti) * h + hi) * w_ + wi) * c + cc];
                                if (round_bf16) xv = round_through_bf16(xv);
                                const double xd = (double)xv;
                                const double* wrow = wt + ((int64_t)cc * Ks + ((int64_t)kt * Kh + kh) * Kw + kw) * M;
                                for (int m = 0; m < M; ++m) acc[m] += xd * wrow[m];
                            }
                        }
                    }
                float* yo = y + ((((int64_t)nn * To + to) * Ho + ho) * Wo + wo) * M;
                for (int m = 0; m < M; ++m) {
                    double v = acc[m] + (bias ? (double)bias[m] : 0.0);
                    if (relu && v < 0.0) v = 0.0;
                    yo[m] = (float)v;
                }
            }
        }
        free(acc);
    }
    free(wt);
    return 0;
}

/* ----------------------------------------------------------- conv3d, scatter form ---- */
/*
 * Brute force with separate index arithmetic: walk every input voxel and every weight,
 * and add the product into the output it lands on ((i + pad - k) must be a
 * non-negative multiple of the stride).  Double accumulators for the whole output.
 * Single-threaded; meant for tiny shapes only.
 */
int oracle_conv3d_scatter(const float* x, int n, int t, int h, int w_, int c,
                          const float* w, const uint8_t* mask, const float* bias,
                          int M, int Kt, int Kh, int Kw,
                          int st, int sh, int sw, int pt, int ph, int pw,
                          int relu, float* y)
{
    const int To = out_extent(t, pt, Kt, st), Ho = out_extent(h, ph, Kh, sh), Wo = out_extent(w_, pw, Kw, sw);
    if (To <= 0 || Ho <= 0 || Wo <= 0) return -1;
    const int64_t total = (int64_t)n * To * Ho * Wo * M;
    double* acc = (double*)calloc((size_t)total, sizeof(double));
    if (!acc) return -1;
    for (int nn = 0; nn < n; ++nn)
      for (int ti = 0; ti < t; ++ti)
        for (int hi = 0; hi < h; ++hi)
          for (int wi = 0; wi < w_; ++wi)
            for (int cc = 0; cc < c; ++cc) {
                const double xv = (double)x[((((int64_t)nn * t + ti) * h + hi) * w_ + wi) * c + cc];
                for (int m = 0; m < M; ++m)
                  for (int kt = 0; kt < Kt; ++kt) {
                    const int a = ti + pt - kt;
                    if (a < 0 || a % st) continue;
                    const int to = a / st;
                    if (to >= To) continue;
                    for (int kh = 0; kh < Kh; ++kh) {
                      const int b = hi + ph - kh;
                      if (b < 0 || b % sh) continue;
                      const int ho = b / sh;
                      if (ho >= Ho) continue;
                      for (int kw = 0; kw < Kw; ++kw) {
                        const int d = wi + pw - kw;
                        if (d < 0 || d % sw) continue;
                        const int wo = d / sw;
                        if (wo >= Wo) continue;
                        const int64_t wi_idx = ((((int64_t)m * c + cc) * Kt + kt) * Kh + kh) * Kw + kw;
                        if (mask && !mask[wi_idx]) continue;
                        acc[((((int64_t)nn * To + to) * Ho + ho) * Wo + wo) * M + m] += xv * (double)w[wi_idx];
                      }
                    }
                  }
            }
    for (int64_t i = 0; i < total; ++i) {
        double v = acc[i] + (bias ? (double)bias[i % M] : 0.0);
        if (relu && v < 0.0) v = 0.0;
        y[i] = (float)v;
    }
    free(acc);
    return 0;
}

/* ------------------------------------------------------------------------ conv2d ---- */
/* Independent 2-D convolution, NHWC activations, weights [M][N][Kh][Kw]; used to pin the
   T = 1 special case of the 3-D routine. */
int oracle_conv2d(const float* x, int n, int h, int w_, int c,
                  const float* w, const float* bias, int M, int Kh, int Kw,
                  int sh, int sw, int ph, int pw, int relu, float* y)
{
    const int Ho = out_extent(h, ph, Kh, sh), Wo = out_extent(w_, pw, Kw, sw);
    if (Ho <= 0 || Wo <= 0) return -1;
    for (int nn = 0; nn < n; ++nn)
      for (int ho = 0; ho < Ho; ++ho)
        for (int wo = 0; wo < Wo; ++wo)
          for (int m = 0; m < M; ++m) {
              double s = bias ? (double)bias[m] : 0.0;
              for (int kh = 0; kh < Kh; ++kh)
                for (int kw = 0; kw < Kw; ++kw) {
                    const int hi = ho * sh - ph + kh, wi = wo * sw - pw + kw;
                    if (hi < 0 || wi < 0 || hi >= h || wi >= w_) continue;
                    for (int cc = 0; cc < c; ++cc)
                        s += (double)x[(((int64_t)nn * h + hi) * w_ + wi) * c + cc] *
                             (double)w[(((int64_t)m * c + cc) * Kh + kh) * Kw + kw];
                }
              if (relu && s < 0.0) s = 0.0;
              y[(((int64_t)nn * Ho + ho) * Wo + wo) * M + m] = (float)s;
          }
    return 0;
}

/* ---------------------------------------------------------------------- KGS pack ---- */
/*
 * Canonical packed form of a KGS-pruned weight tensor (Section 3: within a kernel group
 * of g_m x g_n kernels the same kernel locations are pruned; in the group's weight
 * matrix this is whole-column removal).  Groups are aligned and non-overlapping,
 * P = ceil(M/g_m), Q = ceil(N/g_n) (Section 4); group id = p*Q + q.
 *
 *   group_ptr[P*Q+1]      CSR offsets over kept (group, location) entries
 *   pos_idx[nnz]          kernel location kpos = (kt*Kh + kh)*Kw + kw, ascending in a group
 *   tiles[nnz][g_m][g_n]  tiles[e][i][j] = W[p*g_m+i][q*g_n+j][kpos], 0 where the kernel
 *                         does not exist (ragged last groups); float, or bf16 bits (RNE)
 *
 * The mask is authoritative: a kept location is stored even if its weights are zero.
 * Two-call protocol: with group_ptr == NULL only *nnz_out is written.
 * Returns 0; 1 if the mask differs inside some (group, location) (not a KGS mask);
 * -1 on a bad argument.  *is_vanilla_out = every group keeps all or none.
 */
int oracle_pack_kgs(const float* w, const uint8_t* mask, int M, int N, int Kt, int Kh, int Kw,
                    int g_m, int g_n, int to_bf16,
                    int32_t* group_ptr, uint16_t* pos_idx, void* tiles,
                    int64_t* nnz_out, int* is_vanilla_out)
{
    if (!w || M <= 0 || N <= 0 || g_m <= 0 || g_n <= 0 || Kt <= 0 || Kh <= 0 || Kw <= 0) return -1;
    const int P = (M + g_m - 1) / g_m, Q = (N + g_n - 1) / g_n;
    const int Ks = Kt * Kh * Kw;
    int64_t e = 0;
    int vanilla = 1;
    for (int p = 0; p < P; ++p)
      for (int q = 0; q < Q; ++q) {
          if (group_ptr) group_ptr[p * Q + q] = (int32_t)e;
          int kept_here = 0;
          for (int k = 0; k < Ks; ++k) {
              int first = -1;
              for (int i = 0; i < g_m; ++i)
                for (int j = 0; j < g_n; ++j) {
                    const int m = p * g_m + i, cc = q * g_n + j;
                    if (m >= M || cc >= N) continue;
                    const int bit = mask ? (mask[((int64_t)m * N + cc) * Ks + k] != 0) : 1;
                    if (first < 0) first = bit;
                    else if (bit != first) return 1;
                }
              if (first <= 0) continue;
              ++kept_here;
              if (group_ptr) {
                  pos_idx[e] = (uint16_t)k;
                  for (int i = 0; i < g_m; ++i)
                    for (int j = 0; j < g_n; ++j) {
                        const int m = p * g_m + i, cc = q * g_n + j;
                        const float v = (m < M && cc < N) ? w[((int64_t)m * N + cc) * Ks + k] : 0.0f;
                        const int64_t o = (e * g_m + i) * g_n + j;
                        if (to_bf16) ((uint16_t*)tiles)[o] = oracle_bf16_bits(v);
                        else ((float*)tiles)[o] = v;
                    }
              }
              ++e;
          }
          if (kept_here != 0 && kept_here != Ks) vanilla = 0;
      }
    if (group_ptr) group_ptr[P * Q] = (int32_t)e;
    if (nnz_out) *nnz_out = e;
    if (is_vanilla_out) *is_vanilla_out = vanilla;
    return 0;
}

/* Inverse of the pack: dense [M][N][Kt][Kh][Kw] float with zeros at pruned locations. */
int oracle_unpack_kgs(const int32_t* group_ptr, const uint16_t* pos_idx, const void* tiles,
                      int M, int N, int Kt, int Kh, int Kw, int g_m, int g_n, int is_bf16, float* w_out)
{
    const int P = (M + g_m - 1) / g_m, Q = (N + g_n - 1) / g_n;
    const int Ks = Kt * Kh * Kw;
    memset(w_out, 0, sizeof(float) * (size_t)M * N * Ks);
    for (int p = 0; p < P; ++p)
      for (int q = 0; q < Q; ++q)
        for (int32_t e = group_ptr[p * Q + q]; e < group_ptr[p * Q + q + 1]; ++e)
          for (int i = 0; i < g_m; ++i)
            for (int j = 0; j < g_n; ++j) {
                const int m = p * g_m + i, cc = q * g_n + j;
                if (m >= M || cc >= N) continue;
                const int64_t o = ((int64_t)e * g_m + i) * g_n + j;
                w_out[((int64_t)m * N + cc) * Ks + pos_idx[e]] =
                    is_bf16 ? oracle_bf16_widen(((const uint16_t*)tiles)[o]) : ((const float*)tiles)[o];
            }
    return 0;
}

/* ------------------------------------------------------------- pooling, add+relu ---- */
/* Max-pool over NDHWC; padding positions are ignored (they never win the max).
   A window with no valid input (cannot happen for pad < kernel) would give -inf. */
int oracle_maxpool3d(const float* x, int n, int t, int h, int w_, int c,
                     int kt, int kh, int kw, int st, int sh, int sw, int pt, int ph, int pw, float* y)
{
    const int To = out_extent(t, pt, kt, st), Ho = out_extent(h, ph, kh, sh), Wo = out_extent(w_, pw, kw, sw);
    if (To <= 0 || Ho <= 0 || Wo <= 0) return -1;
    for (int nn = 0; nn < n; ++nn)
      for (int to = 0; to < To; ++to)
        for (int ho = 0; ho < Ho; ++ho)
          for (int wo = 0; wo < Wo; ++wo)
            for (int cc = 0; cc < c; ++cc) {
                float best = -INFINITY;
                for (int a = 0; a < kt; ++a)
                  for (int b = 0; b < kh; ++b)
                    for (int d = 0; d < kw; ++d) {
                        const int ti = to * st - pt + a, hi = ho * sh - ph + b, wi = wo * sw - pw + d;
                        if (ti < 0 || hi < 0 || wi < 0 || ti >= t || hi >= h || wi >= w_) continue;
                        const float v = x[((((int64_t)nn * t + ti) * h + hi) * w_ + wi) * c + cc];
                        if (v > best) best = v;
                    }
                y[((((int64_t)nn * To + to) * Ho + ho) * Wo + wo) * c + cc] = best;
            }
    return 0;
}

/* y = a + b, optionally clamped at zero (residual join of the R(2+1)D-shaped network). */
int oracle_add_relu(const float* a, const float* b, int64_t count, int relu, float* y)
{
    for (int64_t i = 0; i < count; ++i) {
        double v = (double)a[i] + (double)b[i];
        if (relu && v < 0.0) v = 0.0;
        y[i] = (float)v;
    }
    return 0;
}

/* -------------------------------------------- group norms, reweighting, mask (pruning step) ---- */
/*
 * Group-lasso norm of every (kernel group, kernel location), Section 4 (Fig. 2 caption, Eq. 2):
 *   norms[p][q][k] = ( sum over kernels (i,j) of group (p,q) of |W[i][j][k]|^g )^(1/g),  g = 1 or 2.
 * The printed caption drops the (i,j) subscript inside the sum; it is read as the sum over the
 * kernels of the group.  Kernels that do not exist (ragged last groups) contribute nothing.
 * Double accumulation, result cast to float.
 */
int oracle_group_norms(const float* w, int M, int N, int Ks, int g_m, int g_n, int g, float* norms)
{
    if (!w || !norms || (g != 1 && g != 2) || M <= 0 || N <= 0 || Ks <= 0 || g_m <= 0 || g_n <= 0) return -1;
    const int P = (M + g_m - 1) / g_m, Q = (N + g_n - 1) / g_n;
    for (int p = 0; p < P; ++p)
      for (int q = 0; q < Q; ++q)
        for (int k = 0; k < Ks; ++k) {
            double s = 0.0;
            for (int i = 0; i < g_m; ++i)
              for (int j = 0; j < g_n; ++j) {
                  const int m = p * g_m + i, c = q * g_n + j;
                  if (m >= M || c >= N) continue;
                  const double v = fabs((double)w[((int64_t)m * N + c) * Ks + k]);
                  s += (g == 1) ? v : v * v;
              }
            norms[((int64_t)p * Q + q) * Ks + k] = (float)((g == 1) ? s : sqrt(s));
        }
    return 0;
}

/*
 * One reweighting step (the update rule below Eq. 3): penalty = 1 / (norm^2 + eps); and the hard
 * pruning decision that follows the last round ("prune the weights that converge to zero"):
 * keep = norm > threshold.  The comparison is made on the float norm.
 */
int oracle_reweight(const float* norms, int64_t count, float eps, float threshold, float* penalty, uint8_t* keep)
{
    for (int64_t i = 0; i < count; ++i) {
        const double n = (double)norms[i];
        if (penalty) penalty[i] = (float)(1.0 / (n * n + (double)eps));
        if (keep) keep[i] = norms[i] > threshold ? 1 : 0;
    }
    return 0;
}
