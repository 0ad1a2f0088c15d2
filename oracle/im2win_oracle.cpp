// CPU oracle for im2win (transformation + convolution).  TEST INFRASTRUCTURE ONLY:
// see im2win_oracle.h.  Every routine is the paper's definition written out as
// loops in the paper's order and notation, with no blocking, fusion or
// vectorisation.  The only parallelism is an OpenMP "parallel for" on an outer
// loop whose iterations are independent (Algorithm 1 marks the image loop
// parallel; Section III-B observes that all output elements are independent).

#include "im2win_oracle.h"

#include <cstddef>
#include <cstdint>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

bool shape_ok(const oracle_shape* sh) {
  if (!sh) return false;
  if (sh->N < 1 || sh->C < 1 || sh->H < 1 || sh->W < 1) return false;
  if (sh->K < 1 || sh->Fh < 1 || sh->Fw < 1 || sh->s < 1) return false;
  if (sh->Fh > sh->H || sh->Fw > sh->W) return false;
  return true;
}

// Algorithm 1, first line, with integer (floor) division.  Table I's Conv4
// (224, 7x7, stride 2 -> 109) fixes the division as floor.  The paper never
// writes Wo; it is the same expression in the width.
inline int64_t out_h(const oracle_shape* sh) { return (sh->H - sh->Fh) / sh->s + 1; }
inline int64_t out_w(const oracle_shape* sh) { return (sh->W - sh->Fw) / sh->s + 1; }

}  // namespace

extern "C" {

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

int oracle_out_dims(const oracle_shape* sh, int32_t* Ho, int32_t* Wo) {
  if (!shape_ok(sh) || !Ho || !Wo) return -1;
  *Ho = (int32_t)out_h(sh);
  *Wo = (int32_t)out_w(sh);
  return 0;
}

// Section III-A: the im2win tensor has Ni*Ci*Hf*Wi*((Hi-Hf)/s+1) elements and the
// im2col matrix Ci*Hf*Wf*((Hi-Hf)/s+1)*((Wi-Wf)/s+1) per image.
int oracle_counts(const oracle_shape* sh, int64_t* n_input, int64_t* n_im2win,
                  int64_t* n_im2col, int64_t* n_output) {
  if (!shape_ok(sh)) return -1;
  const int64_t N = sh->N, C = sh->C, H = sh->H, W = sh->W, K = sh->K, Fh = sh->Fh, Fw = sh->Fw;
  const int64_t Ho = out_h(sh), Wo = out_w(sh);
  if (n_input) *n_input = N * C * H * W;
  if (n_im2win) *n_im2win = N * C * Fh * W * Ho;
  if (n_im2col) *n_im2col = N * (C * Fh * Fw * Ho * Wo);
  if (n_output) *n_output = N * K * Ho * Wo;
  return 0;
}

// Algorithm 1.  Loop order i, r, m, k, u exactly as printed; the assignment is
//   Ihat[i][r][m][k*Hf + u] = I[i][r][m*s + u][k],   k = 0..Wi-1.
// The tensor is laid out (Ni, Ci, Ho, Wi*Hf) (Section III-A and the first line
// of Algorithm 2), Hf fastest inside a strip.
int64_t oracle_im2win(const float* in, const oracle_shape* sh, float* out) {
  if (!shape_ok(sh) || !in || !out) return -1;
  const int64_t N = sh->N, C = sh->C, H = sh->H, W = sh->W, Fh = sh->Fh, s = sh->s;
  const int64_t Ho = out_h(sh);
  const int64_t L = W * Fh;  // one strip
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < N; ++i)
    for (int64_t r = 0; r < C; ++r)
      for (int64_t m = 0; m < Ho; ++m)
        for (int64_t k = 0; k < W; ++k)
          for (int64_t u = 0; u < Fh; ++u)
            out[((i * C + r) * Ho + m) * L + (k * Fh + u)] =
                in[((i * C + r) * H + (m * s + u)) * W + k];
  return N * C * Ho * L;
}

// Eq. (1):  O(i,j,m,n) = sum_{r,u,v} I(i, r, m*s+u, n*s+v) * F(j, r, u, v).
// (The printed equation reuses j,m,n as summation indices and writes m*s+v for
// the column; the index ranges listed under it, and Algorithms 1 and 2 composed,
// give the form above.)  fp32 x fp32 is exact in double; only the sum rounds.
int oracle_conv_direct(const float* in, const float* f, const oracle_shape* sh, double* out) {
  if (!shape_ok(sh) || !in || !f || !out) return -1;
  const int64_t N = sh->N, C = sh->C, H = sh->H, W = sh->W, K = sh->K, Fh = sh->Fh, Fw = sh->Fw,
                s = sh->s;
  const int64_t Ho = out_h(sh), Wo = out_w(sh);
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t i = 0; i < N; ++i)
    for (int64_t j = 0; j < K; ++j)
      for (int64_t m = 0; m < Ho; ++m)
        for (int64_t n = 0; n < Wo; ++n) {
          double acc = 0.0;
          for (int64_t r = 0; r < C; ++r)
            for (int64_t u = 0; u < Fh; ++u)
              for (int64_t v = 0; v < Fw; ++v)
                acc += (double)in[((i * C + r) * H + (m * s + u)) * W + (n * s + v)] *
                       (double)f[((j * C + r) * Fh + u) * Fw + v];
          out[((i * K + j) * Ho + m) * Wo + n] = acc;
        }
  return 0;
}

// Algorithm 2: seven loops i, j, m, n, r, u, v over the im2win tensor,
//   O[i][j][m][n] += Ihat[i][r][m][(n*s + v)*Hf + u] * F[j][r][u][v].
// The printed strip offset is n*s*Wf + v*Hf + u.  Algorithm 1 stores column k of
// the window row at offset k*Hf, so the window that starts at column n*s starts
// at offset n*s*Hf; the two agree when Hf == Wf (every layer the paper runs)
// and the form used here is the one consistent with Algorithm 1 for Hf != Wf.
int oracle_conv_via_im2win(const float* im2win, const float* f, const oracle_shape* sh,
                           double* out) {
  if (!shape_ok(sh) || !im2win || !f || !out) return -1;
  const int64_t N = sh->N, C = sh->C, W = sh->W, K = sh->K, Fh = sh->Fh, Fw = sh->Fw, s = sh->s;
  const int64_t Ho = out_h(sh), Wo = out_w(sh);
  const int64_t L = W * Fh;
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t i = 0; i < N; ++i)
    for (int64_t j = 0; j < K; ++j)
      for (int64_t m = 0; m < Ho; ++m)
        for (int64_t n = 0; n < Wo; ++n) {
          double acc = 0.0;
          for (int64_t r = 0; r < C; ++r)
            for (int64_t u = 0; u < Fh; ++u)
              for (int64_t v = 0; v < Fw; ++v)
                acc += (double)im2win[((i * C + r) * Ho + m) * L + ((n * s + v) * Fh + u)] *
                       (double)f[((j * C + r) * Fh + u) * Fw + v];
          out[((i * K + j) * Ho + m) * Wo + n] = acc;
        }
  return 0;
}

// Section II-B, one image at a time:
//   M(m*Wo+n, (r*Hf+u)*Wf+v) = I'(r, m*s+u, n*s+v)     (the paper prints the s=1 case)
//   Nmat((r*Hf+u)*Wf+v, j)   = F(j, r, u, v)
//   R' = M x Nmat,   R(j, m, n) = R'(m*Wo+n, j).
// Both matrices are materialised so that M's element count is a fact of the
// construction rather than a formula.
int64_t oracle_conv_via_im2col(const float* in, const float* f, const oracle_shape* sh,
                               double* out) {
  if (!shape_ok(sh) || !in || !f || !out) return -1;
  const int64_t N = sh->N, C = sh->C, H = sh->H, W = sh->W, K = sh->K, Fh = sh->Fh, Fw = sh->Fw,
                s = sh->s;
  const int64_t Ho = out_h(sh), Wo = out_w(sh);
  const int64_t rows = Ho * Wo, cols = C * Fh * Fw;
  std::vector<double> M;
  std::vector<double> Nmat;
  int64_t m_count = 0;
  for (int64_t i = 0; i < N; ++i) {
    const float* img = in + i * C * H * W;
    M.clear();
    M.resize((size_t)(rows * cols));
    for (int64_t m = 0; m < Ho; ++m)
      for (int64_t n = 0; n < Wo; ++n)
        for (int64_t r = 0; r < C; ++r)
          for (int64_t u = 0; u < Fh; ++u)
            for (int64_t v = 0; v < Fw; ++v)
              M[(size_t)((m * Wo + n) * cols + (r * Fh + u) * Fw + v)] =
                  (double)img[(r * H + (m * s + u)) * W + (n * s + v)];
    m_count = (int64_t)M.size();
    Nmat.assign((size_t)(cols * K), 0.0);
    for (int64_t j = 0; j < K; ++j)
      for (int64_t r = 0; r < C; ++r)
        for (int64_t u = 0; u < Fh; ++u)
          for (int64_t v = 0; v < Fw; ++v)
            Nmat[(size_t)(((r * Fh + u) * Fw + v) * K + j)] =
                (double)f[((j * C + r) * Fh + u) * Fw + v];
    for (int64_t p = 0; p < rows; ++p)
      for (int64_t j = 0; j < K; ++j) {
        double acc = 0.0;
        for (int64_t q = 0; q < cols; ++q) acc += M[(size_t)(p * cols + q)] * Nmat[(size_t)(q * K + j)];
        // transpose back: R(j, m, n) = R'(m*Wo+n, j)
        out[(i * K + j) * rows + p] = acc;
      }
  }
  return m_count;
}

int oracle_conv_direct_points(const float* in, const float* f, const oracle_shape* sh,
                              const int32_t* idx, int64_t npoints, double* out) {
  if (!shape_ok(sh) || !in || !f || !idx || !out || npoints < 0) return -1;
  const int64_t N = sh->N, C = sh->C, H = sh->H, W = sh->W, K = sh->K, Fh = sh->Fh, Fw = sh->Fw,
                s = sh->s;
  const int64_t Ho = out_h(sh), Wo = out_w(sh);
  for (int64_t p = 0; p < npoints; ++p) {
    const int64_t i = idx[4 * p], j = idx[4 * p + 1], m = idx[4 * p + 2], n = idx[4 * p + 3];
    if (i < 0 || i >= N || j < 0 || j >= K || m < 0 || m >= Ho || n < 0 || n >= Wo) return -1;
  }
#pragma omp parallel for schedule(static)
  for (int64_t p = 0; p < npoints; ++p) {
    const int64_t i = idx[4 * p], j = idx[4 * p + 1], m = idx[4 * p + 2], n = idx[4 * p + 3];
    double acc = 0.0;
    for (int64_t r = 0; r < C; ++r)
      for (int64_t u = 0; u < Fh; ++u)
        for (int64_t v = 0; v < Fw; ++v)
          acc += (double)in[((i * C + r) * H + (m * s + u)) * W + (n * s + v)] *
                 (double)f[((j * C + r) * Fh + u) * Fw + v];
    out[p] = acc;
  }
  return 0;
}

}  // extern "C"
