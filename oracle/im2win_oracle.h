/*
 * CPU oracle for the im2win transformation and the im2win-based convolution.
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, slow, host-only restatement of the
 * paper's definitions (Eq. 1, Algorithm 1, Algorithm 2, and the im2col
 * formulation of Section II-B).  It shares no code with the CUDA library and
 * must never be linked into, imported by or called from the product path; only
 * the tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * All pointers are HOST pointers.  Tensors are dense, row-major ("stored as a
 * 1D array", Section I): input I[N][C][H][W], filter F[K][C][Fh][Fw], output
 * O[N][K][Ho][Wo], im2win tensor Ihat[N][C][Ho][W*Fh].  Inputs are fp32 (the
 * paper's storage type, Section IV-A); convolution results are returned in
 * double so that the oracle's own rounding is negligible next to the
 * reduced-precision modes it judges.
 *
 * Notation follows the paper: N=Ni, C=Ci, H=Hi, W=Wi, K=Co, Fh=Hf, Fw=Wf, s.
 *
 * Pins (see tests/test_oracle_*.py): the 4x4 / 2x2 worked example's element
 * counts (16 / 36 / 24), the twelve output sizes of Table I, the 2.93x mean
 * size ratio of Section IV-C, the closed-form sizes of Section III-A, the
 * row-overlap property of Section III-A, agreement of the three conv routes,
 * textbook special cases, and an independent library convolution.
 * No function here is "parity unpinned".
 */
#ifndef IM2WIN_ORACLE_H
#define IM2WIN_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
  int32_t N, C, H, W;  /* input  I[N][C][H][W]            */
  int32_t K, Fh, Fw;   /* filter F[K][C][Fh][Fw]          */
  int32_t s;           /* one stride for both directions  */
} oracle_shape;

/* Ho = floor((H-Fh)/s)+1 (Algorithm 1, first line; floor pinned by Table I Conv4),
 * Wo likewise.  Returns 0, or -1 on a null pointer / non-positive size / Fh>H / Fw>W. */
int oracle_out_dims(const oracle_shape* sh, int32_t* Ho, int32_t* Wo);

/* Element counts of Section III-A: im2win N*C*Ho*Fh*W, im2col (all images)
 * N*C*Fh*Fw*Ho*Wo, input N*C*H*W, output N*K*Ho*Wo. */
int oracle_counts(const oracle_shape* sh, int64_t* n_input, int64_t* n_im2win,
                  int64_t* n_im2col, int64_t* n_output);

/* Algorithm 1: Ihat[i][r][m][k*Fh+u] = I[i][r][m*s+u][k].  out holds N*C*Ho*Fh*W floats.
 * Returns the number of elements written, or -1. */
int64_t oracle_im2win(const float* in, const oracle_shape* sh, float* out);

/* Eq. (1), the seven-loop direct convolution on the untransformed input. */
int oracle_conv_direct(const float* in, const float* f, const oracle_shape* sh, double* out);

/* Algorithm 2: the seven loops over the im2win tensor. */
int oracle_conv_via_im2win(const float* im2win, const float* f, const oracle_shape* sh, double* out);

/* Section II-B: per image, materialise the im2col matrix M and the filter matrix,
 * multiply, transpose back.  Returns the element count of ONE image's M, or -1.
 * Meant for tiny inputs only (M is C*Fh*Fw*Ho*Wo doubles). */
int64_t oracle_conv_via_im2col(const float* in, const float* f, const oracle_shape* sh, double* out);

/* Eq. (1) evaluated only at the listed output coordinates; idx holds npoints
 * quadruples (i, j, m, n); out holds npoints doubles. */
int oracle_conv_direct_points(const float* in, const float* f, const oracle_shape* sh,
                              const int32_t* idx, int64_t npoints, double* out);

/* Threads the parallel loops will use (1 when built without OpenMP). */
int oracle_num_threads(void);

#ifdef __cplusplus
}
#endif
#endif
