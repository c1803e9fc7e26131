/*
 * CPU oracle for the fused operator  Y = act(X * W^T + b) * s  followed by a
 * row-wise reduction over N.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the CUDA
 * path is compared against.  It shares no code, header, table or constant with
 * the CUDA library and must never be linked into, or called from, the product
 * path: only the tests, the smoke check and the benchmark's CPU-baseline leg
 * execute it.
 *
 * What it follows.  The paper states the task as: given the reference
 * operator's inputs, return the same outputs (Section 3.1, Verifier; Section
 * 3.3), and names the operator categories (Section 1; Section 4.1, Datasets).
 * It gives no formula for any operator, so the formula here is the operator's
 * plain definition (a linear layer, an element-wise activation, a scale, and a
 * reduction over the last dimension), written as three nested loops in fp64:
 *
 *   z[m,n] = sum_{k = 0 .. K-1, ascending} X[m,k] * W[n,k]
 *   y[m,n] = act(z[m,n] + b[n]) * s[n]  ( + R[m,n] when a residual tensor is given: a skip connection
 *            added after the scale; the reductions then run over this y )
 *   mx[m]  = max_n y[m,n]
 *   LSE        : out[m]   = mx + log( sum_n exp(y - mx) )
 *   SOFTMAX    : P[m,n]   = exp(y - mx) / sum_n exp(y - mx)
 *   MAXSUM     : out[m,:] = ( mx , sum_n y )
 *   MAX_SUMEXP : out[m,:] = ( mx , sum_n exp(y - mx) )
 *   MEANVAR    : out[m,:] = ( mu , (1/N) sum_n (y - mu)^2 ),  mu = (1/N) sum_n y
 *                (the row statistics of a normalisation layer: population variance, two passes)
 *
 *   act: NONE a = u;  RELU a = max(u, 0);
 *        GELU_TANH a = 0.5 u (1 + tanh( sqrt(2/pi) (u + 0.044715 u^3) ))
 *        SIGMOID a = 1 / (1 + e^-u);  TANH a = tanh u;  SILU a = u / (1 + e^-u)
 *
 * Inputs are the very bits the GPU gets: fp32 values, or bf16 bit patterns
 * (uint16) that are widened exactly to fp64 here.  Rows are independent; the
 * only parallelism is over rows, so the result does not depend on the thread
 * count.  No blocking, no fusion, no reordering.
 *
 * Pins (tests/test_oracle_pins.py): identity and zero weights (closed forms),
 * one-hot rows, integer-valued inputs (exact), 4x4x4 brute force in rational
 * arithmetic, hand-computed fixtures (tests/golden/), library routines in fp64,
 * GELU symmetry and limits, LSE bounds and shift, softmax row sums, the GEMV
 * closed form of the row sum.  Every function below is pinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORC_F32 = 0, ORC_BF16 = 1 };
enum { ORC_ACT_NONE = 0, ORC_ACT_RELU = 1, ORC_ACT_GELU_TANH = 2, ORC_ACT_SIGMOID = 3, ORC_ACT_TANH = 4, ORC_ACT_SILU = 5 };
enum { ORC_SCALE_NONE = 0, ORC_SCALE_SCALAR = 1, ORC_SCALE_PER_COLUMN = 2 };
enum { ORC_RED_LSE = 0, ORC_RED_SOFTMAX = 1, ORC_RED_MAXSUM = 2, ORC_RED_MAX_SUMEXP = 3, ORC_RED_MEANVAR = 6 };

typedef struct {
  int32_t batch, M, N, K;
  int32_t dtype, act, scale_kind, reduce;
  double scale;           /* used when scale_kind == ORC_SCALE_SCALAR */
  int32_t bias_per_batch; /* 0: bias[N]; 1: bias[batch, N] */
  int32_t reserved;
} fgr_oracle_problem;

/* bf16 is the upper half of an IEEE fp32: widening is exact. */
static double bf16_to_double(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

static double load_elem(const void* p, int dtype, int64_t i) {
  return dtype == ORC_BF16 ? bf16_to_double(((const uint16_t*)p)[i]) : (double)((const float*)p)[i];
}

/* GELU, tanh form: 0.5 u (1 + tanh( sqrt(2/pi) (u + 0.044715 u^3) )). */
double fgr_oracle_gelu_tanh(double u) {
  const double c = sqrt(2.0 / acos(-1.0));
  return 0.5 * u * (1.0 + tanh(c * (u + 0.044715 * u * u * u)));
}

double fgr_oracle_act(int act, double u) {
  switch (act) {
    case ORC_ACT_RELU: return u > 0.0 ? u : 0.0;
    case ORC_ACT_GELU_TANH: return fgr_oracle_gelu_tanh(u);
    case ORC_ACT_SIGMOID: return 1.0 / (1.0 + exp(-u));          /* logistic function */
    case ORC_ACT_TANH: return tanh(u);
    case ORC_ACT_SILU: return u / (1.0 + exp(-u));             /* u * sigmoid(u) */
    default: return u;
  }
}

/* One row: fills y[0..N) and, when red != NULL, the reduction (1 or 2 values);
 * for SOFTMAX y is overwritten by P. */
static void oracle_row(const fgr_oracle_problem* p, const void* X, const void* W, const float* bias,
                       const float* scale_vec, const void* R, int64_t bt, int64_t m, double* y, double* red) {
  const int64_t N = p->N, K = p->K, M = p->M;
  const int64_t xoff = (bt * M + m) * K;
  const int64_t woff = bt * N * K;
  const float* b = bias ? bias + (p->bias_per_batch ? bt * N : 0) : NULL;
  for (int64_t n = 0; n < N; ++n) {
    double z = 0.0;
    for (int64_t k = 0; k < K; ++k)
      z += load_elem(X, p->dtype, xoff + k) * load_elem(W, p->dtype, woff + n * K + k);
    double a = fgr_oracle_act(p->act, z + (b ? (double)b[n] : 0.0));
    double s = 1.0;
    if (p->scale_kind == ORC_SCALE_SCALAR) s = p->scale;
    else if (p->scale_kind == ORC_SCALE_PER_COLUMN) s = (double)scale_vec[n];
    y[n] = a * s;
    if (R) y[n] += load_elem(R, p->dtype, (bt * M + m) * N + n);
  }
  if (p->reduce == ORC_RED_MEANVAR) {
    double sum = 0.0, dev = 0.0;
    for (int64_t n = 0; n < N; ++n) sum += y[n];
    const double mu = sum / (double)N;
    for (int64_t n = 0; n < N; ++n) dev += (y[n] - mu) * (y[n] - mu);
    if (red) { red[0] = mu; red[1] = dev / (double)N; }
    return;
  }
  double mx = y[0];
  for (int64_t n = 1; n < N; ++n) if (y[n] > mx) mx = y[n];
  if (p->reduce == ORC_RED_MAXSUM) {
    double sum = 0.0;
    for (int64_t n = 0; n < N; ++n) sum += y[n];
    if (red) { red[0] = mx; red[1] = sum; }
    return;
  }
  double l = 0.0;
  for (int64_t n = 0; n < N; ++n) l += exp(y[n] - mx);
  if (p->reduce == ORC_RED_LSE) { if (red) red[0] = mx + log(l); }
  else if (p->reduce == ORC_RED_MAX_SUMEXP) { if (red) { red[0] = mx; red[1] = l; } }
  else if (p->reduce == ORC_RED_SOFTMAX) { for (int64_t n = 0; n < N; ++n) y[n] = exp(y[n] - mx) / l; }
}

static int out_width(int reduce) {
  return reduce == ORC_RED_LSE ? 1 : reduce == ORC_RED_SOFTMAX ? 0 : 2;   /* MAXSUM, MAX_SUMEXP, MEANVAR */
}

/*
 * Computes the operator for a list of rows.
 *   rows      : nrows global row indices r = bt * M + m, or NULL for rows 0 .. nrows-1
 *   Y         : [nrows, N] fp64, y (or P for SOFTMAX); may be NULL
 *   out       : [nrows, width] fp64, width = 1 (LSE), 2 (MAXSUM, MAX_SUMEXP), unused for SOFTMAX; may be NULL
 *   nthreads  : threads over rows (<= 0: the OpenMP default)
 * Returns the number of threads used, or a negative value on a bad argument.
 */
static int oracle_rows(const fgr_oracle_problem* p, const void* X, const void* W, const float* bias,
                       const float* scale_vec, const void* R, const int64_t* rows, int64_t nrows, double* Y, double* out,
                       int nthreads) {
  if (!p || !X || !W || nrows < 0) return -1;
  if (p->batch < 1 || p->M < 1 || p->N < 1 || p->K < 1) return -2;
  if (p->dtype != ORC_F32 && p->dtype != ORC_BF16) return -3;
  if (p->act < 0 || p->act > 5 || p->scale_kind < 0 || p->scale_kind > 2 || p->reduce < 0 || (p->reduce > 3 && p->reduce != ORC_RED_MEANVAR)) return -4;
  if (p->scale_kind == ORC_SCALE_PER_COLUMN && !scale_vec) return -5;
  const int64_t total = (int64_t)p->batch * p->M;
  for (int64_t i = 0; i < nrows; ++i) {
    int64_t r = rows ? rows[i] : i;
    if (r < 0 || r >= total) return -6;
  }
  const int w = out_width(p->reduce);
  int used = 1;
#ifdef _OPENMP
  if (nthreads <= 0) nthreads = omp_get_max_threads();
  if ((int64_t)nthreads > nrows) nthreads = nrows > 0 ? (int)nrows : 1;
  used = nthreads;
#pragma omp parallel num_threads(nthreads)
#endif
  {
    double* ybuf = (double*)malloc(sizeof(double) * (size_t)p->N);
#ifdef _OPENMP
#pragma omp for schedule(dynamic, 1)
#endif
    for (int64_t i = 0; i < nrows; ++i) {
      int64_t r = rows ? rows[i] : i;
      double red[2] = {0.0, 0.0};
      double* y = Y ? Y + i * (int64_t)p->N : ybuf;
      oracle_row(p, X, W, bias, scale_vec, R, r / p->M, r % p->M, y, red);
      if (out) for (int j = 0; j < w; ++j) out[i * w + j] = red[j];
    }
    free(ybuf);
  }
  return used;
}

int fgr_oracle_rows(const fgr_oracle_problem* p, const void* X, const void* W, const float* bias,
                    const float* scale_vec, const int64_t* rows, int64_t nrows, double* Y, double* out,
                    int nthreads) {
  return oracle_rows(p, X, W, bias, scale_vec, NULL, rows, nrows, Y, out, nthreads);
}

/* The same with a residual tensor R [batch, M, N] (packed, in the dtype of X and W), added to y after the scale. */
int fgr_oracle_rows_residual(const fgr_oracle_problem* p, const void* X, const void* W, const float* bias,
                             const float* scale_vec, const void* R, const int64_t* rows, int64_t nrows, double* Y,
                             double* out, int nthreads) {
  return oracle_rows(p, X, W, bias, scale_vec, R, rows, nrows, Y, out, nthreads);
}

int fgr_oracle_out_width(int reduce) { return out_width(reduce); }

/*
 * Stand-alone reduction over the last dimension of a given matrix A[M, N] (the operator category
 * "reduction" of Section 4.1, Datasets; the paper's GPU case study is a max reduction over a
 * dimension, Section 4.4.1).  Same four kinds as above, applied to y = A directly, plus
 *   kind 4 (MAX): out[m] = max_n A[m, n]          kind 5 (SUM): out[m] = sum_n A[m, n]
 *   kind 6 (MEANVAR): out[m, :] = (mean, population variance) of row m, as above
 * P (SOFTMAX) and out are fp64; A is fp32 or bf16 bit patterns, row stride lda elements.
 * Returns 0, or a negative value on a bad argument.
 */
int fgr_oracle_reduce_rows(int32_t M, int32_t N, int32_t dtype, int32_t kind, const void* A, int64_t lda,
                           double* P, double* out) {
  if (M < 1 || N < 1 || !A || lda < N) return -1;
  if (dtype != ORC_F32 && dtype != ORC_BF16) return -3;
  if (kind < 0 || kind > 6) return -4;
  for (int64_t m = 0; m < M; ++m) {
    if (kind == ORC_RED_MEANVAR) {
      double s = 0.0, dev = 0.0;
      for (int64_t n = 0; n < N; ++n) s += load_elem(A, dtype, m * lda + n);
      const double mu = s / (double)N;
      for (int64_t n = 0; n < N; ++n) { double v = load_elem(A, dtype, m * lda + n) - mu; dev += v * v; }
      out[2 * m] = mu; out[2 * m + 1] = dev / (double)N;
      continue;
    }
    double mx = load_elem(A, dtype, m * lda);
    for (int64_t n = 1; n < N; ++n) { double v = load_elem(A, dtype, m * lda + n); if (v > mx) mx = v; }
    double sum = 0.0, l = 0.0;
    for (int64_t n = 0; n < N; ++n) { double v = load_elem(A, dtype, m * lda + n); sum += v; l += exp(v - mx); }
    switch (kind) {
      case ORC_RED_LSE: out[m] = mx + log(l); break;
      case ORC_RED_SOFTMAX: for (int64_t n = 0; n < N; ++n) P[m * N + n] = exp(load_elem(A, dtype, m * lda + n) - mx) / l; break;
      case ORC_RED_MAXSUM: out[2 * m] = mx; out[2 * m + 1] = sum; break;
      case ORC_RED_MAX_SUMEXP: out[2 * m] = mx; out[2 * m + 1] = l; break;
      case 4: out[m] = mx; break;
      default: out[m] = sum; break;
    }
  }
  return 0;
}
