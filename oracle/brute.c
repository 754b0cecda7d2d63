/*
 * Brute-force reference for the kernels of Section 5.1 (test infrastructure).
 *
 * A checker, not a product: only the tests, the smoke check and the
 * benchmark's CPU-baseline leg may build or call it.  It shares no code with
 * the CUDA library.  Each routine is the paper's element-wise equation written
 * as nested loops: no tiling, no reordering, no im2col.  Inputs are float32
 * (every bf16 value is exactly a float32), sums are carried in double unless a
 * routine's name ends in _f32acc.  OpenMP only spreads independent outputs
 * over threads.
 *
 * pad is not in the paper (parity unpinned by the paper): it is the plain
 * textbook border of constant cells.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int o2_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* Constant border around the last two dimensions:
 * out[u, h + ph_lo, w + pw_lo] = in[u, h, w], every other cell = fill. */
void o2_pad_hw(const float* in, float* out, int64_t outer, int64_t H, int64_t W,
               int64_t ph_lo, int64_t ph_hi, int64_t pw_lo, int64_t pw_hi, float fill) {
  const int64_t Hp = H + ph_lo + ph_hi, Wp = W + pw_lo + pw_hi;
#pragma omp parallel for schedule(static)
  for (int64_t u = 0; u < outer; ++u) {
    for (int64_t h = 0; h < Hp; ++h)
      for (int64_t w = 0; w < Wp; ++w) out[(u * Hp + h) * Wp + w] = fill;
    for (int64_t h = 0; h < H; ++h)
      for (int64_t w = 0; w < W; ++w)
        out[(u * Hp + h + ph_lo) * Wp + w + pw_lo] = in[(u * H + h) * W + w];
  }
}

/* Section 5.1, 2D convolution:
 *   out[n,o,x,y] = sum_{dx,dy,c} A[n,c,S0*x+dx,S1*y+dy] * W[o,c,dx,dy]
 * A is (N,C,H,W), Wt is (O,C,Kh,Kw), out is (N,O,Ho,Wo) with
 * Ho = (H-Kh)/S0+1, Wo = (W-Kw)/S1+1 (every window lies inside A). */
static double conv_cell(const float* A, const float* Wt, int64_t C, int64_t H, int64_t W,
                        int64_t Kh, int64_t Kw, int64_t S0, int64_t S1,
                        int64_t n, int64_t o, int64_t x, int64_t y) {
  double acc = 0.0;
  for (int64_t dx = 0; dx < Kh; ++dx)
    for (int64_t dy = 0; dy < Kw; ++dy)
      for (int64_t c = 0; c < C; ++c)
        acc += (double)A[((n * C + c) * H + S0 * x + dx) * W + S1 * y + dy] *
               (double)Wt[((o * C + c) * Kh + dx) * Kw + dy];
  return acc;
}

void o2_conv2d(const float* A, const float* Wt, double* out, int64_t N, int64_t C, int64_t H,
               int64_t W, int64_t O, int64_t Kh, int64_t Kw, int64_t S0, int64_t S1) {
  const int64_t Ho = (H - Kh) / S0 + 1, Wo = (W - Kw) / S1 + 1;
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t n = 0; n < N; ++n)
    for (int64_t o = 0; o < O; ++o)
      for (int64_t x = 0; x < Ho; ++x)
        for (int64_t y = 0; y < Wo; ++y)
          out[((n * O + o) * Ho + x) * Wo + y] = conv_cell(A, Wt, C, H, W, Kh, Kw, S0, S1, n, o, x, y);
}

/* The same equation for a list of output cells given as flat (n,o,x,y) offsets. */
void o2_conv2d_sampled(const float* A, const float* Wt, const int64_t* flat, int64_t count,
                       double* vals, int64_t N, int64_t C, int64_t H, int64_t W, int64_t O,
                       int64_t Kh, int64_t Kw, int64_t S0, int64_t S1) {
  const int64_t Ho = (H - Kh) / S0 + 1, Wo = (W - Kw) / S1 + 1;
  (void)N;
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < count; ++i) {
    int64_t f = flat[i];
    const int64_t y = f % Wo; f /= Wo;
    const int64_t x = f % Ho; f /= Ho;
    const int64_t o = f % O;  f /= O;
    vals[i] = conv_cell(A, Wt, C, H, W, Kh, Kw, S0, S1, f, o, x, y);
  }
}

/* Same equation with a float accumulator in the natural loop order; exact
 * whenever every partial sum is an integer below 2^24. */
void o2_conv2d_f32acc(const float* A, const float* Wt, float* out, int64_t N, int64_t C, int64_t H,
                      int64_t W, int64_t O, int64_t Kh, int64_t Kw, int64_t S0, int64_t S1) {
  const int64_t Ho = (H - Kh) / S0 + 1, Wo = (W - Kw) / S1 + 1;
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t n = 0; n < N; ++n)
    for (int64_t o = 0; o < O; ++o)
      for (int64_t x = 0; x < Ho; ++x)
        for (int64_t y = 0; y < Wo; ++y) {
          float acc = 0.0f;
          for (int64_t dx = 0; dx < Kh; ++dx)
            for (int64_t dy = 0; dy < Kw; ++dy)
              for (int64_t c = 0; c < C; ++c)
                acc += A[((n * C + c) * H + S0 * x + dx) * W + S1 * y + dy] *
                       Wt[((o * C + c) * Kh + dx) * Kw + dy];
          out[((n * O + o) * Ho + x) * Wo + y] = acc;
        }
}

/* Section 3.1: R_ij = sum_k P_ik Q_kj, P is (I,K), Q is (K,J). */
void o2_matmul(const float* P, const float* Q, double* R, int64_t I, int64_t K, int64_t J) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < I; ++i)
    for (int64_t j = 0; j < J; ++j) {
      double acc = 0.0;
      for (int64_t k = 0; k < K; ++k) acc += (double)P[i * K + k] * (double)Q[k * J + j];
      R[i * J + j] = acc;
    }
}

/* Section 3.1, second form: R_ij = P_i . (Q^T)_j with both operands stored as
 * row vectors, A is (M,K), B is (O,K).  `rows` (may be NULL = all M rows)
 * lists the rows of A to evaluate; R holds nrows x O values. */
void o2_rowdot(const float* A, const float* B, double* R, int64_t M, int64_t O, int64_t K,
               const int64_t* rows, int64_t nrows) {
  if (!rows) nrows = M;
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < nrows; ++r) {
    const int64_t m = rows ? rows[r] : r;
    for (int64_t o = 0; o < O; ++o) {
      double acc = 0.0;
      for (int64_t k = 0; k < K; ++k) acc += (double)A[m * K + k] * (double)B[o * K + k];
      R[r * O + o] = acc;
    }
  }
}

/* Section 5.1, max pooling:
 *   out[n,c,x,y] = max_{dx,dy} act[n,c,S0*x+dx,S1*y+dy]
 * act is (NC,H,W) with n and c fused, out is (NC,Ho,Wo). */
void o2_maxpool(const float* act, float* out, int64_t NC, int64_t H, int64_t W, int64_t Kh,
                int64_t Kw, int64_t S0, int64_t S1) {
  const int64_t Ho = (H - Kh) / S0 + 1, Wo = (W - Kw) / S1 + 1;
#pragma omp parallel for schedule(static)
  for (int64_t u = 0; u < NC; ++u)
    for (int64_t x = 0; x < Ho; ++x)
      for (int64_t y = 0; y < Wo; ++y) {
        float best = -INFINITY;
        for (int64_t dx = 0; dx < Kh; ++dx)
          for (int64_t dy = 0; dy < Kw; ++dy) {
            const float v = act[(u * H + S0 * x + dx) * W + S1 * y + dy];
            if (v > best) best = v;
          }
        out[(u * Ho + x) * Wo + y] = best;
      }
}

/* Transformer table, `windows` on ((N),(C,H,W)) with window (C,Kh,Kw) and
 * strides (1,S0,S1), then `flatten`: the im2col matrix
 *   out[(n,x,y), (c,dx,dy)] = A[n,c,S0*x+dx,S1*y+dy]. */
void o2_im2col(const float* A, float* out, int64_t N, int64_t C, int64_t H, int64_t W,
               int64_t Kh, int64_t Kw, int64_t S0, int64_t S1) {
  const int64_t Ho = (H - Kh) / S0 + 1, Wo = (W - Kw) / S1 + 1;
  const int64_t Kd = C * Kh * Kw;
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t n = 0; n < N; ++n)
    for (int64_t x = 0; x < Ho; ++x)
      for (int64_t y = 0; y < Wo; ++y)
        for (int64_t c = 0; c < C; ++c)
          for (int64_t dx = 0; dx < Kh; ++dx)
            for (int64_t dy = 0; dy < Kw; ++dy)
              out[((n * Ho + x) * Wo + y) * Kd + (c * Kh + dx) * Kw + dy] =
                  A[((n * C + c) * H + S0 * x + dx) * W + S1 * y + dy];
}

/* Transformer table, `transpose` with (0 2 1) on a (B,R,C) tensor:
 * out[b,c,r] = in[b,r,c]  (NCHW -> NHWC is B=N, R=C, C=H*W). */
void o2_transpose_021(const float* in, float* out, int64_t B, int64_t R, int64_t C) {
#pragma omp parallel for schedule(static)
  for (int64_t b = 0; b < B; ++b)
    for (int64_t r = 0; r < R; ++r)
      for (int64_t c = 0; c < C; ++c) out[(b * C + c) * R + r] = in[(b * R + r) * C + c];
}
