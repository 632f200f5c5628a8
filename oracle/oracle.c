/* CPU oracle -- TEST INFRASTRUCTURE ONLY (used by tests/, the smoke check and
 * the timed cpu baseline; never by the product path).
 *
 * Every function restates one operation of the replayed training step in the
 * order the paper's auditable regime fixes (Sec. 2.1 conventions; Sec. 3.1/3.2
 * recipe arithmetic; Sec. 6 + Appendix A reduction order).  OpenMP is used only
 * across independent outputs, never across the terms of one reduction, so the
 * bits do not depend on the thread count.
 */
#include "prim.h"
#include <stdio.h>

#define C127 0x1.6b7612p-4f      /* 1/sqrt(127) rounded to binary32 */
#define ATT_SCALE 0x1.6a09e6p-4f /* 1/sqrt(128) rounded to binary32 */

/* ------------------------------------------------------------------ */
/* primitives exposed for tests                                        */
/* ------------------------------------------------------------------ */
void orc_prim(int op, const float *a, const float *b, float *out, size_t n) {
  for (size_t i = 0; i < n; ++i) {
    float x = a[i], y = b ? b[i] : 0.0f, r;
    switch (op) {
      case 0: r = fadd(x, y); break;
      case 1: r = fsub(x, y); break;
      case 2: r = fmul(x, y); break;
      case 3: r = fdiv(x, y); break;
      case 4: r = fsqrt(x); break;
      case 5: r = det_exp(x); break;
      case 6: r = det_log(x); break;
      case 7: r = fmax2(x, y); break;
      case 8: r = bf2f(f2bf(x)); break;
      case 9: r = fadd(fmul(x, y), y); break; /* unfused a*b+b */
      default: r = 0.0f;
    }
    out[i] = r;
  }
}

float orc_det_sum(const float *x, size_t n) { return det_sum(x, n); }

/* sum of squares in the fixed tree (grad-norm building block) */
float orc_sumsq(const float *x, size_t n) {
  float *t = (float *)malloc((n ? n : 1) * sizeof(float));
#pragma omp parallel for
  for (size_t i = 0; i < n; ++i) t[i] = fmul(x[i], x[i]);
  float r = det_sum(t, n);
  free(t);
  return r;
}

void orc_f2bf(const float *x, bf16_t *y, size_t n) { for (size_t i = 0; i < n; ++i) y[i] = f2bf(x[i]); }

/* ------------------------------------------------------------------ */
/* LSQ int8 linear (Sec. 3.1 "int8 quantization-aware training",       */
/* Sec. 3.2 "int8 computation", Sec. 4.4 step-size re-pin)             */
/* ------------------------------------------------------------------ */

/* step = 2*mean(|w|)/sqrt(q_max), q_max = 127, per output channel (row of W)
 * or over the whole tensor; mean = tree sum times a reciprocal constant. */
void orc_lsq_weight_scale(const bf16_t *W, int N, int K, int per_tensor, float *s_w) {
  if (per_tensor) {
    size_t n = (size_t)N * K;
    float *t = (float *)malloc(n * sizeof(float));
    for (size_t i = 0; i < n; ++i) t[i] = fabs1(bf2f(W[i]));
    float s = fmul(fmul(2.0f, fmul(det_sum(t, n), (float)(1.0 / (double)n))), C127);
    s = fmax2(s, 0x1p-40f);
    for (int r = 0; r < N; ++r) s_w[r] = s;
    free(t);
    return;
  }
#pragma omp parallel for
  for (int r = 0; r < N; ++r) {
    float *t = (float *)malloc((size_t)K * sizeof(float));
    for (int k = 0; k < K; ++k) t[k] = fabs1(bf2f(W[(size_t)r * K + k]));
    float s = fmul(fmul(2.0f, fmul(det_sum(t, K), (float)(1.0 / (double)K))), C127);
    s_w[r] = fmax2(s, 0x1p-40f);
    free(t);
  }
}

void orc_lsq_act_scale_init(const bf16_t *X, size_t n, float *s_x) {
  float *t = (float *)malloc(n * sizeof(float));
  for (size_t i = 0; i < n; ++i) t[i] = fabs1(bf2f(X[i]));
  float s = fmul(fmul(2.0f, fmul(det_sum(t, n), (float)(1.0 / (double)n))), C127);
  *s_x = fmax2(s, 0x1p-40f);
  free(t);
}

/* q = rne(clamp(v * (1/s), -128, 127)) */
static inline int8_t quant1(float v, float inv_s) {
  float t = fmul(v, inv_s);
  t = fmin2(fmax2(t, -128.0f), 127.0f);
  return (int8_t)(int)frne(t);
}

void orc_lsq_quantize(const bf16_t *X, int rows, int cols, const float *s, int per_row, int8_t *q) {
#pragma omp parallel for
  for (int r = 0; r < rows; ++r) {
    float inv = fdiv(1.0f, s[per_row ? r : 0]);
    for (int c = 0; c < cols; ++c) q[(size_t)r * cols + c] = quant1(bf2f(X[(size_t)r * cols + c]), inv);
  }
}

/* C[i,j] = sum_k A[i,k] * B[j,k], exact int32 (order-free) */
static void igemm_tn(const int8_t *A, const int8_t *B, int I, int J, int K, int32_t *C) {
#pragma omp parallel for
  for (int i = 0; i < I; ++i)
    for (int j = 0; j < J; ++j) {
      const int8_t *a = A + (size_t)i * K, *b = B + (size_t)j * K;
      int32_t acc = 0;
      for (int k = 0; k < K; ++k) acc += (int32_t)a[k] * (int32_t)b[k];
      C[(size_t)i * J + j] = acc;
    }
}

void orc_igemm_tn(const int8_t *A, const int8_t *B, int I, int J, int K, int32_t *C) { igemm_tn(A, B, I, J, K, C); }

/* forward: Y = bf16( float(acc) * (s_x * s_w[n]) ) */
void orc_linear_fwd(const bf16_t *X, const bf16_t *W, int M, int N, int K, const float *s_x,
                    const float *s_w, bf16_t *Y, int8_t *qX, int8_t *qW) {
  orc_lsq_quantize(X, M, K, s_x, 0, qX);
  orc_lsq_quantize(W, N, K, s_w, 1, qW);
  int32_t *acc = (int32_t *)malloc((size_t)M * N * sizeof(int32_t));
  igemm_tn(qX, qW, M, N, K, acc);
#pragma omp parallel for
  for (int m = 0; m < M; ++m)
    for (int n = 0; n < N; ++n)
      Y[(size_t)m * N + n] = f2bf(fmul(i2f(acc[(size_t)m * N + n]), fmul(*s_x, s_w[n])));
  free(acc);
}

/* Unnormalised Walsh-Hadamard butterflies on a strided vector of length 128:
 * stages h = 1,2,...,64; (a,b) -> (a+b, a-b) for pairs (i, i+h) with i & h == 0. */
static void wht128_f(float *v) {
  for (int h = 1; h < 128; h <<= 1)
    for (int i = 0; i < 128; ++i)
      if (!(i & h)) { float a = v[i], b = v[i + h]; v[i] = fadd(a, b); v[i + h] = fsub(a, b); }
}
static void wht128_i(int32_t *v) {
  for (int h = 1; h < 128; h <<= 1)
    for (int i = 0; i < 128; ++i)
      if (!(i & h)) { int32_t a = v[i], b = v[i + h]; v[i] = a + b; v[i + h] = a - b; }
}
void orc_wht128_f(float *v) { wht128_f(v); }
void orc_wht128_i(int32_t *v) { wht128_i(v); }

/* per-tensor absmax int8 quantiser used by the gradient GEMM operands:
 * s = absmax/127, q = rne(v * (127/absmax)); absmax == 0 gives s = 0, q = 0. */
static void absmax_quant_f(const float *v, size_t n, int8_t *q, float *s) {
  float am = 0.0f;
  for (size_t i = 0; i < n; ++i) am = fmax2(am, fabs1(v[i]));
  float inv = 0.0f;
  *s = 0.0f;
  if (am > 0.0f) { *s = fdiv(am, 127.0f); inv = fdiv(127.0f, am); }
#pragma omp parallel for
  for (size_t i = 0; i < n; ++i) {
    float t = fmin2(fmax2(fmul(v[i], inv), -128.0f), 127.0f);
    q[i] = (int8_t)(int)frne(t);
  }
}

/* backward (straight-through estimator through both quantisers; both gradient
 * contractions in int8 after a block-128 Walsh-Hadamard rotation along the
 * contraction dimension when hb == 128; hb == 0 disables the rotation).
 * Outputs: dX bf16 [M,K], dW f32 [N,K], ds_x f32 scalar.
 * Optional (nullable) debug outputs: Aq [M,N], UqT [K,N], GqT [N,M], ZqT [K,M],
 * scales[4] = {s_a, s_u, s_g, s_z}. */
/* integer operand after the rotation: exact int32 values -> int8 with s = absmax/127 (rotation on), or the values
 * themselves with s = 1 (rotation off) */
static void int_operand_quant(const int32_t *U, size_t n, int hb, int8_t *q, float *s) {
  if (hb) {
    int32_t am = 0;
    for (size_t i = 0; i < n; ++i) { int32_t v = U[i] < 0 ? -U[i] : U[i]; if (v > am) am = v; }
    float inv = 0.0f; *s = 0.0f;
    if (am > 0) { *s = fdiv(i2f(am), 127.0f); inv = fdiv(127.0f, i2f(am)); }
    for (size_t i = 0; i < n; ++i) {
      float t = fmin2(fmax2(fmul(i2f(U[i]), inv), -128.0f), 127.0f);
      q[i] = (int8_t)(int)frne(t);
    }
  } else {
    *s = 1.0f;
    for (size_t i = 0; i < n; ++i) q[i] = (int8_t)U[i];
  }
}

/* operands of the input-gradient GEMM: Aq [M,N] = quant(rotate_n(dY * s_w)), UqT [K,N] = quant(rotate_n(qW)^T) */
static void bwd_operands_x(const bf16_t *dY, const int8_t *qW, int M, int N, int K, const float *s_w, int hb,
                           int8_t *Aq, int8_t *UqT, float *s_a, float *s_u) {
  size_t MN = (size_t)M * N, NK = (size_t)N * K;
  float *a = (float *)malloc(MN * sizeof(float));
#pragma omp parallel for
  for (int m = 0; m < M; ++m) {
    for (int n = 0; n < N; ++n) a[(size_t)m * N + n] = fmul(bf2f(dY[(size_t)m * N + n]), s_w[n]);
    if (hb) for (int n0 = 0; n0 < N; n0 += 128) wht128_f(a + (size_t)m * N + n0);
  }
  absmax_quant_f(a, MN, Aq, s_a);
  free(a);
  /* U = H * qW along n (exact integers), stored transposed [K,N] */
  int32_t *U = (int32_t *)malloc(NK * sizeof(int32_t));
#pragma omp parallel for
  for (int k = 0; k < K; ++k) {
    for (int n = 0; n < N; ++n) U[(size_t)k * N + n] = qW[(size_t)n * K + k];
    if (hb) for (int n0 = 0; n0 < N; n0 += 128) wht128_i(U + (size_t)k * N + n0);
  }
  int_operand_quant(U, NK, hb, UqT, s_u);
  free(U);
}

/* operands of the weight-gradient GEMM: GqT [N,M] = quant(rotate_m(dY)^T), ZqT [K,M] = quant(rotate_m(qX)^T) */
static void bwd_operands_w(const bf16_t *dY, const int8_t *qX, int M, int N, int K, int hb, int8_t *GqT, int8_t *ZqT,
                           float *s_g, float *s_z) {
  size_t MN = (size_t)M * N, MK = (size_t)M * K;
  float *GT = (float *)malloc(MN * sizeof(float)); /* [N,M] */
#pragma omp parallel for
  for (int n = 0; n < N; ++n) {
    for (int m = 0; m < M; ++m) GT[(size_t)n * M + m] = bf2f(dY[(size_t)m * N + n]);
    if (hb) for (int m0 = 0; m0 < M; m0 += 128) wht128_f(GT + (size_t)n * M + m0);
  }
  absmax_quant_f(GT, MN, GqT, s_g);
  free(GT);
  int32_t *Z = (int32_t *)malloc(MK * sizeof(int32_t)); /* [K,M] */
#pragma omp parallel for
  for (int k = 0; k < K; ++k) {
    for (int m = 0; m < M; ++m) Z[(size_t)k * M + m] = qX[(size_t)m * K + k];
    if (hb) for (int m0 = 0; m0 < M; m0 += 128) wht128_i(Z + (size_t)k * M + m0);
  }
  int_operand_quant(Z, MK, hb, ZqT, s_z);
  free(Z);
}

/* dX element and its LSQ step-gradient term from the integer accumulator */
static inline float dx_epilogue(int32_t acc, float cx, float x, float inv_sx, int8_t qx, bf16_t *dx) {
  float gx = fmul(i2f(acc), cx);
  float t = fmul(x, inv_sx);
  int in_range = (t >= -128.0f) && (t <= 127.0f);
  *dx = f2bf(in_range ? gx : 0.0f);
  float phi = t < -128.0f ? -128.0f : (t > 127.0f ? 127.0f : fsub(i2f((int32_t)qx), t));
  return fmul(gx, phi);
}
static inline float dw_epilogue(int32_t acc, float cw, float w, float inv_sw) {
  float t = fmul(w, inv_sw);
  int in_range = (t >= -128.0f) && (t <= 127.0f);
  return in_range ? fmul(i2f(acc), cw) : 0.0f;
}

void orc_linear_bwd(const bf16_t *dY, const bf16_t *X, const bf16_t *W, int M, int N, int K,
                    const float *s_x, const float *s_w, int hb, bf16_t *dX, float *dW, float *ds_x,
                    int8_t *Aq_out, int8_t *UqT_out, int8_t *GqT_out, int8_t *ZqT_out, float *scales) {
  size_t MN = (size_t)M * N, MK = (size_t)M * K, NK = (size_t)N * K;
  int8_t *qX = (int8_t *)malloc(MK), *qW = (int8_t *)malloc(NK);
  orc_lsq_quantize(X, M, K, s_x, 0, qX);
  orc_lsq_quantize(W, N, K, s_w, 1, qW);
  float rot = hb ? 0x1p-7f : 1.0f;
  float s_a, s_u, s_g, s_z;

  /* ---- grad wrt x: contraction over n ---- */
  int8_t *Aq = (int8_t *)malloc(MN), *UqT = (int8_t *)malloc(NK);
  bwd_operands_x(dY, qW, M, N, K, s_w, hb, Aq, UqT, &s_a, &s_u);
  int32_t *acc = (int32_t *)malloc(MK * sizeof(int32_t));
  igemm_tn(Aq, UqT, M, K, N, acc);
  float cx = fmul(fmul(s_a, s_u), rot);
  float inv_sx = fdiv(1.0f, *s_x);
  float *terms = (float *)malloc(MK * sizeof(float));
#pragma omp parallel for
  for (size_t i = 0; i < MK; ++i) terms[i] = dx_epilogue(acc[i], cx, bf2f(X[i]), inv_sx, qX[i], dX + i);
  /* LSQ step-size gradient, scaled by 1/sqrt(M*K*q_max) */
  float gs = (float)(1.0 / sqrt((double)M * (double)K * 127.0));
  *ds_x = fmul(gs, det_sum(terms, MK));
  free(terms); free(acc);

  /* ---- grad wrt W: contraction over tokens m ---- */
  int8_t *GqT = (int8_t *)malloc(MN), *ZqT = (int8_t *)malloc(MK);
  bwd_operands_w(dY, qX, M, N, K, hb, GqT, ZqT, &s_g, &s_z);
  int32_t *accw = (int32_t *)malloc(NK * sizeof(int32_t));
  igemm_tn(GqT, ZqT, N, K, M, accw);
  float cw = fmul(fmul(fmul(s_g, s_z), *s_x), rot);
#pragma omp parallel for
  for (int n = 0; n < N; ++n) {
    float inv_sw = fdiv(1.0f, s_w[n]);
    for (int k = 0; k < K; ++k) {
      size_t i = (size_t)n * K + k;
      dW[i] = dw_epilogue(accw[i], cw, bf2f(W[i]), inv_sw);
    }
  }
  if (Aq_out) memcpy(Aq_out, Aq, MN);
  if (UqT_out) memcpy(UqT_out, UqT, NK);
  if (GqT_out) memcpy(GqT_out, GqT, MN);
  if (ZqT_out) memcpy(ZqT_out, ZqT, MK);
  if (scales) { scales[0] = s_a; scales[1] = s_u; scales[2] = s_g; scales[3] = s_z; }
  free(accw); free(ZqT); free(GqT); free(Aq); free(UqT); free(qX); free(qW);
}

/* The same backward, but only nm rows of dX (token indices rows_m) and nn rows of dW (output channels rows_n) are
 * evaluated: the operands are prepared in full (their scales are whole-tensor maxima), the two integer contractions
 * and epilogues only for the selected rows.  For checks at shapes whose full contractions are too slow on a CPU. */
void orc_linear_bwd_rows(const bf16_t *dY, const bf16_t *X, const bf16_t *W, int M, int N, int K, const float *s_x,
                         const float *s_w, int hb, const int32_t *rows_m, int nm, const int32_t *rows_n, int nn,
                         bf16_t *dX_rows, float *dW_rows) {
  size_t MN = (size_t)M * N, MK = (size_t)M * K, NK = (size_t)N * K;
  int8_t *qX = (int8_t *)malloc(MK), *qW = (int8_t *)malloc(NK);
  orc_lsq_quantize(X, M, K, s_x, 0, qX);
  orc_lsq_quantize(W, N, K, s_w, 1, qW);
  float rot = hb ? 0x1p-7f : 1.0f;
  float s_a, s_u, s_g, s_z;
  int8_t *Aq = (int8_t *)malloc(MN), *UqT = (int8_t *)malloc(NK);
  bwd_operands_x(dY, qW, M, N, K, s_w, hb, Aq, UqT, &s_a, &s_u);
  int8_t *Ar = (int8_t *)malloc((size_t)nm * N);
  for (int i = 0; i < nm; ++i) memcpy(Ar + (size_t)i * N, Aq + (size_t)rows_m[i] * N, N);
  int32_t *acc = (int32_t *)malloc((size_t)nm * K * sizeof(int32_t));
  igemm_tn(Ar, UqT, nm, K, N, acc);
  float cx = fmul(fmul(s_a, s_u), rot);
  float inv_sx = fdiv(1.0f, *s_x);
  for (int i = 0; i < nm; ++i)
    for (int k = 0; k < K; ++k) {
      size_t src = (size_t)rows_m[i] * K + k;
      dx_epilogue(acc[(size_t)i * K + k], cx, bf2f(X[src]), inv_sx, qX[src], dX_rows + (size_t)i * K + k);
    }
  free(acc); free(Ar); free(Aq); free(UqT);
  int8_t *GqT = (int8_t *)malloc(MN), *ZqT = (int8_t *)malloc(MK);
  bwd_operands_w(dY, qX, M, N, K, hb, GqT, ZqT, &s_g, &s_z);
  int8_t *Gr = (int8_t *)malloc((size_t)nn * M);
  for (int i = 0; i < nn; ++i) memcpy(Gr + (size_t)i * M, GqT + (size_t)rows_n[i] * M, M);
  int32_t *accw = (int32_t *)malloc((size_t)nn * K * sizeof(int32_t));
  igemm_tn(Gr, ZqT, nn, K, M, accw);
  float cw = fmul(fmul(fmul(s_g, s_z), *s_x), rot);
  for (int i = 0; i < nn; ++i) {
    float inv_sw = fdiv(1.0f, s_w[rows_n[i]]);
    for (int k = 0; k < K; ++k)
      dW_rows[(size_t)i * K + k] = dw_epilogue(accw[(size_t)i * K + k], cw, bf2f(W[(size_t)rows_n[i] * K + k]), inv_sw);
  }
  free(accw); free(Gr); free(GqT); free(ZqT); free(qX); free(qW);
}

/* ------------------------------------------------------------------ */
/* RMSNorm (Sec. 3.1 "RMSNorm"; FP32 internals)                        */
/* ------------------------------------------------------------------ */
static inline float ld(int bf, const void *p, size_t i) {
  return bf ? bf2f(((const bf16_t *)p)[i]) : ftz(((const float *)p)[i]);
}
static inline void st(int bf, void *p, size_t i, float v) {
  if (bf) ((bf16_t *)p)[i] = f2bf(v); else ((float *)p)[i] = v;
}

void orc_rmsnorm_fwd(int bf, const void *x, const void *gamma, int rows, int D, float eps, void *y, float *rstd) {
  float invD = (float)(1.0 / (double)D);
#pragma omp parallel for
  for (int r = 0; r < rows; ++r) {
    float *t = (float *)malloc((size_t)D * sizeof(float));
    for (int j = 0; j < D; ++j) { float v = ld(bf, x, (size_t)r * D + j); t[j] = fmul(v, v); }
    float ms = fmul(det_sum(t, D), invD);
    float rs = fdiv(1.0f, fsqrt(fadd(ms, eps)));
    rstd[r] = rs;
    for (int j = 0; j < D; ++j) {
      float v = fmul(ld(bf, x, (size_t)r * D + j), rs);
      if (gamma) v = fmul(v, ld(bf, gamma, j));
      st(bf, y, (size_t)r * D + j, v);
    }
    free(t);
  }
}

void orc_rmsnorm_bwd(int bf, const void *dy, const void *x, const void *gamma, const float *rstd, int rows, int D,
                     void *dx, float *dgamma) {
  float invD = (float)(1.0 / (double)D);
#pragma omp parallel for
  for (int r = 0; r < rows; ++r) {
    float *t = (float *)malloc((size_t)D * sizeof(float));
    float rs = rstd[r];
    for (int j = 0; j < D; ++j) {
      float w = ld(bf, dy, (size_t)r * D + j);
      if (gamma) w = fmul(w, ld(bf, gamma, j));
      t[j] = fmul(w, fmul(ld(bf, x, (size_t)r * D + j), rs));
    }
    float c = fmul(det_sum(t, D), invD);
    for (int j = 0; j < D; ++j) {
      float w = ld(bf, dy, (size_t)r * D + j);
      if (gamma) w = fmul(w, ld(bf, gamma, j));
      float xh = fmul(ld(bf, x, (size_t)r * D + j), rs);
      st(bf, dx, (size_t)r * D + j, fmul(rs, fsub(w, fmul(xh, c))));
    }
    free(t);
  }
  if (dgamma) {
#pragma omp parallel for
    for (int j = 0; j < D; ++j) {
      float *t = (float *)malloc((size_t)rows * sizeof(float));
      for (int r = 0; r < rows; ++r)
        t[r] = fmul(ld(bf, dy, (size_t)r * D + j), fmul(ld(bf, x, (size_t)r * D + j), rstd[r]));
      dgamma[j] = det_sum(t, rows);
      free(t);
    }
  }
}

/* ------------------------------------------------------------------ */
/* cross-entropy (+ z-loss) (Sec. 3.1 "Z-loss"; FP32 loss)             */
/* ------------------------------------------------------------------ */
/* returns the number of rows whose target is out of [0,V) (those rows give 0) */
int orc_xent_fwd(const float *logits, const int32_t *target, int rows, int V, float z_weight, float *loss_row,
                 float *lse, float *loss_mean, float *z_mean) {
  int bad = 0;
  float *zr = (float *)malloc((size_t)rows * sizeof(float));
#pragma omp parallel for reduction(+ : bad)
  for (int r = 0; r < rows; ++r) {
    const float *z = logits + (size_t)r * V;
    float *e = (float *)malloc((size_t)V * sizeof(float));
    float m = ftz(z[0]);
    for (int j = 1; j < V; ++j) m = fmax2(m, z[j]);
    for (int j = 0; j < V; ++j) e[j] = det_exp(fsub(z[j], m));
    float S = det_sum(e, V);
    float l = fadd(m, det_log(S));
    lse[r] = l;
    int t = target[r];
    if (t < 0 || t >= V) { loss_row[r] = 0.0f; zr[r] = 0.0f; bad++; }
    else { loss_row[r] = fsub(l, z[t]); zr[r] = fmul(l, l); }
    free(e);
  }
  float inv = (float)(1.0 / (double)rows);
  float ce = fmul(det_sum(loss_row, rows), inv);
  float zm = fmul(det_sum(zr, rows), inv);
  *z_mean = zm;
  *loss_mean = (z_weight != 0.0f) ? fadd(ce, fmul(z_weight, zm)) : ce;
  free(zr);
  return bad;
}

/* dz = (p - onehot [+ 2 w lse p]) * scale, p = exp(z - lse); in place */
void orc_xent_bwd(float *logits, const int32_t *target, const float *lse, int rows, int V, float z_weight, float scale) {
#pragma omp parallel for
  for (int r = 0; r < rows; ++r) {
    float *z = logits + (size_t)r * V;
    int t = target[r];
    int ok = (t >= 0 && t < V);
    float zc = fmul(fmul(2.0f, z_weight), lse[r]);
    for (int j = 0; j < V; ++j) {
      if (!ok) { z[j] = 0.0f; continue; }
      float p = det_exp(fsub(z[j], lse[r]));
      float d = fsub(p, j == t ? 1.0f : 0.0f);
      if (z_weight != 0.0f) d = fadd(d, fmul(zc, p));
      z[j] = fmul(d, scale);
    }
  }
}

/* ------------------------------------------------------------------ */
/* causal attention, head_dim 128, KV tiles of 128 keys in ascending    */
/* order (Sec. 3.2: QK^T and softmax in higher precision, BF16 flash    */
/* backward with recomputed weights)                                    */
/* ------------------------------------------------------------------ */
#define DH 128
#define KT 128
static inline float dot128(const bf16_t *a, const bf16_t *b) {
  float acc = 0.0f;
  for (int c = 0; c < DH; ++c) acc = fadd(acc, fmul(bf2f(a[c]), bf2f(b[c])));
  return acc;
}
static float tree128(float *v) { /* perfect adjacent tree, in place */
  for (int w = 1; w < 128; w <<= 1)
    for (int i = 0; i < 128; i += 2 * w) v[i] = fadd(v[i], v[i + w]);
  return v[0];
}

/* q,k,v: row (b*S+i) at element offset ld*(b*S+i) + h*128; out likewise with ld_out; lse [B,H,S] */
/* Hkv: number of key/value heads (grouped-query attention, Sec. 3.1: query head h reads key/value head
 * h / (H/Hkv)); Hkv == H is ordinary multi-head attention.  W: sliding window (Sec. 3.1: local layers see the
 * last W keys, j in (i - W, i]); W == 0 is full causal attention.  A row visits only the key tiles that hold at
 * least one visible key, in ascending order. */
static inline int visible(int i, int j, int W) { return j <= i && (W == 0 || j > i - W); }
static inline int first_tile(int i, int W) { int lo = (W == 0 || i - W + 1 < 0) ? 0 : i - W + 1; return lo / KT * KT; }

void orc_attn_fwd(const bf16_t *q, const bf16_t *k, const bf16_t *v, int ldq, int B, int H, int Hkv, int S, int W,
                  bf16_t *out, int ld_out, float *lse) {
  const int G = H / Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic, 8)
  for (int bh = 0; bh < B * H; ++bh)
    for (int i = 0; i < S; ++i) {
      int b = bh / H, h = bh % H, hk = h / G;
      const bf16_t *qi = q + (size_t)ldq * (b * S + i) + h * DH;
      float m = -INFINITY, l = 0.0f, o[DH], s[KT], p[KT], pt[KT];
      for (int c = 0; c < DH; ++c) o[c] = 0.0f;
      for (int j0 = first_tile(i, W); j0 <= i; j0 += KT) {
        float mt = m;
        for (int jj = 0; jj < KT; ++jj) {
          int j = j0 + jj;
          if (visible(i, j, W)) {
            s[jj] = fmul(dot128(qi, k + (size_t)ldq * (b * S + j) + hk * DH), ATT_SCALE);
            mt = fmax2(mt, s[jj]);
          }
        }
        float alpha = det_exp(fsub(m, mt));
        for (int jj = 0; jj < KT; ++jj) {
          p[jj] = visible(i, j0 + jj, W) ? det_exp(fsub(s[jj], mt)) : 0.0f;
          pt[jj] = bf2f(f2bf(p[jj]));
        }
        float r = tree128(p);
        l = fadd(fmul(l, alpha), r);
        for (int c = 0; c < DH; ++c) {
          float u = 0.0f;
          for (int jj = 0; jj < KT && j0 + jj <= i; ++jj)
            u = fadd(u, fmul(pt[jj], bf2f(v[(size_t)ldq * (b * S + j0 + jj) + hk * DH + c])));
          o[c] = fadd(fmul(o[c], alpha), u);
        }
        m = mt;
      }
      float il = fdiv(1.0f, l);
      for (int c = 0; c < DH; ++c) out[(size_t)ld_out * (b * S + i) + h * DH + c] = f2bf(fmul(o[c], il));
      lse[(size_t)bh * S + i] = fadd(m, det_log(l));
    }
}

/* Forward with the P.V product of every KV block in int8 (Sec. 3.2: "int8 P.V per block; QK^T and softmax in
 * higher precision").  The paper does not state the scales; this version fixes them as follows.  Per (batch, key/value
 * head, block of 128 keys): s_v = absmax(V block)/127, q_v = rne(clamp(v * (127/absmax))).  Per row and block:
 * q_p = rne(p * 127) with p = exp(s - m) in [0,1] (masked slots 0).  u_c = float(sum_j q_p[j] q_v[j,c]) * (s_v/127)
 * (the integer sum is exact and order-free), then o = o*alpha + u as before.  The row sum l and the logsumexp use
 * the unquantised p, so lse equals that of orc_attn_fwd; the backward pass is unchanged (it recomputes P in full
 * precision and does not see the quantisation).  The scale of a block is shared by all rows that touch it. */
void orc_attn_fwd_int8pv(const bf16_t *q, const bf16_t *k, const bf16_t *v, int ldq, int B, int H, int Hkv, int S, int W,
                         bf16_t *out, int ld_out, float *lse) {
  const int G = H / Hkv, NT = (S + KT - 1) / KT;
  float *sv = (float *)malloc((size_t)B * Hkv * NT * sizeof(float));   /* absmax of every V block */
#pragma omp parallel for
  for (int t = 0; t < B * Hkv * NT; ++t) {
    int b = t / (Hkv * NT), hk = (t / NT) % Hkv, j0 = (t % NT) * KT;
    float am = 0.0f;
    for (int j = j0; j < j0 + KT && j < S; ++j)
      for (int c = 0; c < DH; ++c) am = fmax2(am, fabs1(bf2f(v[(size_t)ldq * (b * S + j) + hk * DH + c])));
    sv[t] = am;
  }
#pragma omp parallel for collapse(2) schedule(dynamic, 8)
  for (int bh = 0; bh < B * H; ++bh)
    for (int i = 0; i < S; ++i) {
      int b = bh / H, h = bh % H, hk = h / G;
      const bf16_t *qi = q + (size_t)ldq * (b * S + i) + h * DH;
      float m = -INFINITY, l = 0.0f, o[DH], s[KT], p[KT];
      int32_t qp[KT];
      for (int c = 0; c < DH; ++c) o[c] = 0.0f;
      for (int j0 = first_tile(i, W); j0 <= i; j0 += KT) {
        float mt = m;
        for (int jj = 0; jj < KT; ++jj) {
          int j = j0 + jj;
          if (visible(i, j, W)) {
            s[jj] = fmul(dot128(qi, k + (size_t)ldq * (b * S + j) + hk * DH), ATT_SCALE);
            mt = fmax2(mt, s[jj]);
          }
        }
        float alpha = det_exp(fsub(m, mt));
        for (int jj = 0; jj < KT; ++jj) {
          p[jj] = visible(i, j0 + jj, W) ? det_exp(fsub(s[jj], mt)) : 0.0f;
          qp[jj] = (int32_t)frne(fmul(p[jj], 127.0f));
        }
        float r = tree128(p);
        l = fadd(fmul(l, alpha), r);
        float am = sv[((size_t)b * Hkv + hk) * NT + j0 / KT];
        float s_v = 0.0f, inv_v = 0.0f;
        if (am > 0.0f) { s_v = fdiv(am, 127.0f); inv_v = fdiv(127.0f, am); }
        float cs = fdiv(s_v, 127.0f);
        for (int c = 0; c < DH; ++c) {
          int32_t acc = 0;
          for (int jj = 0; jj < KT && j0 + jj <= i; ++jj) {
            float t = fmin2(fmax2(fmul(bf2f(v[(size_t)ldq * (b * S + j0 + jj) + hk * DH + c]), inv_v), -128.0f), 127.0f);
            acc += qp[jj] * (int32_t)frne(t);
          }
          o[c] = fadd(fmul(o[c], alpha), fmul(i2f(acc), cs));
        }
        m = mt;
      }
      float il = fdiv(1.0f, l);
      for (int c = 0; c < DH; ++c) out[(size_t)ld_out * (b * S + i) + h * DH + c] = f2bf(fmul(o[c], il));
      lse[(size_t)bh * S + i] = fadd(m, det_log(l));
    }
  free(sv);
}

/* backward: p_ij = exp(s_ij - L_i); Delta_i = tree_c(dO*O); dP = dO.v_j;
 * dS = p (dP - Delta) scale; contraction operands rounded to bf16; all three
 * gradient contractions are sequential ascending sums from +0.  With grouped
 * queries the gradient of a shared key/value head is ONE sequential accumulator
 * over its query heads in ascending order and, within a head, over the queries
 * in ascending order. */
/* Sec. 3.2 names a second accumulator for the query gradient: 64-bit fixed point, so that the sum over the key blocks
   does not depend on their order.  Reading: the contribution of one block of 128 keys is the ordered fp32 sum over the
   block's keys from +0 (the same per-block arithmetic as P.V in the forward); it enters a signed 64-bit accumulator
   with 48 fractional bits as rne(u * 2^48), saturated at the ends of the range (a NaN contributes 0); integer
   additions wrap; the result is the accumulator converted to fp32 (round to nearest even) times 2^-48, then bf16. */
int64_t orc_fix48(float u) {
  float t = fmul(u, 0x1p48f);
  if (t != t) return 0;
  if (t >= 0x1p63f) return INT64_MAX;
  if (t <= -0x1p63f) return INT64_MIN;
  return (int64_t)llrintf(t);
}
float orc_unfix48(int64_t a) { return fmul((float)a, 0x1p-48f); }

static void attn_bwd_impl(const bf16_t *dout, const bf16_t *q, const bf16_t *k, const bf16_t *v, const bf16_t *out,
                          const float *lse, int ldq, int ld_out, int B, int H, int Hkv, int S, int W, bf16_t *dq,
                          bf16_t *dk, bf16_t *dv, int ld_d, int fixq) {
  const int G = H / Hkv;
#pragma omp parallel for schedule(dynamic, 1)
  for (int bk = 0; bk < B * Hkv; ++bk) {
    int b = bk / Hkv, hk = bk % Hkv;
    size_t SS = (size_t)S * S;
    float *Pt = (float *)calloc(SS * G, sizeof(float));  /* bf16-rounded p, widened, per query head of the group */
    float *dSt = (float *)calloc(SS * G, sizeof(float)); /* bf16-rounded dS, widened */
    for (int g = 0; g < G; ++g) {
      int h = hk * G + g;
      for (int i = 0; i < S; ++i) {
        const bf16_t *qi = q + (size_t)ldq * (b * S + i) + h * DH;
        const bf16_t *doi = dout + (size_t)ld_out * (b * S + i) + h * DH;
        const bf16_t *oi = out + (size_t)ld_out * (b * S + i) + h * DH;
        float t[DH];
        for (int c = 0; c < DH; ++c) t[c] = fmul(bf2f(doi[c]), bf2f(oi[c]));
        float delta = tree128(t);
        float L = lse[((size_t)b * H + h) * S + i];
        for (int j = 0; j <= i; ++j) {
          if (!visible(i, j, W)) continue;
          float s = fmul(dot128(qi, k + (size_t)ldq * (b * S + j) + hk * DH), ATT_SCALE);
          float p = det_exp(fsub(s, L));
          float dP = dot128(doi, v + (size_t)ldq * (b * S + j) + hk * DH);
          float dS = fmul(fmul(p, fsub(dP, delta)), ATT_SCALE);
          Pt[g * SS + (size_t)i * S + j] = bf2f(f2bf(p));
          dSt[g * SS + (size_t)i * S + j] = bf2f(f2bf(dS));
        }
      }
    }
    for (int j = 0; j < S; ++j)
      for (int c = 0; c < DH; ++c) {
        float av = 0.0f, ak = 0.0f;
        for (int g = 0; g < G; ++g) {
          int h = hk * G + g;
          for (int i = j; i < S; ++i) {
            if (!visible(i, j, W)) continue;
            av = fadd(av, fmul(Pt[g * SS + (size_t)i * S + j], bf2f(dout[(size_t)ld_out * (b * S + i) + h * DH + c])));
            ak = fadd(ak, fmul(dSt[g * SS + (size_t)i * S + j], bf2f(q[(size_t)ldq * (b * S + i) + h * DH + c])));
          }
        }
        dv[(size_t)ld_d * (b * S + j) + hk * DH + c] = f2bf(av);
        dk[(size_t)ld_d * (b * S + j) + hk * DH + c] = f2bf(ak);
      }
    for (int g = 0; g < G; ++g) {
      int h = hk * G + g;
      for (int i = 0; i < S; ++i)
        for (int c = 0; c < DH; ++c) {
          float aq = 0.0f;
          if (!fixq) {
            for (int j = 0; j <= i; ++j) {
              if (!visible(i, j, W)) continue;
              aq = fadd(aq, fmul(dSt[g * SS + (size_t)i * S + j], bf2f(k[(size_t)ldq * (b * S + j) + hk * DH + c])));
            }
          } else {
            uint64_t fx = 0;
            for (int j0 = 0; j0 <= i; j0 += 128) {   /* blocks of 128 keys; a block without visible keys adds 0 */
              float u = 0.0f;
              for (int j = j0; j < j0 + 128 && j <= i; ++j) {
                if (!visible(i, j, W)) continue;
                u = fadd(u, fmul(dSt[g * SS + (size_t)i * S + j], bf2f(k[(size_t)ldq * (b * S + j) + hk * DH + c])));
              }
              fx += (uint64_t)orc_fix48(u);
            }
            aq = orc_unfix48((int64_t)fx);
          }
          dq[(size_t)ld_d * (b * S + i) + h * DH + c] = f2bf(aq);
        }
    }
    free(Pt); free(dSt);
  }
}
void orc_attn_bwd(const bf16_t *dout, const bf16_t *q, const bf16_t *k, const bf16_t *v, const bf16_t *out,
                  const float *lse, int ldq, int ld_out, int B, int H, int Hkv, int S, int W, bf16_t *dq, bf16_t *dk,
                  bf16_t *dv, int ld_d) {
  attn_bwd_impl(dout, q, k, v, out, lse, ldq, ld_out, B, H, Hkv, S, W, dq, dk, dv, ld_d, 0);
}
void orc_attn_bwd_fixq(const bf16_t *dout, const bf16_t *q, const bf16_t *k, const bf16_t *v, const bf16_t *out,
                       const float *lse, int ldq, int ld_out, int B, int H, int Hkv, int S, int W, bf16_t *dq, bf16_t *dk,
                       bf16_t *dv, int ld_d) {
  attn_bwd_impl(dout, q, k, v, out, lse, ldq, ld_out, B, H, Hkv, S, W, dq, dk, dv, ld_d, 1);
}

/* ------------------------------------------------------------------ */
/* elementwise glue (Sec. 3.1: SwiGLU, residual stream, embedding)      */
/* ------------------------------------------------------------------ */
/* gu [rows, 2F]: gate = columns [0,F), up = columns [F,2F) */
void orc_swiglu_fwd(const bf16_t *gu, int rows, int F, bf16_t *h) {
#pragma omp parallel for
  for (int r = 0; r < rows; ++r)
    for (int j = 0; j < F; ++j) {
      float g = bf2f(gu[(size_t)r * 2 * F + j]), u = bf2f(gu[(size_t)r * 2 * F + F + j]);
      float sg = fdiv(1.0f, fadd(1.0f, det_exp(fneg(g))));
      h[(size_t)r * F + j] = f2bf(fmul(fmul(g, sg), u));
    }
}
void orc_swiglu_bwd(const bf16_t *dh, const bf16_t *gu, int rows, int F, bf16_t *dgu) {
#pragma omp parallel for
  for (int r = 0; r < rows; ++r)
    for (int j = 0; j < F; ++j) {
      float g = bf2f(gu[(size_t)r * 2 * F + j]), u = bf2f(gu[(size_t)r * 2 * F + F + j]);
      float d = bf2f(dh[(size_t)r * F + j]);
      float sg = fdiv(1.0f, fadd(1.0f, det_exp(fneg(g))));
      float du = fmul(d, fmul(g, sg));
      float dg = fmul(fmul(d, u), fmul(sg, fadd(1.0f, fmul(g, fsub(1.0f, sg)))));
      dgu[(size_t)r * 2 * F + j] = f2bf(dg);
      dgu[(size_t)r * 2 * F + F + j] = f2bf(du);
    }
}
void orc_residual_add(const bf16_t *a, const bf16_t *b, size_t n, bf16_t *y) {
#pragma omp parallel for
  for (size_t i = 0; i < n; ++i) y[i] = f2bf(fadd(bf2f(a[i]), bf2f(b[i])));
}
void orc_embed_fwd(const int32_t *tok, int T, const bf16_t *E, int D, bf16_t *y) {
  for (int t = 0; t < T; ++t) memcpy(y + (size_t)t * D, E + (size_t)tok[t] * D, (size_t)D * 2);
}
/* dE[v,:] = sequential sum over positions with tok == v in ascending position, from +0 */
void orc_embed_bwd(const int32_t *tok, int T, const bf16_t *dy, int V, int D, float *dE) {
  memset(dE, 0, (size_t)V * D * sizeof(float));
  for (int t = 0; t < T; ++t) {
    float *row = dE + (size_t)tok[t] * D;
    for (int j = 0; j < D; ++j) row[j] = fadd(row[j], bf2f(dy[(size_t)t * D + j]));
  }
}

/* ------------------------------------------------------------------ */
/* LM head in full precision: ordered f32 sums of exact bf16 products   */
/* (Sec. 3.2: the head is excluded from quantisation)                   */
/* ------------------------------------------------------------------ */
void orc_lmhead_fwd(const bf16_t *Hh, const bf16_t *W, int M, int V, int K, float *logits) {
#pragma omp parallel for
  for (int m = 0; m < M; ++m)
    for (int n = 0; n < V; ++n) {
      float acc = 0.0f;
      for (int k = 0; k < K; ++k) acc = fadd(acc, fmul(bf2f(Hh[(size_t)m * K + k]), bf2f(W[(size_t)n * K + k])));
      logits[(size_t)m * V + n] = acc;
    }
}
/* dlogits rounded to bf16 first; dH bf16 [M,K] (sum over vocabulary ascending);
 * dW f32 [V,K]: sum over tokens ascending, continuing from the value already in
 * dW unless first_chunk (then from +0). */
void orc_lmhead_bwd(const float *dlogits, const bf16_t *Hh, const bf16_t *W, int M, int V, int K, bf16_t *dH,
                    float *dW, int first_chunk) {
  size_t MV = (size_t)M * V;
  float *g = (float *)malloc(MV * sizeof(float));
#pragma omp parallel for
  for (size_t i = 0; i < MV; ++i) g[i] = bf2f(f2bf(dlogits[i]));
#pragma omp parallel for
  for (int m = 0; m < M; ++m)
    for (int k = 0; k < K; ++k) {
      float acc = 0.0f;
      for (int n = 0; n < V; ++n) acc = fadd(acc, fmul(g[(size_t)m * V + n], bf2f(W[(size_t)n * K + k])));
      dH[(size_t)m * K + k] = f2bf(acc);
    }
#pragma omp parallel for
  for (int n = 0; n < V; ++n)
    for (int k = 0; k < K; ++k) {
      float acc = first_chunk ? 0.0f : dW[(size_t)n * K + k];
      for (int m = 0; m < M; ++m) acc = fadd(acc, fmul(g[(size_t)m * V + n], bf2f(Hh[(size_t)m * K + k])));
      dW[(size_t)n * K + k] = acc;
    }
  free(g);
}

/* ------------------------------------------------------------------ */
/* gradient reduction replay: Algorithm 1 (mesh-order loop) + Algorithm */
/* 2 (binary-carry TreeFold); averages are reciprocal multiplies         */
/* (Appendix A.3)                                                       */
/* ------------------------------------------------------------------ */
typedef struct {
  int accum, dp_shard, dp_replicate;
  size_t n;
  int pushes;          /* micro-batch pushes so far */
  float *g_r, *inner;  /* running sums */
  int nstack;
  int level[40];
  float *part[40];
  int resident, max_resident; /* full-size replica partials alive at once */
} orc_accum;

orc_accum *orc_accum_new(int accum, int dp_shard, int dp_replicate, size_t n) {
  orc_accum *a = (orc_accum *)calloc(1, sizeof(orc_accum));
  a->accum = accum; a->dp_shard = dp_shard; a->dp_replicate = dp_replicate; a->n = n;
  a->g_r = (float *)malloc(n * sizeof(float));
  a->inner = NULL;
  return a;
}
static void fold_push(orc_accum *a, float *part) { /* Algorithm 2, Push */
  int level = 0;
  a->resident++;
  if (a->resident > a->max_resident) a->max_resident = a->resident;
  while (a->nstack > 0 && a->level[a->nstack - 1] == level) {
    float *lower = a->part[--a->nstack];
    for (size_t i = 0; i < a->n; ++i) part[i] = fadd(lower[i], part[i]); /* lower replica on the left */
    free(lower);
    a->resident--;
    level++;
  }
  a->level[a->nstack] = level;
  a->part[a->nstack++] = part;
}
/* one micro-batch gradient, in mesh order (replica-major, shard-minor, then k) */
int orc_accum_push(orc_accum *a, const float *g) {
  int per_rank = a->accum, N = a->dp_shard * a->dp_replicate;
  if (a->pushes >= per_rank * N) return -1;
  int r = a->pushes / per_rank, kk = a->pushes % per_rank, shard = r % a->dp_shard;
  float inv_accum = (float)(1.0 / (double)a->accum);
  if (kk == 0) for (size_t i = 0; i < a->n; ++i) a->g_r[i] = 0.0f;
  for (size_t i = 0; i < a->n; ++i) a->g_r[i] = fadd(a->g_r[i], fmul(g[i], inv_accum));
  a->pushes++;
  if (kk == per_rank - 1) {
    if (shard == 0) {
      a->inner = (float *)malloc(a->n * sizeof(float));
      memcpy(a->inner, a->g_r, a->n * sizeof(float));
    } else {
      for (size_t i = 0; i < a->n; ++i) a->inner[i] = fadd(a->inner[i], a->g_r[i]);
    }
    if (shard == a->dp_shard - 1) {
      float inv_shard = (float)(1.0 / (double)a->dp_shard);
      for (size_t i = 0; i < a->n; ++i) a->inner[i] = fmul(a->inner[i], inv_shard);
      fold_push(a, a->inner);
      a->inner = NULL;
    }
  }
  return 0;
}
/* Algorithm 2, Result (pseudo-code reading: start from the lowest level entry,
 * i.e. the top of the stack, and add the higher-level (lower-replica) blocks on
 * the left), then the all-reduce average. */
int orc_accum_result(orc_accum *a, float *out) {
  if (a->pushes != a->accum * a->dp_shard * a->dp_replicate || a->nstack == 0) return -1;
  float inv_rep = (float)(1.0 / (double)a->dp_replicate);
  float *acc = a->part[a->nstack - 1];
  for (int s = a->nstack - 2; s >= 0; --s)
    for (size_t i = 0; i < a->n; ++i) acc[i] = fadd(a->part[s][i], acc[i]);
  for (size_t i = 0; i < a->n; ++i) out[i] = fmul(acc[i], inv_rep);
  return 0;
}
int orc_accum_max_resident(const orc_accum *a) { return a->max_resident; }
int orc_accum_stack_size(const orc_accum *a) { return a->nstack; }
void orc_accum_free(orc_accum *a) {
  for (int s = 0; s < a->nstack; ++s) free(a->part[s]);
  free(a->inner); free(a->g_r); free(a);
}

/* ------------------------------------------------------------------ */
/* global grad-norm + clip, AdamW (Sec. 3.2 "Optimizer",                */
/* "Optimizer-state precision")                                         */
/* ------------------------------------------------------------------ */
void orc_grad_norm(const float *const *g, const size_t *n, int ntensors, float max_norm, float *norm_out,
                   float *coef_out) {
  float *per = (float *)malloc((size_t)(ntensors ? ntensors : 1) * sizeof(float));
  for (int t = 0; t < ntensors; ++t) per[t] = orc_sumsq(g[t], n[t]);
  float norm = fsqrt(det_sum(per, ntensors));
  *norm_out = norm;
  *coef_out = (max_norm > 0.0f) ? fmin2(1.0f, fdiv(max_norm, fadd(norm, 1e-6f))) : 1.0f;
  free(per);
}
void orc_scale(float *g, size_t n, float coef) {
#pragma omp parallel for
  for (size_t i = 0; i < n; ++i) g[i] = fmul(g[i], coef);
}

static double ipow(double b, int e) { /* binary square-and-multiply */
  double r = 1.0;
  while (e > 0) { if (e & 1) r *= b; b *= b; e >>= 1; }
  return r;
}
/* p_is_bf16: parameters stored bf16 (rounded once per step) or f32 */
void orc_adamw(double lr, double beta1, double beta2, double eps, double wd, int step, int p_is_bf16, void *p,
               const float *g, float *m, float *v, size_t n) {
  double bc1 = 1.0 - ipow(beta1, step), bc2 = 1.0 - ipow(beta2, step);
  float stepsz = (float)(lr / bc1), isb2 = (float)(1.0 / sqrt(bc2)), decay = (float)(1.0 - lr * wd);
  float b1 = (float)beta1, b2 = (float)beta2, epsf = (float)eps;
  float omb1 = fsub(1.0f, b1), omb2 = fsub(1.0f, b2);
#pragma omp parallel for
  for (size_t i = 0; i < n; ++i) {
    float pv = p_is_bf16 ? bf2f(((bf16_t *)p)[i]) : ftz(((float *)p)[i]);
    float gi = g[i];
    float mi = fadd(fmul(b1, m[i]), fmul(omb1, gi));
    float vi = fadd(fmul(b2, v[i]), fmul(omb2, fmul(gi, gi)));
    float den = fadd(fmul(fsqrt(vi), isb2), epsf);
    pv = fsub(fmul(pv, decay), fmul(stepsz, fdiv(mi, den)));
    m[i] = mi; v[i] = vi;
    if (p_is_bf16) ((bf16_t *)p)[i] = f2bf(pv); else ((float *)p)[i] = pv;
  }
}

/* ------------------------------------------------------------------ */
/* SHA-256 (FIPS 180-4) and the chunked tensor hash (Appendix B: the    */
/* per-step state hash)                                                 */
/* ------------------------------------------------------------------ */
static const uint32_t KK[64] = {
    0x428a2f98, 0x71374491, 0xb5c0fbcf, 0xe9b5dba5, 0x3956c25b, 0x59f111f1, 0x923f82a4, 0xab1c5ed5, 0xd807aa98,
    0x12835b01, 0x243185be, 0x550c7dc3, 0x72be5d74, 0x80deb1fe, 0x9bdc06a7, 0xc19bf174, 0xe49b69c1, 0xefbe4786,
    0x0fc19dc6, 0x240ca1cc, 0x2de92c6f, 0x4a7484aa, 0x5cb0a9dc, 0x76f988da, 0x983e5152, 0xa831c66d, 0xb00327c8,
    0xbf597fc7, 0xc6e00bf3, 0xd5a79147, 0x06ca6351, 0x14292967, 0x27b70a85, 0x2e1b2138, 0x4d2c6dfc, 0x53380d13,
    0x650a7354, 0x766a0abb, 0x81c2c92e, 0x92722c85, 0xa2bfe8a1, 0xa81a664b, 0xc24b8b70, 0xc76c51a3, 0xd192e819,
    0xd6990624, 0xf40e3585, 0x106aa070, 0x19a4c116, 0x1e376c08, 0x2748774c, 0x34b0bcb5, 0x391c0cb3, 0x4ed8aa4a,
    0x5b9cca4f, 0x682e6ff3, 0x748f82ee, 0x78a5636f, 0x84c87814, 0x8cc70208, 0x90befffa, 0xa4506ceb, 0xbef9a3f7,
    0xc67178f2};
static inline uint32_t rotr(uint32_t x, int r) { return (x >> r) | (x << (32 - r)); }
static void sha_block(uint32_t h[8], const uint8_t *blk) {
  uint32_t w[64];
  for (int i = 0; i < 16; ++i)
    w[i] = ((uint32_t)blk[4 * i] << 24) | ((uint32_t)blk[4 * i + 1] << 16) | ((uint32_t)blk[4 * i + 2] << 8) | blk[4 * i + 3];
  for (int i = 16; i < 64; ++i) {
    uint32_t s0 = rotr(w[i - 15], 7) ^ rotr(w[i - 15], 18) ^ (w[i - 15] >> 3);
    uint32_t s1 = rotr(w[i - 2], 17) ^ rotr(w[i - 2], 19) ^ (w[i - 2] >> 10);
    w[i] = w[i - 16] + s0 + w[i - 7] + s1;
  }
  uint32_t a = h[0], b = h[1], c = h[2], d = h[3], e = h[4], f = h[5], g = h[6], hh = h[7];
  for (int i = 0; i < 64; ++i) {
    uint32_t S1 = rotr(e, 6) ^ rotr(e, 11) ^ rotr(e, 25), ch = (e & f) ^ (~e & g);
    uint32_t t1 = hh + S1 + ch + KK[i] + w[i];
    uint32_t S0 = rotr(a, 2) ^ rotr(a, 13) ^ rotr(a, 22), mj = (a & b) ^ (a & c) ^ (b & c);
    uint32_t t2 = S0 + mj;
    hh = g; g = f; f = e; e = d + t1; d = c; c = b; b = a; a = t1 + t2;
  }
  h[0] += a; h[1] += b; h[2] += c; h[3] += d; h[4] += e; h[5] += f; h[6] += g; h[7] += hh;
}
void orc_sha256(const uint8_t *data, size_t n, uint8_t out[32]) {
  uint32_t h[8] = {0x6a09e667, 0xbb67ae85, 0x3c6ef372, 0xa54ff53a, 0x510e527f, 0x9b05688c, 0x1f83d9ab, 0x5be0cd19};
  size_t full = n / 64;
  for (size_t i = 0; i < full; ++i) sha_block(h, data + 64 * i);
  uint8_t tail[128];
  size_t rem = n - 64 * full;
  memset(tail, 0, sizeof tail);
  memcpy(tail, data + 64 * full, rem);
  tail[rem] = 0x80;
  size_t tl = (rem + 9 <= 64) ? 64 : 128;
  uint64_t bits = (uint64_t)n * 8;
  for (int i = 0; i < 8; ++i) tail[tl - 1 - i] = (uint8_t)(bits >> (8 * i));
  sha_block(h, tail);
  if (tl == 128) sha_block(h, tail + 64);
  for (int i = 0; i < 8; ++i) { out[4 * i] = h[i] >> 24; out[4 * i + 1] = h[i] >> 16; out[4 * i + 2] = h[i] >> 8; out[4 * i + 3] = h[i]; }
}
/* Tree hash of a tensor's raw bytes (the per-step state hash; Appendix B only says "sharded canonical hash"):
 *   level 1: SHA-256 of every 4 KiB chunk of the data (the last chunk may be shorter);
 *   while more than 128 digests remain: SHA-256 of every 4 KiB block (128 digests) of the concatenated digests;
 *   root = SHA-256(remaining digests || u64le(nbytes)). */
static size_t hash_level(const uint8_t *data, size_t n, uint8_t *out) {
  size_t nc = (n + 4095) / 4096;
#pragma omp parallel for
  for (size_t c = 0; c < nc; ++c) {
    size_t len = (c + 1) * 4096 <= n ? 4096 : n - c * 4096;
    orc_sha256(data + c * 4096, len, out + 32 * c);
  }
  return nc;
}
void orc_tensor_hash(const uint8_t *data, size_t n, uint8_t out[32]) {
  size_t cap = ((n + 4095) / 4096) * 32 + 64;
  uint8_t *a = (uint8_t *)malloc(cap), *b = (uint8_t *)malloc(cap);
  size_t nc = hash_level(data, n, a);
  while (nc > 128) {
    nc = hash_level(a, nc * 32, b);
    uint8_t *t = a; a = b; b = t;
  }
  uint64_t nn = n;
  for (int i = 0; i < 8; ++i) a[nc * 32 + i] = (uint8_t)(nn >> (8 * i));
  orc_sha256(a, nc * 32 + 8, out);
  free(a); free(b);
}

/* ------------------------------------------------------------------ */
/* rotary position embedding (Sec. 3.1 "RoPE", theta = 5e5; the tables  */
/* are inputs of the step, generated once in float64 and rounded)       */
/* ------------------------------------------------------------------ */
/* x, y: bf16 [T, nh, 128]; position of token t is t mod S; cos, sin: f32 [S, 64].
 * Pairs are (i, i + 64):  y_i = x_i c_i - x_{i+64} s_i,  y_{i+64} = x_{i+64} c_i + x_i s_i,
 * every product rounded on its own; inverse != 0 rotates by the opposite angle (the backward pass). */
void orc_rope(const bf16_t *x, int T, int nh, int S, const float *cs, const float *sn, int inverse, bf16_t *y) {
#pragma omp parallel for
  for (int t = 0; t < T; ++t) {
    const float *c = cs + (size_t)(t % S) * 64, *s = sn + (size_t)(t % S) * 64;
    for (int h = 0; h < nh; ++h) {
      const bf16_t *xr = x + ((size_t)t * nh + h) * 128;
      bf16_t *yr = y + ((size_t)t * nh + h) * 128;
      for (int i = 0; i < 64; ++i) {
        float a = bf2f(xr[i]), b = bf2f(xr[i + 64]);
        float si = inverse ? -s[i] : s[i];
        float lo = fsub(fmul(a, c[i]), fmul(b, si));
        float hi = fadd(fmul(b, c[i]), fmul(a, si));
        yr[i] = f2bf(lo);
        yr[i + 64] = f2bf(hi);
      }
    }
  }
}
