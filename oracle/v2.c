/* CPU oracle, arithmetic version 2 -- TEST INFRASTRUCTURE ONLY (tests and the timed cpu baseline; never the product path).
 *
 * Version 2 changes ONE definition of the step: the full-precision contraction of the LM head (Sec. 3.2: the head stays
 * out of quantisation) becomes order-free and exactly defined instead of an ordered chain of binary32 roundings, built
 * from the paper's own two devices: integer products of aligned significands that are exact in int32 (Sec. 3.2 "int8
 * computation") and a wide exact integer total that cannot depend on the order of its terms (Sec. 3.2: the query
 * gradient "in 64-bit fixed point for bitwise reproducibility").  Nothing else of version 1 changes.
 *
 *   row exponent   E(x) = the largest biased exponent field among the bf16 values of the row (0 for an all-zero row;
 *                  subnormal bf16 values count as zero, Sec. 2.1 "Subnormal handling")
 *   aligned value  T_k  = ((128 + fraction_k) << 6) >> (E - E_k), a 14-bit magnitude with the sign of x_k (0 if x_k = 0):
 *                  x_k is replaced by T_k 2^(E - 140); values within 2^-6 of the row's largest keep every bit, smaller
 *                  ones are truncated toward zero, and those more than 2^-14 below it vanish
 *   slices         T_k = 128 hi_k + lo_k, hi_k = T_k >> 7, lo_k = T_k & 127 (both carry the sign), each an int8
 *   contraction    I = sum_k Ta_k Tb_k = 2^14 sum(ha hb) + 2^7 (sum(ha lb) + sum(la hb)) + sum(la lb), exact integers in
 *                  any order (each of the four sums fits int32 for K < 2^17, the total fits int64)
 *   result         binary32 nearest-even rounding of I 2^(E(a) + E(b) - 280), ONE rounding; a result below 2^-126 in
 *                  magnitude after that rounding is a signed zero; a row that holds an infinity or a NaN gives NaN
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include "prim.h" /* the version-1 primitives that version 2 keeps: binary32 operations with flushing, det_sum, det_exp, det_log */

/* row exponent; *bad is set when the row holds an infinity or a NaN */
static int row_exponent(const bf16_t *x, int K, int *bad) {
  int e = 0;
  *bad = 0;
  for (int k = 0; k < K; ++k) {
    int ek = (x[k] >> 7) & 0xFF;
    if (ek == 255) *bad = 1;
    if (ek > e) e = ek;
  }
  return e;
}

/* signed aligned 14-bit value of one element against the row exponent E */
static int aligned(bf16_t h, int E) {
  int ek = (h >> 7) & 0xFF;
  if (ek == 0) return 0; /* zero or flushed subnormal */
  int d = E - ek;
  if (d >= 14) return 0;
  int t = ((128 + (h & 0x7F)) << 6) >> d;
  return (h & 0x8000) ? -t : t;
}

/* X bf16 [R,K] -> hi, lo int8 [R,K], E int32 [R] (row exponent; bit 30 set for a row with a non-finite value) */
void orc2_slice_rows(const bf16_t *X, int R, int K, int8_t *hi, int8_t *lo, int32_t *E) {
#pragma omp parallel for
  for (int r = 0; r < R; ++r) {
    int bad;
    const bf16_t *x = X + (size_t)r * K;
    int e = row_exponent(x, K, &bad);
    E[r] = e | (bad ? (1 << 30) : 0);
    for (int k = 0; k < K; ++k) {
      int t = aligned(x[k], e);
      int m = t < 0 ? -t : t;
      int h = m >> 7, l = m & 127;
      hi[(size_t)r * K + k] = (int8_t)(t < 0 ? -h : h);
      lo[(size_t)r * K + k] = (int8_t)(t < 0 ? -l : l);
    }
  }
}

/* the one rounding of the definition: I 2^e as binary32, nearest even, then flush */
static float round_scaled(int64_t I, int e) {
  double v = ldexp((double)I, e); /* exact: |I| < 2^53 and the scaled value is a normal double */
  float r = (float)v;             /* IEEE nearest-even (default rounding mode) */
  if (fabsf(r) < 0x1p-126f) r = copysignf(0.0f, r);
  return r;
}

/* logits[m,n] = version-2 contraction of row m of H with row n of W (both bf16 [.,K]) */
void orc2_lmhead_fwd(const bf16_t *H, const bf16_t *W, int M, int V, int K, float *logits) {
  int32_t *Ta = (int32_t *)malloc((size_t)M * K * sizeof(int32_t));
  int32_t *Tb = (int32_t *)malloc((size_t)V * K * sizeof(int32_t));
  int *Ea = (int *)malloc((size_t)M * sizeof(int)), *Eb = (int *)malloc((size_t)V * sizeof(int));
  int *Ba = (int *)malloc((size_t)M * sizeof(int)), *Bb = (int *)malloc((size_t)V * sizeof(int));
#pragma omp parallel for
  for (int m = 0; m < M; ++m) {
    Ea[m] = row_exponent(H + (size_t)m * K, K, &Ba[m]);
    for (int k = 0; k < K; ++k) Ta[(size_t)m * K + k] = aligned(H[(size_t)m * K + k], Ea[m]);
  }
#pragma omp parallel for
  for (int n = 0; n < V; ++n) {
    Eb[n] = row_exponent(W + (size_t)n * K, K, &Bb[n]);
    for (int k = 0; k < K; ++k) Tb[(size_t)n * K + k] = aligned(W[(size_t)n * K + k], Eb[n]);
  }
#pragma omp parallel for
  for (int m = 0; m < M; ++m)
    for (int n = 0; n < V; ++n) {
      if (Ba[m] || Bb[n]) {
        uint32_t q = 0x7FC00000u;
        memcpy(&logits[(size_t)m * V + n], &q, 4);
        continue;
      }
      int64_t I = 0;
      for (int k = 0; k < K; ++k) I += (int64_t)Ta[(size_t)m * K + k] * (int64_t)Tb[(size_t)n * K + k];
      logits[(size_t)m * V + n] = round_scaled(I, Ea[m] + Eb[n] - 280);
    }
  free(Ta); free(Tb); free(Ea); free(Eb); free(Ba); free(Bb);
}

/* ------------------------------------------------------------------------------------------------------------------
 * Causal attention in arithmetic version 2 (head dimension 128, one key/value head per query head, no window).
 *
 * Version 1 defines the logits, P.V and the online rescaling as ordered chains of binary32 roundings.  Version 2 keeps the
 * softmax arithmetic of version 1 (binary32, det_exp, det_sum, det_log) and replaces the two contractions by the
 * order-free contraction defined at the top of this file; with no order to respect there are no key tiles and no
 * rescaling: a row takes its maximum over all of its keys first.
 *
 *   s_ij  = fmul(C(q_i, k_j), 2^-3.5 rounded to binary32)        j <= i; C = the version-2 contraction over the 128 dimensions,
 *                                                                row exponents over the 128 values of q_i and of k_j
 *   m_i   = max_j s_ij,  p_ij = det_exp(s_ij - m_i),  l_i = det_sum(p_i0 .. p_ii),  lse_i = m_i + det_log(l_i)
 *   P~_ij = bf16(p_ij)                                            (as in version 1; 0 for j > i)
 *   u_ic  = C(P~_i., v_.c) over the keys 0 .. i                   exponent of row i of P~ over its keys, exponent of column c
 *                                                                of v over ALL keys of the sequence (so that it is shared
 *                                                                by every query)
 *   o_ic  = bf16(fmul(u_ic, fdiv(1, l_i)))
 * ------------------------------------------------------------------------------------------------------------------ */
#define A2_SCALE 0x1.6a09e6p-4f /* 1/sqrt(128) rounded to binary32 */

/* exponent over n values spaced `stride` apart; *bad as in row_exponent */
static int strided_exponent(const bf16_t *x, size_t stride, int n, int *bad) {
  int e = 0;
  *bad = 0;
  for (int k = 0; k < n; ++k) {
    int ek = (x[(size_t)k * stride] >> 7) & 0xFF;
    if (ek == 255) *bad = 1;
    if (ek > e) e = ek;
  }
  return e;
}
/* the version-2 contraction of n values of a (stride sa, exponent ea) with n values of b (stride sb, exponent eb) */
static float contract2(const bf16_t *a, size_t sa, int ea, const bf16_t *b, size_t sb, int eb, int n) {
  int64_t I = 0;
  for (int k = 0; k < n; ++k) I += (int64_t)aligned(a[(size_t)k * sa], ea) * (int64_t)aligned(b[(size_t)k * sb], eb);
  return round_scaled(I, ea + eb - 280);
}
static float quiet_nan(void) { uint32_t q = 0x7FC00000u; float f; memcpy(&f, &q, 4); return f; }

void orc2_attn_fwd(const bf16_t *q, const bf16_t *k, const bf16_t *v, int ld, int B, int H, int S, bf16_t *out, int ld_out,
                   float *lse) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int bh = 0; bh < B * H; ++bh) {
    const int b = bh / H, h = bh % H;
    const bf16_t *qb = q + (size_t)ld * b * S + h * 128, *kb = k + (size_t)ld * b * S + h * 128;
    const bf16_t *vb = v + (size_t)ld * b * S + h * 128;
    int *Eq = (int *)malloc(S * sizeof(int)), *Ek = (int *)malloc(S * sizeof(int));
    int *Bq = (int *)malloc(S * sizeof(int)), *Bk = (int *)malloc(S * sizeof(int));
    int Ev[128], Bv[128];
    for (int i = 0; i < S; ++i) {
      Eq[i] = row_exponent(qb + (size_t)ld * i, 128, &Bq[i]);
      Ek[i] = row_exponent(kb + (size_t)ld * i, 128, &Bk[i]);
    }
    for (int c = 0; c < 128; ++c) Ev[c] = strided_exponent(vb + c, (size_t)ld, S, &Bv[c]);
    float *s = (float *)malloc(S * sizeof(float)), *p = (float *)malloc(S * sizeof(float));
    bf16_t *pt = (bf16_t *)malloc(S * sizeof(bf16_t));
    for (int i = 0; i < S; ++i) {
      float m = -INFINITY;
      for (int j = 0; j <= i; ++j) {
        float c = (Bq[i] || Bk[j]) ? quiet_nan() : contract2(qb + (size_t)ld * i, 1, Eq[i], kb + (size_t)ld * j, 1, Ek[j], 128);
        s[j] = fmul(c, A2_SCALE);
        m = fmax2(m, s[j]);
      }
      for (int j = 0; j <= i; ++j) {
        p[j] = det_exp(fsub(s[j], m));
        pt[j] = f2bf(p[j]);
      }
      float l = det_sum(p, (size_t)i + 1);
      int bp, ep = row_exponent(pt, i + 1, &bp);
      float il = fdiv(1.0f, l);
      for (int c = 0; c < 128; ++c) {
        float u = (bp || Bv[c]) ? quiet_nan() : contract2(pt, 1, ep, vb + c, (size_t)ld, Ev[c], i + 1);
        out[(size_t)ld_out * (b * S + i) + h * 128 + c] = f2bf(fmul(u, il));
      }
      lse[(size_t)bh * S + i] = fadd(m, det_log(l));
    }
    free(Eq); free(Ek); free(Bq); free(Bk); free(s); free(p); free(pt);
  }
}
