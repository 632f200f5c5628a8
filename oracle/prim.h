/* CPU oracle -- TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, scalar C restatement of the arithmetic conventions of the
 * paper's reproducible-operations section (Sec. 2.1 "Reproducible Operations":
 * fixed reduction order, unfused multiply-add, subnormals flushed to zero).
 * Nothing in here is shared with the CUDA path and the product never links it.
 *
 * Conventions (each primitive is one IEEE-754 binary32 round-to-nearest-even
 * operation with flush-to-zero applied to its inputs and to its result):
 *   fadd/fsub/fmul/fdiv/fsqrt  - separate roundings, never fused
 *   fmax2/fmin2                - -0 orders below +0; a NaN operand is ignored (the
 *                                other operand is returned), so a running maximum
 *                                does not depend on where a NaN sits in the scan
 *   bf16 widen                 - exact;  narrow - RN-even on the top 16 bits
 *   det_sum                    - level-by-level adjacent pairwise tree; an odd
 *                                trailing element is carried up unchanged
 *   det_exp / det_log          - spelled-out sequences of the primitives above
 */
#ifndef ORACLE_PRIM_H
#define ORACLE_PRIM_H
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef uint16_t bf16_t;

static inline uint32_t f2u(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }
static inline float u2f(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }

/* Sec. 2.1 "Subnormals": every backend flushes subnormals identically.
 * Exponent field zero => signed zero. */
static inline float ftz(float x) {
  uint32_t u = f2u(x);
  return (u & 0x7f800000u) ? x : u2f(u & 0x80000000u);
}

/* Sec. 2.1 "Fused multiply-add": multiply and add round separately.  Built
 * with -ffp-contract=off and without any FMA-capable -march, so the compiler
 * has no fused instruction to pick. */
static inline float fadd(float a, float b) { return ftz(ftz(a) + ftz(b)); }
static inline float fsub(float a, float b) { return ftz(ftz(a) - ftz(b)); }
/* Products and quotients are flushed when their EXACT value is below 2^-126 in magnitude (tininess
 * judged before rounding): an exact value just under the smallest normal that IEEE rounding would
 * lift onto it is still flushed.  This is the "least permissive backend" of Sec. 2.1 "Subnormals";
 * sums and differences that small are exact, so the two ways of judging never differ for them. */
static inline float fmul(float a, float b) {
  double p = (double)ftz(a) * (double)ftz(b); /* exact: 48 significant bits */
  if (fabs(p) < 0x1p-126) return u2f((f2u(a) ^ f2u(b)) & 0x80000000u);
  return (float)p; /* one rounding of the exact product */
}
static inline float fdiv(float a, float b) {
  a = ftz(a); b = ftz(b);
  if (b != 0.0f && a != 0.0f && !isinf(b) && !isinf(a) && fabs((double)a) < ldexp(fabs((double)b), -126))
    return u2f((f2u(a) ^ f2u(b)) & 0x80000000u);
  return ftz(a / b);
}
static inline float fsqrt(float a) { return ftz(sqrtf(ftz(a))); }
static inline float fabs1(float a) { return u2f(f2u(ftz(a)) & 0x7fffffffu); }
static inline float fneg(float a) { return u2f(f2u(ftz(a)) ^ 0x80000000u); }
static inline float fmax2(float a, float b) {
  a = ftz(a); b = ftz(b);
  if (a != a) return b;                    /* a NaN operand is ignored (maxNum); two NaNs give NaN */
  if (b != b) return a;
  if (a == b) return u2f(f2u(a) & f2u(b)); /* max(-0,+0) = +0 */
  return a > b ? a : b;
}
static inline float fmin2(float a, float b) {
  a = ftz(a); b = ftz(b);
  if (a != a) return b;
  if (b != b) return a;
  if (a == b) return u2f(f2u(a) | f2u(b)); /* min(-0,+0) = -0 */
  return a < b ? a : b;
}
/* round to nearest integer, ties to even (default rounding mode) */
static inline float frne(float a) { return rintf(ftz(a)); }
static inline float i2f(int32_t v) { return (float)v; } /* RN-even above 2^24 */

static inline float bf2f(bf16_t h) { return u2f((uint32_t)h << 16); }
static inline bf16_t f2bf(float x) {
  uint32_t u = f2u(ftz(x));
  if ((u & 0x7fffffffu) > 0x7f800000u) return 0x7fff; /* NaN: out of contract */
  u += 0x7fffu + ((u >> 16) & 1u);
  return (bf16_t)(u >> 16);
}

/* Fixed pairwise tree (Sec. 2.1 "Reduction order"; same binary-carry shape as
 * Algorithm 2 applied to elements).  next[i] = cur[2i] + cur[2i+1]; an odd
 * last element moves up unchanged; n == 0 gives +0. */
static inline float det_sum(const float *x, size_t n) {
  if (n == 0) return 0.0f;
  if (n == 1) return ftz(x[0]);
  size_t m = (n + 1) / 2;
  float *t = (float *)malloc(m * sizeof(float));
  for (size_t i = 0; i < n / 2; ++i) t[i] = fadd(x[2 * i], x[2 * i + 1]);
  if (n & 1) t[m - 1] = ftz(x[n - 1]);
  n = m;
  while (n > 1) {
    m = (n + 1) / 2;
    for (size_t i = 0; i < n / 2; ++i) t[i] = fadd(t[2 * i], t[2 * i + 1]);
    if (n & 1) t[m - 1] = t[n - 1];
    n = m;
  }
  float r = t[0];
  free(t);
  return r;
}

/* exp: range reduction x = k ln2 + r, degree-7 Taylor polynomial in Horner
 * form (one fmul and one fadd per step), scaling through the exponent field. */
static inline float det_exp(float x) {
  x = ftz(x);
  if (x > 0x1.62e42ep+6f) return INFINITY;
  if (x < -0x1.5d58a0p+6f) return 0.0f;
  float kf = frne(fmul(x, 0x1.715476p+0f));
  float r = fsub(fsub(x, fmul(kf, 0x1.62e400p-1f)), fmul(kf, 0x1.7f7d1cp-20f));
  float p = 0x1.a01a02p-13f;          /* 1/5040 */
  p = fadd(fmul(p, r), 0x1.6c16c2p-10f); /* 1/720 */
  p = fadd(fmul(p, r), 0x1.111112p-7f);  /* 1/120 */
  p = fadd(fmul(p, r), 0x1.555556p-5f);  /* 1/24 */
  p = fadd(fmul(p, r), 0x1.555556p-3f);  /* 1/6 */
  p = fadd(fmul(p, r), 0.5f);
  p = fadd(fmul(p, r), 1.0f);
  p = fadd(fmul(p, r), 1.0f);
  int k = (int)kf;
  if (k > 127) return fmul(fmul(p, 0x1p127f), 2.0f);
  return fmul(p, u2f((uint32_t)(k + 127) << 23));
}

/* log: the ends of the domain first (0 -> -inf, +inf -> +inf, negative or NaN -> NaN; a flushed subnormal is 0), so that
 * a non-finite operand stays visible instead of turning into an arbitrary finite number; then for normal x > 0: x = 2^e m, m in (sqrt(1/2), sqrt(2)], s = (m-1)/(m+1),
 * log m = 2s (1 + z/3 + z^2/5 + z^3/7 + z^4/9), z = s^2. */
static inline float det_log(float x) {
  x = ftz(x);
  if (!(x > 0.0f)) return x == 0.0f ? -INFINITY : NAN;   /* log 0 = -inf; a negative argument or a NaN gives NaN */
  if (x == INFINITY) return x;
  uint32_t u = f2u(x);
  int e = (int)(u >> 23) - 127;
  float m = u2f((u & 0x007fffffu) | 0x3f800000u);
  if (m > 0x1.6a09e6p+0f) { m = fmul(m, 0.5f); e += 1; }
  float f = fsub(m, 1.0f);
  float s = fdiv(f, fadd(2.0f, f));
  float z = fmul(s, s);
  float p = 0x1.c71c72p-4f;             /* 1/9 */
  p = fadd(fmul(p, z), 0x1.24924ap-3f); /* 1/7 */
  p = fadd(fmul(p, z), 0x1.99999ap-3f); /* 1/5 */
  p = fadd(fmul(p, z), 0x1.555556p-2f); /* 1/3 */
  p = fadd(fmul(p, z), 1.0f);
  float lm = fmul(fmul(2.0f, s), p);
  float ef = i2f(e);
  return fadd(fmul(ef, 0x1.62e400p-1f), fadd(lm, fmul(ef, 0x1.7f7d1cp-20f)));
}

#endif
