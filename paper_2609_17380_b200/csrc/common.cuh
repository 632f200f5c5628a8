// Device-side arithmetic conventions of libdet (Sec. 2.1 "Reproducible Operations").
//
// The library is compiled with -fmad=false -ftz=true -prec-div=true -prec-sqrt=true, and every
// floating-point operation whose rounding matters is written with the explicit round-to-nearest
// intrinsics, so that no multiply-add is ever contracted and subnormal inputs/results are flushed.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/det.h"

#define DET_CHECK_LAUNCH()                                   \
  do {                                                       \
    if (cudaPeekAtLastError() != cudaSuccess) {              \
      cudaGetLastError();                                    \
      return DET_ERR_CUDA;                                   \
    }                                                        \
  } while (0)

namespace det {

__device__ __forceinline__ float fadd(float a, float b) { return __fadd_rn(a, b); }
__device__ __forceinline__ float fsub(float a, float b) { return __fsub_rn(a, b); }
__device__ __forceinline__ float fmul(float a, float b) { return __fmul_rn(a, b); }
__device__ __forceinline__ float fdiv(float a, float b) { return __fdiv_rn(a, b); }
__device__ __forceinline__ float fsqrt(float a) { return __fsqrt_rn(a); }

// bf16 <-> f32 on raw bit patterns.  Widening is exact; narrowing is round-to-nearest-even.
__device__ __forceinline__ float bf2f(uint16_t h) { return __uint_as_float(((uint32_t)h) << 16); }
__device__ __forceinline__ float bflo(uint32_t pair) { return __uint_as_float(pair << 16); }
__device__ __forceinline__ float bfhi(uint32_t pair) { return __uint_as_float(pair & 0xffff0000u); }
__device__ __forceinline__ uint16_t f2bf(float x) { return __bfloat16_as_ushort(__float2bfloat16_rn(x)); }
__device__ __forceinline__ uint32_t pack_bf2(float lo, float hi) {
  return (uint32_t)f2bf(lo) | ((uint32_t)f2bf(hi) << 16);
}

// LSQ quantiser (Sec. 3.1): code = rne(clamp(v * (1/s), -128, 127)); the reciprocal is one division per step size.
__device__ __forceinline__ int8_t quant1(float v, float inv_s) {
  float t = fminf(fmaxf(__fmul_rn(v, inv_s), -128.0f), 127.0f);
  return (int8_t)__float2int_rn(t);
}
// eight values -> eight codes packed low byte first
__device__ __forceinline__ uint2 quant8(const float v[8], float inv_s) {
  uint2 o;
  o.x = ((uint32_t)(uint8_t)quant1(v[0], inv_s)) | ((uint32_t)(uint8_t)quant1(v[1], inv_s) << 8) |
        ((uint32_t)(uint8_t)quant1(v[2], inv_s) << 16) | ((uint32_t)(uint8_t)quant1(v[3], inv_s) << 24);
  o.y = ((uint32_t)(uint8_t)quant1(v[4], inv_s)) | ((uint32_t)(uint8_t)quant1(v[5], inv_s) << 8) |
        ((uint32_t)(uint8_t)quant1(v[6], inv_s) << 16) | ((uint32_t)(uint8_t)quant1(v[7], inv_s) << 24);
  return o;
}

// exp: x = k ln2 + r, degree-7 Taylor polynomial in Horner form, one multiply and one add per step,
// scaled through the exponent field.  Results below 2^-126 flush to +0; above FLT_MAX give +inf.
// Written without branches: the special ranges are chosen by selects, so that several independent evaluations
// interleave in one instruction stream (a kernel that evaluates many exponentials per thread is bound by the latency
// of this chain, not by its instruction count).
//   k = rne(x log2 e): adding 1.5 * 2^23 rounds to the nearest even integer exactly like rintf for |t| < 2^22 (here
//   |t| < 2^8 wherever the result is kept) and leaves k in the low bits of the sum, so neither the rounding nor the
//   conversion needs the conversion pipe.
__device__ __forceinline__ float det_exp(float x) {
  const float km = fadd(fmul(x, 0x1.715476p+0f), 12582912.0f);
  const float kf = fsub(km, 12582912.0f);
  const float r = fsub(fsub(x, fmul(kf, 0x1.62e400p-1f)), fmul(kf, 0x1.7f7d1cp-20f));
  float p = 0x1.a01a02p-13f;
  p = fadd(fmul(p, r), 0x1.6c16c2p-10f);
  p = fadd(fmul(p, r), 0x1.111112p-7f);
  p = fadd(fmul(p, r), 0x1.555556p-5f);
  p = fadd(fmul(p, r), 0x1.555556p-3f);
  p = fadd(fmul(p, r), 0.5f);
  p = fadd(fmul(p, r), 1.0f);
  p = fadd(fmul(p, r), 1.0f);
  const int k = (int)__float_as_uint(km) - 0x4B400000;
  const float big = fmul(fmul(p, 0x1p127f), 2.0f);                              // k = 128
  float v = fmul(p, __int_as_float((min(max(k, -127), 127) + 127) << 23));      // k in [-126, 127] wherever v is kept
  v = (k > 127) ? big : v;
  v = (x < -0x1.5d58a0p+6f) ? 0.0f : v;
  v = (x > 0x1.62e42ep+6f) ? __int_as_float(0x7f800000) : v;
  return v;
}

// The same function for arguments that are never positive (x <= 0, or NaN): a softmax argument z - max.  There k <= 0, so
// neither the k = 128 product nor the overflow select can be chosen and the upper clamp of k never binds; what is left
// is the same sequence, so every result has the bits det_exp gives.  For x > 0 the value is unspecified (no trap).
__device__ __forceinline__ float det_exp_le0(float x) {
  const float km = fadd(fmul(x, 0x1.715476p+0f), 12582912.0f);
  const float kf = fsub(km, 12582912.0f);
  const float r = fsub(fsub(x, fmul(kf, 0x1.62e400p-1f)), fmul(kf, 0x1.7f7d1cp-20f));
  float p = 0x1.a01a02p-13f;
  p = fadd(fmul(p, r), 0x1.6c16c2p-10f);
  p = fadd(fmul(p, r), 0x1.111112p-7f);
  p = fadd(fmul(p, r), 0x1.555556p-5f);
  p = fadd(fmul(p, r), 0x1.555556p-3f);
  p = fadd(fmul(p, r), 0.5f);
  p = fadd(fmul(p, r), 1.0f);
  p = fadd(fmul(p, r), 1.0f);
  // 2^k: the bits of km are 0x4B400000 + k and 0x4B400000 << 23 is 0 mod 2^32, so k << 23 needs no subtraction; and
  // wherever the result is kept (x at or above the flush threshold) k >= -126, so k needs no lower clamp either
  const float v = fmul(p, __int_as_float((int)(__float_as_uint(km) << 23) + 0x3f800000));
  return (x < -0x1.5d58a0p+6f) ? 0.0f : v;
}

// NOTE on the packed two-lane FP32 instructions (mul/add/fma .f32x2): each lane of a single packed instruction
// rounds exactly like the scalar instruction, but ptxas contracts a packed multiply followed by a packed add into one
// fused instruction even when both carry .rn and --fmad=false is given (measured on this toolchain: the result
// equals the true fused multiply-add in every lane).  Packed arithmetic is therefore used only where a fused
// multiply-add is wanted and proven identical; every multiply-then-add whose product must be rounded on its own is
// written with the scalar intrinsics, which ptxas never contracts.

// log: for normal x > 0, x = 2^e m, m in (sqrt(1/2), sqrt(2)], s = (m-1)/(m+1), z = s^2,
// log m = 2 s (1 + z/3 + z^2/5 + z^3/7 + z^4/9).
__device__ __forceinline__ float det_log(float x) {
  // the ends of the domain first: 0 (a flushed subnormal included) -> -inf, +inf -> +inf, negative or NaN -> NaN
  // (comparisons flush subnormal operands like every other instruction here)
  if (!(x > 0.0f)) return x == 0.0f ? __int_as_float(0xff800000) : __int_as_float(0x7fffffff);
  if (x == __int_as_float(0x7f800000)) return x;
  uint32_t u = __float_as_uint(x);
  int e = (int)(u >> 23) - 127;
  float m = __uint_as_float((u & 0x007fffffu) | 0x3f800000u);
  if (m > 0x1.6a09e6p+0f) { m = fmul(m, 0.5f); e += 1; }
  float f = fsub(m, 1.0f);
  float s = fdiv(f, fadd(2.0f, f));
  float z = fmul(s, s);
  float p = 0x1.c71c72p-4f;
  p = fadd(fmul(p, z), 0x1.24924ap-3f);
  p = fadd(fmul(p, z), 0x1.99999ap-3f);
  p = fadd(fmul(p, z), 0x1.555556p-2f);
  p = fadd(fmul(p, z), 1.0f);
  float lm = fmul(fmul(2.0f, s), p);
  float ef = __int2float_rn(e);
  return fadd(fmul(ef, 0x1.62e400p-1f), fadd(lm, fmul(ef, 0x1.7f7d1cp-20f)));
}

// ---------------------------------------------------------------------------------------------
// The fixed pairwise tree.  A node of the tree covers an aligned range of 2^l element indices; it
// exists iff its first index is < n.  Combining a left node with a right node that does not exist
// carries the left value up unchanged; this reproduces the level-by-level "odd element is carried"
// rule for any n, and aligned power-of-two blocks are perfect subtrees.
// ---------------------------------------------------------------------------------------------

// Tree over 8 adjacent values held by one lane; element index of v[0] is `first`, valid iff < n.
__device__ __forceinline__ float tree8(const float v[8], long long first, long long n) {
  float a0 = (first + 1 < n) ? fadd(v[0], v[1]) : v[0];
  float a1 = (first + 3 < n) ? fadd(v[2], v[3]) : v[2];
  float a2 = (first + 5 < n) ? fadd(v[4], v[5]) : v[4];
  float a3 = (first + 7 < n) ? fadd(v[6], v[7]) : v[6];
  float b0 = (first + 2 < n) ? fadd(a0, a1) : a0;
  float b1 = (first + 6 < n) ? fadd(a2, a3) : a2;
  return (first + 4 < n) ? fadd(b0, b1) : b0;
}
__device__ __forceinline__ float tree8_full(const float v[8]) {
  return fadd(fadd(fadd(v[0], v[1]), fadd(v[2], v[3])), fadd(fadd(v[4], v[5]), fadd(v[6], v[7])));
}

// Butterfly over the 32 lanes of a warp: lane l holds the node that starts at element
// `leaf_first + l*stride` (stride = elements per lane).  All lanes end with the warp's node value.
__device__ __forceinline__ float warp_tree(float v, long long leaf_first, long long stride, long long n) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int w = 1; w < 32; w <<= 1) {
    float o = __shfl_xor_sync(0xffffffffu, v, w);
    int right_lane = (lane | w) & ~(w - 1);
    bool right_valid = leaf_first + (long long)right_lane * stride < n;
    bool i_am_left = !(lane & w);
    v = right_valid ? fadd(v, o) : (i_am_left ? v : o);
  }
  return v;
}
__device__ __forceinline__ float warp_tree_full(float v) {
#pragma unroll
  for (int w = 1; w < 32; w <<= 1) v = fadd(v, __shfl_xor_sync(0xffffffffu, v, w));
  return v;
}

// Tree over `cnt` (power of two, <= 32) node values s[0..cnt) held redundantly in registers; node j
// starts at element first + j*stride.
template <int CNT>
__device__ __forceinline__ float reg_tree(float (&s)[CNT], long long first, long long stride, long long n) {
#pragma unroll
  for (int w = 1; w < CNT; w <<= 1)
#pragma unroll
    for (int j = 0; j < CNT; j += 2 * w)
      s[j] = (first + (long long)(j + w) * stride < n) ? fadd(s[j], s[j + w]) : s[j];
  return s[0];
}

// Level-by-level tree over an array in shared memory (any length, carry rule); all threads of the
// CTA must call it; buf is overwritten; result in buf[0] after the call.
__device__ __forceinline__ void smem_tree(float* buf, int n) {
  while (n > 1) {
    int half = n >> 1, m = (n + 1) >> 1;
    float v = 0.0f;
    bool act = (int)threadIdx.x < m;
    // one thread per output; supports n up to 2*blockDim.x
    if (act) v = ((int)threadIdx.x < half) ? fadd(buf[2 * threadIdx.x], buf[2 * threadIdx.x + 1]) : buf[n - 1];
    __syncthreads();
    if (act) buf[threadIdx.x] = v;
    __syncthreads();
    n = m;
  }
}

__device__ __forceinline__ void or_status(int* status, int bit) {
  if (status) atomicOr(status, bit);
}

static inline bool aligned16(const void* p) { return (((uintptr_t)p) & 15u) == 0; }
static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace det
