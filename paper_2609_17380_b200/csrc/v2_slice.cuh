// Arithmetic version 2: the aligned 14-bit value of a bf16 number against the exponent of its row, as two int8 slices
// (shared by the LM head and the attention of version 2).
#pragma once
#include "common.cuh"

namespace det {

// bf16 bit pattern of a binary32 value (subnormal inputs flushed first), as the gradient of the logits is rounded
__device__ __forceinline__ uint32_t bf_bits(float x) {
  if (!(__float_as_uint(x) & 0x7f800000u)) x = __uint_as_float(__float_as_uint(x) & 0x80000000u);
  return (uint32_t)f2bf(x);
}
// signed 14-bit aligned value of one bf16 pattern against the exponent e of its row, as two int8 slices
__device__ __forceinline__ void slice1(uint32_t b, int e, int& h, int& l) {
  const int ek = (b >> 7) & 0xFF, d = e - ek;
  const int t = (ek == 0 || d >= 14) ? 0 : (int)(((128u + (b & 0x7Fu)) << 6) >> d);
  h = t >> 7; l = t & 127;
  if (b & 0x8000u) { h = -h; l = -l; }
}

}  // namespace det
