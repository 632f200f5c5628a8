// LSQ int8 linear layer around the tensor-core GEMM: step sizes, quantisers, Walsh-Hadamard operand
// preparation for the two gradient GEMMs, and the det_linear_fwd / det_linear_bwd entry points
// (Sec. 3.1 "int8 quantization-aware training", Sec. 3.2 "int8 computation", Sec. 4.4 step re-pin).
#include "common.cuh"
#include "internal.h"

namespace det {

#define C127 0x1.6b7612p-4f

__device__ __forceinline__ void unpack8u(const uint4& u, float v[8]) {
  v[0] = bflo(u.x); v[1] = bfhi(u.x); v[2] = bflo(u.y); v[3] = bfhi(u.y);
  v[4] = bflo(u.z); v[5] = bfhi(u.z); v[6] = bflo(u.w); v[7] = bfhi(u.w);
}

// ---- step sizes -------------------------------------------------------------------------------
// per output channel: one warp per row of W, K <= 8192
__global__ void __launch_bounds__(256) k_wscale_rows(const uint16_t* __restrict__ W, int N, int K, float invK,
                                                     float* __restrict__ s_w) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = blockIdx.x * 8 + warp;
  if (row >= N) return;
  const int nl = (K + 255) >> 8;
  float mine = 0.0f;
  for (int j = 0; j < nl; ++j) {
    const int e0 = j * 256 + lane * 8;
    float v[8];
    if (e0 < K) {
      unpack8u(*reinterpret_cast<const uint4*>(W + (size_t)row * K + e0), v);
#pragma unroll
      for (int t = 0; t < 8; ++t) v[t] = fabsf(v[t]);
    } else {
#pragma unroll
      for (int t = 0; t < 8; ++t) v[t] = 0.0f;
    }
    float leaf = warp_tree(tree8_full(v), (long long)j * 256, 8, K);
    if (lane == j) mine = leaf;
  }
  float s = warp_tree(mine, 0, 256, K);
  s = fmaxf(fmul(fmul(2.0f, fmul(s, invK)), C127), 0x1p-40f);
  if (lane == 0) s_w[row] = s;
}

// chunk sums of |x| over a flat bf16 tensor (chunk = 16384 elements), same tree as det_sum
__global__ void __launch_bounds__(256) k_abs_chunk(const uint16_t* __restrict__ x, long long n, float* __restrict__ partial) {
  __shared__ float wsum[8];
  const long long base = (long long)blockIdx.x * 16384;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float s[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const long long lf = base + (warp * 8 + j) * 256;
    const long long e0 = lf + lane * 8;
    float v[8];
    if (e0 + 8 <= n) {
      unpack8u(*reinterpret_cast<const uint4*>(x + e0), v);
    } else {
#pragma unroll
      for (int t = 0; t < 8; ++t) v[t] = (e0 + t < n) ? bf2f(x[e0 + t]) : 0.0f;
    }
#pragma unroll
    for (int t = 0; t < 8; ++t) v[t] = fabsf(v[t]);
    s[j] = warp_tree(tree8(v, e0, n), lf, 8, n);
  }
  float r = reg_tree<8>(s, base + (long long)warp * 2048, 256, n);
  if (lane == 0) wsum[warp] = r;
  __syncthreads();
  if (threadIdx.x == 0) {
    float w[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) w[j] = wsum[j];
    partial[blockIdx.x] = reg_tree<8>(w, base, 2048, n);
  }
}
__global__ void k_scale_finish(const float* sum, float inv_n, float* out, int count) {
  const float s = fmaxf(fmul(fmul(2.0f, fmul(sum[0], inv_n)), C127), 0x1p-40f);
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < count; i += gridDim.x * blockDim.x) out[i] = s;
}

// ---- quantisers ---------------------------------------------------------------------------------
// rows x cols bf16 -> int8, step per row (per_row) or one step for the tensor; cols % 16 == 0
__global__ void __launch_bounds__(256) k_quantize(const uint16_t* __restrict__ X, size_t n16, int cols16,
                                                  const float* __restrict__ s, int per_row, int8_t* __restrict__ q) {
  size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= n16) return;
  const float inv = fdiv(1.0f, s[per_row ? (i / cols16) : 0]);
  const uint4* p = reinterpret_cast<const uint4*>(X) + 2 * i;
  float a[8], b[8];
  unpack8u(__ldg(p), a);
  unpack8u(__ldg(p + 1), b);
  uint32_t o[4];
#pragma unroll
  for (int w = 0; w < 2; ++w) {
    o[w] = ((uint32_t)(uint8_t)quant1(a[4 * w], inv)) | ((uint32_t)(uint8_t)quant1(a[4 * w + 1], inv) << 8) |
           ((uint32_t)(uint8_t)quant1(a[4 * w + 2], inv) << 16) | ((uint32_t)(uint8_t)quant1(a[4 * w + 3], inv) << 24);
    o[2 + w] = ((uint32_t)(uint8_t)quant1(b[4 * w], inv)) | ((uint32_t)(uint8_t)quant1(b[4 * w + 1], inv) << 8) |
               ((uint32_t)(uint8_t)quant1(b[4 * w + 2], inv) << 16) | ((uint32_t)(uint8_t)quant1(b[4 * w + 3], inv) << 24);
  }
  reinterpret_cast<uint4*>(q)[i] = make_uint4(o[0], o[1], o[2], o[3]);
}

// ---- Walsh-Hadamard operand preparation -----------------------------------------------------------
// Unnormalised butterflies, stages h = 1..64, (a, b) -> (a + b, a - b) for index pairs (i, i + h).

// (1) rotation along the row (contiguous) direction: A = rotate_n(dY[m,n] * s_w[n]).
//     A warp owns one 128-element block: a lane holds 4 adjacent elements (stages 1, 2 in registers,
//     stages 4..64 by shuffles).  PASS 0 records the absmax, PASS 1 quantises.
template <int PASS, bool ROT>
__global__ void __launch_bounds__(256) k_rot_rows(const uint16_t* __restrict__ dY, const float* __restrict__ s_w, int M,
                                                  int N, uint32_t* __restrict__ amax, int8_t* __restrict__ Aq) {
  // a warp owns RB consecutive 128-element blocks of one row and issues all its loads before any arithmetic
  constexpr int RB = 8;
  const int lane = threadIdx.x & 31;
  const int gpr = (N / 128 + RB - 1) / RB;  // warp groups per row
  const size_t grp = (size_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  float local = 0.0f;
  if (grp < (size_t)M * gpr) {
    const size_t m = grp / gpr;
    const int nb0 = (int)(grp % gpr) * RB;  // first 128-block of this group
    uint2 u[RB];
    float4 w[RB];
#pragma unroll
    for (int r = 0; r < RB; ++r) {
      const int n0 = (nb0 + r) * 128 + lane * 4;
      if (n0 < N) {
        u[r] = __ldg(reinterpret_cast<const uint2*>(dY + m * N + n0));
        w[r] = __ldg(reinterpret_cast<const float4*>(s_w + n0));
      } else {
        u[r] = make_uint2(0u, 0u);
        w[r] = make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
    float inv = 0.0f;
    if (PASS == 1) {
      const float am = __uint_as_float(amax[0]);
      inv = (am > 0.0f) ? fdiv(127.0f, am) : 0.0f;
    }
#pragma unroll
    for (int r = 0; r < RB; ++r) {
      const int n0 = (nb0 + r) * 128 + lane * 4;
      float v[4] = {fmul(bflo(u[r].x), w[r].x), fmul(bfhi(u[r].x), w[r].y), fmul(bflo(u[r].y), w[r].z), fmul(bfhi(u[r].y), w[r].w)};
      if (ROT) {
        float a0 = fadd(v[0], v[1]), a1 = fsub(v[0], v[1]), a2 = fadd(v[2], v[3]), a3 = fsub(v[2], v[3]);
        v[0] = fadd(a0, a2); v[2] = fsub(a0, a2); v[1] = fadd(a1, a3); v[3] = fsub(a1, a3);
#pragma unroll
        for (int hl = 1; hl < 32; hl <<= 1) {
          const bool upper = lane & hl;
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            float o = __shfl_xor_sync(0xffffffffu, v[e], hl);
            v[e] = upper ? fsub(o, v[e]) : fadd(v[e], o);
          }
        }
      }
      if (PASS == 0) {
        local = fmaxf(local, fmaxf(fmaxf(fabsf(v[0]), fabsf(v[1])), fmaxf(fabsf(v[2]), fabsf(v[3]))));
      } else if (n0 < N) {
        uint32_t o = ((uint32_t)(uint8_t)quant1(v[0], inv)) | ((uint32_t)(uint8_t)quant1(v[1], inv) << 8) |
                     ((uint32_t)(uint8_t)quant1(v[2], inv) << 16) | ((uint32_t)(uint8_t)quant1(v[3], inv) << 24);
        *reinterpret_cast<uint32_t*>(Aq + m * N + n0) = o;
      }
    }
  }
  if (PASS == 0) {
#pragma unroll
    for (int w = 16; w; w >>= 1) local = fmaxf(local, __shfl_xor_sync(0xffffffffu, local, w));
    // non-negative floats order as uints; the plain read filters out almost every atomic (the maximum only grows)
    if (lane == 0 && local > 0.0f && __float_as_uint(local) > *reinterpret_cast<volatile uint32_t*>(amax))
      atomicMax(amax, __float_as_uint(local));
  }
}

// (2) rotation along the row-index (strided) direction with a transposed int8 result:
//     in [R, C] (bf16 for G = dY, int8 for Z = qX and U = qW)  ->  out int8 [C, R],
//     out[c, r] = quantise(rotate_r(in[:, c]))[r].  A thread owns one column of a 128-row block: 128 values in
//     registers (a warp reads 32 adjacent columns of each row, i.e. whole 32/64-byte sectors), the seven butterfly
//     stages run in registers, and the thread writes its 128 quantised values as one contiguous 128-byte run of the
//     transposed output.  Each stage touches disjoint pairs, so the rounding order per element is fixed.
template <bool ISF, int PASS, bool ROT>
__global__ void __launch_bounds__(128) k_rotc(const void* __restrict__ in, int R, int C, uint32_t* __restrict__ amax,
                                              int8_t* __restrict__ outT) {
  const int col = blockIdx.x * 128 + threadIdx.x;
  const int r0 = blockIdx.y * 128;
  float vf[ISF ? 128 : 1];
  int vi[ISF ? 1 : 128];
  if (ISF) {
    const uint16_t* p = reinterpret_cast<const uint16_t*>(in) + (size_t)r0 * C + col;
#pragma unroll
    for (int i = 0; i < 128; ++i) vf[i] = bf2f(__ldg(p + (size_t)i * C));
  } else {
    const int8_t* p = reinterpret_cast<const int8_t*>(in) + (size_t)r0 * C + col;
#pragma unroll
    for (int i = 0; i < 128; ++i) vi[i] = (int)__ldg(p + (size_t)i * C);
  }
  if (ROT) {
#pragma unroll
    for (int h = 1; h < 128; h <<= 1) {
#pragma unroll
      for (int i = 0; i < 128; ++i) {
        if (!(i & h)) {
          if (ISF) { const float a = vf[i], b = vf[i + h]; vf[i] = fadd(a, b); vf[i + h] = fsub(a, b); }
          else { const int a = vi[i], b = vi[i + h]; vi[i] = a + b; vi[i + h] = a - b; }
        }
      }
    }
  }
  if (PASS == 0) {
    uint32_t local = 0;
#pragma unroll
    for (int i = 0; i < 128; ++i) {
      if (ISF) local = max(local, __float_as_uint(fabsf(vf[i])));
      else local = max(local, (uint32_t)abs(vi[i]));
    }
#pragma unroll
    for (int w = 16; w; w >>= 1) local = max(local, __shfl_xor_sync(0xffffffffu, local, w));
    if ((threadIdx.x & 31) == 0 && local > *reinterpret_cast<volatile uint32_t*>(amax)) atomicMax(amax, local);
  } else {
    float inv = 0.0f;
    if (ISF) {
      const float am = __uint_as_float(amax[0]);
      inv = (am > 0.0f) ? fdiv(127.0f, am) : 0.0f;
    } else if (ROT) {
      const int am = (int)amax[0];
      inv = (am > 0) ? fdiv(127.0f, __int2float_rn(am)) : 0.0f;
    }
    uint4* dst = reinterpret_cast<uint4*>(outT + (size_t)col * R + r0);
#pragma unroll
    for (int g = 0; g < 8; ++g) {
      uint32_t w[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        uint32_t o = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int i = g * 16 + k * 4 + e;
          int8_t qv;
          if (ISF) qv = quant1(vf[i], inv);
          else if (ROT) qv = quant1(__int2float_rn(vi[i]), inv);
          else qv = (int8_t)vi[i];
          o |= ((uint32_t)(uint8_t)qv) << (8 * e);
        }
        w[k] = o;
      }
      dst[g] = make_uint4(w[0], w[1], w[2], w[3]);
    }
  }
}

// (2b) the int8 operands (Z = qX, U = qW) through shared memory: the CTA loads its 128 x 128 tile with whole 128-byte row
//      segments (eight lanes per row), every thread takes one column from the tile (a warp reads 32 adjacent bytes of a
//      row: one wavefront), rotates it in registers (exact integers, |value| <= 2^14), and in PASS 1 the quantised columns
//      go back through the tile so that the transposed output is written as whole 128-byte lines as well (the version this
//      replaced read one byte and wrote sixteen per lane in 32 different lines per instruction; the values are the same).
template <int PASS, bool ROT>
__global__ void __launch_bounds__(128) k_rotc8(const int8_t* __restrict__ in, int R, int C, uint32_t* __restrict__ amax,
                                               int8_t* __restrict__ outT) {
  __shared__ __align__(16) uint8_t tile[128 * 128];
  const int t = threadIdx.x, c0 = blockIdx.x * 128, r0 = blockIdx.y * 128;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int r = i * 16 + (t >> 3), ch = t & 7;
    *reinterpret_cast<uint4*>(tile + r * 128 + ch * 16) =
        __ldg(reinterpret_cast<const uint4*>(in + (size_t)(r0 + r) * C + c0 + ch * 16));
  }
  __syncthreads();
  int vi[128];
#pragma unroll
  for (int i = 0; i < 128; ++i) vi[i] = (int)(int8_t)tile[i * 128 + t];
  if (ROT) {
#pragma unroll
    for (int h = 1; h < 128; h <<= 1) {
#pragma unroll
      for (int i = 0; i < 128; ++i) {
        if (!(i & h)) { const int a = vi[i], b = vi[i + h]; vi[i] = a + b; vi[i + h] = a - b; }
      }
    }
  }
  if (PASS == 0) {
    uint32_t local = 0;
#pragma unroll
    for (int i = 0; i < 128; ++i) local = max(local, (uint32_t)abs(vi[i]));
#pragma unroll
    for (int w = 16; w; w >>= 1) local = max(local, __shfl_xor_sync(0xffffffffu, local, w));
    if ((t & 31) == 0 && local > *reinterpret_cast<volatile uint32_t*>(amax)) atomicMax(amax, local);
    return;
  }
  float inv = 0.0f;
  if (ROT) {
    const int am = (int)amax[0];
    inv = (am > 0) ? fdiv(127.0f, __int2float_rn(am)) : 0.0f;
  }
  __syncthreads();                       // everybody has read its column: the tile becomes the transposed output tile
#pragma unroll
  for (int g = 0; g < 8; ++g) {
    uint32_t w[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      uint32_t o = 0;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int i = g * 16 + k * 4 + e;
        const int8_t qv = ROT ? quant1(__int2float_rn(vi[i]), inv) : (int8_t)vi[i];
        o |= ((uint32_t)(uint8_t)qv) << (8 * e);
      }
      w[k] = o;
    }
    // row t of the transposed tile (column c0 + t of the input), sixteen-byte pieces XOR-swizzled by row
    *reinterpret_cast<uint4*>(tile + t * 128 + ((g ^ (t & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int r = i * 16 + (t >> 3), ch = t & 7;
    *reinterpret_cast<uint4*>(outT + (size_t)(c0 + r) * R + r0 + ch * 16) =
        *reinterpret_cast<const uint4*>(tile + r * 128 + ((ch ^ (r & 7)) << 4));
  }
}

// (3) both rotations of dY from one read: a CTA stages a 128 x 128 tile of dY in shared memory (raw bf16), then every thread
//     rotates one row of dY * s_w along n (the A operand of the input-gradient GEMM) and one column of dY along the
//     token index (the G operand of the weight-gradient GEMM, written transposed).  128 values per thread in registers,
//     butterflies on register pairs with packed arithmetic: a + b is one packed add, a - b one packed fused
//     multiply-add b * (-1) + a, which rounds exactly like the subtraction.  PASS 0 records both absmax values,
//     PASS 1 quantises with them.  dY is read twice per backward pass instead of four times.
constexpr int PT = 128;

__device__ __forceinline__ void wht128_pairs(float2 (&v)[64]) {
#pragma unroll
  for (int p = 0; p < 64; ++p) v[p] = make_float2(fadd(v[p].x, v[p].y), fsub(v[p].x, v[p].y));   // stage h = 1
  const float2 m1 = make_float2(-1.0f, -1.0f);
#pragma unroll
  for (int hp = 1; hp < 64; hp <<= 1) {                                                        // stages h = 2 .. 64
#pragma unroll
    for (int p = 0; p < 64; ++p) {
      if (!(p & hp)) {
        const float2 a = v[p], b = v[p + hp];
        v[p] = __fadd2_rn(a, b);
        v[p + hp] = __ffma2_rn(b, m1, a);
      }
    }
  }
}
__device__ __forceinline__ float absmax128(const float2 (&v)[64]) {
  float m = 0.0f;
#pragma unroll
  for (int p = 0; p < 64; ++p) m = fmaxf(m, fmaxf(fabsf(v[p].x), fabsf(v[p].y)));
  return m;
}
// 128 rotated values -> 32 words of int8 codes clamp(rne(v * inv), -128, 127).
// FAST: every product is finite and at most 127 (1 + 2^-22) in magnitude (the caller checked: the step comes from the
// absmax of these very values, and the first rotated value, the plain sum that every input reaches through additions
// only, is finite), so the clamp cannot act; adding 1.5 * 2^23 rounds to nearest-even exactly like the conversion and
// leaves the code in the low byte of the float's bits.  The multiply stays a scalar instruction of its own (rounded
// before the add); otherwise the generic path.
template <bool FAST>
__device__ __forceinline__ void quant_pack128(const float2 (&v)[64], float inv, uint32_t (&w)[32]) {
  const float2 magic = make_float2(12582912.0f, 12582912.0f);
#pragma unroll
  for (int k = 0; k < 32; ++k) {
    const float2 lo = v[2 * k], hi = v[2 * k + 1];
    if (FAST) {
      const float2 a = __fadd2_rn(make_float2(fmul(lo.x, inv), fmul(lo.y, inv)), magic);
      const float2 b = __fadd2_rn(make_float2(fmul(hi.x, inv), fmul(hi.y, inv)), magic);
      const uint32_t t1 = __byte_perm(__float_as_uint(a.x), __float_as_uint(a.y), 0x0040);
      const uint32_t t2 = __byte_perm(__float_as_uint(b.x), __float_as_uint(b.y), 0x0040);
      w[k] = __byte_perm(t1, t2, 0x5410);
    } else {
      w[k] = ((uint32_t)(uint8_t)quant1(lo.x, inv)) | ((uint32_t)(uint8_t)quant1(lo.y, inv) << 8) |
             ((uint32_t)(uint8_t)quant1(hi.x, inv) << 16) | ((uint32_t)(uint8_t)quant1(hi.y, inv) << 24);
    }
  }
}
__device__ __forceinline__ bool finite1(float x) { return (__float_as_uint(x) & 0x7f800000u) != 0x7f800000u; }
__device__ __forceinline__ void amax_publish(float local, uint32_t* amax) {
#pragma unroll
  for (int w = 16; w; w >>= 1) local = fmaxf(local, __shfl_xor_sync(0xffffffffu, local, w));
  if ((threadIdx.x & 31) == 0 && local > 0.0f && __float_as_uint(local) > *reinterpret_cast<volatile uint32_t*>(amax))
    atomicMax(amax, __float_as_uint(local));
}

//     The kernel is persistent and software-pipelined: a CTA walks over tiles, the raw bf16 tile of the NEXT step travels
//     into the other half of a double buffer (16-byte asynchronous copies, chunks XOR-swizzled by row so that a thread reads
//     its row with conflict-free 16-byte loads and its column with 2-byte loads) while the current one is rotated, so no
//     global-load latency and no convert-and-store pass sits between the butterflies; the finished int8 rows leave through
//     the buffer that has just been consumed, as whole 128-byte lines.
constexpr size_t PREP2_SMEM = (size_t)2 * PT * 256 + 2 * PT * sizeof(float);

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async4(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}

template <int PASS>
__global__ void __launch_bounds__(PT, 3) k_prep_dy2(const uint16_t* __restrict__ dY, const float* __restrict__ s_w, int M, int N,
                                                    uint32_t* __restrict__ amax, int8_t* __restrict__ Aq,
                                                    int8_t* __restrict__ GqT) {
  extern __shared__ __align__(16) uint8_t pbuf[];
  float* swb = reinterpret_cast<float*>(pbuf + 2 * PT * 256);      // [2][128]
  const int t = threadIdx.x;
  const int ntn = N / PT, ntiles = ntn * (M / PT);
  auto issue = [&](int tile, int b) {
    const int n0 = (tile % ntn) * PT, m0 = (tile / ntn) * PT;
    uint8_t* dst = pbuf + b * (PT * 256);
#pragma unroll
    for (int it = 0; it < 16; ++it) {
      const int r = it * 8 + (t >> 4), c = t & 15;
      cp_async16(dst + r * 256 + ((c ^ (r & 7)) << 4), dY + (size_t)(m0 + r) * N + n0 + c * 8);
    }
    cp_async4(swb + b * PT + t, s_w + n0 + t);
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  float invA = 0.0f, invG = 0.0f;
  bool fastA = false, fastG = false;
  if (PASS == 1) {
    const float a = __uint_as_float(amax[0]), g = __uint_as_float(amax[1]);
    invA = (a > 0.0f) ? fdiv(127.0f, a) : 0.0f;
    invG = (g > 0.0f) ? fdiv(127.0f, g) : 0.0f;
    fastA = finite1(a) && finite1(invA);
    fastG = finite1(g) && finite1(invG);
  }
  float maxA = 0.0f, maxG = 0.0f;
  if ((int)blockIdx.x < ntiles) issue(blockIdx.x, 0);
  int i = 0;
  for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++i) {
    const int b = i & 1, next = tile + gridDim.x;
    __syncthreads();                                   // the other buffer (tile i - 1: operands and staging) is free
    if (next < ntiles) {
      issue(next, b ^ 1);
      asm volatile("cp.async.wait_group 1;" ::: "memory");
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();                                   // tile i has landed for every thread
    const uint8_t* buf = pbuf + b * (PT * 256);
    const float* sw = swb + b * PT;
    const int n0 = (tile % ntn) * PT, m0 = (tile / ntn) * PT;
    float2 v[64];
    uint32_t qa[32], qg[32];
    // row t of the tile, scaled by the weight steps (scalar multiplies: the products are rounded before any add)
#pragma unroll
    for (int c = 0; c < 16; ++c) {
      const uint4 u = *reinterpret_cast<const uint4*>(buf + t * 256 + ((c ^ (t & 7)) << 4));
      const float4 w0 = *reinterpret_cast<const float4*>(&sw[8 * c]), w1 = *reinterpret_cast<const float4*>(&sw[8 * c + 4]);
      v[4 * c] = make_float2(fmul(bflo(u.x), w0.x), fmul(bfhi(u.x), w0.y));
      v[4 * c + 1] = make_float2(fmul(bflo(u.y), w0.z), fmul(bfhi(u.y), w0.w));
      v[4 * c + 2] = make_float2(fmul(bflo(u.z), w1.x), fmul(bfhi(u.z), w1.y));
      v[4 * c + 3] = make_float2(fmul(bflo(u.w), w1.z), fmul(bfhi(u.w), w1.w));
    }
    wht128_pairs(v);
    if (PASS == 0) maxA = fmaxf(maxA, absmax128(v));
    else if (fastA && finite1(v[0].x)) quant_pack128<true>(v, invA, qa);
    else quant_pack128<false>(v, invA, qa);
    // column t of the tile, transposed output
    const int cc = t >> 3, cw = (t & 7) * 2;
#pragma unroll
    for (int p = 0; p < 64; ++p) {
      const uint16_t lo = *reinterpret_cast<const uint16_t*>(buf + (2 * p) * 256 + ((cc ^ ((2 * p) & 7)) << 4) + cw);
      const uint16_t hi = *reinterpret_cast<const uint16_t*>(buf + (2 * p + 1) * 256 + ((cc ^ ((2 * p + 1) & 7)) << 4) + cw);
      v[p] = make_float2(bf2f(lo), bf2f(hi));
    }
    wht128_pairs(v);
    if (PASS == 0) { maxG = fmaxf(maxG, absmax128(v)); continue; }
    if (fastG && finite1(v[0].x)) quant_pack128<true>(v, invG, qg);
    else quant_pack128<false>(v, invG, qg);
    // hand-over through the consumed buffer: two tiles of 128 rows x 128 bytes, sixteen-byte pieces XOR-swizzled by row
    __syncthreads();
    uint8_t* stg = pbuf + b * (PT * 256);
#pragma unroll
    for (int g = 0; g < 8; ++g) {
      const int off = t * 128 + ((g ^ (t & 7)) << 4);
      *reinterpret_cast<uint4*>(stg + off) = make_uint4(qa[4 * g], qa[4 * g + 1], qa[4 * g + 2], qa[4 * g + 3]);
      *reinterpret_cast<uint4*>(stg + 16384 + off) = make_uint4(qg[4 * g], qg[4 * g + 1], qg[4 * g + 2], qg[4 * g + 3]);
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int idx = k * PT + t, r = idx >> 3, piece = idx & 7;
      const int off = r * 128 + ((piece ^ (r & 7)) << 4);
      *reinterpret_cast<uint4*>(Aq + (size_t)(m0 + r) * N + n0 + piece * 16) = *reinterpret_cast<const uint4*>(stg + off);
      *reinterpret_cast<uint4*>(GqT + (size_t)(n0 + r) * M + m0 + piece * 16) = *reinterpret_cast<const uint4*>(stg + 16384 + off);
    }
  }
  if (PASS == 0) {
    amax_publish(maxA, amax + 0);
    amax_publish(maxG, amax + 1);
  }
}

__global__ void k_su_finish(const uint32_t* amax, int rotated, float* s_u) {
  if (!rotated) { s_u[0] = 1.0f; return; }
  const int am = (int)amax[0];
  s_u[0] = (am > 0) ? fdiv(__int2float_rn(am), 127.0f) : 0.0f;
}
__global__ void k_dsx_finish(const float* sum, float gs, float* ds_x) { ds_x[0] = fmul(gs, sum[0]); }

}  // namespace det

using namespace det;

extern "C" size_t det_lsq_weight_scale_ws_bytes(int N, int K) {
  size_t n = (size_t)N * K;
  size_t c = (n + 16383) / 16384;
  return (align_up(c, 64) + 64 + sum_ws_floats(c)) * sizeof(float);
}
static int abs_mean_scale(const det_bf16* X, size_t n, float* out, int count, float* ws, cudaStream_t st) {
  const size_t c = (n + 16383) / 16384;
  float* partial = ws;
  float* total = partial + align_up(c, 64);
  float* scratch = total + 64;
  k_abs_chunk<<<DET_L((unsigned)c), 256, 0, st>>>(X, (long long)n, partial);
  sum_launch(partial, c, 0, total, scratch, st);
  k_scale_finish<<<DET_L((count + 255) / 256 < 64 ? (count + 255) / 256 : 64), 256, 0, st>>>(total, (float)(1.0 / (double)n), out, count);
  return DET_OK;
}
extern "C" int det_lsq_weight_scale(const det_bf16* W, int N, int K, int per_tensor, float* s_w, void* ws,
                                    size_t ws_bytes, void* stream) {
  if (!W || !s_w || N <= 0 || K <= 0) return DET_ERR_ARG;
  if (K % 8 || (!per_tensor && K > 8192)) return DET_ERR_SHAPE;
  if (!aligned16(W)) return DET_ERR_ALIGN;
  cudaStream_t st = (cudaStream_t)stream;
  if (per_tensor) {
    if (!ws || ws_bytes < det_lsq_weight_scale_ws_bytes(N, K)) return DET_ERR_WORKSPACE;
    abs_mean_scale(W, (size_t)N * K, s_w, N, (float*)ws, st);
  } else {
    k_wscale_rows<<<DET_L((N + 7) / 8), 256, 0, st>>>(W, N, K, (float)(1.0 / (double)K), s_w);
  }
  DET_CHECK_LAUNCH();
  return DET_OK;
}
extern "C" size_t det_lsq_act_scale_init_ws_bytes(size_t n) { return det_lsq_weight_scale_ws_bytes(1, (int)1) + ((n + 16383) / 16384 + 128) * 2 * sizeof(float); }
extern "C" int det_lsq_act_scale_init(const det_bf16* X, size_t n, float* s_x, void* ws, size_t ws_bytes, void* stream) {
  if (!X || !s_x || n == 0) return DET_ERR_ARG;
  if (!aligned16(X)) return DET_ERR_ALIGN;
  if (!ws || ws_bytes < det_lsq_act_scale_init_ws_bytes(n)) return DET_ERR_WORKSPACE;
  abs_mean_scale(X, n, s_x, 1, (float*)ws, (cudaStream_t)stream);
  DET_CHECK_LAUNCH();
  return DET_OK;
}

extern "C" size_t det_lsq_quantize_weight_ws_bytes(int N, int K) { (void)N; (void)K; return 256; }
extern "C" int det_lsq_quantize_weight(const det_bf16* W, const float* s_w, int N, int K, int hadamard_block, int8_t* qW,
                                       int8_t* qWt_bwd, float* s_u, void* ws, size_t ws_bytes, void* stream) {
  if (!W || !s_w || !qW || N <= 0 || K <= 0 || (qWt_bwd && !s_u)) return DET_ERR_ARG;
  if (N % 128 || K % 128 || (hadamard_block != 0 && hadamard_block != 128)) return DET_ERR_SHAPE;
  if (!aligned16(W) || !aligned16(qW) || (qWt_bwd && !aligned16(qWt_bwd))) return DET_ERR_ALIGN;
  if (qWt_bwd && (!ws || ws_bytes < 256)) return DET_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t n16 = (size_t)N * K / 16;
  k_quantize<<<DET_L((unsigned)((n16 + 255) / 256)), 256, 0, st>>>(W, n16, K / 16, s_w, 1, qW);
  if (qWt_bwd) {
    uint32_t* amax = (uint32_t*)ws;
    cudaMemsetAsync(amax, 0, 256, st);
    dim3 grid(K / 128, N / 128);
    if (hadamard_block) {
      k_rotc8<0, true><<<DET_L(grid), 128, 0, st>>>(qW, N, K, amax, nullptr);
      k_rotc8<1, true><<<DET_L(grid), 128, 0, st>>>(qW, N, K, amax, qWt_bwd);
    } else {
      k_rotc8<1, false><<<DET_L(grid), 128, 0, st>>>(qW, N, K, amax, qWt_bwd);
    }
    k_su_finish<<<DET_L(1), 1, 0, st>>>(amax, hadamard_block != 0, s_u);
  }
  DET_CHECK_LAUNCH();
  return DET_OK;
}

extern "C" int det_linear_fwd(const det_bf16* X, const int8_t* qW, const float* s_x, const float* s_w, int M, int N, int K,
                              det_bf16* Y, int8_t* qX_save, void* stream, int* status_dev) {
  if (!X || !qW || !s_x || !s_w || !Y || !qX_save || M <= 0 || N <= 0 || K <= 0) return DET_ERR_ARG;
  if (M % 128 || N % 128 || K % 128) return DET_ERR_SHAPE;
  if (K >= (1 << 17)) return DET_ERR_RANGE;
  if (!aligned16(X) || !aligned16(qW) || !aligned16(Y) || !aligned16(qX_save) || !aligned16(s_w)) return DET_ERR_ALIGN;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t n16 = (size_t)M * K / 16;
  k_quantize<<<DET_L((unsigned)((n16 + 255) / 256)), 256, 0, st>>>(X, n16, K / 16, s_x, 0, qX_save);
  DET_CHECK_LAUNCH();
  EpiParams ep = {};
  ep.out = Y; ep.s_x = s_x; ep.s_w = s_w;
  return igemm_launch(EPI_FWD, qX_save, qW, M, N, K, ep, status_dev, st);
}

extern "C" int det_linear_fwd_q(const int8_t* qX, const int8_t* qW, const float* s_x, const float* s_w, int M, int N, int K,
                                det_bf16* Y, void* stream, int* status_dev) {
  if (!qX || !qW || !s_x || !s_w || !Y || M <= 0 || N <= 0 || K <= 0) return DET_ERR_ARG;
  if (M % 128 || N % 128 || K % 128) return DET_ERR_SHAPE;
  if (K >= (1 << 17)) return DET_ERR_RANGE;
  if (!aligned16(qX) || !aligned16(qW) || !aligned16(Y) || !aligned16(s_w)) return DET_ERR_ALIGN;
  EpiParams ep = {};
  ep.out = Y; ep.s_x = s_x; ep.s_w = s_w;
  return igemm_launch(EPI_FWD, qX, qW, M, N, K, ep, status_dev, (cudaStream_t)stream);
}

static size_t bwd_ws_layout(int M, int N, int K, size_t* oA, size_t* oG, size_t* oZ, size_t* oP, size_t* oS) {
  size_t off = 256;
  *oA = off; off += align_up((size_t)M * N, 256);
  *oG = off; off += align_up((size_t)M * N, 256);
  *oZ = off; off += align_up((size_t)M * K, 256);
  const size_t np = (size_t)M * (K / 128);
  *oP = off; off += align_up(np * sizeof(float), 256);
  *oS = off; off += align_up((sum_ws_floats(np) + 64) * sizeof(float), 256);
  return off;
}
extern "C" size_t det_linear_bwd_ws_bytes(int M, int N, int K) {
  size_t a, g, z, p, s;
  return bwd_ws_layout(M, N, K, &a, &g, &z, &p, &s);
}
extern "C" int det_linear_bwd(const det_bf16* dY, const det_bf16* X, const int8_t* qX, const det_bf16* W,
                              const int8_t* qWt_bwd, const float* s_x, const float* s_w, const float* s_u, int M, int N,
                              int K, int hadamard_block, det_bf16* dX, float* dW, float* ds_x, void* ws, size_t ws_bytes,
                              void* stream, int* status_dev) {
  if (!dY || !X || !qX || !W || !qWt_bwd || !s_x || !s_w || !s_u || !dX || !dW || !ds_x || M <= 0 || N <= 0 || K <= 0)
    return DET_ERR_ARG;
  if (M % 128 || N % 128 || K % 128 || (hadamard_block != 0 && hadamard_block != 128)) return DET_ERR_SHAPE;
  if (K >= (1 << 17) || N >= (1 << 17) || M >= (1 << 17)) return DET_ERR_RANGE;
  if (!aligned16(dY) || !aligned16(X) || !aligned16(qX) || !aligned16(W) || !aligned16(qWt_bwd) || !aligned16(dX) ||
      !aligned16(dW) || !aligned16(s_w) || !aligned16(ws))
    return DET_ERR_ALIGN;
  size_t oA, oG, oZ, oP, oS;
  if (!ws || ws_bytes < bwd_ws_layout(M, N, K, &oA, &oG, &oZ, &oP, &oS)) return DET_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  uint8_t* base = (uint8_t*)ws;
  uint32_t* amax = (uint32_t*)base;  // [0] A (float bits), [1] G (float bits), [2] Z (int)
  int8_t* Aq = (int8_t*)(base + oA);
  int8_t* GqT = (int8_t*)(base + oG);
  int8_t* ZqT = (int8_t*)(base + oZ);
  float* partial = (float*)(base + oP);
  float* sscr = (float*)(base + oS);
  const bool rot = hadamard_block != 0;
  cudaMemsetAsync(amax, 0, 256, st);
  const size_t ngrp = (size_t)M * ((N / 128 + 7) / 8);  // warp groups of 8 blocks
  const unsigned g1 = (unsigned)((ngrp + 7) / 8);
  dim3 gG(N / 128, M / 128), gZ(K / 128, M / 128);
  if (rot) {
    static DevOnce once0 = {}, once1 = {};
    if (dev_ensure_smem(once0, (const void*)k_prep_dy2<0>, PREP2_SMEM) != DET_OK ||
        dev_ensure_smem(once1, (const void*)k_prep_dy2<1>, PREP2_SMEM) != DET_OK)
      return DET_ERR_CUDA;
    const int sms = dev_sm_count();
    if (sms <= 0) return DET_ERR_CUDA;
    const int ptiles = (M / PT) * (N / PT);
    const unsigned gP = (unsigned)(ptiles < 3 * sms ? ptiles : 3 * sms);   // persistent: three CTAs per SM
    // the rotation of the saved int8 activations does not depend on dY: it runs beside the two passes over dY
    AuxScope az(st);
    cudaStream_t sz = az.aux(1);
    k_prep_dy2<0><<<DET_L(gP), PT, PREP2_SMEM, st>>>(dY, s_w, M, N, amax, nullptr, nullptr);
    k_rotc8<0, true><<<DET_L(gZ), 128, 0, sz>>>(qX, M, K, amax + 2, nullptr);
    k_prep_dy2<1><<<DET_L(gP), PT, PREP2_SMEM, st>>>(dY, s_w, M, N, amax, Aq, GqT);
    k_rotc8<1, true><<<DET_L(gZ), 128, 0, sz>>>(qX, M, K, amax + 2, ZqT);
    if (!az.join()) return DET_ERR_CUDA;
  } else {
    k_rot_rows<0, false><<<DET_L(g1), 256, 0, st>>>(dY, s_w, M, N, amax + 0, nullptr);
    k_rotc<true, 0, false><<<DET_L(gG), 128, 0, st>>>(dY, M, N, amax + 1, nullptr);
    k_rot_rows<1, false><<<DET_L(g1), 256, 0, st>>>(dY, s_w, M, N, amax + 0, Aq);
    k_rotc<true, 1, false><<<DET_L(gG), 128, 0, st>>>(dY, M, N, amax + 1, GqT);
    k_rotc8<1, false><<<DET_L(gZ), 128, 0, st>>>(qX, M, K, amax + 2, ZqT);
  }
  DET_CHECK_LAUNCH();
  const float rotf = rot ? 0x1p-7f : 1.0f;
  // The two gradient GEMMs are independent.  Each is a persistent grid whose blocks leave as their tiles run out, so the
  // weight-gradient GEMM, queued on an auxiliary stream, moves onto the SMs that the input-gradient GEMM's last
  // partial round leaves idle.
  AuxScope aux(st);   // joined again on every way out
  // grad wrt W: [N,K] = G_q^T [N,M] . (Z_q^T [K,M])^T
  EpiParams ew = {};
  ew.out = dW; ew.s_x = s_x; ew.s_w = s_w; ew.amax1 = amax + 1; ew.amax2 = rot ? amax + 2 : nullptr; ew.ref = W; ew.rot = rotf;
  // grad wrt x: [M,K] = A_q [M,N] . (U_q^T [K,N])^T
  EpiParams ex = {};
  ex.out = dX; ex.s_x = s_x; ex.amax1 = amax + 0; ex.s_u = s_u; ex.ref = X; ex.rot = rotf; ex.ds_partial = partial;
  int rc = igemm_launch(EPI_DX, Aq, qWt_bwd, M, K, N, ex, status_dev, st);
  if (rc != DET_OK) return rc;
  rc = igemm_launch(EPI_DW, GqT, ZqT, N, K, M, ew, status_dev, aux.aux(0));
  if (rc != DET_OK) return rc;
  const size_t np = (size_t)M * (K / 128);
  sum_launch(partial, np, 0, sscr, sscr + 64, st);
  k_dsx_finish<<<DET_L(1), 1, 0, st>>>(sscr, (float)(1.0 / sqrt((double)M * (double)K * 127.0)), ds_x);
  DET_CHECK_LAUNCH();
  if (!aux.join()) return DET_ERR_CUDA;
  return DET_OK;
}
