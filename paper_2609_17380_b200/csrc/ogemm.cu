// Ordered full-precision contractions for the LM head (Sec. 3.2: the head stays out of quantisation).
//
// Every output is ONE f32 accumulator that starts at +0 (or at the value already in the output) and
// receives its terms in ascending order of the contraction index, each term an exact bf16 x bf16 product
// added with a separate rounding (no FMA).  That fixes the order, so these GEMMs run on the FP32 ALUs:
// 128x128 output tile per CTA, 8x8 register tile per thread, 16-deep slabs staged through shared memory
// as f32, software-pipelined global loads.
#include "common.cuh"
#include "internal.h"

namespace det {

constexpr int OT = 128;  // tile edge
constexpr int OK = 16;   // slab depth

// Operand access modes.  C[i,j] = sum_c A(i,c) * B(j,c).
//   CONTIG : operand stored [rows, contraction] (contraction index contiguous)
//   STRIDED: operand stored [contraction, rows] (row index contiguous)
enum { CONTIG = 0, STRIDED = 1 };

template <bool F32IN>
__device__ __forceinline__ void load8_any(const void* base, size_t idx, bool ok, float v[8]) {
  if (!ok) {
#pragma unroll
    for (int t = 0; t < 8; ++t) v[t] = 0.0f;
    return;
  }
  if (F32IN) {
    const float4* p = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(base) + idx);
    float4 a = __ldg(p), b = __ldg(p + 1);
    // operands of the gradient contractions are rounded to bf16 first
    v[0] = bf2f(f2bf(a.x)); v[1] = bf2f(f2bf(a.y)); v[2] = bf2f(f2bf(a.z)); v[3] = bf2f(f2bf(a.w));
    v[4] = bf2f(f2bf(b.x)); v[5] = bf2f(f2bf(b.y)); v[6] = bf2f(f2bf(b.z)); v[7] = bf2f(f2bf(b.w));
  } else {
    uint4 u = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const uint16_t*>(base) + idx));
    v[0] = bflo(u.x); v[1] = bfhi(u.x); v[2] = bflo(u.y); v[3] = bfhi(u.y);
    v[4] = bflo(u.z); v[5] = bfhi(u.z); v[6] = bflo(u.w); v[7] = bfhi(u.w);
  }
}

// fetch this thread's 8 values of a 128 x 16 operand slab
template <int MODE, bool F32IN>
__device__ __forceinline__ void slab_fetch(const void* base, int rows, int C, int ld, int r0, int c0, float v[8]) {
  const int tid = threadIdx.x;
  if (MODE == CONTIG) {
    const int r = r0 + (tid & 127), c = c0 + (tid >> 7) * 8;
    load8_any<F32IN>(base, (size_t)r * ld + c, r < rows && c < C, v);
  } else {
    const int c = c0 + (tid >> 4), r = r0 + (tid & 15) * 8;
    load8_any<F32IN>(base, (size_t)c * ld + r, c < C && r < rows, v);
  }
}
template <int MODE>
__device__ __forceinline__ void slab_store(float (*s)[OT + 4], const float v[8]) {
  const int tid = threadIdx.x;
  if (MODE == CONTIG) {
    const int r = tid & 127, k0 = (tid >> 7) * 8;
#pragma unroll
    for (int t = 0; t < 8; ++t) s[k0 + t][r] = v[t];
  } else {
    const int k = tid >> 4, r = (tid & 15) * 8;
    *reinterpret_cast<float4*>(&s[k][r]) = make_float4(v[0], v[1], v[2], v[3]);
    *reinterpret_cast<float4*>(&s[k][r + 4]) = make_float4(v[4], v[5], v[6], v[7]);
  }
}

// rows of A: I, rows of B: J, contraction length C.  lda/ldb: leading dimensions of the stored operands.
// OUT_BF16: output bf16 else f32.  INIT: start accumulators from the values in `out` (f32 only).
template <int AMODE, int BMODE, bool AF32, bool OUT_BF16>
__global__ void __launch_bounds__(256) k_ogemm(const void* __restrict__ A, const void* __restrict__ B, int I, int J, int C,
                                               int lda, int ldb, void* __restrict__ out, int ldo, int init) {
  __shared__ __align__(16) float As[2][OK][OT + 4];
  __shared__ __align__(16) float Bs[2][OK][OT + 4];
  const int i0 = blockIdx.y * OT, j0 = blockIdx.x * OT;
  const int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
  float acc[8][8];
#pragma unroll
  for (int a = 0; a < 8; ++a)
#pragma unroll
    for (int b = 0; b < 8; ++b) acc[a][b] = 0.0f;
  if (init && !OUT_BF16) {
#pragma unroll
    for (int a = 0; a < 8; ++a) {
      const int r = i0 + (a >> 2) * 64 + ty * 4 + (a & 3);
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int c = j0 + h * 64 + tx * 4;
        if (r < I && c < J) {
          float4 t = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(out) + (size_t)r * ldo + c);
          acc[a][4 * h] = t.x; acc[a][4 * h + 1] = t.y; acc[a][4 * h + 2] = t.z; acc[a][4 * h + 3] = t.w;
        }
      }
    }
  }
  float va[8], vb[8];
  slab_fetch<AMODE, AF32>(A, I, C, lda, i0, 0, va);
  slab_fetch<BMODE, false>(B, J, C, ldb, j0, 0, vb);
  slab_store<AMODE>(As[0], va);
  slab_store<BMODE>(Bs[0], vb);
  __syncthreads();
  const int nslab = (C + OK - 1) / OK;
  for (int s = 0; s < nslab; ++s) {
    const int cur = s & 1;
    if (s + 1 < nslab) {
      slab_fetch<AMODE, AF32>(A, I, C, lda, i0, (s + 1) * OK, va);
      slab_fetch<BMODE, false>(B, J, C, ldb, j0, (s + 1) * OK, vb);
    }
#pragma unroll
    for (int k = 0; k < OK; ++k) {
      const float4 a0 = *reinterpret_cast<const float4*>(&As[cur][k][ty * 4]);
      const float4 a1 = *reinterpret_cast<const float4*>(&As[cur][k][64 + ty * 4]);
      const float4 b0 = *reinterpret_cast<const float4*>(&Bs[cur][k][tx * 4]);
      const float4 b1 = *reinterpret_cast<const float4*>(&Bs[cur][k][64 + tx * 4]);
      const float ar[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      const float br[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
      for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int b = 0; b < 8; ++b) acc[a][b] = fadd(acc[a][b], fmul(ar[a], br[b]));
    }
    if (s + 1 < nslab) {
      slab_store<AMODE>(As[cur ^ 1], va);
      slab_store<BMODE>(Bs[cur ^ 1], vb);
    }
    __syncthreads();
  }
#pragma unroll
  for (int a = 0; a < 8; ++a) {
    const int r = i0 + (a >> 2) * 64 + ty * 4 + (a & 3);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int c = j0 + h * 64 + tx * 4;
      if (r < I && c < J) {
        if (OUT_BF16) {
          uint2 u;
          u.x = pack_bf2(acc[a][4 * h], acc[a][4 * h + 1]);
          u.y = pack_bf2(acc[a][4 * h + 2], acc[a][4 * h + 3]);
          *reinterpret_cast<uint2*>(reinterpret_cast<uint16_t*>(out) + (size_t)r * ldo + c) = u;
        } else {
          *reinterpret_cast<float4*>(reinterpret_cast<float*>(out) + (size_t)r * ldo + c) =
              make_float4(acc[a][4 * h], acc[a][4 * h + 1], acc[a][4 * h + 2], acc[a][4 * h + 3]);
        }
      }
    }
  }
}

}  // namespace det

using namespace det;

extern "C" int det_lmhead_fwd(const det_bf16* H, const det_bf16* W, int M, int V, int K, float* logits, void* stream) {
  if (!H || !W || !logits || M <= 0 || V <= 0 || K <= 0) return DET_ERR_ARG;
  if (K % 16 || V % 4) return DET_ERR_SHAPE;
  if (!aligned16(H) || !aligned16(W) || !aligned16(logits)) return DET_ERR_ALIGN;
  dim3 grid((V + OT - 1) / OT, (M + OT - 1) / OT);
  k_ogemm<CONTIG, CONTIG, false, false><<<DET_L(grid), 256, 0, (cudaStream_t)stream>>>(H, W, M, V, K, K, K, logits, V, 0);
  DET_CHECK_LAUNCH();
  return DET_OK;
}

extern "C" int det_lmhead_bwd(const float* dlogits, const det_bf16* H, const det_bf16* W, int M, int V, int K, det_bf16* dH,
                              float* dW, int first_chunk, void* stream) {
  if (!dlogits || !H || !W || !dH || !dW || M <= 0 || V <= 0 || K <= 0) return DET_ERR_ARG;
  if (K % 16 || V % 8 || M % 8) return DET_ERR_SHAPE;
  if (!aligned16(dlogits) || !aligned16(H) || !aligned16(W) || !aligned16(dH) || !aligned16(dW)) return DET_ERR_ALIGN;
  cudaStream_t st = (cudaStream_t)stream;
  // dH[m,k] = sum over v ascending of bf16(dlogits[m,v]) * W[v,k]
  dim3 g1((K + OT - 1) / OT, (M + OT - 1) / OT);
  k_ogemm<CONTIG, STRIDED, true, true><<<DET_L(g1), 256, 0, st>>>(dlogits, W, M, K, V, V, K, dH, K, 0);
  // dW[v,k] (+)= sum over m ascending of bf16(dlogits[m,v]) * H[m,k]
  dim3 g2((K + OT - 1) / OT, (V + OT - 1) / OT);
  k_ogemm<STRIDED, STRIDED, true, false><<<DET_L(g2), 256, 0, st>>>(dlogits, H, V, K, M, V, K, dW, K, first_chunk ? 0 : 1);
  DET_CHECK_LAUNCH();
  return DET_OK;
}
