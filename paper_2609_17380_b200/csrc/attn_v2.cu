// Causal attention, arithmetic version 2 (optional mode): both contractions of the forward pass as order-free, exactly
// defined sums on the int8 tensor cores (the construction of lmhead_v2.cu; Sec. 3.2: int8 products accumulated exactly,
// a wide exact integer total "for bitwise reproducibility"), the softmax in the binary32 arithmetic of version 1.
//
//   s_ij  = fmul(C(q_i, k_j), 1/sqrt(128))    C = the version-2 contraction over the 128 dimensions (row exponents over
//                                             the 128 values of q_i and of k_j), one rounding
//   m_i   = max_j s_ij, p_ij = det_exp(s_ij - m_i), l_i = det_sum(p_i0 .. p_ii), lse_i = m_i + det_log(l_i)
//   P~    = bf16(p)
//   u_ic  = C(P~_i., v_.c) over the keys 0 .. i (exponent of row i of P~ over its keys; exponent of column c of v over all
//           keys of the sequence), one rounding;  o_ic = bf16(fmul(u_ic, fdiv(1, l_i)))
//
// With no order to respect there are no key tiles and no rescaling.  The pass is a chain of plain launches:
//   k_slice_heads      q, k: one warp per (head, position) row -> two int8 slices + exponent
//   k_col_exp_heads, k_slice_cols_heads   v: exponent per (head, dimension) over the keys, slices transposed [dim][key]
//   k_igemm_sl         S = Q K^T for the causal tiles of every head (lmhead_v2.cu), f32 to the workspace
//   k_softmax_v2       one CTA per row: maximum, exponentials, the fixed tree, lse, 1/l, and P~ as slices + exponent
//   k_igemm_sl         U = P~ V over the keys up to the row tile's own, times 1/l, bf16 into the head's columns of out
#include "internal.h"
#include "v2_slice.cuh"

namespace det {

constexpr float ATT2_SCALE = 0x1.6a09e6p-4f;  // 1/sqrt(128) rounded to binary32

// element (position i, dimension c) of head z = b*H + h: X[ld * (b*S + i) + h*128 + c]
__device__ __forceinline__ const uint16_t* head_row(const uint16_t* X, int ld, int H, int S, int z, int i) {
  const int b = z / H, h = z - b * H;
  return X + (size_t)ld * ((size_t)b * S + i) + h * 128;
}

// rows of a head-packed bf16 tensor -> slices [Z*S, 128] and exponents [Z*S]; one warp per row, four values per lane
__global__ void __launch_bounds__(256) k_slice_heads(const uint16_t* __restrict__ X, int ld, int H, int S, int rows,
                                                     int8_t* __restrict__ hi, int8_t* __restrict__ lo, int32_t* __restrict__ E) {
  const int r = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (r >= rows) return;
  const int z = r / S, i = r - z * S;
  const uint2 w = __ldg(reinterpret_cast<const uint2*>(head_row(X, ld, H, S, z, i) + lane * 4));
  const uint32_t b4[4] = {w.x & 0xFFFFu, w.x >> 16, w.y & 0xFFFFu, w.y >> 16};
  int e = 0, bad = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int ej = (b4[j] >> 7) & 0xFF;
    bad |= (ej == 255);
    e = max(e, ej);
  }
#pragma unroll
  for (int s = 16; s; s >>= 1) {
    e = max(e, __shfl_xor_sync(0xffffffffu, e, s));
    bad |= __shfl_xor_sync(0xffffffffu, bad, s);
  }
  if (lane == 0) E[r] = e | (bad ? (1 << 30) : 0);
  uint32_t h4 = 0u, l4 = 0u;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    int h, l;
    slice1(b4[j], e, h, l);
    h4 |= (uint32_t)(uint8_t)(int8_t)h << (8 * j);
    l4 |= (uint32_t)(uint8_t)(int8_t)l << (8 * j);
  }
  *reinterpret_cast<uint32_t*>(hi + (size_t)r * 128 + lane * 4) = h4;
  *reinterpret_cast<uint32_t*>(lo + (size_t)r * 128 + lane * 4) = l4;
}

// Slicing along the positions (for an operand contracted over keys or queries): exponent of (head z, dimension c) over
// all S positions (integer maximum through atomicMax: order-free; E zero before), slices written transposed
// [z*128 + c][position].  grid (1, S/128, Z), thread = dimension.
__global__ void __launch_bounds__(128) k_col_exp_heads(const uint16_t* __restrict__ X, int ld, int H, int S,
                                                       int32_t* __restrict__ E) {
  const int c = threadIdx.x, r0 = blockIdx.y * 128, z = blockIdx.z;
  const uint16_t* base = head_row(X, ld, H, S, z, r0) + c;
  int key = 0;
#pragma unroll 8
  for (int i = 0; i < 128; ++i) {
    const uint32_t b = (uint32_t)__ldg(base + (size_t)i * ld);
    const int e = (b >> 7) & 0xFF;
    key = max(key, e | (e == 255 ? (1 << 30) : 0));
  }
  if (key > *reinterpret_cast<volatile int32_t*>(E + z * 128 + c)) atomicMax(E + z * 128 + c, key);
}
__global__ void __launch_bounds__(128) k_slice_cols_heads(const uint16_t* __restrict__ X, int ld, int H, int S,
                                                          const int32_t* __restrict__ E, int8_t* __restrict__ hiT,
                                                          int8_t* __restrict__ loT) {
  __shared__ __align__(16) uint8_t tile[2][128 * 128];
  const int t = threadIdx.x, r0 = blockIdx.y * 128, z = blockIdx.z;
  const uint16_t* base = head_row(X, ld, H, S, z, r0) + t;
  const int e = E[z * 128 + t] & 0xFF;
  uint32_t hw[32], lw[32];
#pragma unroll
  for (int i = 0; i < 128; ++i) {
    const uint32_t b = (uint32_t)__ldg(base + (size_t)i * ld);
    int h, l;
    slice1(b, e, h, l);
    if ((i & 3) == 0) { hw[i >> 2] = 0u; lw[i >> 2] = 0u; }
    hw[i >> 2] |= (uint32_t)(uint8_t)(int8_t)h << (8 * (i & 3));
    lw[i >> 2] |= (uint32_t)(uint8_t)(int8_t)l << (8 * (i & 3));
  }
#pragma unroll
  for (int g = 0; g < 8; ++g) {   // row t of the transposed tiles, sixteen-byte pieces XOR-swizzled by row
    const int off = t * 128 + ((g ^ (t & 7)) << 4);
    *reinterpret_cast<uint4*>(tile[0] + off) = make_uint4(hw[4 * g], hw[4 * g + 1], hw[4 * g + 2], hw[4 * g + 3]);
    *reinterpret_cast<uint4*>(tile[1] + off) = make_uint4(lw[4 * g], lw[4 * g + 1], lw[4 * g + 2], lw[4 * g + 3]);
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int r = i * 16 + (t >> 3), ch = t & 7;
    const int off = r * 128 + ((ch ^ (r & 7)) << 4);
    *reinterpret_cast<uint4*>(hiT + ((size_t)z * 128 + r) * S + r0 + ch * 16) = *reinterpret_cast<const uint4*>(tile[0] + off);
    *reinterpret_cast<uint4*>(loT + ((size_t)z * 128 + r) * S + r0 + ch * 16) = *reinterpret_cast<const uint4*>(tile[1] + off);
  }
}

// One CTA per row (head z, query i) of the logits: a warp owns the leaves w, w + 8, ... of 256 keys, a lane 8 adjacent keys
// of a leaf, as in every fixed tree of this library; at most LPW leaves per warp (S <= 2048 LPW).  Only the warps that
// own a leaf of the row take part: the others leave at once and the barriers count the rest.
//   * every weight is at most 1 and the maximum's own weight is exactly 1 (det_exp(0)), so the largest exponent among
//     the bf16 weights equals the largest binary32 exponent field among the unrounded ones (rounding can lift a weight to
//     1.0 but not beyond), and a NaN shows as 255 in both
//   * the weights are not negative, so their slices carry no sign
constexpr int SM2_LPW = 4;
__device__ __forceinline__ void a2_bar(int nthreads) { asm volatile("bar.sync 1, %0;" ::"r"(nthreads) : "memory"); }
template <int LPW>
__global__ void __launch_bounds__(256) k_softmax_v2(const float* __restrict__ Sraw, int S, float* __restrict__ lse,
                                                    float* __restrict__ inv_l, int8_t* __restrict__ Ph, int8_t* __restrict__ Pl,
                                                    int32_t* __restrict__ Ep) {
  __shared__ float leafs[32];
  __shared__ float redf[8];
  __shared__ int redi[8];
  const int row = blockIdx.x, i = row % S, n = i + 1;
  const int kend = ((i >> 7) + 1) << 7;           // the keys the row tile's contraction runs over
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nl = (n + 255) >> 8;                  // leaves of the row
  const int nw = nl < 8 ? nl : 8;                 // warps that own one
  if (warp >= nw) return;
  const float* s = Sraw + (size_t)row * S;
  const float NEG_INF = __int_as_float(0xff800000);
  float pv[LPW][8];
  float m = NEG_INF;
#pragma unroll
  for (int t = 0; t < LPW; ++t) {
    const int e0 = (warp + 8 * t) * 256 + lane * 8;
    if (e0 < n) {                                 // e0 + 7 < kend: inside the tiles that were computed
      const float4 a = *reinterpret_cast<const float4*>(s + e0), b = *reinterpret_cast<const float4*>(s + e0 + 4);
      const float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
      if (e0 + 8 <= n) {
#pragma unroll
        for (int x = 0; x < 8; ++x) { pv[t][x] = fmul(v[x], ATT2_SCALE); m = fmaxf(m, pv[t][x]); }
      } else {
#pragma unroll
        for (int x = 0; x < 8; ++x) { pv[t][x] = (e0 + x < n) ? fmul(v[x], ATT2_SCALE) : NEG_INF; m = fmaxf(m, pv[t][x]); }
      }
    } else {
#pragma unroll
      for (int x = 0; x < 8; ++x) pv[t][x] = NEG_INF;
    }
  }
#pragma unroll
  for (int w = 16; w; w >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, w));
  if (nw > 1) {
    if (lane == 0) redf[warp] = m;
    a2_bar(nw * 32);
    m = redf[0];
    for (int w = 1; w < nw; ++w) m = fmaxf(m, redf[w]);
  }
  // exponentials (arguments <= 0; an invisible key has -inf and gives +0), leaf sums of the fixed tree over the keys 0 .. i
  int e = 0;
#pragma unroll
  for (int t = 0; t < LPW; ++t) {
    const int leaf = warp + 8 * t, e0 = leaf * 256 + lane * 8;
    if (leaf < nl) {                               // whole warp
#pragma unroll
      for (int x = 0; x < 8; ++x) pv[t][x] = det_exp_le0(fsub(pv[t][x], m));
      const bool whole = leaf * 256 + 256 <= n;    // no existence tests inside a complete leaf
      const float sum = whole ? warp_tree_full(tree8_full(pv[t])) : warp_tree(tree8(pv[t], e0, n), (long long)leaf * 256, 8, n);
      if (lane == 0) leafs[leaf] = sum;
#pragma unroll
      for (int x = 0; x < 8; ++x) e = max(e, (int)((__float_as_uint(pv[t][x]) >> 23) & 0xFFu));
    } else {
#pragma unroll
      for (int x = 0; x < 8; ++x) pv[t][x] = 0.0f;
    }
  }
#pragma unroll
  for (int w = 16; w; w >>= 1) e = max(e, __shfl_xor_sync(0xffffffffu, e, w));
  if (nw > 1) {
    if (lane == 0) redi[warp] = e;
    a2_bar(nw * 32);                               // leaf sums and exponents are published
    for (int w = 0; w < nw; ++w) e = max(e, redi[w]);
  } else {
    __syncwarp();
  }
  if (warp == 0) {   // the tree over the leaf sums (at most 32 nodes of 256 keys) by one warp: no further barrier
    const float l = warp_tree(lane < nl ? leafs[lane] : 0.0f, 0, 256, n);
    if (lane == 0) {
      lse[row] = fadd(m, det_log(l));
      inv_l[row] = fdiv(1.0f, l);
      Ep[row] = (e == 255) ? (255 | (1 << 30)) : e;
    }
  }
  // slices of bf16(p) for the keys below kend (zeros from i + 1 on)
  const int ee = e == 255 ? 255 : e;
#pragma unroll
  for (int t = 0; t < LPW; ++t) {
    const int e0 = (warp + 8 * t) * 256 + lane * 8;
    if (e0 < kend) {
      uint32_t h8[2] = {0u, 0u}, l8[2] = {0u, 0u};
#pragma unroll
      for (int x = 0; x < 8; ++x) {
        const uint32_t b = bf_bits(pv[t][x]);
        const int ek = (int)(b >> 7) & 0xFF, d = ee - ek;
        const uint32_t tt = (ek == 0 || d >= 14) ? 0u : (((128u + (b & 0x7Fu)) << 6) >> d);
        h8[x >> 2] |= (tt >> 7) << (8 * (x & 3));
        l8[x >> 2] |= (tt & 127u) << (8 * (x & 3));
      }
      *reinterpret_cast<uint2*>(Ph + (size_t)row * S + e0) = make_uint2(h8[0], h8[1]);
      *reinterpret_cast<uint2*>(Pl + (size_t)row * S + e0) = make_uint2(l8[0], l8[1]);
    }
  }
}

struct A2Layout {
  size_t Qh, Ql, Kh, Kl, Eq, Ek, VTh, VTl, Ev, Sraw, Ph, Pl, Ep, invl, total;
};
static A2Layout a2_layout(int B, int H, int S) {
  const size_t Z = (size_t)B * H, rows = Z * S;
  A2Layout L;
  size_t off = 0;
  auto take = [&](size_t bytes) { const size_t o = off; off += align_up(bytes, 256); return o; };
  L.Qh = take(rows * 128); L.Ql = take(rows * 128); L.Kh = take(rows * 128); L.Kl = take(rows * 128);
  L.Eq = take(rows * 4); L.Ek = take(rows * 4);
  L.VTh = take(rows * 128); L.VTl = take(rows * 128); L.Ev = take(Z * 128 * 4);
  L.Sraw = take(rows * S * 4);
  L.Ph = take(rows * S); L.Pl = take(rows * S);
  L.Ep = take(rows * 4); L.invl = take(rows * 4);
  L.total = off;
  return L;
}

}  // namespace det

using namespace det;

extern "C" size_t det_attn_fwd_v2_ws_bytes(int B, int H, int S) {
  if (B <= 0 || H <= 0 || S <= 0) return 0;
  return a2_layout(B, H, S).total;
}

extern "C" int det_attn_fwd_v2(const det_bf16* q, const det_bf16* k, const det_bf16* v, int ld, int B, int H, int S,
                               det_bf16* out, int ld_out, float* lse, void* ws, size_t ws_bytes, void* stream,
                               int* status_dev) {
  if (!q || !k || !v || !out || !lse || B <= 0 || H <= 0 || S <= 0) return DET_ERR_ARG;
  if (S % 128 || S > 256 * 8 * SM2_LPW || ld % 8 || ld_out % 8 || ld < H * 128 || ld_out < H * 128) return DET_ERR_SHAPE;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(ws)) return DET_ERR_ALIGN;
  const A2Layout L = a2_layout(B, H, S);
  if (!ws || ws_bytes < L.total) return DET_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  uint8_t* w = (uint8_t*)ws;
  const int Z = B * H, rows = Z * S;
  int8_t *Qh = (int8_t*)(w + L.Qh), *Ql = (int8_t*)(w + L.Ql), *Kh = (int8_t*)(w + L.Kh), *Kl = (int8_t*)(w + L.Kl);
  int8_t *VTh = (int8_t*)(w + L.VTh), *VTl = (int8_t*)(w + L.VTl), *Ph = (int8_t*)(w + L.Ph), *Pl = (int8_t*)(w + L.Pl);
  int32_t *Eq = (int32_t*)(w + L.Eq), *Ek = (int32_t*)(w + L.Ek), *Ev = (int32_t*)(w + L.Ev), *Ep = (int32_t*)(w + L.Ep);
  float *Sraw = (float*)(w + L.Sraw), *invl = (float*)(w + L.invl);
  if (cudaMemsetAsync(Ev, 0, (size_t)Z * 128 * 4, st) != cudaSuccess) return DET_ERR_CUDA;
  k_slice_heads<<<DET_L((rows + 7) / 8), 256, 0, st>>>(q, ld, H, S, rows, Qh, Ql, Eq);
  k_slice_heads<<<DET_L((rows + 7) / 8), 256, 0, st>>>(k, ld, H, S, rows, Kh, Kl, Ek);
  k_col_exp_heads<<<DET_L(dim3(1, S / 128, Z)), 128, 0, st>>>(v, ld, H, S, Ev);
  k_slice_cols_heads<<<DET_L(dim3(1, S / 128, Z)), 128, 0, st>>>(v, ld, H, S, Ev, VTh, VTl);
  DET_CHECK_LAUNCH();
  SlArgs a = {};
  a.Ea = Eq; a.Eb = Ek; a.out = Sraw; a.rowscale = nullptr;
  a.I = S; a.J = S; a.K = 128; a.Z = Z; a.hdiv = 1; a.o_b = (long long)S * S; a.o_h = 0; a.ldo = S;
  a.causal_tiles = 1; a.krange = 0; a.epi = SL_F32;
  int rc = sliced_gemm_launch(Qh, Ql, Kh, Kl, a, status_dev, st);
  if (rc != DET_OK) return rc;
  if (S <= 2048) k_softmax_v2<1><<<DET_L(rows), 256, 0, st>>>(Sraw, S, lse, invl, Ph, Pl, Ep);
  else k_softmax_v2<SM2_LPW><<<DET_L(rows), 256, 0, st>>>(Sraw, S, lse, invl, Ph, Pl, Ep);
  DET_CHECK_LAUNCH();
  SlArgs u = {};
  u.Ea = Ep; u.Eb = Ev; u.out = out; u.rowscale = invl;
  u.I = S; u.J = 128; u.K = S; u.Z = Z; u.hdiv = H; u.o_b = (long long)S * ld_out; u.o_h = 128; u.ldo = ld_out;
  u.causal_tiles = 0; u.krange = 1; u.epi = SL_BF16_ROWSCALE;
  return sliced_gemm_launch(Ph, Pl, VTh, VTl, u, status_dev, st);
}
