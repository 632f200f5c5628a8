// Elementwise glue (SwiGLU, residual, embedding), the gradient-reduction replay (Algorithm 1 and the
// TreeFold of Algorithm 2), AdamW, and the chunked SHA-256 tensor hash.  All HBM-bound.
#include "common.cuh"
#include "internal.h"

namespace det {

// ------------------------------------------------------------------------------------------------
// SwiGLU: gu [rows, 2F] = (gate | up);  h = silu(gate) * up
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ float sigmoid_det(float g) { return fdiv(1.0f, fadd(1.0f, det_exp(-g))); }

__device__ __forceinline__ void unpack8(const uint4& u, float v[8]) {
  v[0] = bflo(u.x); v[1] = bfhi(u.x); v[2] = bflo(u.y); v[3] = bfhi(u.y);
  v[4] = bflo(u.z); v[5] = bfhi(u.z); v[6] = bflo(u.w); v[7] = bfhi(u.w);
}
__device__ __forceinline__ uint4 pack8(const float v[8]) {
  uint4 u;
  u.x = pack_bf2(v[0], v[1]); u.y = pack_bf2(v[2], v[3]); u.z = pack_bf2(v[4], v[5]); u.w = pack_bf2(v[6], v[7]);
  return u;
}

__global__ void __launch_bounds__(256) k_swiglu_fwd(const uint16_t* __restrict__ gu, int rows, int F,
                                                    uint16_t* __restrict__ h, const float* __restrict__ s_q = nullptr,
                                                    int8_t* __restrict__ qh = nullptr) {
  const size_t per_row = (size_t)F / 8;
  size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= per_row * rows) return;
  size_t r = i / per_row, c = (i % per_row) * 8;
  float g[8], u[8], o[8];
  unpack8(*reinterpret_cast<const uint4*>(gu + r * 2 * F + c), g);
  unpack8(*reinterpret_cast<const uint4*>(gu + r * 2 * F + F + c), u);
#pragma unroll
  for (int t = 0; t < 8; ++t) o[t] = fmul(fmul(g[t], sigmoid_det(g[t])), u[t]);
  *reinterpret_cast<uint4*>(h + r * F + c) = pack8(o);
  if (qh) {   // the next linear's quantiser, applied to the bf16 values just stored
    const float inv_q = fdiv(1.0f, s_q[0]);
#pragma unroll
    for (int t = 0; t < 8; ++t) o[t] = bf2f(f2bf(o[t]));
    *reinterpret_cast<uint2*>(qh + r * F + c) = quant8(o, inv_q);
  }
}

__global__ void __launch_bounds__(256) k_swiglu_bwd(const uint16_t* __restrict__ dh, const uint16_t* __restrict__ gu,
                                                    int rows, int F, uint16_t* __restrict__ dgu) {
  const size_t per_row = (size_t)F / 8;
  size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= per_row * rows) return;
  size_t r = i / per_row, c = (i % per_row) * 8;
  float g[8], u[8], d[8], dg[8], du[8];
  unpack8(*reinterpret_cast<const uint4*>(gu + r * 2 * F + c), g);
  unpack8(*reinterpret_cast<const uint4*>(gu + r * 2 * F + F + c), u);
  unpack8(*reinterpret_cast<const uint4*>(dh + r * F + c), d);
#pragma unroll
  for (int t = 0; t < 8; ++t) {
    float sg = sigmoid_det(g[t]);
    du[t] = fmul(d[t], fmul(g[t], sg));
    dg[t] = fmul(fmul(d[t], u[t]), fmul(sg, fadd(1.0f, fmul(g[t], fsub(1.0f, sg)))));
  }
  *reinterpret_cast<uint4*>(dgu + r * 2 * F + c) = pack8(dg);
  *reinterpret_cast<uint4*>(dgu + r * 2 * F + F + c) = pack8(du);
}

__global__ void __launch_bounds__(256) k_residual(const uint16_t* a, const uint16_t* b, size_t n8, uint16_t* y) {
  size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= n8) return;
  float x[8], z[8], o[8];
  unpack8(reinterpret_cast<const uint4*>(a)[i], x);
  unpack8(reinterpret_cast<const uint4*>(b)[i], z);
#pragma unroll
  for (int t = 0; t < 8; ++t) o[t] = fadd(x[t], z[t]);
  reinterpret_cast<uint4*>(y)[i] = pack8(o);
}

__global__ void __launch_bounds__(256) k_embed_fwd(const int32_t* __restrict__ tok, const uint16_t* __restrict__ E, int V,
                                                   int D, uint16_t* __restrict__ y) {
  const int t = blockIdx.x;
  int v = tok[t];
  v = v < 0 ? 0 : (v >= V ? V - 1 : v);
  const uint4* src = reinterpret_cast<const uint4*>(E + (size_t)v * D);
  uint4* dst = reinterpret_cast<uint4*>(y + (size_t)t * D);
  for (int i = threadIdx.x; i < D / 8; i += 256) dst[i] = src[i];
}

// One CTA per position p.  Only the first occurrence of a token does work: it walks the later
// positions in ascending order and adds the rows of every occurrence sequentially.
__global__ void __launch_bounds__(256) k_embed_bwd(const int32_t* __restrict__ tok, int T, const uint16_t* __restrict__ dy,
                                                   int V, int D, float* __restrict__ dE) {
  __shared__ int s_flag;
  __shared__ int s_list[256];
  __shared__ int s_cnt;
  const int p = blockIdx.x;
  const int v = tok[p];
  if (v < 0 || v >= V) return;
  if (threadIdx.x == 0) s_flag = 0;
  __syncthreads();
  for (int q = threadIdx.x; q < p; q += 256)
    if (tok[q] == v) s_flag = 1;
  __syncthreads();
  if (s_flag) return;
  // accumulators: each thread owns columns threadIdx.x*4 + k*1024
  const int ncol4 = D / 4;
  float4 acc[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int q0 = p; q0 < T; q0 += 256) {
    // ordered list of matches in [q0, q0+256)
    if (threadIdx.x == 0) s_cnt = 0;
    __syncthreads();
    const int q = q0 + threadIdx.x;
    const bool hit = q < T && tok[q] == v;
    const unsigned bal = __ballot_sync(0xffffffffu, hit);
    __shared__ int s_wcnt[8];
    if ((threadIdx.x & 31) == 0) s_wcnt[threadIdx.x >> 5] = __popc(bal);
    __syncthreads();
    int off = 0;
    for (int w = 0; w < (int)(threadIdx.x >> 5); ++w) off += s_wcnt[w];
    if (hit) s_list[off + __popc(bal & ((1u << (threadIdx.x & 31)) - 1))] = q;
    if (threadIdx.x == 255) s_cnt = off + __popc(bal);
    __syncthreads();
    const int cnt = s_cnt;
    for (int j = 0; j < cnt; ++j) {
      const uint16_t* row = dy + (size_t)s_list[j] * D;
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        int c4 = threadIdx.x + k * 256;
        if (c4 < ncol4) {
          uint2 u = *reinterpret_cast<const uint2*>(row + c4 * 4);
          acc[k].x = fadd(acc[k].x, bflo(u.x)); acc[k].y = fadd(acc[k].y, bfhi(u.x));
          acc[k].z = fadd(acc[k].z, bflo(u.y)); acc[k].w = fadd(acc[k].w, bfhi(u.y));
        }
      }
    }
    __syncthreads();
  }
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    int c4 = threadIdx.x + k * 256;
    if (c4 < ncol4) reinterpret_cast<float4*>(dE + (size_t)v * D)[c4] = acc[k];
  }
}

// ------------------------------------------------------------------------------------------------
// Gradient reduction replay (Algorithm 1 + Algorithm 2), fused into one elementwise pass per push:
//   v = (first ? +0 : g_r) + g * (1/accum)
//   at the end of a virtual rank:  v = shard0 ? v : inner + v;  at the last shard: v *= 1/dp_shard and
//   v = lower_k + v for every stack entry that Push pops (top of stack first).
// ------------------------------------------------------------------------------------------------
struct AccumOp {
  const float* g;       // micro-batch gradient
  const float* g_r;     // running per-rank sum (NULL on the first micro-batch of a rank)
  const float* inner;   // running shard sum (NULL at shard 0 or when the rank is not finished)
  const float* lower[8];
  int nlower;
  int rank_end, last_shard;
  float inv_accum, inv_shard;
  float* dst;
};
__global__ void __launch_bounds__(256) k_accum(AccumOp op, size_t n) {
  size_t i = ((size_t)blockIdx.x * 256 + threadIdx.x) * 4;
  if (i >= n) return;
  float4 g = *reinterpret_cast<const float4*>(op.g + i);
  float v[4] = {g.x, g.y, g.z, g.w};
  float r[4] = {0.f, 0.f, 0.f, 0.f};
  if (op.g_r) { float4 t = *reinterpret_cast<const float4*>(op.g_r + i); r[0] = t.x; r[1] = t.y; r[2] = t.z; r[3] = t.w; }
#pragma unroll
  for (int k = 0; k < 4; ++k) v[k] = fadd(r[k], fmul(v[k], op.inv_accum));
  if (op.rank_end) {
    if (op.inner) {
      float4 t = *reinterpret_cast<const float4*>(op.inner + i);
      v[0] = fadd(t.x, v[0]); v[1] = fadd(t.y, v[1]); v[2] = fadd(t.z, v[2]); v[3] = fadd(t.w, v[3]);
    }
    if (op.last_shard) {
#pragma unroll
      for (int k = 0; k < 4; ++k) v[k] = fmul(v[k], op.inv_shard);
#pragma unroll
      for (int l = 0; l < 8; ++l) {  // static indices: the parameter struct must stay in constant space
        if (l < op.nlower) {
          float4 t = *reinterpret_cast<const float4*>(op.lower[l] + i);
          v[0] = fadd(t.x, v[0]); v[1] = fadd(t.y, v[1]); v[2] = fadd(t.z, v[2]); v[3] = fadd(t.w, v[3]);
        }
      }
    }
  }
  *reinterpret_cast<float4*>(op.dst + i) = make_float4(v[0], v[1], v[2], v[3]);
}
struct ResultOp {
  const float* part[34];
  int n;
  float inv_rep;
  float* dst;
};
__global__ void __launch_bounds__(256) k_accum_result(ResultOp op, size_t n) {
  size_t i = ((size_t)blockIdx.x * 256 + threadIdx.x) * 4;
  if (i >= n) return;
  float4 a = *reinterpret_cast<const float4*>(op.part[0] + i);
  float v[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
  for (int s = 1; s < 34; ++s) {
    if (s < op.n) {
      float4 t = *reinterpret_cast<const float4*>(op.part[s] + i);
      v[0] = fadd(t.x, v[0]); v[1] = fadd(t.y, v[1]); v[2] = fadd(t.z, v[2]); v[3] = fadd(t.w, v[3]);
    }
  }
  *reinterpret_cast<float4*>(op.dst + i) =
      make_float4(fmul(v[0], op.inv_rep), fmul(v[1], op.inv_rep), fmul(v[2], op.inv_rep), fmul(v[3], op.inv_rep));
}

// ------------------------------------------------------------------------------------------------
// AdamW
// ------------------------------------------------------------------------------------------------
struct AdamScalars { float b1, b2, omb1, omb2, eps, stepsz, isb2, decay; };
template <bool BF>
__global__ void __launch_bounds__(256) k_adamw(AdamScalars h, void* __restrict__ p, const float* __restrict__ g,
                                               float* __restrict__ m, float* __restrict__ v, size_t n) {
  size_t i = ((size_t)blockIdx.x * 256 + threadIdx.x) * 4;
  if (i >= n) return;
  const int cnt = (n - i) < 4 ? (int)(n - i) : 4;
  float pv[4], gv[4], mv[4], vv[4];
  if (cnt == 4) {
    float4 t = *reinterpret_cast<const float4*>(g + i); gv[0] = t.x; gv[1] = t.y; gv[2] = t.z; gv[3] = t.w;
    t = *reinterpret_cast<const float4*>(m + i); mv[0] = t.x; mv[1] = t.y; mv[2] = t.z; mv[3] = t.w;
    t = *reinterpret_cast<const float4*>(v + i); vv[0] = t.x; vv[1] = t.y; vv[2] = t.z; vv[3] = t.w;
    if (BF) {
      uint2 u = *reinterpret_cast<const uint2*>(reinterpret_cast<uint16_t*>(p) + i);
      pv[0] = bflo(u.x); pv[1] = bfhi(u.x); pv[2] = bflo(u.y); pv[3] = bfhi(u.y);
    } else {
      t = *reinterpret_cast<const float4*>(reinterpret_cast<float*>(p) + i); pv[0] = t.x; pv[1] = t.y; pv[2] = t.z; pv[3] = t.w;
    }
  } else {
    for (int k = 0; k < 4; ++k) {
      bool ok = k < cnt;
      gv[k] = ok ? g[i + k] : 0.f; mv[k] = ok ? m[i + k] : 0.f; vv[k] = ok ? v[i + k] : 0.f;
      pv[k] = ok ? (BF ? bf2f(reinterpret_cast<uint16_t*>(p)[i + k]) : reinterpret_cast<float*>(p)[i + k]) : 0.f;
    }
  }
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    mv[k] = fadd(fmul(h.b1, mv[k]), fmul(h.omb1, gv[k]));
    vv[k] = fadd(fmul(h.b2, vv[k]), fmul(h.omb2, fmul(gv[k], gv[k])));
    float den = fadd(fmul(fsqrt(vv[k]), h.isb2), h.eps);
    pv[k] = fsub(fmul(pv[k], h.decay), fmul(h.stepsz, fdiv(mv[k], den)));
  }
  if (cnt == 4) {
    *reinterpret_cast<float4*>(m + i) = make_float4(mv[0], mv[1], mv[2], mv[3]);
    *reinterpret_cast<float4*>(v + i) = make_float4(vv[0], vv[1], vv[2], vv[3]);
    if (BF) {
      uint2 u; u.x = pack_bf2(pv[0], pv[1]); u.y = pack_bf2(pv[2], pv[3]);
      *reinterpret_cast<uint2*>(reinterpret_cast<uint16_t*>(p) + i) = u;
    } else {
      *reinterpret_cast<float4*>(reinterpret_cast<float*>(p) + i) = make_float4(pv[0], pv[1], pv[2], pv[3]);
    }
  } else {
    for (int k = 0; k < cnt; ++k) {
      m[i + k] = mv[k]; v[i + k] = vv[k];
      if (BF) reinterpret_cast<uint16_t*>(p)[i + k] = f2bf(pv[k]); else reinterpret_cast<float*>(p)[i + k] = pv[k];
    }
  }
}

// ------------------------------------------------------------------------------------------------
// SHA-256 of 4 KiB chunks (of the data at level 1, of the concatenated digests above it): one thread per chunk,
// message words fetched with 128-bit loads.  A chunk is one sequential chain of 64 compressions (~0.1 ms), so the
// small chunk both bounds the latency of the short upper levels and gives a multi-gigabyte tensor hundreds of
// thousands of independent chains to fill the integer pipes.
// ------------------------------------------------------------------------------------------------
__constant__ uint32_t c_K[64] = {
    0x428a2f98, 0x71374491, 0xb5c0fbcf, 0xe9b5dba5, 0x3956c25b, 0x59f111f1, 0x923f82a4, 0xab1c5ed5, 0xd807aa98,
    0x12835b01, 0x243185be, 0x550c7dc3, 0x72be5d74, 0x80deb1fe, 0x9bdc06a7, 0xc19bf174, 0xe49b69c1, 0xefbe4786,
    0x0fc19dc6, 0x240ca1cc, 0x2de92c6f, 0x4a7484aa, 0x5cb0a9dc, 0x76f988da, 0x983e5152, 0xa831c66d, 0xb00327c8,
    0xbf597fc7, 0xc6e00bf3, 0xd5a79147, 0x06ca6351, 0x14292967, 0x27b70a85, 0x2e1b2138, 0x4d2c6dfc, 0x53380d13,
    0x650a7354, 0x766a0abb, 0x81c2c92e, 0x92722c85, 0xa2bfe8a1, 0xa81a664b, 0xc24b8b70, 0xc76c51a3, 0xd192e819,
    0xd6990624, 0xf40e3585, 0x106aa070, 0x19a4c116, 0x1e376c08, 0x2748774c, 0x34b0bcb5, 0x391c0cb3, 0x4ed8aa4a,
    0x5b9cca4f, 0x682e6ff3, 0x748f82ee, 0x78a5636f, 0x84c87814, 0x8cc70208, 0x90befffa, 0xa4506ceb, 0xbef9a3f7,
    0xc67178f2};
__device__ __forceinline__ uint32_t rotr32(uint32_t x, int r) { return __funnelshift_r(x, x, r); }
__device__ __forceinline__ uint32_t bswap(uint32_t x) { return __byte_perm(x, 0, 0x0123); }

__device__ __forceinline__ void sha_rounds(uint32_t h[8], uint32_t w[16]) {
  uint32_t a = h[0], b = h[1], c = h[2], d = h[3], e = h[4], f = h[5], g = h[6], hh = h[7];
#pragma unroll
  for (int i = 0; i < 64; ++i) {
    if (i >= 16) {
      uint32_t w15 = w[(i + 1) & 15], w2 = w[(i + 14) & 15];
      uint32_t s0 = rotr32(w15, 7) ^ rotr32(w15, 18) ^ (w15 >> 3);
      uint32_t s1 = rotr32(w2, 17) ^ rotr32(w2, 19) ^ (w2 >> 10);
      w[i & 15] = w[i & 15] + s0 + w[(i + 9) & 15] + s1;
    }
    uint32_t t1 = hh + (rotr32(e, 6) ^ rotr32(e, 11) ^ rotr32(e, 25)) + ((e & f) ^ (~e & g)) + c_K[i] + w[i & 15];
    uint32_t t2 = (rotr32(a, 2) ^ rotr32(a, 13) ^ rotr32(a, 22)) + ((a & b) ^ (a & c) ^ (b & c));
    hh = g; g = f; f = e; e = d + t1; d = c; c = b; b = a; a = t1 + t2;
  }
  h[0] += a; h[1] += b; h[2] += c; h[3] += d; h[4] += e; h[5] += f; h[6] += g; h[7] += hh;
}

__global__ void __launch_bounds__(64) k_sha_chunks(const uint8_t* __restrict__ data, size_t nbytes, size_t nchunks,
                                                   uint8_t* __restrict__ digests) {
  size_t c = (size_t)blockIdx.x * 64 + threadIdx.x;
  if (c >= nchunks) return;
  const size_t CH = 4096;
  const uint8_t* p = data + c * CH;
  const size_t len = (c + 1) * CH <= nbytes ? CH : nbytes - c * CH;
  uint32_t h[8] = {0x6a09e667, 0xbb67ae85, 0x3c6ef372, 0xa54ff53a, 0x510e527f, 0x9b05688c, 0x1f83d9ab, 0x5be0cd19};
  uint32_t w[16];
  const size_t full = len / 64;
  // the next 64-byte block is fetched while the 64 rounds of the current one run
  uint4 nx[4];
  if (full) {
#pragma unroll
    for (int k = 0; k < 4; ++k) nx[k] = __ldg(reinterpret_cast<const uint4*>(p) + k);
  }
  for (size_t b = 0; b < full; ++b) {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint4 u = nx[k];
      w[4 * k] = bswap(u.x); w[4 * k + 1] = bswap(u.y); w[4 * k + 2] = bswap(u.z); w[4 * k + 3] = bswap(u.w);
    }
    if (b + 1 < full) {
      const uint4* q = reinterpret_cast<const uint4*>(p + (b + 1) * 64);
#pragma unroll
      for (int k = 0; k < 4; ++k) nx[k] = __ldg(q + k);
    }
    sha_rounds(h, w);
  }
  // tail with padding (one or two blocks)
  const size_t rem = len - full * 64;
  uint8_t tail[128];
  for (int i = 0; i < 128; ++i) tail[i] = 0;
  for (size_t i = 0; i < rem; ++i) tail[i] = p[full * 64 + i];
  tail[rem] = 0x80;
  const int tl = (rem + 9 <= 64) ? 64 : 128;
  const unsigned long long bits = (unsigned long long)len * 8ull;
  for (int i = 0; i < 8; ++i) tail[tl - 1 - i] = (uint8_t)(bits >> (8 * i));
  for (int b = 0; b < tl / 64; ++b) {
    for (int k = 0; k < 16; ++k)
      w[k] = ((uint32_t)tail[b * 64 + 4 * k] << 24) | ((uint32_t)tail[b * 64 + 4 * k + 1] << 16) |
             ((uint32_t)tail[b * 64 + 4 * k + 2] << 8) | (uint32_t)tail[b * 64 + 4 * k + 3];
    sha_rounds(h, w);
  }
  uint4* o = reinterpret_cast<uint4*>(digests + c * 32);
  o[0] = make_uint4(bswap(h[0]), bswap(h[1]), bswap(h[2]), bswap(h[3]));
  o[1] = make_uint4(bswap(h[4]), bswap(h[5]), bswap(h[6]), bswap(h[7]));
}

// Root of the tree: SHA-256(the nd <= 128 remaining digests || u64le(nbytes)), one thread (at most 65 compressions).
__global__ void k_sha_root(const uint8_t* __restrict__ digests, int nd, unsigned long long nbytes, uint8_t* __restrict__ out32) {
  uint32_t h[8] = {0x6a09e667, 0xbb67ae85, 0x3c6ef372, 0xa54ff53a, 0x510e527f, 0x9b05688c, 0x1f83d9ab, 0x5be0cd19};
  uint32_t w[16];
  const uint4* d4 = reinterpret_cast<const uint4*>(digests);
  for (int b = 0; b < nd / 2; ++b) {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint4 u = d4[4 * b + k];
      w[4 * k] = bswap(u.x); w[4 * k + 1] = bswap(u.y); w[4 * k + 2] = bswap(u.z); w[4 * k + 3] = bswap(u.w);
    }
    sha_rounds(h, w);
  }
  // last block: an odd digest (32 bytes), the length word (8 bytes, little endian), 0x80, zeros, the bit count
#pragma unroll
  for (int k = 0; k < 16; ++k) w[k] = 0;
  int pos = 0;   // words filled
  if (nd & 1) {
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const uint4 u = d4[2 * (nd - 1) + k];
      w[4 * k] = bswap(u.x); w[4 * k + 1] = bswap(u.y); w[4 * k + 2] = bswap(u.z); w[4 * k + 3] = bswap(u.w);
    }
    pos = 8;
  }
  const uint32_t lo = (uint32_t)nbytes, hi = (uint32_t)(nbytes >> 32);
  const uint32_t wl = bswap(lo), wh = bswap(hi), pad = 0x80000000u;
  if (pos == 0) { w[0] = wl; w[1] = wh; w[2] = pad; } else { w[8] = wl; w[9] = wh; w[10] = pad; }
  const unsigned long long bits = ((unsigned long long)nd * 32ull + 8ull) * 8ull;
  w[14] = (uint32_t)(bits >> 32);
  w[15] = (uint32_t)bits;
  sha_rounds(h, w);
  uint4* o = reinterpret_cast<uint4*>(out32);
  o[0] = make_uint4(bswap(h[0]), bswap(h[1]), bswap(h[2]), bswap(h[3]));
  o[1] = make_uint4(bswap(h[4]), bswap(h[5]), bswap(h[6]), bswap(h[7]));
}

static double ipow(double b, int e) {
  double r = 1.0;
  while (e > 0) { if (e & 1) r *= b; b *= b; e >>= 1; }
  return r;
}

}  // namespace det

using namespace det;

extern "C" int det_swiglu_fwd(const det_bf16* gu, int rows, int F, det_bf16* h, void* stream) {
  if (!gu || !h || rows < 0 || F <= 0) return DET_ERR_ARG;
  if (F % 8) return DET_ERR_SHAPE;
  if (!aligned16(gu) || !aligned16(h)) return DET_ERR_ALIGN;
  size_t n = (size_t)rows * (F / 8);
  if (!n) return DET_OK;
  k_swiglu_fwd<<<DET_L((unsigned)((n + 255) / 256)), 256, 0, (cudaStream_t)stream>>>(gu, rows, F, h);
  DET_CHECK_LAUNCH();
  return DET_OK;
}
extern "C" int det_swiglu_fwd_q(const det_bf16* gu, int rows, int F, det_bf16* h, const float* s_q, int8_t* qh, void* stream) {
  if (!gu || !h || !s_q || !qh || rows < 0 || F <= 0) return DET_ERR_ARG;
  if (F % 8) return DET_ERR_SHAPE;
  if (!aligned16(gu) || !aligned16(h) || (((uintptr_t)qh) & 7u)) return DET_ERR_ALIGN;
  size_t n = (size_t)rows * (F / 8);
  if (!n) return DET_OK;
  k_swiglu_fwd<<<DET_L((unsigned)((n + 255) / 256)), 256, 0, (cudaStream_t)stream>>>(gu, rows, F, h, s_q, qh);
  DET_CHECK_LAUNCH();
  return DET_OK;
}
extern "C" int det_swiglu_bwd(const det_bf16* dh, const det_bf16* gu, int rows, int F, det_bf16* dgu, void* stream) {
  if (!gu || !dh || !dgu || rows < 0 || F <= 0) return DET_ERR_ARG;
  if (F % 8) return DET_ERR_SHAPE;
  if (!aligned16(gu) || !aligned16(dh) || !aligned16(dgu)) return DET_ERR_ALIGN;
  size_t n = (size_t)rows * (F / 8);
  if (!n) return DET_OK;
  k_swiglu_bwd<<<DET_L((unsigned)((n + 255) / 256)), 256, 0, (cudaStream_t)stream>>>(dh, gu, rows, F, dgu);
  DET_CHECK_LAUNCH();
  return DET_OK;
}
extern "C" int det_residual_add(const det_bf16* a, const det_bf16* b, size_t n, det_bf16* y, void* stream) {
  if ((n && (!a || !b || !y))) return DET_ERR_ARG;
  if (n % 8) return DET_ERR_SHAPE;
  if (!aligned16(a) || !aligned16(b) || !aligned16(y)) return DET_ERR_ALIGN;
  if (!n) return DET_OK;
  k_residual<<<DET_L((unsigned)((n / 8 + 255) / 256)), 256, 0, (cudaStream_t)stream>>>(a, b, n / 8, y);
  DET_CHECK_LAUNCH();
  return DET_OK;
}
extern "C" int det_embed_fwd(const int32_t* tok, int T, const det_bf16* E, int V, int D, det_bf16* y, void* stream) {
  if (!tok || !E || !y || T < 0 || V <= 0 || D <= 0) return DET_ERR_ARG;
  if (D % 8) return DET_ERR_SHAPE;
  if (!aligned16(E) || !aligned16(y)) return DET_ERR_ALIGN;
  if (!T) return DET_OK;
  k_embed_fwd<<<DET_L(T), 256, 0, (cudaStream_t)stream>>>(tok, E, V, D, y);
  DET_CHECK_LAUNCH();
  return DET_OK;
}
extern "C" int det_embed_bwd(const int32_t* tok, int T, const det_bf16* dy, int V, int D, float* dE, void* stream) {
  if (!tok || !dy || !dE || T < 0 || V <= 0 || D <= 0) return DET_ERR_ARG;
  if (D % 4 || D > 8192) return DET_ERR_SHAPE;
  if (!aligned16(dy) || !aligned16(dE)) return DET_ERR_ALIGN;
  cudaStream_t st = (cudaStream_t)stream;
  cudaMemsetAsync(dE, 0, (size_t)V * D * sizeof(float), st);
  if (T) k_embed_bwd<<<DET_L(T), 256, 0, st>>>(tok, T, dy, V, D, dE);
  DET_CHECK_LAUNCH();
  return DET_OK;
}

extern "C" int det_grad_accum_nbufs(int dp_replicate) {
  if (dp_replicate < 1) return DET_ERR_ARG;
  int lg = 0;
  while ((1 << (lg + 1)) <= dp_replicate) ++lg;
  return 2 + lg;
}
extern "C" int det_grad_accum_init(det_accum* st, int accum, int dp_shard, int dp_replicate, size_t n, float* bufs) {
  if (!st || accum < 1 || dp_shard < 1 || dp_replicate < 1 || !bufs) return DET_ERR_ARG;
  if (n % 4) return DET_ERR_SHAPE;
  if (!aligned16(bufs)) return DET_ERR_ALIGN;
  int nb = det_grad_accum_nbufs(dp_replicate);
  if (nb > 34) return DET_ERR_SHAPE;
  st->accum = accum; st->dp_shard = dp_shard; st->dp_replicate = dp_replicate;
  st->pushes = 0; st->nstack = 0; st->n = n; st->bufs = bufs; st->inner_slot = -1; st->gr_slot = -1;
  st->free_mask = (nb >= 64) ? ~0ull : ((1ull << nb) - 1ull);
  return DET_OK;
}
static int take_slot(det_accum* st) {
  for (int s = 0; s < 64; ++s)
    if (st->free_mask & (1ull << s)) { st->free_mask &= ~(1ull << s); return s; }
  return -1;
}
extern "C" int det_grad_accum_push(det_accum* st, const float* g, void* stream) {
  if (!st || !g) return DET_ERR_ARG;
  if (!aligned16(g)) return DET_ERR_ALIGN;
  const int N = st->dp_shard * st->dp_replicate;
  if (st->pushes >= st->accum * N) return DET_ERR_ARG;
  const int r = st->pushes / st->accum, kk = st->pushes % st->accum, shard = r % st->dp_shard;
  const size_t n = st->n;
  AccumOp op;
  op.g = g;
  op.inv_accum = (float)(1.0 / (double)st->accum);
  op.inv_shard = (float)(1.0 / (double)st->dp_shard);
  op.nlower = 0;
  op.rank_end = (kk == st->accum - 1);
  op.last_shard = (shard == st->dp_shard - 1);
  op.inner = nullptr;
  op.g_r = (kk == 0) ? nullptr : st->bufs + (size_t)st->gr_slot * n;
  if (kk == 0) st->gr_slot = -1;
  int dst_slot;
  int popped[34], npop = 0;
  if (!op.rank_end) {
    dst_slot = (st->gr_slot >= 0) ? st->gr_slot : take_slot(st);
    st->gr_slot = dst_slot;
  } else {
    if (shard != 0) {
      // inner <- inner + g_r, written over the inner buffer; the g_r buffer goes back to the pool
      op.inner = st->bufs + (size_t)st->inner_slot * n;
      dst_slot = st->inner_slot;
      if (st->gr_slot >= 0) st->free_mask |= (1ull << st->gr_slot);
    } else {
      // inner <- g_r: the g_r buffer simply becomes the inner buffer (no copy)
      dst_slot = (st->gr_slot >= 0) ? st->gr_slot : take_slot(st);
    }
    st->gr_slot = -1;
    if (op.last_shard) {
      int level = 0;
      while (st->nstack > 0 && st->level[st->nstack - 1] == level) {
        --st->nstack;
        popped[npop++] = st->slot[st->nstack];
        ++level;
      }
      if (npop > 8) return DET_ERR_SHAPE;
      for (int l = 0; l < npop; ++l) op.lower[l] = st->bufs + (size_t)popped[l] * n;
      op.nlower = npop;
      st->level[st->nstack] = level;
      st->slot[st->nstack] = dst_slot;
      ++st->nstack;
      st->inner_slot = -1;
    } else {
      st->inner_slot = dst_slot;
    }
  }
  if (dst_slot < 0) return DET_ERR_ARG;
  op.dst = st->bufs + (size_t)dst_slot * n;
  if (n) k_accum<<<DET_L((unsigned)((n / 4 + 255) / 256)), 256, 0, (cudaStream_t)stream>>>(op, n);
  for (int l = 0; l < npop; ++l) st->free_mask |= (1ull << popped[l]);
  st->pushes++;
  DET_CHECK_LAUNCH();
  return DET_OK;
}
extern "C" int det_grad_accum_result(det_accum* st, float* g_out, void* stream) {
  if (!st || !g_out) return DET_ERR_ARG;
  if (!aligned16(g_out)) return DET_ERR_ALIGN;
  if (st->pushes != st->accum * st->dp_shard * st->dp_replicate || st->nstack < 1) return DET_ERR_ARG;
  ResultOp op;
  op.n = st->nstack;
  // lowest level (top of the stack) first, then ascending level
  for (int s = 0; s < st->nstack; ++s) op.part[s] = st->bufs + (size_t)st->slot[st->nstack - 1 - s] * st->n;
  op.inv_rep = (float)(1.0 / (double)st->dp_replicate);
  op.dst = g_out;
  if (st->n) k_accum_result<<<DET_L((unsigned)((st->n / 4 + 255) / 256)), 256, 0, (cudaStream_t)stream>>>(op, st->n);
  DET_CHECK_LAUNCH();
  return DET_OK;
}

extern "C" int det_adamw_step(const det_adamw_desc* d, int pdtype, void* p, const float* g, float* m, float* v,
                              size_t n, void* stream) {
  if (!d || !p || !g || !m || !v || d->step < 1 || (pdtype != DET_F32 && pdtype != DET_BF16)) return DET_ERR_ARG;
  if (!aligned16(g) || !aligned16(m) || !aligned16(v) || (((uintptr_t)p) & 7u)) return DET_ERR_ALIGN;
  if (pdtype == DET_F32 && !aligned16(p)) return DET_ERR_ALIGN;
  if (!n) return DET_OK;
  const double bc1 = 1.0 - ipow(d->beta1, d->step), bc2 = 1.0 - ipow(d->beta2, d->step);
  AdamScalars h;
  h.b1 = (float)d->beta1; h.b2 = (float)d->beta2;
  h.omb1 = 1.0f - h.b1; h.omb2 = 1.0f - h.b2;
  h.eps = (float)d->eps;
  h.stepsz = (float)(d->lr / bc1);
  h.isb2 = (float)(1.0 / sqrt(bc2));
  h.decay = (float)(1.0 - d->lr * d->weight_decay);
  unsigned grid = (unsigned)((n + 1023) / 1024);
  if (pdtype == DET_BF16) k_adamw<true><<<DET_L(grid), 256, 0, (cudaStream_t)stream>>>(h, p, g, m, v, n);
  else k_adamw<false><<<DET_L(grid), 256, 0, (cudaStream_t)stream>>>(h, p, g, m, v, n);
  DET_CHECK_LAUNCH();
  return DET_OK;
}

// Workspace: two areas of level-1 size, ping-ponged by the levels, and 256 bytes for the root of the synchronising call.
static inline size_t hash_l1_bytes(size_t nbytes) { return align_up(((nbytes + 4095) / 4096) * 32 + 32, 256); }
extern "C" size_t det_tensor_hash_ws_bytes(size_t nbytes) {
  return hash_l1_bytes(nbytes) + hash_l1_bytes(hash_l1_bytes(nbytes)) + 256;
}

extern "C" int det_tensor_hash_async(const void* p, size_t nbytes, uint8_t* out32_dev, void* ws, size_t ws_bytes,
                                     void* stream) {
  if ((nbytes && !p) || !out32_dev) return DET_ERR_ARG;
  if ((nbytes && !aligned16(p)) || !aligned16(out32_dev)) return DET_ERR_ALIGN;
  if (ws_bytes < det_tensor_hash_ws_bytes(nbytes) || !ws || !aligned16(ws)) return DET_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  uint8_t* a = (uint8_t*)ws;
  uint8_t* b = a + hash_l1_bytes(nbytes);
  size_t nc = (nbytes + 4095) / 4096;
  if (nc) k_sha_chunks<<<DET_L((unsigned)((nc + 63) / 64)), 64, 0, st>>>((const uint8_t*)p, nbytes, nc, a);
  DET_CHECK_LAUNCH();
  while (nc > 128) {
    const size_t lb = nc * 32, m = (lb + 4095) / 4096;
    k_sha_chunks<<<DET_L((unsigned)((m + 63) / 64)), 64, 0, st>>>(a, lb, m, b);
    DET_CHECK_LAUNCH();
    uint8_t* t = a; a = b; b = t;
    nc = m;
  }
  k_sha_root<<<DET_L(1), 1, 0, st>>>(a, (int)nc, (unsigned long long)nbytes, out32_dev);
  DET_CHECK_LAUNCH();
  return DET_OK;
}

extern "C" int det_tensor_hash(const void* p, size_t nbytes, uint8_t* out32_host, void* ws, size_t ws_bytes,
                               void* stream) {
  if (!out32_host) return DET_ERR_ARG;
  if (ws_bytes < det_tensor_hash_ws_bytes(nbytes) || !ws || !aligned16(ws)) return DET_ERR_WORKSPACE;
  uint8_t* root = (uint8_t*)ws + det_tensor_hash_ws_bytes(nbytes) - 256;
  int rc = det_tensor_hash_async(p, nbytes, root, ws, ws_bytes, stream);
  if (rc != DET_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMemcpyAsync(out32_host, root, 32, cudaMemcpyDeviceToHost, st) != cudaSuccess) return DET_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return DET_ERR_CUDA;
  return DET_OK;
}
