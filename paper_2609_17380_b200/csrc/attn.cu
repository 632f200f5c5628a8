// Causal attention, head_dim 128, in a fixed order on the FP32 ALUs (Sec. 3.2: QK^T and softmax stay in
// higher precision; the backward recomputes the weights in full precision and is not quantised).
//
// Forward: online softmax over KV tiles of 128 keys in ascending order.  Each logit is a sequential
// ascending sum over the 128 head dimensions of exact bf16 products; the tile's row sum is the adjacent
// pairwise tree over its 128 slots (masked slots are +0); P is rounded to bf16 before P.V; P.V is a
// sequential ascending sum over the tile's keys from +0, then o = o*alpha + u.
// Backward: P = exp(S - L) recomputed; dV, dK (per key) and dQ (per query) are single accumulators fed in
// ascending order of the contraction index; bf16(dS) goes through global scratch from the dK/dV kernel to
// the dQ kernel, so nothing is accumulated with atomics.
#include "common.cuh"
#include "internal.h"

namespace det {

#define ATT_SCALE 0x1.6a09e6p-4f
constexpr int DH = 128;

__device__ __forceinline__ void unpack8a(const uint4& u, float v[8]) {
  v[0] = bflo(u.x); v[1] = bfhi(u.x); v[2] = bflo(u.y); v[3] = bfhi(u.y);
  v[4] = bflo(u.z); v[5] = bfhi(u.z); v[6] = bflo(u.w); v[7] = bfhi(u.w);
}

// ---------------------------------------------------------------------------------------------
// forward: CTA = 64 queries of one (batch, head); 256 threads, thread = 4 queries x 8 keys / 8 dims
// ---------------------------------------------------------------------------------------------
constexpr int FQ = 64, FK = 128;
constexpr int LQ = FQ + 4, LK = FK + 4;
constexpr size_t FWD_SMEM = (size_t)(DH * LQ + DH * LK + FK * LQ + FK * LK) * sizeof(float);

__global__ void __launch_bounds__(256, 1) k_attn_fwd(const uint16_t* __restrict__ q, const uint16_t* __restrict__ k,
                                                     const uint16_t* __restrict__ v, int ld, int H, int S,
                                                     uint16_t* __restrict__ out, int ld_out, float* __restrict__ lse) {
  extern __shared__ __align__(16) float sm[];
  float(*Qs)[LQ] = reinterpret_cast<float(*)[LQ]>(sm);                                   // [dim][query]
  float(*Ks)[LK] = reinterpret_cast<float(*)[LK]>(sm + DH * LQ);                         // [dim][key]
  float(*Ps)[LQ] = reinterpret_cast<float(*)[LQ]>(sm + DH * LQ + DH * LK);               // [key][query]
  float(*Vs)[LK] = reinterpret_cast<float(*)[LK]>(sm + DH * LQ + DH * LK + FK * LQ);     // [key][dim]
  const int qb = gridDim.x - 1 - blockIdx.x;  // longest rows first
  const int h = blockIdx.y, b = blockIdx.z;
  const int q0 = qb * FQ;
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const size_t row0 = (size_t)b * S;
  const uint16_t* qp = q + row0 * ld + (size_t)h * DH;
  const uint16_t* kp = k + row0 * ld + (size_t)h * DH;
  const uint16_t* vp = v + row0 * ld + (size_t)h * DH;

  for (int idx = tid; idx < FQ * 16; idx += 256) {
    const int r = idx & 63, ch = idx >> 6;
    float t[8];
    unpack8a(__ldg(reinterpret_cast<const uint4*>(qp + (size_t)(q0 + r) * ld + ch * 8)), t);
#pragma unroll
    for (int e = 0; e < 8; ++e) Qs[ch * 8 + e][r] = t[e];
  }
  float m[4], l[4], o[4][8];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    m[i] = __int_as_float(0xff800000);
    l[i] = 0.0f;
#pragma unroll
    for (int e = 0; e < 8; ++e) o[i][e] = 0.0f;
  }
  const int ntiles = q0 / FK + 1;
  for (int jt = 0; jt < ntiles; ++jt) {
    const int j0 = jt * FK;
    const int kmax = min(FK, q0 + FQ - j0);  // keys of this tile that some row of the block can see
    __syncthreads();
    for (int idx = tid; idx < FK * 16; idx += 256) {
      const int key = idx & 127, ch = idx >> 7;
      float t[8];
      if (j0 + key < S) unpack8a(__ldg(reinterpret_cast<const uint4*>(kp + (size_t)(j0 + key) * ld + ch * 8)), t);
      else {
#pragma unroll
        for (int e = 0; e < 8; ++e) t[e] = 0.0f;
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) Ks[ch * 8 + e][key] = t[e];
    }
    for (int idx = tid; idx < FK * 16; idx += 256) {
      const int key = idx >> 4, ch = idx & 15;
      float t[8];
      if (j0 + key < S) unpack8a(__ldg(reinterpret_cast<const uint4*>(vp + (size_t)(j0 + key) * ld + ch * 8)), t);
      else {
#pragma unroll
        for (int e = 0; e < 8; ++e) t[e] = 0.0f;
      }
      *reinterpret_cast<float4*>(&Vs[key][ch * 8]) = make_float4(t[0], t[1], t[2], t[3]);
      *reinterpret_cast<float4*>(&Vs[key][ch * 8 + 4]) = make_float4(t[4], t[5], t[6], t[7]);
    }
    __syncthreads();
    // logits
    float s[4][8];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int e = 0; e < 8; ++e) s[i][e] = 0.0f;
    if (kmax > 64) {
#pragma unroll 4
      for (int d = 0; d < DH; ++d) {
        const float4 a = *reinterpret_cast<const float4*>(&Qs[d][ty * 4]);
        const float4 b0 = *reinterpret_cast<const float4*>(&Ks[d][tx * 4]);
        const float4 b1 = *reinterpret_cast<const float4*>(&Ks[d][64 + tx * 4]);
        const float ar[4] = {a.x, a.y, a.z, a.w};
        const float br[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int e = 0; e < 8; ++e) s[i][e] = fadd(s[i][e], fmul(ar[i], br[e]));
      }
    } else {
#pragma unroll 4
      for (int d = 0; d < DH; ++d) {
        const float4 a = *reinterpret_cast<const float4*>(&Qs[d][ty * 4]);
        const float4 b0 = *reinterpret_cast<const float4*>(&Ks[d][tx * 4]);
        const float ar[4] = {a.x, a.y, a.z, a.w};
        const float br[4] = {b0.x, b0.y, b0.z, b0.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int e = 0; e < 4; ++e) s[i][e] = fadd(s[i][e], fmul(ar[i], br[e]));
      }
    }
    // online softmax statistics per row
    float alpha[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int row = q0 + ty * 4 + i;
      float mt = m[i];
      bool valid[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int key = j0 + ((e < 4) ? (tx * 4 + e) : (64 + tx * 4 + e - 4));
        valid[e] = key <= row;
        s[i][e] = fmul(s[i][e], ATT_SCALE);
        if (valid[e]) mt = fmaxf(mt, s[i][e]);
      }
#pragma unroll
      for (int w = 1; w < 16; w <<= 1) mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, w));
      alpha[i] = det_exp(fsub(m[i], mt));
      float p[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) p[e] = valid[e] ? det_exp(fsub(s[i][e], mt)) : 0.0f;
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int kl = (e < 4) ? (tx * 4 + e) : (64 + tx * 4 + e - 4);
        Ps[kl][ty * 4 + i] = bf2f(f2bf(p[e]));
      }
      float h0 = fadd(fadd(p[0], p[1]), fadd(p[2], p[3]));
      float h1 = fadd(fadd(p[4], p[5]), fadd(p[6], p[7]));
#pragma unroll
      for (int w = 1; w < 16; w <<= 1) {
        h0 = fadd(h0, __shfl_xor_sync(0xffffffffu, h0, w));
        h1 = fadd(h1, __shfl_xor_sync(0xffffffffu, h1, w));
      }
      l[i] = fadd(fmul(l[i], alpha[i]), fadd(h0, h1));
      m[i] = mt;
    }
    __syncthreads();
    // u = P~ . V over the tile's keys in ascending order, then o = o*alpha + u
    float u[4][8];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int e = 0; e < 8; ++e) u[i][e] = 0.0f;
#pragma unroll 4
    for (int j = 0; j < kmax; ++j) {
      const float4 a = *reinterpret_cast<const float4*>(&Ps[j][ty * 4]);
      const float4 b0 = *reinterpret_cast<const float4*>(&Vs[j][tx * 4]);
      const float4 b1 = *reinterpret_cast<const float4*>(&Vs[j][64 + tx * 4]);
      const float ar[4] = {a.x, a.y, a.z, a.w};
      const float br[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int e = 0; e < 8; ++e) u[i][e] = fadd(u[i][e], fmul(ar[i], br[e]));
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int e = 0; e < 8; ++e) o[i][e] = fadd(fmul(o[i][e], alpha[i]), u[i][e]);
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int row = q0 + ty * 4 + i;
    const float il = fdiv(1.0f, l[i]);
    uint16_t* op = out + (row0 + row) * ld_out + (size_t)h * DH;
    uint2 w0, w1;
    w0.x = pack_bf2(fmul(o[i][0], il), fmul(o[i][1], il)); w0.y = pack_bf2(fmul(o[i][2], il), fmul(o[i][3], il));
    w1.x = pack_bf2(fmul(o[i][4], il), fmul(o[i][5], il)); w1.y = pack_bf2(fmul(o[i][6], il), fmul(o[i][7], il));
    *reinterpret_cast<uint2*>(op + tx * 4) = w0;
    *reinterpret_cast<uint2*>(op + 64 + tx * 4) = w1;
    if (tx == 0) lse[((size_t)b * H + h) * S + row] = fadd(m[i], det_log(l[i]));
  }
}

// ---------------------------------------------------------------------------------------------
// backward
// ---------------------------------------------------------------------------------------------
// Delta_i = adjacent tree over the 128 dims of dO_ic * O_ic; one warp per (b, h, i)
__global__ void __launch_bounds__(256) k_attn_delta(const uint16_t* __restrict__ dout, const uint16_t* __restrict__ out,
                                                    int ld_out, int H, int S, size_t nrows, float* __restrict__ delta) {
  const size_t w = (size_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (w >= nrows) return;  // w = (b*H + h)*S + i
  const size_t i = w % S, bh = w / S, b = bh / H, h = bh % H;
  const size_t off = (b * S + i) * ld_out + h * DH + lane * 4;
  const uint2 a = __ldg(reinterpret_cast<const uint2*>(dout + off));
  const uint2 c = __ldg(reinterpret_cast<const uint2*>(out + off));
  float t = fadd(fadd(fmul(bflo(a.x), bflo(c.x)), fmul(bfhi(a.x), bfhi(c.x))),
                 fadd(fmul(bflo(a.y), bflo(c.y)), fmul(bfhi(a.y), bfhi(c.y))));
  t = warp_tree_full(t);
  if (lane == 0) delta[w] = t;
}

constexpr int BT = 64;        // tile edge for the backward
constexpr int LN = DH + 4;    // row pitch of [row][dim] tiles
constexpr int LP = BT + 4;    // row pitch of [query][key] tiles
constexpr size_t DKDV_SMEM = (size_t)(4 * BT * LN + 2 * BT * LP + 2 * BT) * sizeof(float);
constexpr size_t DQ_SMEM = (size_t)(BT * LN + BT * LP) * sizeof(float);

__device__ __forceinline__ void load_tile_nat(float (*dst)[LN], const uint16_t* base, int ld, int r0, int S) {
  for (int idx = threadIdx.x; idx < BT * 16; idx += 256) {
    const int r = idx >> 4, ch = idx & 15;
    float t[8];
    if (r0 + r < S) unpack8a(__ldg(reinterpret_cast<const uint4*>(base + (size_t)(r0 + r) * ld + ch * 8)), t);
    else {
#pragma unroll
      for (int e = 0; e < 8; ++e) t[e] = 0.0f;
    }
    *reinterpret_cast<float4*>(&dst[r][ch * 8]) = make_float4(t[0], t[1], t[2], t[3]);
    *reinterpret_cast<float4*>(&dst[r][ch * 8 + 4]) = make_float4(t[4], t[5], t[6], t[7]);
  }
}

// CTA = 64 keys of one (batch, head); loops over query tiles in ascending order
__global__ void __launch_bounds__(256, 1)
    k_attn_dkdv(const uint16_t* __restrict__ dout, const uint16_t* __restrict__ q, const uint16_t* __restrict__ k,
                const uint16_t* __restrict__ v, const float* __restrict__ lse, const float* __restrict__ delta, int ld,
                int ld_out, int H, int S, uint16_t* __restrict__ dk, uint16_t* __restrict__ dv, int ld_d,
                uint16_t* __restrict__ dS) {
  extern __shared__ __align__(16) float sm[];
  float(*Kn)[LN] = reinterpret_cast<float(*)[LN]>(sm);
  float(*Vn)[LN] = reinterpret_cast<float(*)[LN]>(sm + BT * LN);
  float(*Qn)[LN] = reinterpret_cast<float(*)[LN]>(sm + 2 * BT * LN);
  float(*On)[LN] = reinterpret_cast<float(*)[LN]>(sm + 3 * BT * LN);
  float(*Pt)[LP] = reinterpret_cast<float(*)[LP]>(sm + 4 * BT * LN);
  float(*St)[LP] = reinterpret_cast<float(*)[LP]>(sm + 4 * BT * LN + BT * LP);
  float* Ls = sm + 4 * BT * LN + 2 * BT * LP;
  float* Ds = Ls + BT;
  const int jb = blockIdx.x;  // small jb = most query tiles; blocks are issued in that order
  const int h = blockIdx.y, b = blockIdx.z;
  const int j0 = jb * BT;
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const size_t row0 = (size_t)b * S;
  const size_t bh = (size_t)b * H + h;
  load_tile_nat(Kn, k + row0 * ld + (size_t)h * DH, ld, j0, S);
  load_tile_nat(Vn, v + row0 * ld + (size_t)h * DH, ld, j0, S);
  float dvv[4][8], dkk[4][8];
#pragma unroll
  for (int e = 0; e < 4; ++e)
#pragma unroll
    for (int c = 0; c < 8; ++c) { dvv[e][c] = 0.0f; dkk[e][c] = 0.0f; }
  const int nt = S / BT;
  for (int it = jb; it < nt; ++it) {
    const int i0 = it * BT;
    __syncthreads();
    load_tile_nat(Qn, q + row0 * ld + (size_t)h * DH, ld, i0, S);
    load_tile_nat(On, dout + row0 * ld_out + (size_t)h * DH, ld_out, i0, S);
    if (tid < BT) { Ls[tid] = lse[bh * S + i0 + tid]; Ds[tid] = delta[bh * S + i0 + tid]; }
    __syncthreads();
    // S = q.k and dP = dO.v, thread = queries ty+16e x keys tx+16f, sequential over the 128 dims
    float s[4][4], dp[4][4];
#pragma unroll
    for (int e = 0; e < 4; ++e)
#pragma unroll
      for (int f = 0; f < 4; ++f) { s[e][f] = 0.0f; dp[e][f] = 0.0f; }
#pragma unroll 2
    for (int d = 0; d < DH; d += 4) {
      float4 qa[4], ka[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        qa[e] = *reinterpret_cast<const float4*>(&Qn[ty + 16 * e][d]);
        ka[e] = *reinterpret_cast<const float4*>(&Kn[tx + 16 * e][d]);
      }
#pragma unroll
      for (int e = 0; e < 4; ++e)
#pragma unroll
        for (int f = 0; f < 4; ++f) {
          s[e][f] = fadd(s[e][f], fmul(qa[e].x, ka[f].x));
          s[e][f] = fadd(s[e][f], fmul(qa[e].y, ka[f].y));
          s[e][f] = fadd(s[e][f], fmul(qa[e].z, ka[f].z));
          s[e][f] = fadd(s[e][f], fmul(qa[e].w, ka[f].w));
        }
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        qa[e] = *reinterpret_cast<const float4*>(&On[ty + 16 * e][d]);
        ka[e] = *reinterpret_cast<const float4*>(&Vn[tx + 16 * e][d]);
      }
#pragma unroll
      for (int e = 0; e < 4; ++e)
#pragma unroll
        for (int f = 0; f < 4; ++f) {
          dp[e][f] = fadd(dp[e][f], fmul(qa[e].x, ka[f].x));
          dp[e][f] = fadd(dp[e][f], fmul(qa[e].y, ka[f].y));
          dp[e][f] = fadd(dp[e][f], fmul(qa[e].z, ka[f].z));
          dp[e][f] = fadd(dp[e][f], fmul(qa[e].w, ka[f].w));
        }
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int il = ty + 16 * e;
      const float L = Ls[il], dl = Ds[il];
#pragma unroll
      for (int f = 0; f < 4; ++f) {
        const int jl = tx + 16 * f;
        float p = 0.0f, ds = 0.0f;
        if (j0 + jl <= i0 + il) {
          p = det_exp(fsub(fmul(s[e][f], ATT_SCALE), L));
          ds = fmul(fmul(p, fsub(dp[e][f], dl)), ATT_SCALE);
        }
        Pt[il][jl] = bf2f(f2bf(p));
        St[il][jl] = bf2f(f2bf(ds));
      }
    }
    __syncthreads();
    // bf16(dS) tile to global scratch for the dQ kernel: row = tid/4, 16 columns
    {
      const int r = tid >> 2, c0 = (tid & 3) * 16;
      uint32_t w[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) w[e] = pack_bf2(St[r][c0 + 2 * e], St[r][c0 + 2 * e + 1]);
      uint4* dst = reinterpret_cast<uint4*>(dS + (bh * S + i0 + r) * S + j0 + c0);
      dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
      dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
    }
    // dV += P~^T dO, dK += dS~^T q: thread = keys tx+16e x dims {4ty.., 64+4ty..}, queries ascending
#pragma unroll 2
    for (int i = 0; i < BT; ++i) {
      float pa[4], sa[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) { pa[e] = Pt[i][tx + 16 * e]; sa[e] = St[i][tx + 16 * e]; }
      const float4 o0 = *reinterpret_cast<const float4*>(&On[i][ty * 4]);
      const float4 o1 = *reinterpret_cast<const float4*>(&On[i][64 + ty * 4]);
      const float4 q0v = *reinterpret_cast<const float4*>(&Qn[i][ty * 4]);
      const float4 q1v = *reinterpret_cast<const float4*>(&Qn[i][64 + ty * 4]);
      const float ob[8] = {o0.x, o0.y, o0.z, o0.w, o1.x, o1.y, o1.z, o1.w};
      const float qbv[8] = {q0v.x, q0v.y, q0v.z, q0v.w, q1v.x, q1v.y, q1v.z, q1v.w};
#pragma unroll
      for (int e = 0; e < 4; ++e)
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          dvv[e][c] = fadd(dvv[e][c], fmul(pa[e], ob[c]));
          dkk[e][c] = fadd(dkk[e][c], fmul(sa[e], qbv[c]));
        }
    }
  }
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const size_t r = (row0 + j0 + tx + 16 * e) * ld_d + (size_t)h * DH;
    uint2 a, c;
    a.x = pack_bf2(dvv[e][0], dvv[e][1]); a.y = pack_bf2(dvv[e][2], dvv[e][3]);
    c.x = pack_bf2(dvv[e][4], dvv[e][5]); c.y = pack_bf2(dvv[e][6], dvv[e][7]);
    *reinterpret_cast<uint2*>(dv + r + ty * 4) = a;
    *reinterpret_cast<uint2*>(dv + r + 64 + ty * 4) = c;
    a.x = pack_bf2(dkk[e][0], dkk[e][1]); a.y = pack_bf2(dkk[e][2], dkk[e][3]);
    c.x = pack_bf2(dkk[e][4], dkk[e][5]); c.y = pack_bf2(dkk[e][6], dkk[e][7]);
    *reinterpret_cast<uint2*>(dk + r + ty * 4) = a;
    *reinterpret_cast<uint2*>(dk + r + 64 + ty * 4) = c;
  }
}

// CTA = 64 queries; dQ_ic = sum over keys ascending of dS~_ij k_jc
__global__ void __launch_bounds__(256, 1)
    k_attn_dq(const uint16_t* __restrict__ k, const uint16_t* __restrict__ dS, int ld, int H, int S,
              uint16_t* __restrict__ dq, int ld_d) {
  extern __shared__ __align__(16) float sm[];
  float(*Kn)[LN] = reinterpret_cast<float(*)[LN]>(sm);
  float(*St)[LP] = reinterpret_cast<float(*)[LP]>(sm + BT * LN);
  const int ib = gridDim.x - 1 - blockIdx.x;
  const int h = blockIdx.y, b = blockIdx.z;
  const int i0 = ib * BT;
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const size_t row0 = (size_t)b * S;
  const size_t bh = (size_t)b * H + h;
  float acc[4][8];
#pragma unroll
  for (int e = 0; e < 4; ++e)
#pragma unroll
    for (int c = 0; c < 8; ++c) acc[e][c] = 0.0f;
  for (int jt = 0; jt <= ib; ++jt) {
    const int j0 = jt * BT;
    __syncthreads();
    load_tile_nat(Kn, k + row0 * ld + (size_t)h * DH, ld, j0, S);
    {
      const int r = tid >> 2, c0 = (tid & 3) * 16;
      const uint4* src = reinterpret_cast<const uint4*>(dS + (bh * S + i0 + r) * S + j0 + c0);
      float t[8];
      unpack8a(__ldg(src), t);
#pragma unroll
      for (int e = 0; e < 8; ++e) St[r][c0 + e] = t[e];
      unpack8a(__ldg(src + 1), t);
#pragma unroll
      for (int e = 0; e < 8; ++e) St[r][c0 + 8 + e] = t[e];
    }
    __syncthreads();
#pragma unroll 2
    for (int j = 0; j < BT; ++j) {
      float sa[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) sa[e] = St[ty + 16 * e][j];
      const float4 k0 = *reinterpret_cast<const float4*>(&Kn[j][tx * 4]);
      const float4 k1 = *reinterpret_cast<const float4*>(&Kn[j][64 + tx * 4]);
      const float kb[8] = {k0.x, k0.y, k0.z, k0.w, k1.x, k1.y, k1.z, k1.w};
#pragma unroll
      for (int e = 0; e < 4; ++e)
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[e][c] = fadd(acc[e][c], fmul(sa[e], kb[c]));
    }
  }
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const size_t r = (row0 + i0 + ty + 16 * e) * ld_d + (size_t)h * DH;
    uint2 a, c;
    a.x = pack_bf2(acc[e][0], acc[e][1]); a.y = pack_bf2(acc[e][2], acc[e][3]);
    c.x = pack_bf2(acc[e][4], acc[e][5]); c.y = pack_bf2(acc[e][6], acc[e][7]);
    *reinterpret_cast<uint2*>(dq + r + tx * 4) = a;
    *reinterpret_cast<uint2*>(dq + r + 64 + tx * 4) = c;
  }
}

static int set_smem(const void* fn, size_t bytes) {
  return cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) == cudaSuccess ? 0 : -1;
}

}  // namespace det

using namespace det;

extern "C" int det_attn_fwd(const det_bf16* q, const det_bf16* k, const det_bf16* v, int ld, int B, int H, int S,
                            det_bf16* out, int ld_out, float* lse, void* stream) {
  if (!q || !k || !v || !out || !lse || B <= 0 || H <= 0 || S <= 0) return DET_ERR_ARG;
  if (S % 64 || ld % 8 || ld_out % 8 || ld < H * DH || ld_out < H * DH || H > 65535 || B > 65535) return DET_ERR_SHAPE;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return DET_ERR_ALIGN;
  static bool cfg = false;
  if (!cfg) { if (set_smem((const void*)k_attn_fwd, FWD_SMEM)) return DET_ERR_CUDA; cfg = true; }
  dim3 grid(S / FQ, H, B);
  k_attn_fwd<<<DET_L(grid), 256, FWD_SMEM, (cudaStream_t)stream>>>(q, k, v, ld, H, S, out, ld_out, lse);
  DET_CHECK_LAUNCH();
  return DET_OK;
}

extern "C" size_t det_attn_bwd_ws_bytes(int B, int H, int S) {
  return align_up((size_t)B * H * S * S * 2, 256) + align_up((size_t)B * H * S * 4, 256);
}

extern "C" int det_attn_bwd(const det_bf16* dout, const det_bf16* q, const det_bf16* k, const det_bf16* v,
                            const det_bf16* out, const float* lse, int ld, int ld_out, int B, int H, int S, det_bf16* dq,
                            det_bf16* dk, det_bf16* dv, int ld_d, void* ws, size_t ws_bytes, void* stream) {
  if (!dout || !q || !k || !v || !out || !lse || !dq || !dk || !dv || B <= 0 || H <= 0 || S <= 0) return DET_ERR_ARG;
  if (S % 64 || ld % 8 || ld_out % 8 || ld_d % 8 || H > 65535 || B > 65535) return DET_ERR_SHAPE;
  if (!aligned16(dout) || !aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(dq) ||
      !aligned16(dk) || !aligned16(dv) || !aligned16(ws))
    return DET_ERR_ALIGN;
  if (!ws || ws_bytes < det_attn_bwd_ws_bytes(B, H, S)) return DET_ERR_WORKSPACE;
  static bool cfg = false;
  if (!cfg) {
    if (set_smem((const void*)k_attn_dkdv, DKDV_SMEM) || set_smem((const void*)k_attn_dq, DQ_SMEM)) return DET_ERR_CUDA;
    cfg = true;
  }
  cudaStream_t st = (cudaStream_t)stream;
  uint16_t* dS = (uint16_t*)ws;
  float* delta = (float*)((uint8_t*)ws + align_up((size_t)B * H * S * S * 2, 256));
  const size_t nrows = (size_t)B * H * S;
  k_attn_delta<<<DET_L((unsigned)((nrows + 7) / 8)), 256, 0, st>>>(dout, out, ld_out, H, S, nrows, delta);
  dim3 grid(S / BT, H, B);
  k_attn_dkdv<<<DET_L(grid), 256, DKDV_SMEM, st>>>(dout, q, k, v, lse, delta, ld, ld_out, H, S, dk, dv, ld_d, dS);
  k_attn_dq<<<DET_L(grid), 256, DQ_SMEM, st>>>(k, dS, ld, H, S, dq, ld_d);
  DET_CHECK_LAUNCH();
  return DET_OK;
}
