// Attention forward with the P.V product of every block of 128 keys on the int8 tensor cores (Sec. 3.2: "int8 P.V per
// block; QK^T and softmax in higher precision").
//
// Per (batch, key/value head, block of 128 keys): s_v = absmax(V block) / 127, q_v = rne(clamp(v * (127 / absmax))).
// Per query row and block: q_p = rne(p * 127), p = exp(s - m) in [0, 1].  u = float(sum_j q_p q_v) * (s_v / 127): the
// integer sum is exact, so the tensor core's accumulation order does not matter.  Logits, running maximum, row sums
// and the rescale o = o * alpha + u stay in ordered f32 exactly as in the full-precision kernel (attn.cu); lse is the
// same as there.
//
// CTA = 128 queries of one (batch, head), 512 threads, one CTA per SM.  Logits: 4 x 8 register tiles on the FP32 pipe
// as in attn.cu.  The quantised weights (A operand, [query][key]) and the quantised, transposed values (B operand,
// [dim][key]) are written by the threads into shared memory in the 128-byte-swizzled K-major layout the MMA expects;
// one thread issues four tcgen05.mma.kind::i8 (M = N = 128, K = 32 each) into a 128-column TMEM accumulator and
// commits to an mbarrier; every warp then loads its 32 lanes x 32 columns of the accumulator.  In that phase a thread
// owns one query row and 32 output dimensions.  The wait on the mbarrier is bounded: on expiry the kernel raises
// DET_DEV_TIMEOUT in *status, skips the remaining tiles, frees its TMEM and returns.
#include "tc05.cuh"
#include "internal.h"

namespace det {

#define ATT_SCALE 0x1.6a09e6p-4f
constexpr int PD = 128;                 // head dimension
constexpr int PQ = 128, PK = 128, PTH = 512;
constexpr int PLQ = PQ + 4;
// shared memory: Q f32 [dim][query], K f32 [dim][key], then (1024-byte aligned) q_p int8 [query][key], q_v int8 [dim][key]
constexpr size_t PV8_SMEM = (size_t)(2 * PD * PLQ) * sizeof(float) + 1024 + 2 * PQ * PK;

__device__ __forceinline__ void unpack8p(const uint4& u, float v[8]) {
  v[0] = bflo(u.x); v[1] = bfhi(u.x); v[2] = bflo(u.y); v[3] = bfhi(u.y);
  v[4] = bflo(u.z); v[5] = bfhi(u.z); v[6] = bflo(u.w); v[7] = bfhi(u.w);
}
__device__ __forceinline__ bool tiny1p(float v) { return (__float_as_uint(v) * 2u - 1u) < 0x3fffffffu; }

// byte offset of element (row, col) of a 128 x 128 int8 K-major tile with 128-byte swizzle (16-byte chunks of a row
// are permuted by the row index modulo 8)
__device__ __forceinline__ int swz(int row, int col) { return row * 128 + ((((col >> 4) ^ (row & 7))) << 4) + (col & 15); }

template <bool FUSED>
__device__ __forceinline__ void mac_4x8p(const float (*As)[PLQ], const float (*Bs)[PLQ], int ty, int tx, float2 (&acc)[4][4]) {
#pragma unroll 8
  for (int k = 0; k < PD; ++k) {
    const float4 a0 = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
    const float4 b0 = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
    const float4 b1 = *reinterpret_cast<const float4*>(&Bs[k][64 + tx * 4]);
    const float av[4] = {a0.x, a0.y, a0.z, a0.w};
    const float2 b[4] = {make_float2(b0.x, b0.y), make_float2(b0.z, b0.w), make_float2(b1.x, b1.y), make_float2(b1.z, b1.w)};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 a = make_float2(av[i], av[i]);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (FUSED) {
          acc[i][j] = __ffma2_rn(a, b[j], acc[i][j]);
        } else {  // scalar on purpose: a packed multiply + add pair would be contracted by ptxas
          acc[i][j].x = fadd(acc[i][j].x, fmul(av[i], b[j].x));
          acc[i][j].y = fadd(acc[i][j].y, fmul(av[i], b[j].y));
        }
      }
    }
  }
}

__global__ void __launch_bounds__(PTH, 1)
    k_attn_fwd_pv8(const uint16_t* __restrict__ q, const uint16_t* __restrict__ k, const uint16_t* __restrict__ v, int ld, int H,
                   int Hkv, int S, int W, uint16_t* __restrict__ out, int ld_out, float* __restrict__ lse, int* status) {
  extern __shared__ __align__(16) unsigned char psm8[];
  float(*Qs)[PLQ] = reinterpret_cast<float(*)[PLQ]>(psm8);
  float(*Ks)[PLQ] = reinterpret_cast<float(*)[PLQ]>(psm8 + (size_t)PD * PLQ * sizeof(float));
  uint8_t* ops = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(psm8 + (size_t)2 * PD * PLQ * sizeof(float)) + 1023) &
                                            ~(uintptr_t)1023);
  int8_t* Pq = reinterpret_cast<int8_t*>(ops);              // A operand: [query][key]
  int8_t* Vq = reinterpret_cast<int8_t*>(ops + PQ * PK);    // B operand: [dim][key]
  __shared__ float alpha_s[PQ], l_s[PQ], m_s[PQ];
  __shared__ uint32_t vmax_s, tmem_base_s;
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_s;
  volatile int* abort_flag = &abort_s;

  const int qb = gridDim.y - 1 - blockIdx.y;  // longest rows first
  const int h = blockIdx.x % H, b = blockIdx.x / H;
  const int q0 = qb * PQ;
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15, warp = tid >> 5, lane = tid & 31;
  const size_t row0 = (size_t)b * S;
  const int hk = h / (H / Hkv);
  const uint16_t* qp = q + row0 * ld + (size_t)h * PD;
  const uint16_t* kp = k + row0 * ld + (size_t)hk * PD;
  const uint16_t* vp = v + row0 * ld + (size_t)hk * PD;

  if (tid == 0) {
    mbar_init(&bar, 1);
    abort_s = 0;
    vmax_s = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(128u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  // accumulator phase: this thread owns query row orow and the 32 output dimensions starting at ocol
  const int orow = (warp & 3) * 32 + lane, ocol = (warp >> 2) * 32;
  const uint32_t taddr = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)ocol;

  uint4 rw[4];
  auto fetch = [&](const uint16_t* base, int j0, bool key_major) {
#pragma unroll
    for (int it = 0; it < 4; ++it) {
      const int idx = tid + PTH * it;
      const int key = key_major ? (idx & 127) : (idx >> 4), ch = key_major ? (idx >> 7) : (idx & 15);
      rw[it] = (j0 + key < S) ? __ldg(reinterpret_cast<const uint4*>(base + (size_t)(j0 + key) * ld + ch * 8))
                              : make_uint4(0u, 0u, 0u, 0u);
    }
  };
  const int jt0 = (W > 0 && q0 > W) ? (q0 - W) / PK : 0;
  fetch(kp, jt0 * PK, true);
  bool tq = false;
#pragma unroll
  for (int it = 0; it < 4; ++it) {
    const int idx = tid + PTH * it, r = idx & 127, ch = idx >> 7;
    float t[8];
    if (q0 + r < S) unpack8p(__ldg(reinterpret_cast<const uint4*>(qp + (size_t)(q0 + r) * ld + ch * 8)), t);
    else {
#pragma unroll
      for (int e = 0; e < 8; ++e) t[e] = 0.0f;
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) { tq |= tiny1p(t[e]); Qs[ch * 8 + e][r] = t[e]; }
  }
  const int tiny_q = __syncthreads_or(tq);
  float m[4], l[4], o[32];
#pragma unroll
  for (int i = 0; i < 4; ++i) { m[i] = __int_as_float(0xff800000); l[i] = 0.0f; }
#pragma unroll
  for (int c = 0; c < 32; ++c) o[c] = 0.0f;
  const int ntiles = q0 / PK + 1;
  constexpr uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(PD >> 3) << 17) | ((uint32_t)(PQ >> 4) << 24);
  uint32_t phase = 0;
  bool ok = true;
  for (int jt = jt0; jt < ntiles; ++jt) {
    const int j0 = jt * PK;
    // ---- K tile (fetched during the previous tile), transposed, f32 ----
    bool tk = false;
#pragma unroll
    for (int it = 0; it < 4; ++it) {
      const int idx = tid + PTH * it, key = idx & 127, ch = idx >> 7;
      float t[8];
      unpack8p(rw[it], t);
#pragma unroll
      for (int e = 0; e < 8; ++e) { tk |= tiny1p(t[e]); Ks[ch * 8 + e][key] = t[e]; }
    }
    fetch(vp, j0, false);   // V words travel while the logits are computed
    const int tiny_k = __syncthreads_or(tk);
    float2 s[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int e = 0; e < 4; ++e) s[i][e] = make_float2(0.0f, 0.0f);
    if (tiny_q || tiny_k) mac_4x8p<false>(Qs, Ks, ty, tx, s);
    else mac_4x8p<true>(Qs, Ks, ty, tx, s);
    // ---- block absmax of V (all 128 keys x 128 dims of the tile) ----
    float vm = 0.0f;
#pragma unroll
    for (int it = 0; it < 4; ++it) {
      float t[8];
      unpack8p(rw[it], t);
#pragma unroll
      for (int e = 0; e < 8; ++e) vm = fmaxf(vm, fabsf(t[e]));
    }
#pragma unroll
    for (int w = 16; w; w >>= 1) vm = fmaxf(vm, __shfl_xor_sync(0xffffffffu, vm, w));
    if (lane == 0 && vm > 0.0f) atomicMax(&vmax_s, __float_as_uint(vm));
    // ---- online softmax statistics per row; quantised weights to the A operand ----
    const bool diag = (jt == ntiles - 1);
    const bool edge = W > 0 && j0 <= q0 + PQ - 1 - W;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int rl = ty * 4 + i;
      const int row = q0 + rl;
      const bool rowvalid = !(edge && j0 + PK - 1 <= row - W);
      float sv[8] = {s[i][0].x, s[i][0].y, s[i][1].x, s[i][1].y, s[i][2].x, s[i][2].y, s[i][3].x, s[i][3].y};
      float mt = m[i];
      bool valid[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int key = j0 + ((e < 4) ? (tx * 4 + e) : (64 + tx * 4 + e - 4));
        valid[e] = (!diag || key <= row) && (!edge || key > row - W);
        sv[e] = fmul(sv[e], ATT_SCALE);
        if (valid[e]) mt = fmaxf(mt, sv[e]);
      }
#pragma unroll
      for (int w = 1; w < 16; w <<= 1) mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, w));
      const float al0 = det_exp_le0(fsub(m[i], mt));
      const float al = rowvalid ? al0 : 1.0f;
      float p[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) p[e] = det_exp_le0(fsub(sv[e], mt));   // branch-free, so the eight chains interleave
#pragma unroll
      for (int e = 0; e < 8; ++e) p[e] = valid[e] ? p[e] : 0.0f;
      uint32_t w0 = 0, w1 = 0;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        w0 |= ((uint32_t)(int)rintf(fmul(p[e], 127.0f))) << (8 * e);
        w1 |= ((uint32_t)(int)rintf(fmul(p[4 + e], 127.0f))) << (8 * e);
      }
      *reinterpret_cast<uint32_t*>(Pq + swz(rl, tx * 4)) = w0;
      *reinterpret_cast<uint32_t*>(Pq + swz(rl, 64 + tx * 4)) = w1;
      float h0 = fadd(fadd(p[0], p[1]), fadd(p[2], p[3]));
      float h1 = fadd(fadd(p[4], p[5]), fadd(p[6], p[7]));
#pragma unroll
      for (int w = 1; w < 16; w <<= 1) {
        h0 = fadd(h0, __shfl_xor_sync(0xffffffffu, h0, w));
        h1 = fadd(h1, __shfl_xor_sync(0xffffffffu, h1, w));
      }
      l[i] = fadd(fmul(l[i], al), fadd(h0, h1));
      m[i] = mt;
      if (tx == 0) alpha_s[rl] = al;
    }
    __syncthreads();  // vmax_s is complete; every thread is done with K
    const float am = __uint_as_float(vmax_s);
    const float s_v = (am > 0.0f) ? fdiv(am, 127.0f) : 0.0f, inv_v = (am > 0.0f) ? fdiv(127.0f, am) : 0.0f;
    const float cs = fdiv(s_v, 127.0f);
    // ---- quantised, transposed values to the B operand ----
#pragma unroll
    for (int it = 0; it < 4; ++it) {
      const int idx = tid + PTH * it, key = idx >> 4, ch = idx & 15;
      float vv[8];
      unpack8p(rw[it], vv);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float t = fminf(fmaxf(fmul(vv[e], inv_v), -128.0f), 127.0f);
        Vq[swz(ch * 8 + e, key)] = (int8_t)(int)rintf(t);
      }
    }
    if (jt + 1 < ntiles) fetch(kp, j0 + PK, true);   // next K travels during the tensor-core product
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      vmax_s = 0;
      tc_fence_after();
      const uint64_t da = make_smem_desc(smem_u32(Pq)), db = make_smem_desc(smem_u32(Vq));
#pragma unroll
      for (int k4 = 0; k4 < PK / 32; ++k4) umma_i8(tmem_base, da + (uint64_t)(k4 * 2), db + (uint64_t)(k4 * 2), idesc, k4 ? 1u : 0u);
      umma_commit(&bar);
    }
    if (ok && !mbar_wait(&bar, phase, abort_flag, status)) ok = false;
    ok = __all_sync(0xffffffffu, ok);   // the TMEM load below is warp-collective
    phase ^= 1u;
    tc_fence_after();
    if (ok) {
      uint32_t r[32];
      tmem_ld32(taddr, r);
      const float al = alpha_s[orow];
#pragma unroll
      for (int c = 0; c < 32; ++c) o[c] = fadd(fmul(o[c], al), fmul(__int2float_rn((int)r[c]), cs));
    }
    tc_fence_before();
    if (!__syncthreads_and(ok)) break;   // operands, alpha and the accumulator may be overwritten by the next tile
  }
  // row statistics travel from the logit mapping (4 rows per thread) to the accumulator mapping (1 row per thread)
  if (tx == 0) {
#pragma unroll
    for (int i = 0; i < 4; ++i) { l_s[ty * 4 + i] = l[i]; m_s[ty * 4 + i] = m[i]; }
  }
  __syncthreads();
  const int row = q0 + orow;
  if (row < S && !abort_s) {
    const float lr = l_s[orow];
    const float il = fdiv(1.0f, lr);
    uint16_t* op = out + (row0 + row) * ld_out + (size_t)h * PD + ocol;
#pragma unroll
    for (int c = 0; c < 32; c += 8) {
      uint4 w;
      w.x = pack_bf2(fmul(o[c], il), fmul(o[c + 1], il)); w.y = pack_bf2(fmul(o[c + 2], il), fmul(o[c + 3], il));
      w.z = pack_bf2(fmul(o[c + 4], il), fmul(o[c + 5], il)); w.w = pack_bf2(fmul(o[c + 6], il), fmul(o[c + 7], il));
      *reinterpret_cast<uint4*>(op + c) = w;
    }
    if (ocol == 0) lse[((size_t)b * H + h) * S + row] = fadd(m_s[orow], det_log(lr));
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(128u) : "memory");
}

}  // namespace det

using namespace det;

extern "C" int det_attn_fwd_int8pv(const det_bf16* q, const det_bf16* k, const det_bf16* v, int ld, int B, int H, int Hkv, int S,
                                   int window, det_bf16* out, int ld_out, float* lse, void* stream, int* status_dev) {
  if (!q || !k || !v || !out || !lse || B <= 0 || H <= 0 || Hkv <= 0 || S <= 0 || window < 0) return DET_ERR_ARG;
  if (S % 64 || ld % 8 || ld_out % 8 || ld < H * PD || ld_out < H * PD || H % Hkv || window % 128) return DET_ERR_SHAPE;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return DET_ERR_ALIGN;
  static DevOnce once = {};
  if (dev_ensure_smem(once, (const void*)k_attn_fwd_pv8, PV8_SMEM) != DET_OK) return DET_ERR_CUDA;
  dim3 grid(H * B, (S + PQ - 1) / PQ);
  k_attn_fwd_pv8<<<DET_L(grid), PTH, PV8_SMEM, (cudaStream_t)stream>>>(q, k, v, ld, H, Hkv, S, window, out, ld_out, lse, status_dev);
  DET_CHECK_LAUNCH();
  return DET_OK;
}
