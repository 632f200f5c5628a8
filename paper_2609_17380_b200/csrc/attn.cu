// Causal attention, head_dim 128, in a fixed order on the FP32 ALUs (Sec. 3.2: QK^T and softmax stay in
// higher precision; the backward recomputes the weights in full precision and is not quantised).
//
// Forward: online softmax over KV tiles of 128 keys in ascending order.  Each logit is a sequential
// ascending sum over the 128 head dimensions of exact bf16 products; the tile's row sum is the adjacent
// pairwise tree over its 128 slots (masked slots are +0); P is rounded to bf16 before P.V; P.V is a
// sequential ascending sum over the tile's keys from +0, then o = o*alpha + u.
// Backward: P = exp(S*scale - L) recomputed; every one of the five contractions (S, dP, dV, dK, dQ) is a batched
// ordered contraction with one sequential accumulator per output (ogemm_core.cuh); bf16(P) and bf16(dS) go through
// global scratch, so nothing is accumulated with atomics.
#include "ogemm_core.cuh"

namespace det {

#define ATT_SCALE 0x1.6a09e6p-4f
constexpr int DH = 128;

__device__ __forceinline__ void unpack8a(const uint4& u, float v[8]) {
  v[0] = bflo(u.x); v[1] = bfhi(u.x); v[2] = bflo(u.y); v[3] = bfhi(u.y);
  v[4] = bflo(u.z); v[5] = bfhi(u.z); v[6] = bflo(u.w); v[7] = bfhi(u.w);
}

// ---------------------------------------------------------------------------------------------
// forward: CTA = 128 queries of one (batch, head); 512 threads (four warps per scheduler, so that the softmax and
// staging phases, which are chains of dependent instructions, overlap across warps), thread = 4 queries x 8 keys /
// 8 dims.  Shared memory (f32): Q [dim][query], one buffer that holds K [dim][key] during the logits and V [key][dim]
// during P.V, and P~ [key][query].  Multiply-adds use the fused instruction whenever no factor of the tile is
// below 2^-63 in magnitude (then the exact bf16 x bf16 product cannot be subnormal and fused = unfused bit for bit).
// ---------------------------------------------------------------------------------------------
constexpr int FQ = 128, FK = 128, FT = 512;
constexpr int LQ = FQ + 4;
constexpr size_t FWD_SMEM = (size_t)(3 * DH * LQ) * sizeof(float);

// conservative test for 0 < |v| < 2^-63 (also true for subnormal v, which only selects the slower exact path)
__device__ __forceinline__ bool tiny1(float v) { return (__float_as_uint(v) * 2u - 1u) < 0x3fffffffu; }
__device__ __forceinline__ bool tiny8a(const float v[8]) {
  bool t = false;
#pragma unroll
  for (int i = 0; i < 8; ++i) t |= tiny1(v[i]);
  return t;
}

// acc[i][j] += A[k][ty*4 + i] * B[k][{tx*4.., 64 + tx*4..}] for k ascending
template <bool FUSED>
__device__ __forceinline__ void mac_4x8(const float (*As)[LQ], const float (*Bs)[LQ], int n, int ty, int tx,
                                        float2 (&acc)[4][4]) {
#pragma unroll 8
  for (int k = 0; k < n; ++k) {
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

// Hkv key/value heads serve H query heads (head h reads key/value head h / (H/Hkv)); W > 0 restricts row i to the keys
// j in (i - W, i] (W a multiple of 128): the tile loop then starts at the tile of q0 - W, and a row skips a tile that
// holds none of its keys (its statistics stay untouched: alpha = 1, all weights 0).
template <bool WIN>
__global__ void __launch_bounds__(FT, 1) k_attn_fwd(const uint16_t* __restrict__ q, const uint16_t* __restrict__ k,
                                                    const uint16_t* __restrict__ v, int ld, int H, int Hkv, int S, int Warg,
                                                    uint16_t* __restrict__ out, int ld_out, float* __restrict__ lse,
                                                    const float* __restrict__ s_q, int8_t* __restrict__ qout) {
  const int W = WIN ? Warg : 0;
  extern __shared__ __align__(16) float sm[];
  float(*Qs)[LQ] = reinterpret_cast<float(*)[LQ]>(sm);                 // [dim][query]
  float(*KV)[LQ] = reinterpret_cast<float(*)[LQ]>(sm + DH * LQ);       // K: [dim][key]; V: [key][dim]
  float(*Ps)[LQ] = reinterpret_cast<float(*)[LQ]>(sm + 2 * DH * LQ);   // [key][query]
  // blocks are handed out in linear order: the query block is the slow index and runs from the longest rows to the
  // shortest, so the blocks that are still running at the end are the short ones
  const int qb = gridDim.y - 1 - blockIdx.y;
  const int h = blockIdx.x % H, b = blockIdx.x / H;
  const int q0 = qb * FQ;
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const size_t row0 = (size_t)b * S;
  const uint16_t* qp = q + row0 * ld + (size_t)h * DH;
  const int hk = h / (H / Hkv);
  const uint16_t* kp = k + row0 * ld + (size_t)hk * DH;
  const uint16_t* vp = v + row0 * ld + (size_t)hk * DH;

  // one 128 x 128 bf16 tile in flight: 4 sixteen-byte words per thread
  uint4 rw[4];
  auto fetch_k = [&](int j0) {
#pragma unroll
    for (int it = 0; it < 4; ++it) {
      const int idx = tid + FT * it, key = idx & 127, ch = idx >> 7;
      rw[it] = (j0 + key < S) ? __ldg(reinterpret_cast<const uint4*>(kp + (size_t)(j0 + key) * ld + ch * 8))
                              : make_uint4(0u, 0u, 0u, 0u);
    }
  };
  const int jt0 = (WIN && q0 > W) ? (q0 - W) / FK : 0;
  fetch_k(jt0 * FK);
  bool tq = false;
#pragma unroll
  for (int it = 0; it < 4; ++it) {
    const int idx = tid + FT * it, r = idx & 127, ch = idx >> 7;
    float t[8];
    if (q0 + r < S) unpack8a(__ldg(reinterpret_cast<const uint4*>(qp + (size_t)(q0 + r) * ld + ch * 8)), t);
    else {
#pragma unroll
      for (int e = 0; e < 8; ++e) t[e] = 0.0f;
    }
    tq |= tiny8a(t);
#pragma unroll
    for (int e = 0; e < 8; ++e) Qs[ch * 8 + e][r] = t[e];
  }
  const int tiny_q = __syncthreads_or(tq);
  float m[4], l[4];
  float2 o[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    m[i] = __int_as_float(0xff800000);
    l[i] = 0.0f;
#pragma unroll
    for (int e = 0; e < 4; ++e) o[i][e] = make_float2(0.0f, 0.0f);
  }
  const int ntiles = q0 / FK + 1;
  for (int jt = jt0; jt < ntiles; ++jt) {
    const int j0 = jt * FK;
    // ---- K tile (fetched during the previous tile's P.V), transposed ----
    bool tk = false;
#pragma unroll
    for (int it = 0; it < 4; ++it) {
      const int idx = tid + FT * it, key = idx & 127, ch = idx >> 7;
      float t[8];
      unpack8a(rw[it], t);
      tk |= tiny8a(t);
#pragma unroll
      for (int e = 0; e < 8; ++e) KV[ch * 8 + e][key] = t[e];
    }
    // V words of this tile travel while the logits are computed
#pragma unroll
    for (int it = 0; it < 4; ++it) {
      const int idx = tid + FT * it, key = idx >> 4, ch = idx & 15;
      rw[it] = (j0 + key < S) ? __ldg(reinterpret_cast<const uint4*>(vp + (size_t)(j0 + key) * ld + ch * 8))
                              : make_uint4(0u, 0u, 0u, 0u);
    }
    const int tiny_k = __syncthreads_or(tk);
    float2 s[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int e = 0; e < 4; ++e) s[i][e] = make_float2(0.0f, 0.0f);
    if (tiny_q || tiny_k) mac_4x8<false>(Qs, KV, DH, ty, tx, s);
    else mac_4x8<true>(Qs, KV, DH, ty, tx, s);
    // ---- online softmax statistics per row; P~ to shared memory ----
    float alpha[4];
    bool tp = false;
    const bool diag = (jt == ntiles - 1);  // only the last tile of a row block reaches past the diagonal
    const bool edge = WIN && j0 <= q0 + FQ - 1 - W;  // some row's window starts inside or after this tile
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int rl = ty * 4 + i;
      const int row = q0 + rl;
      const bool rowvalid = !(edge && j0 + FK - 1 <= row - W);
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
      const float al = det_exp_le0(fsub(m[i], mt));
      alpha[i] = rowvalid ? al : 1.0f;
      float p[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) p[e] = det_exp_le0(fsub(sv[e], mt));   // branch-free, so the eight chains interleave
#pragma unroll
      for (int e = 0; e < 8; ++e) p[e] = valid[e] ? p[e] : 0.0f;
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int kl = (e < 4) ? (tx * 4 + e) : (64 + tx * 4 + e - 4);
        const float pt = bf2f(f2bf(p[e]));
        tp |= tiny1(pt);
        Ps[kl][rl] = pt;
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
    __syncthreads();  // every thread is done with K; P~ is complete
    // ---- V tile, natural layout, into the same buffer ----
    bool tv = false;
#pragma unroll
    for (int it = 0; it < 4; ++it) {
      const int idx = tid + FT * it, key = idx >> 4, ch = idx & 15;
      float t[8];
      unpack8a(rw[it], t);
      tv |= tiny8a(t);
      *reinterpret_cast<float4*>(&KV[key][ch * 8]) = make_float4(t[0], t[1], t[2], t[3]);
      *reinterpret_cast<float4*>(&KV[key][ch * 8 + 4]) = make_float4(t[4], t[5], t[6], t[7]);
    }
    // K words of the next tile travel during P.V
    if (jt + 1 < ntiles) fetch_k(j0 + FK);
    const int tiny_pv = __syncthreads_or(tp || tv);
    // ---- u = P~ . V over the tile's keys in ascending order, then o = o*alpha + u ----
    float2 u[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int e = 0; e < 4; ++e) u[i][e] = make_float2(0.0f, 0.0f);
    const int kmax = min(FK, q0 + FQ - j0);
    if (tiny_pv) mac_4x8<false>(Ps, KV, kmax, ty, tx, u);
    else mac_4x8<true>(Ps, KV, kmax, ty, tx, u);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {  // scalar: the product o*alpha is rounded before the add
        o[i][e].x = fadd(fmul(o[i][e].x, alpha[i]), u[i][e].x);
        o[i][e].y = fadd(fmul(o[i][e].y, alpha[i]), u[i][e].y);
      }
    }
    __syncthreads();  // V and P~ may be overwritten by the next tile
  }
  const float inv_q = qout ? fdiv(1.0f, s_q[0]) : 0.0f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int row = q0 + ty * 4 + i;
    if (row >= S) continue;
    const float il = fdiv(1.0f, l[i]);
    uint16_t* op = out + (row0 + row) * ld_out + (size_t)h * DH;
    uint2 w0, w1;
    w0.x = pack_bf2(fmul(o[i][0].x, il), fmul(o[i][0].y, il)); w0.y = pack_bf2(fmul(o[i][1].x, il), fmul(o[i][1].y, il));
    w1.x = pack_bf2(fmul(o[i][2].x, il), fmul(o[i][2].y, il)); w1.y = pack_bf2(fmul(o[i][3].x, il), fmul(o[i][3].y, il));
    *reinterpret_cast<uint2*>(op + tx * 4) = w0;
    *reinterpret_cast<uint2*>(op + 64 + tx * 4) = w1;
    if (qout) {   // the output projection's quantiser, applied to the bf16 values just stored
      const float f[8] = {bflo(w0.x), bfhi(w0.x), bflo(w0.y), bfhi(w0.y), bflo(w1.x), bfhi(w1.x), bflo(w1.y), bfhi(w1.y)};
      const uint2 c = quant8(f, inv_q);
      int8_t* qp8 = qout + (row0 + row) * ld_out + (size_t)h * DH;
      *reinterpret_cast<uint32_t*>(qp8 + tx * 4) = c.x;
      *reinterpret_cast<uint32_t*>(qp8 + 64 + tx * 4) = c.y;
    }
    if (tx == 0) lse[((size_t)b * H + h) * S + row] = fadd(m[i], det_log(l[i]));
  }
}

// ---------------------------------------------------------------------------------------------
// forward, warp-specialised (full causal attention; the windowed layers keep k_attn_fwd<true>).
//
// What bounds the kernel above is shared-memory bandwidth: a 16-byte load costs the port one cycle per 128 distinct
// bytes of every half-warp, its 4 x 8 register tiles need three such loads (10 port cycles per warp) for 16 packed
// multiply-adds, and its phases (logits, softmax, P.V) are block-wide, so the FP32 pipe idles during every softmax.
// Here a consumer warp owns 16 whole query rows: a lane holds 16 rows x 4 adjacent columns (keys while the logits are
// formed, head dimensions during P.V), so the row operand is one address for the whole warp (q^T [dim][query] and
// P~ [key][query] in shared memory) and the column operand one 16-byte word per lane: five loads (12 port cycles) per 32
// packed multiply-adds.  A row's 128 logits of a key block sit in one warp, so its maximum and its row sum (the
// adjacent pairwise tree: four slots in the lane, then lanes 1, 2, 4, 8, 16 apart) are warp shuffles, P~ of the warp's
// rows is written and read by that warp alone, and the running maximum, sum and rescale factor of row i live in lane i.
// K and V arrive through an mbarrier-guarded ring of 16-deep slabs filled by four producer warps (K: 16 head dimensions
// x 128 keys, eight per block; V: 16 keys x 128 dimensions, eight per block), so no block-wide barrier is left in the
// loop and consumer warps are not coupled to each other.  The softmax evaluates its 64 exponentials per lane as one
// straight-line block of branch-free chains and reduces the 16 rows with 16 shuffles per reduction.
// On the diagonal block a warp stops P.V after the last key any of its rows may see.
// Arithmetic and order per output are exactly those of k_attn_fwd (and of the definition): bit-identical results.
// ---------------------------------------------------------------------------------------------
constexpr int AF_RW = 8;                      // query rows per consumer warp (8: sixteen consumer warps, 16: eight)
constexpr int AF_SLOTS = 8, AF_PF = 4, AF_CONS = (FQ / AF_RW) * 32, AF_PROD = 128, AF_THREADS = AF_CONS + AF_PROD;
constexpr size_t AFW_SMEM = (size_t)(DH * LQ + FK * FQ + AF_SLOTS * OK * (OT + 4)) * sizeof(float);

// one 16-deep slab: (row i, column c) += A[k][row i of the warp] * B[k][4 lane + c], accumulators laid out as RP() says.  A chunk g (rows 4g..4g+3) of step k is at ap + k * a_ld + ((chunk0 + g) ^ (PSWZ ? swizzle of the key : 0)) * 4.
template <bool FUSED, bool PSWZ>
__device__ __forceinline__ void mac_16x4(const float* __restrict__ ap, int a_ld, int chunk0, int key0,
                                         const float (*Bs)[OT + 4], int lane, float2 (&acc)[AF_RW / 2][4]) {
#pragma unroll
  for (int k = 0; k < OK; ++k) {
    const int sw = PSWZ ? (((key0 + k) >> 2) & 7) : 0;
    float4 a[AF_RW / 4];
#pragma unroll
    for (int g = 0; g < AF_RW / 4; ++g) a[g] = *reinterpret_cast<const float4*>(ap + (size_t)k * a_ld + (((chunk0 + g) ^ sw) << 2));
    const float4 bv = *reinterpret_cast<const float4*>(&Bs[k][4 * lane]);
    const float bs[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const float2 bb = make_float2(bs[c], bs[c]);
#pragma unroll
      for (int g = 0; g < AF_RW / 4; ++g) {
        if (FUSED) {
          acc[2 * g][c] = __ffma2_rn(make_float2(a[g].x, a[g].y), bb, acc[2 * g][c]);
          acc[2 * g + 1][c] = __ffma2_rn(make_float2(a[g].z, a[g].w), bb, acc[2 * g + 1][c]);
        } else {  // scalar on purpose: a packed multiply + add pair would be contracted by ptxas
          acc[2 * g][c].x = fadd(acc[2 * g][c].x, fmul(a[g].x, bs[c]));
          acc[2 * g][c].y = fadd(acc[2 * g][c].y, fmul(a[g].y, bs[c]));
          acc[2 * g + 1][c].x = fadd(acc[2 * g + 1][c].x, fmul(a[g].z, bs[c]));
          acc[2 * g + 1][c].y = fadd(acc[2 * g + 1][c].y, fmul(a[g].w, bs[c]));
        }
      }
    }
  }
}
// element (row i, column c) of a row-paired accumulator set (pair [i/2][c] holds rows i, i+1 of column c, so the row
// operand's register pairs come straight out of its 16-byte loads and only the four column values are duplicated into
// pairs); i is a compile-time constant wherever this is used
#define RP(acc, i, c) (((i) & 1) ? (acc)[(i) >> 1][c].y : (acc)[(i) >> 1][c].x)
// Reduction of 16 rows across the warp (x[i]: this lane's value for row i) with partners 1, 2, 4, 8, 16 lanes apart in that
// order, which for sums is the adjacent pairwise tree over the lanes.  Instead of 16 butterflies of five shuffles every
// stage halves the rows a lane carries (it sends its partner the half the partner keeps): 8 + 4 + 2 + 1 + 1 shuffles, and
// lane L ends with the result of row ROW_OF_LANE(L); both operand orders of an addition or a maximum give the same bits.
#define ROW_OF_LANE(L) (AF_RW == 16 ? ((((L) & 1) << 3) | (((L) & 2) << 1) | (((L) & 4) >> 1) | (((L) & 8) >> 3)) \
                                    : ((((L) & 1) << 2) | ((L) & 2) | (((L) & 4) >> 2)))
#define ROW_LANE(i) ROW_OF_LANE(i)   /* a lane that holds row i (the bit reversal is its own inverse) */
template <bool SUM>
__device__ __forceinline__ float rows_reduce(const float (&x)[AF_RW], int lane) {
  auto op = [](float a, float b) { return SUM ? fadd(a, b) : fmaxf(a, b); };
  const bool b0 = lane & 1, b1 = lane & 2, b2 = lane & 4, b3 = lane & 8;
  float d;
  if (AF_RW == 16) {
    float a[8], b[4], c[2];
#pragma unroll
    for (int j = 0; j < 8; ++j) a[j] = op(b0 ? x[(8 + j) % AF_RW] : x[j], __shfl_xor_sync(0xffffffffu, b0 ? x[j] : x[(8 + j) % AF_RW], 1));
#pragma unroll
    for (int j = 0; j < 4; ++j) b[j] = op(b1 ? a[4 + j] : a[j], __shfl_xor_sync(0xffffffffu, b1 ? a[j] : a[4 + j], 2));
#pragma unroll
    for (int j = 0; j < 2; ++j) c[j] = op(b2 ? b[2 + j] : b[j], __shfl_xor_sync(0xffffffffu, b2 ? b[j] : b[2 + j], 4));
    d = op(b3 ? c[1] : c[0], __shfl_xor_sync(0xffffffffu, b3 ? c[0] : c[1], 8));
  } else {
    float b[4], c[2];
#pragma unroll
    for (int j = 0; j < 4; ++j) b[j] = op(b0 ? x[4 + j] : x[j], __shfl_xor_sync(0xffffffffu, b0 ? x[j] : x[4 + j], 1));
#pragma unroll
    for (int j = 0; j < 2; ++j) c[j] = op(b1 ? b[2 + j] : b[j], __shfl_xor_sync(0xffffffffu, b1 ? b[j] : b[2 + j], 2));
    d = op(b2 ? c[1] : c[0], __shfl_xor_sync(0xffffffffu, b2 ? c[0] : c[1], 4));
    d = op(d, __shfl_xor_sync(0xffffffffu, d, 8));
  }
  return op(d, __shfl_xor_sync(0xffffffffu, d, 16));
}
// Register hand-over between the roles (setmaxnreg): the counts after it must fit into what the block was launched with
// (threads x the launch-time register count: 384 x 168 for 16 rows per warp, 640 x 96 for 8), or the increase never returns.
static_assert(AF_RW == 16 ? (AF_CONS * 216 + AF_PROD * 72 <= AF_THREADS * 168) : (AF_CONS * 104 + AF_PROD * 64 <= AF_THREADS * 96),
              "register hand-over exceeds the block's allocation");
__global__ void __launch_bounds__(AF_THREADS, 1)
    k_attn_fwd_ws(const uint16_t* __restrict__ q, const uint16_t* __restrict__ k, const uint16_t* __restrict__ v, int ld,
                  int H, int Hkv, int S, uint16_t* __restrict__ out, int ld_out, float* __restrict__ lse,
                  const float* __restrict__ s_q, int8_t* __restrict__ qout) {
  extern __shared__ __align__(16) float sm[];
  float(*Qs)[LQ] = reinterpret_cast<float(*)[LQ]>(sm);                         // [dim][query]
  float* Ps = sm + DH * LQ;                                                    // [key][query], 16-byte chunks swizzled
  float(*Ring)[OK][OT + 4] = reinterpret_cast<float(*)[OK][OT + 4]>(sm + DH * LQ + FK * FQ);
  __shared__ int tiny_s[AF_SLOTS][AF_PROD / 32];
  __shared__ int tiny_q_s, abort_s;
  __shared__ __align__(8) uint64_t bar_full[AF_SLOTS], bar_empty[AF_SLOTS];
  volatile int* abort_flag = &abort_s;
  const int qb = gridDim.y - 1 - blockIdx.y;          // longest rows first
  const int h = blockIdx.x % H, b = blockIdx.x / H, hk = h / (H / Hkv);
  const int q0 = qb * FQ;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const size_t row0 = (size_t)b * S;
  const uint16_t* qp = q + row0 * ld + (size_t)h * DH;
  const uint16_t* kp = k + row0 * ld + (size_t)hk * DH;
  const uint16_t* vp = v + row0 * ld + (size_t)hk * DH;
  const int ntiles = q0 / FK + 1, nslab = ntiles * 16;
  if (tid == 0) {
    for (int s = 0; s < AF_SLOTS; ++s) { mbar_init(&bar_full[s], AF_PROD / 32); mbar_init(&bar_empty[s], AF_CONS / 32); }
    tiny_q_s = 0;
    abort_s = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  {  // q^T of the query block, staged once by everybody
    bool tq = false;
    for (int idx = tid; idx < FQ * 16; idx += AF_THREADS) {
      const int r = idx & 127, ch = idx >> 7;
      float t[8];
      if (q0 + r < S) unpack8a(__ldg(reinterpret_cast<const uint4*>(qp + (size_t)(q0 + r) * ld + ch * 8)), t);
      else {
#pragma unroll
        for (int x = 0; x < 8; ++x) t[x] = 0.0f;
      }
#pragma unroll
      for (int x = 0; x < 8; ++x) { tq |= tiny1(t[x]); Qs[ch * 8 + x][r] = t[x]; }
    }
    if (__any_sync(0xffffffffu, tq) && lane == 0) atomicOr(&tiny_q_s, 1);
  }
  __syncthreads();
  if (tid >= AF_CONS) {
    // ------------------------------- producers -------------------------------
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(AF_RW == 16 ? 72 : 64));
    const int pt = tid - AF_CONS, pw = pt >> 5;
    // Slab s of the block sequence: block s / 16; s % 16 < 8: K, head dimensions 16 (s % 16) .. (thread = key, two
    // 16-byte words); else V, keys 16 (s % 16 - 8) .. (thread = four dimensions of keys kk, kk + 4, kk + 8, kk + 12).
    // AF_PF slabs are in flight in registers, so that the latency of a global load is spread over several slabs.
    // Both kinds are two 16-byte words per thread, so one register array holds whichever kind slab s is.
    uint4 raw[AF_PF][2];
    const int vf = pt & 31, vk = pt >> 5;            // V: dimensions 4 vf .. 4 vf + 3 of keys vk, vk + 4, vk + 8, vk + 12
    auto fetch = [&](int sn, uint4 (&w)[2]) {
      if (sn >= nslab) return;
      const int j0n = (sn >> 4) * FK, phn = sn & 15;
      if (phn < 8) {
        const int key = j0n + pt;
        const uint4* src = reinterpret_cast<const uint4*>(kp + (size_t)key * ld + phn * OK);
        const bool in = key < S;
        w[0] = in ? __ldg(src) : make_uint4(0u, 0u, 0u, 0u);
        w[1] = in ? __ldg(src + 1) : make_uint4(0u, 0u, 0u, 0u);
      } else {
        const int key0 = j0n + (phn - 8) * OK + vk;
        uint2 u[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int key = key0 + 4 * i;
          u[i] = key < S ? __ldg(reinterpret_cast<const uint2*>(vp + (size_t)key * ld + 4 * vf)) : make_uint2(0u, 0u);
        }
        w[0] = make_uint4(u[0].x, u[0].y, u[1].x, u[1].y);
        w[1] = make_uint4(u[2].x, u[2].y, u[3].x, u[3].y);
      }
    };
    // unpack, test for factors below 2^-63 and store: K as [dimension][key] (thread = key), V as [key][dimension]
    auto store = [&](int ph, float (*dst)[OT + 4], const uint4 (&w)[2]) -> bool {
      bool tiny = false;
      if (ph < 8) {
#pragma unroll
        for (int x = 0; x < 2; ++x) {
          float t[8];
          unpack8a(w[x], t);
#pragma unroll
          for (int e = 0; e < 8; ++e) { tiny |= tiny1(t[e]); dst[x * 8 + e][pt] = t[e]; }
        }
      } else {
        const uint32_t words[8] = {w[0].x, w[0].y, w[0].z, w[0].w, w[1].x, w[1].y, w[1].z, w[1].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float4 t = make_float4(bflo(words[2 * i]), bfhi(words[2 * i]), bflo(words[2 * i + 1]), bfhi(words[2 * i + 1]));
          tiny |= tiny1(t.x) | tiny1(t.y) | tiny1(t.z) | tiny1(t.w);
          *reinterpret_cast<float4*>(&dst[vk + 4 * i][4 * vf]) = t;
        }
      }
      return tiny;
    };
#pragma unroll
    for (int d = 0; d < AF_PF; ++d) fetch(d, raw[d]);
    for (int s0 = 0; s0 < nslab; s0 += AF_PF) {
#pragma unroll
      for (int d = 0; d < AF_PF; ++d) {
        const int s = s0 + d, slot = s % AF_SLOTS, ph = s & 15;
        if (s >= AF_SLOTS && !mbar_wait(&bar_empty[slot], (uint32_t)((s / AF_SLOTS - 1) & 1), abort_flag, nullptr)) return;
        const bool tiny = store(ph, Ring[slot], raw[d]);
        fetch(s + AF_PF, raw[d]);
        const int any = __any_sync(0xffffffffu, tiny);
        if (lane == 0) tiny_s[slot][pw] = any;
        __syncwarp();
        if (lane == 0) mbar_arrive(&bar_full[slot]);
      }
    }
    return;
  }
  // --------------------------------- consumers ---------------------------------
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(AF_RW == 16 ? 216 : 104));
  const int tiny_q = tiny_q_s;
  const int wrow = warp * AF_RW;                      // first row of this warp inside the query block
  float m_mine = __int_as_float(0xff800000), l_mine = 0.0f, alpha_mine = 0.0f;   // row (lane & 15) of the warp
  float2 o[AF_RW / 2][4];                                   // rows (2a, 2a+1) x column c
#pragma unroll
  for (int a = 0; a < AF_RW / 2; ++a)
#pragma unroll
    for (int c = 0; c < 4; ++c) o[a][c] = make_float2(0.0f, 0.0f);
  int s = 0;
  bool ok = true;
  // slab s is waited for (and its below-2^-63 flags fetched) one slab ahead of its use
  int tiny_cur = 0;
  auto acquire = [&](int sn) -> bool {
    if (sn >= nslab) return true;
    const int slot = sn % AF_SLOTS;
    if (!mbar_wait(&bar_full[slot], (uint32_t)((sn / AF_SLOTS) & 1), abort_flag, nullptr)) return false;
    tiny_cur = tiny_s[slot][0] | tiny_s[slot][1] | tiny_s[slot][2] | tiny_s[slot][3];
    return true;
  };
  ok = acquire(0);
  for (int jt = 0; jt < ntiles && ok; ++jt) {
    const int j0 = jt * FK;
    const bool diag = (jt == ntiles - 1);           // only the last block of a row block reaches past the diagonal
    // ---- logits: acc[i] = sum over the 128 dimensions ascending of q[row i][d] k[key][d], keys 4 lane .. 4 lane + 3 ----
    float2 acc[AF_RW / 2][4];
#pragma unroll
    for (int a = 0; a < AF_RW / 2; ++a)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[a][c] = make_float2(0.0f, 0.0f);
    for (int sl = 0; sl < 8; ++sl, ++s) {
      const int slot = s % AF_SLOTS;
      const int tiny = tiny_q | tiny_cur;
      if (!acquire(s + 1)) { ok = false; break; }     // the next slab's flags travel while this one is multiplied
      const float* ap = &Qs[sl * OK][wrow];
      if (tiny) mac_16x4<false, false>(ap, LQ, 0, 0, Ring[slot], lane, acc);
      else mac_16x4<true, false>(ap, LQ, 0, 0, Ring[slot], lane, acc);
      __syncwarp();
      if (lane == 0) mbar_arrive(&bar_empty[slot]);
    }
    if (!ok) break;
    // ---- online softmax of the warp's 16 rows ----
    float rm[AF_RW];
#pragma unroll
    for (int i = 0; i < AF_RW; ++i) {
      const int row = q0 + wrow + i;
      float mt = __int_as_float(0xff800000);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float sv = fmul(RP(acc, i, e), ATT_SCALE);
        RP(acc, i, e) = sv;
        if (!diag || j0 + 4 * lane + e <= row) mt = fmaxf(mt, sv);
      }
      rm[i] = mt;
    }
    // the lane that owns row r (see rows16_reduce) updates its running maximum (every row sees at least key 0 of the
    // first block, so the maximum of a block it visits is a number) and the rescale factor of what it has accumulated
    const float m_new = fmaxf(m_mine, rows_reduce<false>(rm, lane));
    alpha_mine = det_exp_le0(fsub(m_mine, m_new));
    m_mine = m_new;
#pragma unroll
    for (int i = 0; i < AF_RW; ++i) rm[i] = __shfl_sync(0xffffffffu, m_new, ROW_LANE(i));
    bool tp = false;
    // 64 independent exponentials in one straight-line block (no branch, no shuffle in between), so that their
    // dependent chains interleave; invisible pairs are zeroed afterwards (their arguments may be anything)
#pragma unroll
    for (int i = 0; i < AF_RW; ++i)
#pragma unroll
      for (int e = 0; e < 4; ++e) RP(acc, i, e) = det_exp_le0(fsub(RP(acc, i, e), rm[i]));
    if (diag) {
#pragma unroll
      for (int i = 0; i < AF_RW; ++i)
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if (j0 + 4 * lane + e > q0 + wrow + i) RP(acc, i, e) = 0.0f;
    }
#pragma unroll
    for (int i = 0; i < AF_RW; ++i) {
      float p[4] = {RP(acc, i, 0), RP(acc, i, 1), RP(acc, i, 2), RP(acc, i, 3)};
      rm[i] = fadd(fadd(p[0], p[1]), fadd(p[2], p[3]));      // the lane's four adjacent slots of the block's row sum
#pragma unroll
      for (int e = 0; e < 4; ++e) { p[e] = bf2f(f2bf(p[e])); tp |= tiny1(p[e]); RP(acc, i, e) = p[e]; }
    }
    // the rest of the adjacent tree over the block's 128 slots: lanes 1, 2, 4, 8, 16 apart
    l_mine = fadd(fmul(l_mine, alpha_mine), rows_reduce<true>(rm, lane));
    // P~ of the warp's rows: key row 4 lane + e, chunk of rows 4g .. 4g+3
    __syncwarp();                                    // the previous block's P.V loads are done
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      float* prow = Ps + (size_t)(4 * lane + e) * FQ;
#pragma unroll
      for (int g = 0; g < AF_RW / 4; ++g) {
        const float4 t = make_float4(RP(acc, 4 * g, e), RP(acc, 4 * g + 1, e), RP(acc, 4 * g + 2, e), RP(acc, 4 * g + 3, e));
        *reinterpret_cast<float4*>(prow + ((((wrow >> 2) + g) ^ (lane & 7)) << 2)) = t;
      }
    }
    const int tiny_p = __any_sync(0xffffffffu, tp);  // also orders the stores before the loads below
    __syncwarp();
    // ---- u = P~ . V over the block's keys ascending from +0, then o = o * alpha + u ----
#pragma unroll
    for (int a = 0; a < AF_RW / 2; ++a)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[a][c] = make_float2(0.0f, 0.0f);
    const int last_slab = diag ? (wrow + AF_RW - 1) / OK : 7;          // on the diagonal the warp's rows see no key past 16 (warp + 1)
    for (int sl = 0; sl < 8; ++sl, ++s) {
      const int slot = s % AF_SLOTS;
      const int tiny = tiny_p | tiny_cur;
      if (!acquire(s + 1)) { ok = false; break; }
      if (sl <= last_slab) {
        const float* ap = Ps + (size_t)(sl * OK) * FQ;
        if (tiny) mac_16x4<false, true>(ap, FQ, wrow >> 2, sl * OK, Ring[slot], lane, acc);
        else mac_16x4<true, true>(ap, FQ, wrow >> 2, sl * OK, Ring[slot], lane, acc);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&bar_empty[slot]);
    }
    if (!ok) break;
#pragma unroll
    for (int i = 0; i < AF_RW; ++i) {  // scalar: the product o * alpha is rounded before the add
      const float al = __shfl_sync(0xffffffffu, alpha_mine, ROW_LANE(i));
#pragma unroll
      for (int c = 0; c < 4; ++c) RP(o, i, c) = fadd(fmul(RP(o, i, c), al), RP(acc, i, c));
    }
  }
  if (!ok) return;
  const float il_mine = fdiv(1.0f, l_mine);
  const float lse_mine = fadd(m_mine, det_log(l_mine));
  if (lane < AF_RW && q0 + wrow + ROW_OF_LANE(lane) < S) lse[((size_t)b * H + h) * S + q0 + wrow + ROW_OF_LANE(lane)] = lse_mine;
  const float inv_q = qout ? fdiv(1.0f, s_q[0]) : 0.0f;
#pragma unroll
  for (int i = 0; i < AF_RW; ++i) {
    const int row = q0 + wrow + i;
    const float il = __shfl_sync(0xffffffffu, il_mine, ROW_LANE(i));
    if (row >= S) continue;
    uint2 w0;
    w0.x = pack_bf2(fmul(RP(o, i, 0), il), fmul(RP(o, i, 1), il));
    w0.y = pack_bf2(fmul(RP(o, i, 2), il), fmul(RP(o, i, 3), il));
    *reinterpret_cast<uint2*>(out + (row0 + row) * ld_out + (size_t)h * DH + 4 * lane) = w0;
    if (qout) {   // the output projection's quantiser, applied to the bf16 values just stored
      const float f0 = bflo(w0.x), f1 = bfhi(w0.x), f2 = bflo(w0.y), f3 = bfhi(w0.y);
      const uint32_t c = ((uint32_t)(uint8_t)quant1(f0, inv_q)) | ((uint32_t)(uint8_t)quant1(f1, inv_q) << 8) |
                         ((uint32_t)(uint8_t)quant1(f2, inv_q) << 16) | ((uint32_t)(uint8_t)quant1(f3, inv_q) << 24);
      *reinterpret_cast<uint32_t*>(qout + (row0 + row) * ld_out + (size_t)h * DH + 4 * lane) = c;
    }
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

// ---------------------------------------------------------------------------------------------
// backward, first half: P and dS of one block of 128 queries against every visible block of 128 keys.
// Warp-specialised like the LM-head kernel: the CTA keeps q^T and dO^T of its query block in shared memory; four
// producer warps stream the key and value blocks through a three-slot ring of 16-dimension slabs (a "full" and an
// "empty" mbarrier per slot, bounded waits); eight consumer warps accumulate S = q.k^T and dP = dO.v^T together (two
// 8 x 8 register tiles per thread, each logit one ascending sum over the 128 dimensions) and, per key block, apply
// P = exp(S*scale - L) and dS = (P (dP - Delta)) scale and store bf16(P) and bf16(dS).  The producers already fetch
// the next key block while the consumers are in that epilogue, and consumer warps are not coupled to each other.
// ---------------------------------------------------------------------------------------------
constexpr size_t SDP_SMEM = (size_t)(2 * DH * (OT + 4) + 2 * WS_STAGES * OK * (OT + 4)) * sizeof(float);

__global__ void __launch_bounds__(WS_THREADS, 1)
    k_attn_sdp_ws(const uint16_t* __restrict__ dout, const uint16_t* __restrict__ q, const uint16_t* __restrict__ k,
                  const uint16_t* __restrict__ v, const float* __restrict__ lse, const float* __restrict__ delta, int ld,
                  int ld_out, int H, int Hkv, int S, int W, uint16_t* __restrict__ Pb, uint16_t* __restrict__ dSt) {
  extern __shared__ __align__(16) unsigned char osm[];
  typedef float(*Full)[OT + 4];
  Full Qs = reinterpret_cast<Full>(osm);                                            // [dim][query]
  Full Os = reinterpret_cast<Full>(osm + (size_t)DH * (OT + 4) * sizeof(float));    // [dim][query] of dO
  float(*Ks)[OK][OT + 4] = reinterpret_cast<float(*)[OK][OT + 4]>(osm + (size_t)2 * DH * (OT + 4) * sizeof(float));
  float(*Vs)[OK][OT + 4] = Ks + WS_STAGES;
  __shared__ int tiny_s[WS_STAGES][WS_PROD / 32];
  __shared__ int tiny_qo, abort_s;
  __shared__ __align__(8) uint64_t bar_full[WS_STAGES], bar_empty[WS_STAGES];
  volatile int* abort_flag = &abort_s;
  const int it = gridDim.y - 1 - blockIdx.y;        // longest rows first
  const int h = blockIdx.x % H, b = blockIdx.x / H, hk = h / (H / Hkv);
  const int i0 = it * OT;
  const int tid = threadIdx.x, lane = tid & 31;
  const size_t row0 = (size_t)b * S;
  const uint16_t* qp = q + row0 * ld + (size_t)h * DH;
  const uint16_t* op = dout + row0 * ld_out + (size_t)h * DH;
  const uint16_t* kp = k + row0 * ld + (size_t)hk * DH;
  const uint16_t* vp = v + row0 * ld + (size_t)hk * DH;
  const int jt_lo = (W > 0 && i0 > W) ? (i0 - W) / OT : 0;
  const int ntile = it - jt_lo + 1, nslab = ntile * (DH / OK);
  if (tid == 0) {
    for (int s = 0; s < WS_STAGES; ++s) { mbar_init(&bar_full[s], WS_PROD / 32); mbar_init(&bar_empty[s], WS_CONS / 32); }
    tiny_qo = 0;
    abort_s = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  {  // q^T and dO^T of the query block, staged once by everybody
    bool tq = false;
    for (int idx = tid; idx < 2 * OT * 16; idx += WS_THREADS) {
      const int which = idx >= OT * 16, e = idx - which * OT * 16, r = e & 127, ch = e >> 7;
      const uint16_t* src = which ? op + (size_t)(i0 + r) * ld_out : qp + (size_t)(i0 + r) * ld;
      float t[8];
      if (i0 + r < S) unpack8a(__ldg(reinterpret_cast<const uint4*>(src + ch * 8)), t);
      else {
#pragma unroll
        for (int x = 0; x < 8; ++x) t[x] = 0.0f;
      }
      Full dst = which ? Os : Qs;
#pragma unroll
      for (int x = 0; x < 8; ++x) { tq |= tiny1(t[x]); dst[ch * 8 + x][r] = t[x]; }
    }
    if (__any_sync(0xffffffffu, tq) && lane == 0) atomicOr(&tiny_qo, 1);
  }
  __syncthreads();
  if (tid >= WS_CONS) {
    // ------------------------------- producers -------------------------------
    asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
    const int pt = tid - WS_CONS, pw = pt >> 5;
    WsRaw<CONTIG, false, OT> rk, rv;
    ws_fetch<CONTIG, false, OT>(kp, S, DH, ld, jt_lo * OT, 0, pt, rk);
    ws_fetch<CONTIG, false, OT>(vp, S, DH, ld, jt_lo * OT, 0, pt, rv);
    for (int s = 0; s < nslab; ++s) {
      const int slot = s % WS_STAGES;
      if (s >= WS_STAGES && !mbar_wait(&bar_empty[slot], (uint32_t)((s / WS_STAGES - 1) & 1), abort_flag, nullptr)) break;
      bool tiny = ws_store<CONTIG, false, OT>(Ks[slot], pt, rk);
      tiny |= ws_store<CONTIG, false, OT>(Vs[slot], pt, rv);
      if (s + 1 < nslab) {
        const int j0n = (jt_lo + (s + 1) / (DH / OK)) * OT, c0n = ((s + 1) % (DH / OK)) * OK;
        ws_fetch<CONTIG, false, OT>(kp, S, DH, ld, j0n, c0n, pt, rk);
        ws_fetch<CONTIG, false, OT>(vp, S, DH, ld, j0n, c0n, pt, rv);
      }
      const int any = __any_sync(0xffffffffu, tiny);
      if (lane == 0) tiny_s[slot][pw] = any;
      __syncwarp();
      if (lane == 0) mbar_arrive(&bar_full[slot]);
    }
    return;
  }
  // --------------------------------- consumers ---------------------------------
  asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
  const int ty = tid >> 4, tx = tid & 15;
  const int tqo = tiny_qo;
  const size_t bh = (size_t)b * H + h;
  float Lr[8], Dr[8];
#pragma unroll
  for (int a = 0; a < 8; ++a) {
    const int i = i0 + (a >> 2) * 64 + ty * 4 + (a & 3);
    Lr[a] = i < S ? lse[bh * S + i] : 0.0f;
    Dr[a] = i < S ? delta[bh * S + i] : 0.0f;
  }
  int s = 0;
  bool ok = true;
  for (int jt = jt_lo; jt <= it && ok; ++jt) {
    const int j0 = jt * OT;
    float2 sa[8][4], da[8][4];
#pragma unroll
    for (int a = 0; a < 8; ++a)
#pragma unroll
      for (int c = 0; c < 4; ++c) { sa[a][c] = make_float2(0.f, 0.f); da[a][c] = make_float2(0.f, 0.f); }
    for (int sl = 0; sl < DH / OK; ++sl, ++s) {
      const int slot = s % WS_STAGES;
      if (!mbar_wait(&bar_full[slot], (uint32_t)((s / WS_STAGES) & 1), abort_flag, nullptr)) { ok = false; break; }
      const int tiny = tqo | tiny_s[slot][0] | tiny_s[slot][1] | tiny_s[slot][2] | tiny_s[slot][3];
      if (tiny) { slab_mac<false, OT>(Qs + sl * OK, Ks[slot], ty, tx, sa); slab_mac<false, OT>(Os + sl * OK, Vs[slot], ty, tx, da); }
      else { slab_mac<true, OT>(Qs + sl * OK, Ks[slot], ty, tx, sa); slab_mac<true, OT>(Os + sl * OK, Vs[slot], ty, tx, da); }
      __syncwarp();
      if (lane == 0) mbar_arrive(&bar_empty[slot]);
    }
    if (!ok) break;
#pragma unroll
    for (int a = 0; a < 8; ++a) {
      const int i = i0 + (a >> 2) * 64 + ty * 4 + (a & 3);
      if (i >= S) continue;
#pragma unroll
      for (int g = 0; g < 2; ++g) {
        const int jb = j0 + g * 64 + tx * 4;
        if (jb >= S) continue;
        const float sv[4] = {sa[a][2 * g].x, sa[a][2 * g].y, sa[a][2 * g + 1].x, sa[a][2 * g + 1].y};
        const float dv4[4] = {da[a][2 * g].x, da[a][2 * g].y, da[a][2 * g + 1].x, da[a][2 * g + 1].y};
        float pv[4], dsv[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {   // branch-free (selects), so that the exponentials' chains interleave
          const bool vis = jb + e <= i && (W == 0 || jb + e > i - W);
          const float pe = det_exp(fsub(fmul(sv[e], ATT_SCALE), Lr[a]));
          const float de = fmul(fmul(pe, fsub(dv4[e], Dr[a])), ATT_SCALE);
          pv[e] = vis ? pe : 0.0f;
          dsv[e] = vis ? de : 0.0f;
        }
        const size_t off = (bh * S + i) * S + jb;
        uint2 u;
        u.x = pack_bf2(pv[0], pv[1]); u.y = pack_bf2(pv[2], pv[3]);        // P~ = bf16(P) is all the value gradient needs
        *reinterpret_cast<uint2*>(Pb + off) = u;
        u.x = pack_bf2(dsv[0], dsv[1]); u.y = pack_bf2(dsv[2], dsv[3]);
        *reinterpret_cast<uint2*>(dSt + off) = u;
      }
    }
  }
}


}  // namespace det

using namespace det;

static int attn_fwd_impl(const det_bf16* q, const det_bf16* k, const det_bf16* v, int ld, int B, int H, int Hkv, int S,
                         int window, det_bf16* out, int ld_out, float* lse, const float* s_q, int8_t* qout, void* stream) {
  if (!q || !k || !v || !out || !lse || B <= 0 || H <= 0 || Hkv <= 0 || S <= 0 || window < 0) return DET_ERR_ARG;
  if (qout && (!s_q || (((uintptr_t)qout) & 3u))) return qout && !s_q ? DET_ERR_ARG : DET_ERR_ALIGN;
  if (S % 64 || ld % 8 || ld_out % 8 || ld < H * DH || ld_out < H * DH || H % Hkv || window % 128) return DET_ERR_SHAPE;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return DET_ERR_ALIGN;
  static DevOnce once_win = {};
  if (dev_ensure_smem(once_win, (const void*)k_attn_fwd<true>, FWD_SMEM) != DET_OK) return DET_ERR_CUDA;
  dim3 grid(H * B, (S + FQ - 1) / FQ);
  static DevOnce once_ws = {};
  if (dev_ensure_smem(once_ws, (const void*)k_attn_fwd_ws, AFW_SMEM) != DET_OK) return DET_ERR_CUDA;
  if (window) k_attn_fwd<true><<<DET_L(grid), FT, FWD_SMEM, (cudaStream_t)stream>>>(q, k, v, ld, H, Hkv, S, window, out, ld_out, lse, s_q, qout);
  else k_attn_fwd_ws<<<DET_L(grid), AF_THREADS, AFW_SMEM, (cudaStream_t)stream>>>(q, k, v, ld, H, Hkv, S, out, ld_out, lse, s_q, qout);
  DET_CHECK_LAUNCH();
  return DET_OK;
}

extern "C" int det_attn_fwd(const det_bf16* q, const det_bf16* k, const det_bf16* v, int ld, int B, int H, int Hkv, int S,
                            int window, det_bf16* out, int ld_out, float* lse, void* stream) {
  return attn_fwd_impl(q, k, v, ld, B, H, Hkv, S, window, out, ld_out, lse, nullptr, nullptr, stream);
}
extern "C" int det_attn_fwd_q(const det_bf16* q, const det_bf16* k, const det_bf16* v, int ld, int B, int H, int Hkv, int S,
                              int window, det_bf16* out, int ld_out, float* lse, const float* s_q, int8_t* qout, void* stream) {
  if (!s_q || !qout) return DET_ERR_ARG;
  return attn_fwd_impl(q, k, v, ld, B, H, Hkv, S, window, out, ld_out, lse, s_q, qout, stream);
}

// workspace: bf16(P) and bf16(dS), [B*H, S, S] each, Delta f32 [B*H, S], and with grouped queries the f32 accumulators
// [B*Hkv, S, 128] that carry dK / dV from one query head of a group to the next
extern "C" size_t det_attn_bwd_ws_bytes(int B, int H, int Hkv, int S) {
  return 2 * align_up((size_t)B * H * S * S * 2, 256) +
         align_up((size_t)B * H * S * 4, 256) + (Hkv < H ? align_up((size_t)B * Hkv * S * DH * 4, 256) : 0);
}

// the fixed-point variant keeps its 64-bit accumulators in registers: no extra scratch
extern "C" size_t det_attn_bwd_fixq_ws_bytes(int B, int H, int Hkv, int S) { return det_attn_bwd_ws_bytes(B, H, Hkv, S); }

static int attn_bwd_impl(const det_bf16* dout, const det_bf16* q, const det_bf16* k, const det_bf16* v,
                         const det_bf16* out, const float* lse, int ld, int ld_out, int B, int H, int Hkv, int S,
                         int window, det_bf16* dq, det_bf16* dk, det_bf16* dv, int ld_d, void* ws, size_t ws_bytes,
                         void* stream, bool fixq) {
  if (!dout || !q || !k || !v || !out || !lse || !dq || !dk || !dv || B <= 0 || H <= 0 || Hkv <= 0 || S <= 0 || window < 0)
    return DET_ERR_ARG;
  if (S % 64 || ld % 8 || ld_out % 8 || ld_d % 8 || (long long)B * H > 65535 || H % Hkv || window % 128) return DET_ERR_SHAPE;
  if (!aligned16(dout) || !aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(dq) ||
      !aligned16(dk) || !aligned16(dv) || !aligned16(ws))
    return DET_ERR_ALIGN;
  if (!ws || ws_bytes < (fixq ? det_attn_bwd_fixq_ws_bytes(B, H, Hkv, S) : det_attn_bwd_ws_bytes(B, H, Hkv, S)))
    return DET_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  const int G = H / Hkv;
  const size_t matP = align_up((size_t)B * H * S * S * 2, 256), matS = matP;
  const size_t dl = align_up((size_t)B * H * S * 4, 256);
  uint16_t* Pb = (uint16_t*)ws;
  uint16_t* dSt = (uint16_t*)((uint8_t*)ws + matP);
  float* delta = (float*)((uint8_t*)ws + matP + matS);
  float* carry = (float*)((uint8_t*)ws + matP + matS + dl);
  const size_t nrows = (size_t)B * H * S;
  k_attn_delta<<<DET_L((unsigned)((nrows + 7) / 8)), 256, 0, st>>>(dout, out, ld_out, H, S, nrows, delta);
  DET_CHECK_LAUNCH();
  // P[i,j] = exp(scale * sum_d q[i,d] k[j,d] - L_i) for visible (i,j) (f32; tiles without a visible pair are never
  // touched) and dS[i,j] = bf16((P[i,j] * (sum_d dO[i,d] v[j,d] - Delta_i)) * scale); both sums ascend over the 128 dims
  static DevOnce once_sdp = {};
  if (dev_ensure_smem(once_sdp, (const void*)k_attn_sdp_ws, SDP_SMEM) != DET_OK) return DET_ERR_CUDA;
  dim3 gsdp(H * B, (S + OT - 1) / OT);
  k_attn_sdp_ws<<<DET_L(gsdp), WS_THREADS, SDP_SMEM, st>>>(dout, q, k, v, lse, delta, ld, ld_out, H, Hkv, S, window, Pb, dSt);
  DET_CHECK_LAUNCH();
  int rc = DET_OK;
  // dV[j,c] = sum over the query heads g of the group, then over queries i >= j ascending, of P~[i,j] dO[i,c];
  // dK[j,c] likewise with dS~ and q.  One accumulator per output: with G > 1 it travels through `carry` in f32, and
  // the two chains then share that scratch and run one after the other.  dV, dK (for G == 1) and dQ are independent of
  // each other and run side by side on auxiliary streams, so that the short blocks at the end of one grid overlap
  // with the long blocks at the start of the next.
  AuxScope aux(st);   // joined again on every way out
  for (int which = 0; which < 2; ++which) {
    cudaStream_t sk = (G == 1 && which == 1) ? aux.aux(0) : st;
    for (int g = 0; g < G; ++g) {
      OgemmArgs p = {};
      p.I = S; p.J = DH; p.C = S; p.lda = S; p.H = Hkv; p.a_b = (long long)H * S * S; p.a_h = (long long)S * S;
      p.h_mul = G; p.h_add = g; p.range_mode = 1; p.window = window;
      p.A = which == 0 ? (const void*)Pb : (const void*)dSt;
      if (which == 0) { p.B = dout; p.ldb = ld_out; p.b_b = (long long)S * ld_out; }
      else { p.B = q; p.ldb = ld; p.b_b = (long long)S * ld; }
      p.b_h = DH;
      if (g > 0) { p.acc_in = carry; p.acc_ld = DH; p.acc_b = (long long)Hkv * S * DH; p.acc_h = (long long)S * DH; }
      if (g == G - 1) {
        p.out = which == 0 ? dv : dk; p.ldo = ld_d; p.o_b = (long long)S * ld_d; p.o_h = DH;
        rc = ogemm_wb_launch<STRIDED, STRIDED, false, true>(p, B * Hkv, sk);
      } else {
        p.out = carry; p.ldo = DH; p.o_b = (long long)Hkv * S * DH; p.o_h = (long long)S * DH;
        rc = ogemm_wb_launch<STRIDED, STRIDED, false, false>(p, B * Hkv, sk);
      }
      if (rc != DET_OK) return rc;
    }
  }
  // dQ[i,c] = sum over visible keys j ascending of dS~[i,j] k[j,c]
  OgemmArgs p = {};
  p.I = S; p.J = DH; p.C = S; p.lda = S; p.H = H; p.a_b = (long long)H * S * S; p.a_h = (long long)S * S;
  p.A = dSt; p.B = k; p.ldb = ld; p.b_b = (long long)S * ld; p.b_h = DH; p.b_div = G;
  p.out = dq; p.ldo = ld_d; p.o_b = (long long)S * ld_d; p.o_h = DH; p.range_mode = 2; p.window = window;
  if (fixq) {
    // per block of 128 keys the ordered f32 sum, accumulated over the blocks in 64-bit fixed point (Sec. 3.2)
    rc = ogemm_fix_launch<CONTIG, STRIDED, false>(p, B * H, aux.aux(1));
  } else {
    rc = ogemm_wb_launch<CONTIG, STRIDED, false, true>(p, B * H, aux.aux(1));
  }
  if (rc != DET_OK) return rc;
  if (!aux.join()) return DET_ERR_CUDA;
  DET_CHECK_LAUNCH();
  return DET_OK;
}

extern "C" int det_attn_bwd(const det_bf16* dout, const det_bf16* q, const det_bf16* k, const det_bf16* v,
                            const det_bf16* out, const float* lse, int ld, int ld_out, int B, int H, int Hkv, int S,
                            int window, det_bf16* dq, det_bf16* dk, det_bf16* dv, int ld_d, void* ws, size_t ws_bytes,
                            void* stream) {
  return attn_bwd_impl(dout, q, k, v, out, lse, ld, ld_out, B, H, Hkv, S, window, dq, dk, dv, ld_d, ws, ws_bytes, stream, false);
}
extern "C" int det_attn_bwd_fixq(const det_bf16* dout, const det_bf16* q, const det_bf16* k, const det_bf16* v,
                                 const det_bf16* out, const float* lse, int ld, int ld_out, int B, int H, int Hkv, int S,
                                 int window, det_bf16* dq, det_bf16* dk, det_bf16* dv, int ld_d, void* ws,
                                 size_t ws_bytes, void* stream) {
  return attn_bwd_impl(dout, q, k, v, out, lse, ld, ld_out, B, H, Hkv, S, window, dq, dk, dv, ld_d, ws, ws_bytes, stream, true);
}
