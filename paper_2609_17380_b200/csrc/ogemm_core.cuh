// The ordered FP32-ALU contractions (LM head, attention backward): C[i,j] = sum over c ascending of A(i,c) B(j,c), one
// sequential accumulator per output.  Operand slabs are staged through shared memory as f32 by producer warps, consumer
// warps hold 8 x 16 (or two 8 x 8) register tiles and use packed two-lane arithmetic; a per-slab check decides between the
// fused and the two-instruction multiply-add (identical bits, see ogemm.cu).
#pragma once
#include "tc05.cuh"
#include "internal.h"

namespace det {

constexpr int OT = 128;  // tile edge
constexpr int OK = 16;   // slab depth

// Operand access modes.  C[i,j] = sum_c A(i,c) * B(j,c).
//   CONTIG : operand stored [rows, contraction] (contraction index contiguous)
//   STRIDED: operand stored [contraction, rows] (row index contiguous)
enum { CONTIG = 0, STRIDED = 1 };

// One 16-deep slab for this thread's 8 x (TN/16) outputs.  FUSED: a*b+acc in one instruction, used only for slabs in
// which no product can be subnormal (every non-zero factor is at least 2^-63 in magnitude), where it gives exactly the
// bits of the unfused sequence because a product of two bf16 values is exact in binary32.  Two accumulators are
// processed per instruction (packed f32x2 arithmetic, each lane rounded on its own).
template <bool FUSED, int TN>
__device__ __forceinline__ void slab_mac(const float (*As)[OT + 4], const float (*Bs)[TN + 4], int ty, int tx,
                                         float2 (&acc)[8][TN / 32]) {
#pragma unroll
  for (int k = 0; k < OK; ++k) {
    const float4 a0 = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
    const float4 a1 = *reinterpret_cast<const float4*>(&As[k][64 + ty * 4]);
    const float av[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
    float2 b[TN / 32];
#pragma unroll
    for (int g = 0; g < TN / 64; ++g) {
      const float4 bv = *reinterpret_cast<const float4*>(&Bs[k][g * 64 + tx * 4]);
      b[2 * g] = make_float2(bv.x, bv.y);
      b[2 * g + 1] = make_float2(bv.z, bv.w);
    }
    // column pairs outermost: each pair of B values meets the eight rows back to back (measured a few percent faster
    // than rows outermost); the order in which different accumulators are visited has no effect on any result
#pragma unroll
    for (int j = 0; j < TN / 32; ++j) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (FUSED) {
          acc[i][j] = __ffma2_rn(make_float2(av[i], av[i]), b[j], acc[i][j]);
        } else {  // scalar on purpose: a packed multiply + add pair would be contracted by ptxas
          acc[i][j].x = fadd(acc[i][j].x, fmul(av[i], b[j].x));
          acc[i][j].y = fadd(acc[i][j].y, fmul(av[i], b[j].y));
        }
      }
    }
  }
}

// C[i,j] = sum over c in [c_lo, c_hi) ascending of A(i,c) B(j,c), one accumulator per output.
struct OgemmArgs {
  const void* A;
  const void* B;
  void* out;
  int I, J, C;          // rows of A, rows of B, contraction length
  int lda, ldb, ldo;    // leading dimensions of the stored operands / output
  int init;             // f32 output only: start from the values already in out
  int H;                // batching: blockIdx.z = b * H + h
  long long a_b, a_h, b_b, b_h, o_b, o_h;  // element offsets per batch index / head index
  // head mapping for grouped-query attention (0 = identity): A reads head hA = h * h_mul + h_add, B reads head
  // hA / b_div, the output (and acc_in) belongs to head h
  int h_mul, h_add, b_div;
  // optional f32 accumulators to start from (any output type): one sequential accumulator can be carried through
  // several launches this way; batched with acc_b / acc_h, leading dimension acc_ld
  const float* acc_in;
  int acc_ld;
  long long acc_b, acc_h;
  int window;           // sliding window W (multiple of 128; 0 = none): only |query - key| < W contributes
  int range_mode;       // 0: whole contraction; 1: c >= first row of the tile (causal, per key); 2: c < last row + 1 of the tile
                        // (with a window, mode 1 also stops at c < i0 + W + 128 and mode 2 starts at c >= i0 - W)
};

// ---------------------------------------------------------------------------------------------------------------
// Warp-specialised variant for the long contractions of the LM head: 128 x 256 tile, eight consumer warps that only
// multiply (8 x 16 register tiles fed from shared memory) and four producer warps that only stage (global loads,
// unpacking, the below-2^-63 test, shared-memory stores) into a three-slab ring.  Each ring slot has a "full" and an
// "empty" mbarrier: a producer warp arrives on "full" after its stores, a consumer warp arrives on "empty" after its
// last read, and everybody only waits for the other side, so consumer warps are not coupled to each other and the
// multiply pipe never waits for staging instructions of its own warp.  All waits are bounded.  Plain contraction only
// (no batching, ranges or epilogues).
// ---------------------------------------------------------------------------------------------------------------
constexpr int WS_STAGES = 3, WS_CONS = 256, WS_PROD = 128, WS_THREADS = WS_CONS + WS_PROD, WS_TN = 256;
constexpr size_t WS_SMEM = (size_t)WS_STAGES * OK * ((OT + 4) + (WS_TN + 4)) * sizeof(float);


// One producer thread's share of a slab of ROWS rows x 16 contraction steps, as raw words.
//   CONTIG : rows pt + 128*g (g < ROWS/128), all 16 contraction indices (two 16-byte words of bf16, four of f32, per row)
//   STRIDED: four consecutive rows 4f .. 4f+3 (f = pt mod ROWS/4) at the contraction indices kk + KPP*i, kk = pt / (ROWS/4),
//            KPP = 512/ROWS, i < 16/KPP: consecutive lanes read and store consecutive words, so the shared-memory stores
//            are free of bank conflicts
template <int MODE, bool F32IN, int ROWS>
struct WsRaw {
  static constexpr int NW = MODE == CONTIG ? (ROWS / 128) * 2 * (F32IN ? 2 : 1) : (16 * ROWS / 512) / (F32IN ? 1 : 2);
  uint4 w[NW];   // STRIDED bf16: two passes share one 16-byte register group (8 bytes each)
};
template <int MODE, bool F32IN, int ROWS>
__device__ __forceinline__ void ws_fetch(const void* base, int rows, int C, int ld, int r0, int c0, int pt,
                                         WsRaw<MODE, F32IN, ROWS>& raw) {
  constexpr int ESZ = F32IN ? 4 : 2;
  const char* b = reinterpret_cast<const char*>(base);
  if (MODE == CONTIG) {
    constexpr int EPW = F32IN ? 4 : 8;    // elements per 16-byte word
    constexpr int WPR = 16 / EPW;        // words per row
#pragma unroll
    for (int g = 0; g < ROWS / 128; ++g) {
      const int r = r0 + pt + 128 * g;
#pragma unroll
      for (int w = 0; w < WPR; ++w) {
        const int c = c0 + w * EPW;
        raw.w[g * WPR + w] = (r < rows && c < C) ? __ldg(reinterpret_cast<const uint4*>(b + ((size_t)r * ld + c) * ESZ))
                                                 : make_uint4(0u, 0u, 0u, 0u);
      }
    }
  } else {
    constexpr int F4 = ROWS / 4, KPP = 128 / F4, NP = 16 / KPP;
    const int f = pt % F4, kk = pt / F4;
    const int r = r0 + 4 * f;
#pragma unroll
    for (int i = 0; i < NP; ++i) {
      const int c = c0 + kk + KPP * i;
      const bool ok = c < C && r < rows;
      const char* src = b + ((size_t)c * ld + r) * ESZ;
      if (F32IN) {
        raw.w[i] = ok ? __ldg(reinterpret_cast<const uint4*>(src)) : make_uint4(0u, 0u, 0u, 0u);
      } else {
        const uint2 u = ok ? __ldg(reinterpret_cast<const uint2*>(src)) : make_uint2(0u, 0u);
        if (i & 1) { raw.w[i >> 1].z = u.x; raw.w[i >> 1].w = u.y; }
        else { raw.w[i >> 1].x = u.x; raw.w[i >> 1].y = u.y; }
      }
    }
  }
}
template <bool F32IN>
__device__ __forceinline__ void ws_unpack_word(const uint4& u, float* v) {   // 8 (bf16) or 4 (f32, rounded to bf16) values
  if (F32IN) {
    v[0] = bf2f(f2bf(__uint_as_float(u.x))); v[1] = bf2f(f2bf(__uint_as_float(u.y)));
    v[2] = bf2f(f2bf(__uint_as_float(u.z))); v[3] = bf2f(f2bf(__uint_as_float(u.w)));
  } else {
    v[0] = bflo(u.x); v[1] = bfhi(u.x); v[2] = bflo(u.y); v[3] = bfhi(u.y);
    v[4] = bflo(u.z); v[5] = bfhi(u.z); v[6] = bflo(u.w); v[7] = bfhi(u.w);
  }
}
// unpack, test and store one thread's share; returns the below-2^-63 flag of its values
template <int MODE, bool F32IN, int ROWS>
__device__ __forceinline__ bool ws_store(float (*s)[ROWS + 4], int pt, const WsRaw<MODE, F32IN, ROWS>& raw) {
  bool tiny = false;
  if (MODE == CONTIG) {
    constexpr int EPW = F32IN ? 4 : 8;
    constexpr int WPR = 16 / EPW;
#pragma unroll
    for (int g = 0; g < ROWS / 128; ++g)
#pragma unroll
      for (int w = 0; w < WPR; ++w) {
        float v[8];
        ws_unpack_word<F32IN>(raw.w[g * WPR + w], v);
#pragma unroll
        for (int e = 0; e < EPW; ++e) {
          tiny |= (__float_as_uint(v[e]) * 2u - 1u) < 0x3fffffffu;
          s[w * EPW + e][pt + 128 * g] = v[e];
        }
      }
  } else {
    constexpr int F4 = ROWS / 4, KPP = 128 / F4, NP = 16 / KPP;
    const int f = pt % F4, kk = pt / F4;
#pragma unroll
    for (int i = 0; i < NP; ++i) {
      float v[4];
      if (F32IN) {
        float t[8];
        ws_unpack_word<true>(raw.w[i], t);
        v[0] = t[0]; v[1] = t[1]; v[2] = t[2]; v[3] = t[3];
      } else {
        const uint32_t lo = (i & 1) ? raw.w[i >> 1].z : raw.w[i >> 1].x, hi = (i & 1) ? raw.w[i >> 1].w : raw.w[i >> 1].y;
        v[0] = bflo(lo); v[1] = bfhi(lo); v[2] = bflo(hi); v[3] = bfhi(hi);
      }
#pragma unroll
      for (int e = 0; e < 4; ++e) tiny |= (__float_as_uint(v[e]) * 2u - 1u) < 0x3fffffffu;
      *reinterpret_cast<float4*>(&s[kk + KPP * i][4 * f]) = make_float4(v[0], v[1], v[2], v[3]);
    }
  }
  return tiny;
}

template <int AMODE, int BMODE, bool AF32, bool OUT_BF16>
__global__ void __launch_bounds__(WS_THREADS, 1) k_ogemm_ws(OgemmArgs p) {
  extern __shared__ __align__(16) unsigned char osm[];
  float(*As)[OK][OT + 4] = reinterpret_cast<float(*)[OK][OT + 4]>(osm);
  float(*Bs)[OK][WS_TN + 4] = reinterpret_cast<float(*)[OK][WS_TN + 4]>(osm + (size_t)WS_STAGES * OK * (OT + 4) * sizeof(float));
  __shared__ int tiny_s[WS_STAGES][WS_PROD / 32];
  __shared__ __align__(8) uint64_t bar_full[WS_STAGES], bar_empty[WS_STAGES];
  __shared__ int abort_s;
  volatile int* abort_flag = &abort_s;
  const int i0 = blockIdx.y * OT, j0 = blockIdx.x * WS_TN;
  const int I = p.I, J = p.J, C = p.C, lda = p.lda, ldb = p.ldb, ldo = p.ldo;
  const int nslab = (C + OK - 1) / OK;
  const int tid = threadIdx.x, lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < WS_STAGES; ++s) { mbar_init(&bar_full[s], WS_PROD / 32); mbar_init(&bar_empty[s], WS_CONS / 32); }
    abort_s = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  // use n of a slot (slabs slot, slot + 3, ...) completes phase n of its barriers: the wait parity is n & 1
  if (tid >= WS_CONS) {
    // ------------------------------- producers -------------------------------
    // the producer warpgroup hands most of its registers to the two consumer warpgroups
    asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
    const int pt = tid - WS_CONS, pw = pt >> 5;
    WsRaw<AMODE, AF32, OT> ra;
    WsRaw<BMODE, false, WS_TN> rb;
    ws_fetch<AMODE, AF32, OT>(p.A, I, C, lda, i0, 0, pt, ra);
    ws_fetch<BMODE, false, WS_TN>(p.B, J, C, ldb, j0, 0, pt, rb);
    for (int s = 0; s < nslab; ++s) {
      const int slot = s % WS_STAGES;
      if (s >= WS_STAGES &&                                          // the consumers have left this slot
          !mbar_wait(&bar_empty[slot], (uint32_t)((s / WS_STAGES - 1) & 1), abort_flag, nullptr))
        break;
      bool tiny = ws_store<AMODE, AF32, OT>(As[slot], pt, ra);
      tiny |= ws_store<BMODE, false, WS_TN>(Bs[slot], pt, rb);
      if (s + 1 < nslab) {                                           // next slab's words travel during the handshake
        ws_fetch<AMODE, AF32, OT>(p.A, I, C, lda, i0, (s + 1) * OK, pt, ra);
        ws_fetch<BMODE, false, WS_TN>(p.B, J, C, ldb, j0, (s + 1) * OK, pt, rb);
      }
      const int any = __any_sync(0xffffffffu, tiny);
      if (lane == 0) tiny_s[slot][pw] = any;
      __syncwarp();
      if (lane == 0) mbar_arrive(&bar_full[slot]);                   // slot is full (releases the warp's stores)
    }
    return;
  }
  // --------------------------------- consumers ---------------------------------
  asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
  const int ty = tid >> 4, tx = tid & 15;
  float2 acc[8][WS_TN / 32];
#pragma unroll
  for (int a = 0; a < 8; ++a)
#pragma unroll
    for (int b = 0; b < WS_TN / 32; ++b) acc[a][b] = make_float2(0.0f, 0.0f);
  float* outf = reinterpret_cast<float*>(p.out);
  if (p.init && !OUT_BF16) {
#pragma unroll
    for (int a = 0; a < 8; ++a) {
      const int r = i0 + (a >> 2) * 64 + ty * 4 + (a & 3);
#pragma unroll
      for (int g = 0; g < WS_TN / 64; ++g) {
        const int c = j0 + g * 64 + tx * 4;
        if (r < I && c < J) {
          const float4 t = *reinterpret_cast<const float4*>(outf + (size_t)r * ldo + c);
          acc[a][2 * g] = make_float2(t.x, t.y);
          acc[a][2 * g + 1] = make_float2(t.z, t.w);
        }
      }
    }
  }
  for (int s = 0; s < nslab; ++s) {
    const int slot = s % WS_STAGES;
    if (!mbar_wait(&bar_full[slot], (uint32_t)((s / WS_STAGES) & 1), abort_flag, nullptr)) break;   // slot is full
    const int tiny = tiny_s[slot][0] | tiny_s[slot][1] | tiny_s[slot][2] | tiny_s[slot][3];
    if (tiny) slab_mac<false, WS_TN>(As[slot], Bs[slot], ty, tx, acc);
    else slab_mac<true, WS_TN>(As[slot], Bs[slot], ty, tx, acc);
    __syncwarp();
    if (lane == 0) mbar_arrive(&bar_empty[slot]);                    // slot may be refilled
  }
#pragma unroll
  for (int a = 0; a < 8; ++a) {
    const int r = i0 + (a >> 2) * 64 + ty * 4 + (a & 3);
#pragma unroll
    for (int g = 0; g < WS_TN / 64; ++g) {
      const int c = j0 + g * 64 + tx * 4;
      if (r < I && c < J) {
        const float2 lo = acc[a][2 * g], hi = acc[a][2 * g + 1];
        if (OUT_BF16) {
          uint2 u;
          u.x = pack_bf2(lo.x, lo.y);
          u.y = pack_bf2(hi.x, hi.y);
          *reinterpret_cast<uint2*>(reinterpret_cast<uint16_t*>(p.out) + (size_t)r * ldo + c) = u;
        } else {
          *reinterpret_cast<float4*>(outf + (size_t)r * ldo + c) = make_float4(lo.x, lo.y, hi.x, hi.y);
        }
      }
    }
  }
}

template <int AMODE, int BMODE, bool AF32, bool OUT_BF16>
static int ogemm_ws_launch(const OgemmArgs& p, cudaStream_t st) {
  static DevOnce once = {};
  if (dev_ensure_smem(once, (const void*)k_ogemm_ws<AMODE, BMODE, AF32, OUT_BF16>, WS_SMEM) != DET_OK) return DET_ERR_CUDA;
  dim3 grid((p.J + WS_TN - 1) / WS_TN, (p.I + OT - 1) / OT, 1);
  k_ogemm_ws<AMODE, BMODE, AF32, OUT_BF16><<<DET_L(grid), WS_THREADS, WS_SMEM, st>>>(p);
  return DET_OK;
}

// ---------------------------------------------------------------------------------------------------------------
// Warp-specialised batched variant for the causal contractions of the attention backward: 128 x 128 tile, four consumer
// warps with 8 x 16 register tiles (rows {ty*4.., 64 + ty*4..}, columns g*32 + tx*4.., g < 4, eight threads across the
// columns), four producer warps, the same mbarrier-guarded ring; two CTAs per SM.  Batching, head mapping, causal ranges,
// windows and carried accumulators as in k_ogemm.
// ---------------------------------------------------------------------------------------------------------------
constexpr int WB_CONS = 128, WB_THREADS = WB_CONS + WS_PROD;
constexpr size_t WB_SMEM = (size_t)WS_STAGES * OK * 2 * (OT + 4) * sizeof(float);

// Which tile a CTA of the batched kernels works on, and over which part of the contraction.
struct WbTile {
  int i0, j0, zidx, c_lo, C, nslab;
  long long zb, zh, hA, hB;
};
__device__ __forceinline__ WbTile wb_tile(const OgemmArgs& p) {
  WbTile t;
  // row tile on the slowest grid index, longest contraction first
  const bool causal = p.range_mode == 1 || p.range_mode == 2;
  const int ti = causal ? (p.range_mode == 2 ? (int)(gridDim.z - 1 - blockIdx.z) : (int)blockIdx.z) : (int)blockIdx.y;
  t.zidx = causal ? (int)blockIdx.y : (int)blockIdx.z;
  t.i0 = ti * OT;
  t.j0 = blockIdx.x * OT;
  const int W = p.window;
  t.zb = t.zidx / p.H;
  t.zh = t.zidx % p.H;
  t.hA = t.zh * (p.h_mul ? p.h_mul : 1) + p.h_add;
  t.hB = t.hA / (p.b_div ? p.b_div : 1);
  t.c_lo = 0;
  t.C = p.C;
  if (p.range_mode == 1) { t.c_lo = t.i0; if (W) t.C = min(p.C, t.i0 + W + OT); }
  if (p.range_mode == 2) { t.C = min(p.C, t.i0 + OT); if (W) t.c_lo = max(0, t.i0 - W); }
  t.nslab = (t.C - t.c_lo + OK - 1) / OK;
  return t;
}
// The producer warps of the batched kernels: 16-deep slabs of both operands into the ring, one slab ahead in registers.
template <int AMODE, int BMODE, bool AF32>
__device__ __forceinline__ void wb_produce(const OgemmArgs& p, const WbTile& t, float (*As)[OK][OT + 4], float (*Bs)[OK][OT + 4],
                                           int (*tiny_s)[WS_PROD / 32], uint64_t* bar_full, uint64_t* bar_empty,
                                           volatile int* abort_flag, int pt) {
  const int lane = pt & 31, pw = pt >> 5;
  const void* A = AF32 ? (const void*)(reinterpret_cast<const float*>(p.A) + t.zb * p.a_b + t.hA * p.a_h)
                       : (const void*)(reinterpret_cast<const uint16_t*>(p.A) + t.zb * p.a_b + t.hA * p.a_h);
  const void* B = reinterpret_cast<const uint16_t*>(p.B) + t.zb * p.b_b + t.hB * p.b_h;
  WsRaw<AMODE, AF32, OT> ra;
  WsRaw<BMODE, false, OT> rb;
  if (t.nslab > 0) {
    ws_fetch<AMODE, AF32, OT>(A, p.I, t.C, p.lda, t.i0, t.c_lo, pt, ra);
    ws_fetch<BMODE, false, OT>(B, p.J, t.C, p.ldb, t.j0, t.c_lo, pt, rb);
  }
  for (int s = 0; s < t.nslab; ++s) {
    const int slot = s % WS_STAGES;
    if (s >= WS_STAGES && !mbar_wait(&bar_empty[slot], (uint32_t)((s / WS_STAGES - 1) & 1), abort_flag, nullptr)) break;
    bool tiny = ws_store<AMODE, AF32, OT>(As[slot], pt, ra);
    tiny |= ws_store<BMODE, false, OT>(Bs[slot], pt, rb);
    if (s + 1 < t.nslab) {
      ws_fetch<AMODE, AF32, OT>(A, p.I, t.C, p.lda, t.i0, t.c_lo + (s + 1) * OK, pt, ra);
      ws_fetch<BMODE, false, OT>(B, p.J, t.C, p.ldb, t.j0, t.c_lo + (s + 1) * OK, pt, rb);
    }
    const int any = __any_sync(0xffffffffu, tiny);
    if (lane == 0) tiny_s[slot][pw] = any;
    __syncwarp();
    if (lane == 0) mbar_arrive(&bar_full[slot]);
  }
}

template <bool FUSED>
__device__ __forceinline__ void slab_mac_8x16n(const float (*As)[OT + 4], const float (*Bs)[OT + 4], int ty, int tx,
                                               float2 (&acc)[8][8]) {
#pragma unroll
  for (int k = 0; k < OK; ++k) {
    const float4 a0 = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
    const float4 a1 = *reinterpret_cast<const float4*>(&As[k][64 + ty * 4]);
    const float av[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
    float2 b[8];
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      const float4 bv = *reinterpret_cast<const float4*>(&Bs[k][g * 32 + tx * 4]);
      b[2 * g] = make_float2(bv.x, bv.y);
      b[2 * g + 1] = make_float2(bv.z, bv.w);
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (FUSED) {
          acc[i][j] = __ffma2_rn(make_float2(av[i], av[i]), b[j], acc[i][j]);
        } else {  // scalar on purpose: a packed multiply + add pair would be contracted by ptxas
          acc[i][j].x = fadd(acc[i][j].x, fmul(av[i], b[j].x));
          acc[i][j].y = fadd(acc[i][j].y, fmul(av[i], b[j].y));
        }
      }
    }
  }
}

// f32 -> signed 64-bit fixed point with 48 fractional bits: round to nearest even, saturate, NaN -> 0
__device__ __forceinline__ long long fix48(float u) {
  const float t = fmul(u, 0x1p48f);
  if (t != t) return 0;
  if (t >= 0x1p63f) return 0x7fffffffffffffffll;
  if (t <= -0x1p63f) return (long long)0x8000000000000000ull;
  return __float2ll_rn(t);
}
__device__ __forceinline__ float unfix48(long long a) { return fmul(__ll2float_rn(a), 0x1p-48f); }

template <int AMODE, int BMODE, bool AF32, bool OUT_BF16>
__global__ void __launch_bounds__(WB_THREADS, 2) k_ogemm_wb(OgemmArgs p) {
  extern __shared__ __align__(16) unsigned char osm[];
  float(*As)[OK][OT + 4] = reinterpret_cast<float(*)[OK][OT + 4]>(osm);
  float(*Bs)[OK][OT + 4] = As + WS_STAGES;
  __shared__ int tiny_s[WS_STAGES][WS_PROD / 32];
  __shared__ __align__(8) uint64_t bar_full[WS_STAGES], bar_empty[WS_STAGES];
  __shared__ int abort_s;
  volatile int* abort_flag = &abort_s;
  const WbTile t = wb_tile(p);
  const int i0 = t.i0, j0 = t.j0, nslab = t.nslab;
  const long long zb = t.zb, zh = t.zh;
  const int I = p.I, J = p.J, ldo = p.ldo;
  const int tid = threadIdx.x, lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < WS_STAGES; ++s) { mbar_init(&bar_full[s], WS_PROD / 32); mbar_init(&bar_empty[s], WB_CONS / 32); }
    abort_s = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (tid >= WB_CONS) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 40;");
    wb_produce<AMODE, BMODE, AF32>(p, t, As, Bs, tiny_s, bar_full, bar_empty, abort_flag, tid - WB_CONS);
    return;
  }
  // --------------------------------- consumers ---------------------------------
  asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
  const int ty = tid >> 3, tx = tid & 7;
  void* out = OUT_BF16 ? (void*)(reinterpret_cast<uint16_t*>(p.out) + zb * p.o_b + zh * p.o_h)
                       : (void*)(reinterpret_cast<float*>(p.out) + zb * p.o_b + zh * p.o_h);
  float2 acc[8][8];
#pragma unroll
  for (int a = 0; a < 8; ++a)
#pragma unroll
    for (int b = 0; b < 8; ++b) acc[a][b] = make_float2(0.0f, 0.0f);
  const float* accp = p.acc_in ? p.acc_in + zb * p.acc_b + zh * p.acc_h
                               : ((p.init && !OUT_BF16) ? reinterpret_cast<const float*>(out) : nullptr);
  if (accp) {
    const int ldacc = p.acc_in ? p.acc_ld : ldo;
#pragma unroll
    for (int a = 0; a < 8; ++a) {
      const int r = i0 + (a >> 2) * 64 + ty * 4 + (a & 3);
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        const int c = j0 + g * 32 + tx * 4;
        if (r < I && c < J) {
          const float4 t = *reinterpret_cast<const float4*>(accp + (size_t)r * ldacc + c);
          acc[a][2 * g] = make_float2(t.x, t.y);
          acc[a][2 * g + 1] = make_float2(t.z, t.w);
        }
      }
    }
  }
  for (int s = 0; s < nslab; ++s) {
    const int slot = s % WS_STAGES;
    if (!mbar_wait(&bar_full[slot], (uint32_t)((s / WS_STAGES) & 1), abort_flag, nullptr)) break;
    const int tiny = tiny_s[slot][0] | tiny_s[slot][1] | tiny_s[slot][2] | tiny_s[slot][3];
    if (tiny) slab_mac_8x16n<false>(As[slot], Bs[slot], ty, tx, acc);
    else slab_mac_8x16n<true>(As[slot], Bs[slot], ty, tx, acc);
    __syncwarp();
    if (lane == 0) mbar_arrive(&bar_empty[slot]);
  }
#pragma unroll
  for (int a = 0; a < 8; ++a) {
    const int r = i0 + (a >> 2) * 64 + ty * 4 + (a & 3);
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      const int c = j0 + g * 32 + tx * 4;
      if (r < I && c < J) {
        const float2 lo = acc[a][2 * g], hi = acc[a][2 * g + 1];
        if (OUT_BF16) {
          uint2 u;
          u.x = pack_bf2(lo.x, lo.y);
          u.y = pack_bf2(hi.x, hi.y);
          *reinterpret_cast<uint2*>(reinterpret_cast<uint16_t*>(out) + (size_t)r * ldo + c) = u;
        } else {
          *reinterpret_cast<float4*>(reinterpret_cast<float*>(out) + (size_t)r * ldo + c) = make_float4(lo.x, lo.y, hi.x, hi.y);
        }
      }
    }
  }
}

template <int AMODE, int BMODE, bool AF32, bool OUT_BF16>
static int ogemm_wb_launch(const OgemmArgs& p, int batches, cudaStream_t st) {
  static DevOnce once = {};
  if (dev_ensure_smem(once, (const void*)k_ogemm_wb<AMODE, BMODE, AF32, OUT_BF16>, WB_SMEM) != DET_OK) return DET_ERR_CUDA;
  const bool causal = p.range_mode == 1 || p.range_mode == 2;
  const unsigned ni = (unsigned)((p.I + OT - 1) / OT);
  dim3 grid((p.J + OT - 1) / OT, causal ? (unsigned)batches : ni, causal ? ni : (unsigned)batches);
  k_ogemm_wb<AMODE, BMODE, AF32, OUT_BF16><<<DET_L(grid), WB_THREADS, WB_SMEM, st>>>(p);
  return DET_OK;
}

// ---------------------------------------------------------------------------------------------------------------
// Fixed-point variant with the 64-bit accumulators in registers: 128 x 128 tile, eight consumer warps with 8 x 8 register
// tiles (64 f32 partial sums + 64 signed 64-bit accumulators per thread), four producer warps, one CTA per SM.  After
// every block of 128 contraction indices the partial sums are converted (48 fractional bits) and added; nothing leaves
// the registers until the converted total is written.  Same arguments, ranges and batching as k_ogemm_wb.
// ---------------------------------------------------------------------------------------------------------------
template <int AMODE, int BMODE, bool AF32>
__global__ void __launch_bounds__(WS_THREADS, 1) k_ogemm_fix(OgemmArgs p) {
  extern __shared__ __align__(16) unsigned char osm[];
  float(*As)[OK][OT + 4] = reinterpret_cast<float(*)[OK][OT + 4]>(osm);
  float(*Bs)[OK][OT + 4] = As + WS_STAGES;
  __shared__ int tiny_s[WS_STAGES][WS_PROD / 32];
  __shared__ __align__(8) uint64_t bar_full[WS_STAGES], bar_empty[WS_STAGES];
  __shared__ int abort_s;
  volatile int* abort_flag = &abort_s;
  const WbTile t = wb_tile(p);
  const int i0 = t.i0, j0 = t.j0, nslab = t.nslab;
  const long long zb = t.zb, zh = t.zh;
  const int I = p.I, J = p.J, ldo = p.ldo;
  const int tid = threadIdx.x, lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < WS_STAGES; ++s) { mbar_init(&bar_full[s], WS_PROD / 32); mbar_init(&bar_empty[s], WS_CONS / 32); }
    abort_s = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (tid >= WS_CONS) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 40;");
    wb_produce<AMODE, BMODE, AF32>(p, t, As, Bs, tiny_s, bar_full, bar_empty, abort_flag, tid - WS_CONS);
    return;
  }
  asm volatile("setmaxnreg.inc.sync.aligned.u32 232;");
  const int ty = tid >> 4, tx = tid & 15;
  float2 acc[8][4];
  long long fx[8][8];
#pragma unroll
  for (int a = 0; a < 8; ++a) {
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = make_float2(0.0f, 0.0f);
#pragma unroll
    for (int b = 0; b < 8; ++b) fx[a][b] = 0;
  }
  for (int s = 0; s < nslab; ++s) {
    const int slot = s % WS_STAGES;
    if (!mbar_wait(&bar_full[slot], (uint32_t)((s / WS_STAGES) & 1), abort_flag, nullptr)) return;
    const int tiny = tiny_s[slot][0] | tiny_s[slot][1] | tiny_s[slot][2] | tiny_s[slot][3];
    if (tiny) slab_mac<false, OT>(As[slot], Bs[slot], ty, tx, acc);
    else slab_mac<true, OT>(As[slot], Bs[slot], ty, tx, acc);
    __syncwarp();
    if (lane == 0) mbar_arrive(&bar_empty[slot]);
    if ((s & 7) == 7 || s == nslab - 1) {
#pragma unroll
      for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          fx[a][2 * b] = (long long)((unsigned long long)fx[a][2 * b] + (unsigned long long)fix48(acc[a][b].x));
          fx[a][2 * b + 1] = (long long)((unsigned long long)fx[a][2 * b + 1] + (unsigned long long)fix48(acc[a][b].y));
          acc[a][b] = make_float2(0.0f, 0.0f);
        }
    }
  }
  uint16_t* out = reinterpret_cast<uint16_t*>(p.out) + zb * p.o_b + zh * p.o_h;
#pragma unroll
  for (int a = 0; a < 8; ++a) {
    const int r = i0 + (a >> 2) * 64 + ty * 4 + (a & 3);
#pragma unroll
    for (int g = 0; g < 2; ++g) {
      const int c = j0 + g * 64 + tx * 4;
      if (r < I && c < J) {
        uint2 u;
        u.x = pack_bf2(unfix48(fx[a][4 * g]), unfix48(fx[a][4 * g + 1]));
        u.y = pack_bf2(unfix48(fx[a][4 * g + 2]), unfix48(fx[a][4 * g + 3]));
        *reinterpret_cast<uint2*>(out + (size_t)r * ldo + c) = u;
      }
    }
  }
}

template <int AMODE, int BMODE, bool AF32>
static int ogemm_fix_launch(const OgemmArgs& p, int batches, cudaStream_t st) {
  static DevOnce once = {};
  if (dev_ensure_smem(once, (const void*)k_ogemm_fix<AMODE, BMODE, AF32>, WB_SMEM) != DET_OK) return DET_ERR_CUDA;
  const bool causal = p.range_mode == 1 || p.range_mode == 2;
  const unsigned ni = (unsigned)((p.I + OT - 1) / OT);
  dim3 grid((p.J + OT - 1) / OT, causal ? (unsigned)batches : ni, causal ? ni : (unsigned)batches);
  k_ogemm_fix<AMODE, BMODE, AF32><<<DET_L(grid), WS_THREADS, WB_SMEM, st>>>(p);
  return DET_OK;
}

}  // namespace det
