// LM head, arithmetic version 2 (optional mode): an order-free, exactly defined contraction on the int8 tensor cores.
//
// Version 1 defines every logit as an ordered chain of binary32 roundings, which only the FP32 ALUs can replay.  Version 2
// uses the paper's own two devices instead (Sec. 3.2: int8 products accumulated exactly in int32; a wide exact integer
// total "for bitwise reproducibility"): every row of H and of W is aligned to its largest exponent and cut into two signed
// 7-bit slices (T = 128 hi + lo, a 14-bit magnitude: values within 2^-6 of the row's largest are kept exactly, smaller
// ones truncated toward zero), the four slice products are exact int32 sums on tcgen05.mma.kind::i8 in whatever order the
// hardware takes them, and the epilogue forms I = 2^14 hh + 2^7 (hl + lh) + ll in 64 bits and rounds I 2^(Ea + Eb - 280)
// to binary32 ONCE.  Nothing about the result depends on tiling, order or hardware.
//
//   k_slice_rows   one warp per row: row exponent (integer maximum), then the two int8 slices
//   k_igemm_sl     persistent, one CTA per SM, 128 x 128 output tile; warp 0 streams the FOUR operand tiles of a 128-deep
//                  step (H hi, H lo, W hi, W lo: 64 KiB) through a three-stage TMA ring, warp 1 issues the sixteen MMAs of
//                  the step into three TMEM accumulators (hh | hl + lh | ll, 128 columns each), warps 2-5 combine and round.
// Every mbarrier wait is bounded (DET_DEV_TIMEOUT), as in igemm.cu.
#include "tc05.cuh"
#include "internal.h"
#include "v2_slice.cuh"

namespace det {

// ---- slicing (bf_bits, slice1: v2_slice.cuh) ------------------------------------------------------------------------------
// eight values of a row as four words of packed bf16 patterns: bf16 source as stored, f32 source rounded to bf16
template <bool F32>
__device__ __forceinline__ void load8_bits(const void* X, size_t idx, uint32_t (&w)[4]) {
  if (F32) {
    const float4 a = __ldg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(X) + idx));
    const float4 b = __ldg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(X) + idx) + 1);
    w[0] = bf_bits(a.x) | (bf_bits(a.y) << 16); w[1] = bf_bits(a.z) | (bf_bits(a.w) << 16);
    w[2] = bf_bits(b.x) | (bf_bits(b.y) << 16); w[3] = bf_bits(b.z) | (bf_bits(b.w) << 16);
  } else {
    const uint4 u = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const uint16_t*>(X) + idx));
    w[0] = u.x; w[1] = u.y; w[2] = u.z; w[3] = u.w;
  }
}
template <bool F32>
__global__ void __launch_bounds__(256) k_slice_rows(const void* __restrict__ X, int R, int K, int8_t* __restrict__ hi,
                                                    int8_t* __restrict__ lo, int32_t* __restrict__ E) {
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= R) return;
  int e = 0, bad = 0;
  for (int i = lane; i < K / 8; i += 32) {
    uint32_t w[4];
    load8_bits<F32>(X, (size_t)row * K + 8 * (size_t)i, w);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int e0 = (w[j] >> 7) & 0xFF, e1 = (w[j] >> 23) & 0xFF;
      bad |= (e0 == 255) | (e1 == 255);
      e = max(e, max(e0, e1));
    }
  }
#pragma unroll
  for (int s = 16; s; s >>= 1) {
    e = max(e, __shfl_xor_sync(0xffffffffu, e, s));
    bad |= __shfl_xor_sync(0xffffffffu, bad, s);
  }
  if (lane == 0) E[row] = e | (bad ? (1 << 30) : 0);
  for (int i = lane; i < K / 8; i += 32) {
    uint32_t w[4];
    load8_bits<F32>(X, (size_t)row * K + 8 * (size_t)i, w);
    uint32_t h8[2] = {0u, 0u}, l8[2] = {0u, 0u};
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const uint32_t b = (j & 1) ? (w[j >> 1] >> 16) : (w[j >> 1] & 0xFFFFu);
      int h, l;
      slice1(b, e, h, l);
      h8[j >> 2] |= (uint32_t)(uint8_t)(int8_t)h << (8 * (j & 3));
      l8[j >> 2] |= (uint32_t)(uint8_t)(int8_t)l << (8 * (j & 3));
    }
    *reinterpret_cast<uint2*>(hi + (size_t)row * K + 8 * i) = make_uint2(h8[0], h8[1]);
    *reinterpret_cast<uint2*>(lo + (size_t)row * K + 8 * i) = make_uint2(l8[0], l8[1]);
  }
}

// Slicing along the OTHER index, for the gradient contractions: the exponent of column c is taken over the rows r, and the
// slices are written transposed ([C, R], so that the contracted index r is contiguous for the tensor core).
//   k_col_exp     E[c] = max over r (integer maximum through atomicMax: order-free); E must be zero before
//   k_slice_cols  a CTA takes a 128 x 128 tile: thread = column (a warp reads 32 adjacent values of a row), 128 rows in
//                 registers as packed bytes, out through a swizzled shared-memory tile as whole 128-byte lines
template <bool F32>
__global__ void __launch_bounds__(128) k_col_exp(const void* __restrict__ X, int R, int C, int32_t* __restrict__ E) {
  const int c = blockIdx.x * 128 + threadIdx.x, r0 = blockIdx.y * 128;
  int key = 0;
#pragma unroll 8
  for (int i = 0; i < 128; ++i) {
    const size_t idx = (size_t)(r0 + i) * C + c;
    const uint32_t b = F32 ? bf_bits(__ldg(reinterpret_cast<const float*>(X) + idx)) : (uint32_t)__ldg(reinterpret_cast<const uint16_t*>(X) + idx);
    const int e = (b >> 7) & 0xFF;
    key = max(key, e | (e == 255 ? (1 << 30) : 0));
  }
  if (key > *reinterpret_cast<volatile int32_t*>(E + c)) atomicMax(E + c, key);
}
template <bool F32>
__global__ void __launch_bounds__(128) k_slice_cols(const void* __restrict__ X, int R, int C, const int32_t* __restrict__ E,
                                                    int8_t* __restrict__ hiT, int8_t* __restrict__ loT) {
  __shared__ __align__(16) uint8_t tile[2][128 * 128];
  const int t = threadIdx.x, c0 = blockIdx.x * 128, r0 = blockIdx.y * 128;
  const int e = E[c0 + t] & 0xFF;
  uint32_t hw[32], lw[32];
#pragma unroll
  for (int i = 0; i < 128; ++i) {
    const size_t idx = (size_t)(r0 + i) * C + c0 + t;
    const uint32_t b = F32 ? bf_bits(__ldg(reinterpret_cast<const float*>(X) + idx)) : (uint32_t)__ldg(reinterpret_cast<const uint16_t*>(X) + idx);
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
    *reinterpret_cast<uint4*>(hiT + (size_t)(c0 + r) * R + r0 + ch * 16) = *reinterpret_cast<const uint4*>(tile[0] + off);
    *reinterpret_cast<uint4*>(loT + (size_t)(c0 + r) * R + r0 + ch * 16) = *reinterpret_cast<const uint4*>(tile[1] + off);
  }
}

// ---- sliced contraction -------------------------------------------------------------------------------------------------
constexpr int SL_T = 128;                     // tile edge (rows of H x rows of W)
constexpr int SL_BK = 128;                    // bytes (= int8 elements) per step along K
constexpr int SL_STAGES = 3;
constexpr int SL_TILE = SL_T * SL_BK;         // one operand tile: 16 KiB
constexpr int SL_STAGE_BYTES = 4 * SL_TILE;   // H hi | H lo | W hi | W lo
constexpr int SL_EPI_WARPS = 16;              // warp & 3 = TMEM lane quarter, four warps per quarter take 32 columns each
constexpr int SL_THREADS = 64 + 32 * SL_EPI_WARPS;
constexpr size_t SL_SMEM = (size_t)SL_STAGES * SL_STAGE_BYTES + SL_EPI_WARPS * 2048 + 1024;   // ring + a staging tile per epilogue warp

// the one rounding of the definition: I 2^e as binary32, nearest even; results below 2^-126 after the rounding are zeros.
// The conversion of the integer rounds once (nearest even) and a scaling by 2^e is exact while the result stays a
// normal number, so the exponent is simply added; near the ends of the range the rounding is done in binary64 instead
// (exact product, one conversion), where the subnormal grid decides what reaches 2^-126.
__device__ __forceinline__ float round_scaled(long long I, int e) {
  if (I == 0) return 0.0f;
  const float f = __ll2float_rn(I);
  const int ef = (int)((__float_as_uint(f) >> 23) & 0xFFu) + e;
  if ((unsigned)(ef - 2) <= 252u) return __uint_as_float(__float_as_uint(f) + ((uint32_t)e << 23));
  const double v = (double)I * __longlong_as_double((long long)(e + 1023) << 52);   // exact: |I| < 2^53, e + 1023 in [745, 1253]
  float r = __double2float_rn(v);
  if (fabsf(r) < 0x1p-126f) r = copysignf(0.0f, r);
  return r;
}

// One launch covers Z independent problems of the same shape (the operands of problem z are rows z*I.. of A and z*J.. of
// B; the result goes to out + (z / hdiv) * o_b + (z % hdiv) * o_h + i * ldo + j).  causal_tiles: only the tiles with
// j0 <= i0 exist.  krange: 0 the whole contraction; 1 only the steps up to and including the row tile's own (a causal
// product whose contracted index is the key); 2 only the steps from the row tile's own on (contracted index = query).
// epi: SL_F32 | SL_BF16 | SL_BF16_ROWSCALE (the rounded result times rowscale[z*I + i] in binary32, then bf16).
__global__ void __launch_bounds__(SL_THREADS, 1)
    k_igemm_sl(const __grid_constant__ CUtensorMap tmAh, const __grid_constant__ CUtensorMap tmAl,
               const __grid_constant__ CUtensorMap tmBh, const __grid_constant__ CUtensorMap tmBl, const SlArgs p, int* status) {
  const int32_t* __restrict__ Ea = p.Ea;
  const int32_t* __restrict__ Eb = p.Eb;
  const int I = p.I, J = p.J, K = p.K;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  __shared__ __align__(8) uint64_t bar_full[SL_STAGES], bar_empty[SL_STAGES], bar_tfull, bar_tempty;
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;
  volatile int* abort_flag = &abort_s;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < SL_STAGES; ++s) { mbar_init(&bar_full[s], 1); mbar_init(&bar_empty[s], 1); }
    mbar_init(&bar_tfull, 1);
    mbar_init(&bar_tempty, SL_EPI_WARPS);
    abort_s = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  const int tiles_i = I / SL_T, tiles_j = J / SL_T, per_z = tiles_i * tiles_j, num_tiles = p.Z * per_z, kblocks = K / SL_BK;
  // tile t -> problem z, row tile it, column tile jt (the rows run fastest: the CTAs resident at one time share a tile of
  // B and stream A through L2); false when the tile does not exist; [k_lo, k_hi) = its steps along the contraction
  auto tile_of = [&](int t, int& z, int& i0, int& j0, int& k_lo, int& k_hi) {
    z = t / per_z;
    const int r = t - z * per_z, it = r % tiles_i, jt = r / tiles_i;
    i0 = it * SL_T; j0 = jt * SL_T;
    k_lo = (p.krange == 2) ? it : 0;
    k_hi = (p.krange == 1) ? min(kblocks, it + 1) : kblocks;
    return !(p.causal_tiles && jt > it);
  };

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        int z, i0, j0, k_lo, k_hi;
        if (!tile_of(tile, z, i0, j0, k_lo, k_hi)) continue;
        for (int kb = k_lo; kb < k_hi; ++kb) {
          if (!mbar_wait(&bar_empty[stage], phase ^ 1u, abort_flag, status)) { ok = false; break; }
          mbar_expect_tx(&bar_full[stage], SL_STAGE_BYTES);
          uint8_t* sa = smem + stage * SL_STAGE_BYTES;
          tma_load_2d(sa, &tmAh, kb * SL_BK, z * I + i0, &bar_full[stage]);
          tma_load_2d(sa + SL_TILE, &tmAl, kb * SL_BK, z * I + i0, &bar_full[stage]);
          tma_load_2d(sa + 2 * SL_TILE, &tmBh, kb * SL_BK, z * J + j0, &bar_full[stage]);
          tma_load_2d(sa + 3 * SL_TILE, &tmBl, kb * SL_BK, z * J + j0, &bar_full[stage]);
          if (++stage == SL_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // instruction descriptor: D = S32, A = B = signed 8-bit, both K-major, N = 128, M = 128
      constexpr uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(SL_T >> 3) << 17) | ((uint32_t)(SL_T >> 4) << 24);
      int stage = 0, it = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        int z, i0, j0, k_lo, k_hi;
        if (!tile_of(tile, z, i0, j0, k_lo, k_hi)) continue;
        if (!mbar_wait(&bar_tempty, ((uint32_t)it & 1u) ^ 1u, abort_flag, status)) { ok = false; break; }   // accumulators drained
        ++it;
        tc_fence_after();
        for (int kb = k_lo; kb < k_hi; ++kb) {
          if (!mbar_wait(&bar_full[stage], phase, abort_flag, status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + stage * SL_STAGE_BYTES);
          const uint64_t ah = make_smem_desc(sa), al = make_smem_desc(sa + SL_TILE);
          const uint64_t bh = make_smem_desc(sa + 2 * SL_TILE), bl = make_smem_desc(sa + 3 * SL_TILE);
#pragma unroll
          for (int k4 = 0; k4 < SL_BK / 32; ++k4) {
            const uint64_t o = (uint64_t)(k4 * 2);
            const uint32_t first = (kb != k_lo || k4) ? 1u : 0u;
            umma_i8(tmem_base, ah + o, bh + o, idesc, first);              // hh
            umma_i8(tmem_base + 128u, ah + o, bl + o, idesc, first);       // hl starts the cross accumulator ...
            umma_i8(tmem_base + 128u, al + o, bh + o, idesc, 1u);          // ... lh adds to it
            umma_i8(tmem_base + 256u, al + o, bl + o, idesc, first);       // ll
          }
          umma_commit(&bar_empty[stage]);
          if (++stage == SL_STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) umma_commit(&bar_tfull);
      }
    }
  } else {
    const int q = warp & 3, part = (warp - 2) >> 2;  // TMEM lane quarter this warp may read; its 32 of the 128 columns
    uint8_t* stage = smem + SL_STAGES * SL_STAGE_BYTES + (warp - 2) * 2048;
    int it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
      int z, i0, j0, k_lo, k_hi;
      if (!tile_of(tile, z, i0, j0, k_lo, k_hi)) continue;
      if (!mbar_wait(&bar_tfull, (uint32_t)it & 1u, abort_flag, status)) { ok = false; break; }
      ++it;
      tc_fence_after();
      const int row = i0 + q * 32 + lane;
      const int ea = Ea[(size_t)z * I + row];
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
      // the warp's first row: whole row segments leave through the staging tile (tc05.cuh: store_rows32)
      const size_t wbase = (size_t)(z / p.hdiv) * p.o_b + (size_t)(z % p.hdiv) * p.o_h + (size_t)(row - lane) * p.ldo + j0;
      const float rsc = (p.epi == SL_BF16_ROWSCALE) ? p.rowscale[(size_t)z * I + row] : 1.0f;
      // the exponents of the warp's 32 columns, one load per tile: lane l keeps column l's, a shuffle hands column c's to
      // every row
      const int ebv = Eb[(size_t)z * J + j0 + part * 32 + lane];
      const int any_bad = __any_sync(0xffffffffu, ((ea | ebv) >> 30) != 0);
      const int ea280 = (ea & 0xFF) - 280;
#pragma unroll 1
      for (int sub = 0; sub < 2; ++sub) {
        const int c0 = part * 32 + sub * 16;
        uint32_t hh[16], cr[16], ll[16];
        tmem_ld16_nowait(taddr + (uint32_t)c0, hh);
        tmem_ld16_nowait(taddr + 128u + (uint32_t)c0, cr);
        tmem_ld16_nowait(taddr + 256u + (uint32_t)c0, ll);
        tmem_wait_ld();
        float f[16];
#pragma unroll
        for (int c = 0; c < 16; ++c) {
          const long long Iv = ((long long)(int)hh[c] << 14) + ((long long)(int)cr[c] << 7) + (long long)(int)ll[c];
          f[c] = round_scaled(Iv, ea280 + (__shfl_sync(0xffffffffu, ebv, sub * 16 + c) & 0xFF));
        }
        if (any_bad) {   // a row or a column of the tile holds an infinity or a NaN: its results are NaN
#pragma unroll
          for (int c = 0; c < 16; ++c)
            if ((ea | __shfl_sync(0xffffffffu, ebv, sub * 16 + c)) >> 30) f[c] = __int_as_float(0x7FC00000);
        }
        if (p.epi == SL_BF16_ROWSCALE) {
#pragma unroll
          for (int c = 0; c < 16; ++c) f[c] = fmul(f[c], rsc);
        }
        if (p.epi != SL_F32) {
          uint4 o[2];
#pragma unroll
          for (int v = 0; v < 2; ++v)
            o[v] = make_uint4(pack_bf2(f[8 * v], f[8 * v + 1]), pack_bf2(f[8 * v + 2], f[8 * v + 3]),
                              pack_bf2(f[8 * v + 4], f[8 * v + 5]), pack_bf2(f[8 * v + 6], f[8 * v + 7]));
          store_rows32<2>(stage, reinterpret_cast<uint8_t*>(reinterpret_cast<uint16_t*>(p.out) + wbase + c0), (size_t)p.ldo * 2, o);
        } else {
          uint4 o[4];
#pragma unroll
          for (int v = 0; v < 4; ++v)
            o[v] = make_uint4(__float_as_uint(f[4 * v]), __float_as_uint(f[4 * v + 1]), __float_as_uint(f[4 * v + 2]),
                              __float_as_uint(f[4 * v + 3]));
          store_rows32<4>(stage, reinterpret_cast<uint8_t*>(reinterpret_cast<float*>(p.out) + wbase + c0), (size_t)p.ldo * 4, o);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bar_tempty);
    }
  }
  __syncthreads();
  if (abort_s) {
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000ll) { }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// host: Z sliced contractions in one launch (see k_igemm_sl); the slices of problem z are rows z*I.. / z*J.. of A / B
int sliced_gemm_launch(const int8_t* Ah, const int8_t* Al, const int8_t* Bh, const int8_t* Bl, const SlArgs& p, int* status,
                       cudaStream_t st) {
  if (p.I % SL_T || p.J % SL_T || p.K % SL_BK || p.Z <= 0 || p.hdiv <= 0) return DET_ERR_SHAPE;
  if (p.K >= (1 << 16)) return DET_ERR_RANGE;   // the cross accumulator holds two products: 2 K 127^2 must stay below 2^31
  CUtensorMap tAh, tAl, tBh, tBl;
  if (!make_map(&tAh, Ah, p.Z * p.I, p.K, SL_T) || !make_map(&tAl, Al, p.Z * p.I, p.K, SL_T) ||
      !make_map(&tBh, Bh, p.Z * p.J, p.K, SL_T) || !make_map(&tBl, Bl, p.Z * p.J, p.K, SL_T))
    return DET_ERR_CUDA;
  static DevOnce once = {};
  if (dev_ensure_smem(once, (const void*)k_igemm_sl, SL_SMEM) != DET_OK) return DET_ERR_CUDA;
  const int sms = dev_sm_count();
  if (sms <= 0) return DET_ERR_CUDA;
  const long long tiles = (long long)p.Z * (p.I / SL_T) * (p.J / SL_T);
  k_igemm_sl<<<DET_L((unsigned)(tiles < sms ? tiles : sms)), SL_THREADS, SL_SMEM, st>>>(tAh, tAl, tBh, tBl, p, status);
  if (cudaPeekAtLastError() != cudaSuccess) { cudaGetLastError(); return DET_ERR_CUDA; }
  return DET_OK;
}

}  // namespace det

using namespace det;

// one sliced contraction out[i,j] = round(I 2^(Ea[i] + Eb[j] - 280)) from the slices of both operands ([I,K] and [J,K] int8)
template <bool OUT_BF16>
static int sliced_gemm(const int8_t* Ah, const int8_t* Al, const int8_t* Bh, const int8_t* Bl, const int32_t* Ea, const int32_t* Eb,
                       void* out, int I, int J, int K, int* status, cudaStream_t st) {
  SlArgs p = {};
  p.Ea = Ea; p.Eb = Eb; p.out = out; p.rowscale = nullptr;
  p.I = I; p.J = J; p.K = K; p.Z = 1; p.hdiv = 1; p.o_b = 0; p.o_h = 0; p.ldo = J;
  p.causal_tiles = 0; p.krange = 0; p.epi = OUT_BF16 ? SL_BF16 : SL_F32;
  return sliced_gemm_launch(Ah, Al, Bh, Bl, p, status, st);
}

static size_t v2_layout(int M, int V, int K, size_t* oAh, size_t* oAl, size_t* oBh, size_t* oBl, size_t* oEa, size_t* oEb) {
  size_t off = 0;
  *oAh = off; off += align_up((size_t)M * K, 256);
  *oAl = off; off += align_up((size_t)M * K, 256);
  *oBh = off; off += align_up((size_t)V * K, 256);
  *oBl = off; off += align_up((size_t)V * K, 256);
  *oEa = off; off += align_up((size_t)M * 4, 256);
  *oEb = off; off += align_up((size_t)V * 4, 256);
  return off;
}
extern "C" size_t det_lmhead_fwd_v2_ws_bytes(int M, int V, int K) {
  size_t a, b, c, d, e, f;
  return v2_layout(M, V, K, &a, &b, &c, &d, &e, &f);
}
extern "C" int det_lmhead_fwd_v2(const det_bf16* H, const det_bf16* W, int M, int V, int K, float* logits, void* ws,
                                 size_t ws_bytes, void* stream, int* status_dev) {
  if (!H || !W || !logits || M <= 0 || V <= 0 || K <= 0) return DET_ERR_ARG;
  if (M % SL_T || V % SL_T || K % SL_BK) return DET_ERR_SHAPE;
  if (K >= (1 << 16)) return DET_ERR_RANGE;   // the cross accumulator holds two products: 2 K 127^2 must stay below 2^31
  if (!aligned16(H) || !aligned16(W) || !aligned16(logits) || !aligned16(ws)) return DET_ERR_ALIGN;
  size_t oAh, oAl, oBh, oBl, oEa, oEb;
  if (!ws || ws_bytes < v2_layout(M, V, K, &oAh, &oAl, &oBh, &oBl, &oEa, &oEb)) return DET_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  uint8_t* base = (uint8_t*)ws;
  int8_t *Ah = (int8_t*)(base + oAh), *Al = (int8_t*)(base + oAl), *Bh = (int8_t*)(base + oBh), *Bl = (int8_t*)(base + oBl);
  int32_t *Ea = (int32_t*)(base + oEa), *Eb = (int32_t*)(base + oEb);
  k_slice_rows<false><<<DET_L((M + 7) / 8), 256, 0, st>>>(H, M, K, Ah, Al, Ea);
  k_slice_rows<false><<<DET_L((V + 7) / 8), 256, 0, st>>>(W, V, K, Bh, Bl, Eb);
  DET_CHECK_LAUNCH();
  return sliced_gemm<false>(Ah, Al, Bh, Bl, Ea, Eb, logits, M, V, K, status_dev, st);
}

// ---- gradients (version 2): the same contraction on transposed operands -------------------------------------------------
static size_t v2b_layout(int M, int V, int K, size_t (&o)[12]) {
  size_t off = 0;
  const size_t sz[12] = {(size_t)M * V, (size_t)M * V,      // g = bf16(dlogits), rows (exponent per token): hi, lo [M,V]
                         (size_t)M * V, (size_t)M * V,      // g columns, transposed (exponent per vocabulary entry): hi, lo [V,M]
                         (size_t)V * K, (size_t)V * K,      // W columns, transposed: hi, lo [K,V]
                         (size_t)M * K, (size_t)M * K,      // H columns, transposed: hi, lo [K,M]
                         (size_t)M * 4, (size_t)V * 4, (size_t)K * 4, (size_t)K * 4};   // exponents: g rows, g columns, W columns, H columns
  for (int i = 0; i < 12; ++i) { o[i] = off; off += align_up(sz[i], 256); }
  return off;
}
extern "C" size_t det_lmhead_bwd_v2_ws_bytes(int M, int V, int K) {
  size_t o[12];
  return v2b_layout(M, V, K, o);
}
extern "C" int det_lmhead_bwd_v2(const float* dlogits, const det_bf16* H, const det_bf16* W, int M, int V, int K, det_bf16* dH,
                                 float* dW, void* ws, size_t ws_bytes, void* stream, int* status_dev) {
  if (!dlogits || !H || !W || !dH || !dW || M <= 0 || V <= 0 || K <= 0) return DET_ERR_ARG;
  if (M % SL_T || V % SL_T || K % SL_BK) return DET_ERR_SHAPE;
  if (M >= (1 << 16) || V >= (1 << 16)) return DET_ERR_RANGE;   // contraction lengths of the two gradients
  if (!aligned16(dlogits) || !aligned16(H) || !aligned16(W) || !aligned16(dH) || !aligned16(dW) || !aligned16(ws)) return DET_ERR_ALIGN;
  size_t o[12];
  if (!ws || ws_bytes < v2b_layout(M, V, K, o)) return DET_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  uint8_t* b = (uint8_t*)ws;
  int8_t *gh = (int8_t*)(b + o[0]), *gl = (int8_t*)(b + o[1]), *gTh = (int8_t*)(b + o[2]), *gTl = (int8_t*)(b + o[3]);
  int8_t *WTh = (int8_t*)(b + o[4]), *WTl = (int8_t*)(b + o[5]), *HTh = (int8_t*)(b + o[6]), *HTl = (int8_t*)(b + o[7]);
  int32_t *Eg = (int32_t*)(b + o[8]), *EgT = (int32_t*)(b + o[9]), *EWT = (int32_t*)(b + o[10]), *EHT = (int32_t*)(b + o[11]);
  cudaMemsetAsync(EgT, 0, o[11] - o[9] + align_up((size_t)K * 4, 256), st);        // the three column-exponent arrays
  k_slice_rows<true><<<DET_L((M + 7) / 8), 256, 0, st>>>(dlogits, M, V, gh, gl, Eg);
  k_col_exp<true><<<DET_L(dim3(V / 128, M / 128)), 128, 0, st>>>(dlogits, M, V, EgT);
  k_col_exp<false><<<DET_L(dim3(K / 128, V / 128)), 128, 0, st>>>(W, V, K, EWT);
  k_col_exp<false><<<DET_L(dim3(K / 128, M / 128)), 128, 0, st>>>(H, M, K, EHT);
  k_slice_cols<true><<<DET_L(dim3(V / 128, M / 128)), 128, 0, st>>>(dlogits, M, V, EgT, gTh, gTl);
  k_slice_cols<false><<<DET_L(dim3(K / 128, V / 128)), 128, 0, st>>>(W, V, K, EWT, WTh, WTl);
  k_slice_cols<false><<<DET_L(dim3(K / 128, M / 128)), 128, 0, st>>>(H, M, K, EHT, HTh, HTl);
  DET_CHECK_LAUNCH();
  // dH[m,k] = bf16(contraction over the vocabulary of row m of g with column k of W)
  int rc = sliced_gemm<true>(gh, gl, WTh, WTl, Eg, EWT, dH, M, K, V, status_dev, st);
  if (rc != DET_OK) return rc;
  // dW[v,k] = contraction over the tokens of column v of g with column k of H
  return sliced_gemm<false>(gTh, gTl, HTh, HTl, EgT, EHT, dW, V, K, M, status_dev, st);
}
