// int8 x int8 -> int32 contraction on the 5th-generation tensor cores (tcgen05), used by the three GEMMs
// of every LSQ linear layer (Sec. 3.2 "int8 computation": forward, grad-x and grad-W all run in int8 and
// accumulate in int32, which is exact and therefore order-free).
//
//   C[i,j] = sum_k A[i,k] * B[j,k]        A: int8 [I,K] row-major, B: int8 [J,K] row-major (both K-major)
//
// One persistent CTA per SM, 192 threads:
//   warp 0    TMA producer: 128-byte-swizzled tiles of A (128 x 128 B) and B (BN x 128 B) into a 4-stage ring
//   warp 1    allocates TMEM (512 columns = two BN=256 accumulators) and issues tcgen05.mma.kind::i8
//             (M=128, N=BN, K=32 per instruction, 4 per stage); tcgen05.commit releases ring slots
//   warps 2-5 epilogue: tcgen05.ld of the int32 accumulator (lane = row), dequantise / mask in registers,
//             stores; overlaps with the next tile's MMAs through the second accumulator
// Every mbarrier wait is bounded: on expiry the kernel raises DET_DEV_TIMEOUT in *status, stops issuing
// work, lets in-flight copies land, frees its TMEM and returns.
#include "tc05.cuh"
#include "internal.h"
#include "../../include/det_test.h"

namespace det {

constexpr int BM = 128;
constexpr int BK = 128;  // bytes (= int8 elements) per stage along K
constexpr int STAGES = 4;
constexpr int GEMM_THREADS = 192;
// Tile order: the dimension with fewer tiles runs fastest, so that the CTAs resident at one time share the smaller
// operand's tiles and the larger operand streams through L2 once.
__device__ __forceinline__ void tile_origin(int tile, int tiles_i, int tiles_j, int bn, int& i0, int& j0) {
  if (tiles_j <= tiles_i) { j0 = (tile % tiles_j) * bn; i0 = (tile / tiles_j) * BM; }
  else { i0 = (tile % tiles_i) * BM; j0 = (tile / tiles_i) * bn; }
}

// data-dependent scalars of the epilogue, read once per CTA from device memory
template <int EPI>
__device__ __forceinline__ void epi_scalars(const EpiParams& ep, float& cscale, float& inv_s, float& sx) {
  cscale = 1.0f; inv_s = 1.0f; sx = 1.0f;
    if (EPI == EPI_FWD) sx = ep.s_x[0];
    if (EPI == EPI_DX) {
      const float am = __uint_as_float(ep.amax1[0]);
      const float s_a = (am > 0.0f) ? fdiv(am, 127.0f) : 0.0f;
      cscale = fmul(fmul(s_a, ep.s_u[0]), ep.rot);
      inv_s = fdiv(1.0f, ep.s_x[0]);
    }
    if (EPI == EPI_DW) {
      const float am = __uint_as_float(ep.amax1[0]);
      const float s_g = (am > 0.0f) ? fdiv(am, 127.0f) : 0.0f;
      float s_z = 1.0f;
      if (ep.amax2) {
        const int az = (int)ep.amax2[0];
        s_z = (az > 0) ? fdiv(__int2float_rn(az), 127.0f) : 0.0f;
      }
      cscale = fmul(fmul(fmul(s_g, s_z), ep.s_x[0]), ep.rot);
    }
}

// The reverse for the bf16 reference operand of the gradient epilogues: `pre` holds sixteen-byte pieces fetched with whole
// 64-byte row segments per quad of lanes (fetch_rows32); rows32_to_lanes hands every lane the four words of its own row.
__device__ __forceinline__ void fetch_rows32(const uint8_t* gbase, size_t row_pitch_bytes, uint4 (&pre)[4]) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int i = 0; i < 4; ++i)
    pre[i] = __ldg(reinterpret_cast<const uint4*>(gbase + (size_t)(i * 8 + (lane >> 2)) * row_pitch_bytes + (lane & 3) * 16));
}
__device__ __forceinline__ void rows32_to_lanes(uint8_t* stage, const uint4 (&pre)[4], uint4 (&w)[4]) {
  const int lane = threadIdx.x & 31;
  __syncwarp();
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = i * 8 + (lane >> 2), piece = lane & 3;
    *reinterpret_cast<uint4*>(stage + r * 64 + ((piece ^ ((r >> 1) & 3)) << 4)) = pre[i];
  }
  __syncwarp();
#pragma unroll
  for (int v = 0; v < 4; ++v) w[v] = *reinterpret_cast<const uint4*>(stage + lane * 64 + ((v ^ ((lane >> 1) & 3)) << 4));
}

// Epilogue of one accumulator row: this lane owns TMEM lane `taddr`'s row (output row `row`), columns j0 .. j0+BN.
// With a staging tile (`stage`, 4 KiB per warp) the outputs are written through store_rows32.
template <int BN, int EPI>
__device__ __forceinline__ void epi_row(const EpiParams& ep, uint32_t taddr, int row, int J, int j0, float cscale,
                                        float inv_s, float sx, uint8_t* stage = nullptr) {
      const size_t rbase = (size_t)row * J + j0;
      const size_t wbase = (size_t)(row - (int)(threadIdx.x & 31)) * J + j0;  // the warp's first row
      if (EPI == EPI_DW) inv_s = fdiv(1.0f, ep.s_w[row]);
#pragma unroll 1
      for (int h = 0; h < BN / 128; ++h) {
      float grp[4];
      uint4 pre[4];
      const bool staged_ref = (EPI == EPI_DX || EPI == EPI_DW) && stage != nullptr;
      if (staged_ref) fetch_rows32(reinterpret_cast<const uint8_t*>(ep.ref + wbase + h * 128), (size_t)J * 2, pre);
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) {
        const int c0 = h * 128 + cc * 32;
        uint32_t r[32];
        tmem_ld32(taddr + (uint32_t)c0, r);
        uint4 refw[4];
        if (EPI == EPI_DX || EPI == EPI_DW) {
          if (staged_ref) {
            rows32_to_lanes(stage, pre, refw);
            if (cc < 3) fetch_rows32(reinterpret_cast<const uint8_t*>(ep.ref + wbase + c0 + 32), (size_t)J * 2, pre);
          } else {
            const uint4* rr = reinterpret_cast<const uint4*>(ep.ref + rbase + c0);
#pragma unroll
            for (int v = 0; v < 4; ++v) refw[v] = __ldg(rr + v);
          }
        }
        if (EPI == EPI_RAW) {
          uint4 o[8];
#pragma unroll
          for (int v = 0; v < 8; ++v) o[v] = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
          if (stage) store_rows32<8>(stage, reinterpret_cast<uint8_t*>(reinterpret_cast<int32_t*>(ep.out) + wbase + c0), (size_t)J * 4, o);
          else {
            uint4* og = reinterpret_cast<uint4*>(reinterpret_cast<int32_t*>(ep.out) + rbase + c0);
#pragma unroll
            for (int v = 0; v < 8; ++v) og[v] = o[v];
          }
        } else if (EPI == EPI_FWD) {
          const float4* sw = reinterpret_cast<const float4*>(ep.s_w + j0 + c0);
          uint4 o[4];
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            float4 w0 = __ldg(sw + 2 * v), w1 = __ldg(sw + 2 * v + 1);
            float f[8];
            f[0] = fmul(__int2float_rn((int)r[8 * v + 0]), fmul(sx, w0.x));
            f[1] = fmul(__int2float_rn((int)r[8 * v + 1]), fmul(sx, w0.y));
            f[2] = fmul(__int2float_rn((int)r[8 * v + 2]), fmul(sx, w0.z));
            f[3] = fmul(__int2float_rn((int)r[8 * v + 3]), fmul(sx, w0.w));
            f[4] = fmul(__int2float_rn((int)r[8 * v + 4]), fmul(sx, w1.x));
            f[5] = fmul(__int2float_rn((int)r[8 * v + 5]), fmul(sx, w1.y));
            f[6] = fmul(__int2float_rn((int)r[8 * v + 6]), fmul(sx, w1.z));
            f[7] = fmul(__int2float_rn((int)r[8 * v + 7]), fmul(sx, w1.w));
            o[v] = make_uint4(pack_bf2(f[0], f[1]), pack_bf2(f[2], f[3]), pack_bf2(f[4], f[5]), pack_bf2(f[6], f[7]));
          }
          if (stage) store_rows32<4>(stage, reinterpret_cast<uint8_t*>(reinterpret_cast<uint16_t*>(ep.out) + wbase + c0), (size_t)J * 2, o);
          else {
            uint4* og = reinterpret_cast<uint4*>(reinterpret_cast<uint16_t*>(ep.out) + rbase + c0);
#pragma unroll
            for (int v = 0; v < 4; ++v) og[v] = o[v];
          }
        } else if (EPI == EPI_DX) {
          uint4 o[4];
          float term[32];
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            uint4 xu = refw[v];
            const uint32_t xs[4] = {xu.x, xu.y, xu.z, xu.w};
            float g[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const float xv = (e & 1) ? bfhi(xs[e >> 1]) : bflo(xs[e >> 1]);
              const float gx = fmul(__int2float_rn((int)r[8 * v + e]), cscale);
              const float t = fmul(xv, inv_s);
              const bool in_range = (t >= -128.0f) && (t <= 127.0f);
              const float phi = t < -128.0f ? -128.0f : (t > 127.0f ? 127.0f : fsub(rintf(t), t));
              g[e] = in_range ? gx : 0.0f;
              term[8 * v + e] = fmul(gx, phi);
            }
            o[v] = make_uint4(pack_bf2(g[0], g[1]), pack_bf2(g[2], g[3]), pack_bf2(g[4], g[5]), pack_bf2(g[6], g[7]));
          }
          if (stage) store_rows32<4>(stage, reinterpret_cast<uint8_t*>(reinterpret_cast<uint16_t*>(ep.out) + wbase + c0), (size_t)J * 2, o);
          else {
            uint4* og = reinterpret_cast<uint4*>(reinterpret_cast<uint16_t*>(ep.out) + rbase + c0);
#pragma unroll
            for (int v = 0; v < 4; ++v) og[v] = o[v];
          }
          // adjacent tree over this lane's 32 columns
#pragma unroll
          for (int w = 1; w < 32; w <<= 1)
#pragma unroll
            for (int e = 0; e < 32; e += 2 * w) term[e] = fadd(term[e], term[e + w]);
          grp[cc] = term[0];
        } else {  // EPI_DW
          uint4 o[8];
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            uint4 wu = refw[v];
            const uint32_t wsr[4] = {wu.x, wu.y, wu.z, wu.w};
            float g[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const float wv = (e & 1) ? bfhi(wsr[e >> 1]) : bflo(wsr[e >> 1]);
              const float t = fmul(wv, inv_s);
              const bool in_range = (t >= -128.0f) && (t <= 127.0f);
              g[e] = in_range ? fmul(__int2float_rn((int)r[8 * v + e]), cscale) : 0.0f;
            }
            o[2 * v] = make_uint4(__float_as_uint(g[0]), __float_as_uint(g[1]), __float_as_uint(g[2]), __float_as_uint(g[3]));
            o[2 * v + 1] = make_uint4(__float_as_uint(g[4]), __float_as_uint(g[5]), __float_as_uint(g[6]), __float_as_uint(g[7]));
          }
          if (stage) store_rows32<8>(stage, reinterpret_cast<uint8_t*>(reinterpret_cast<float*>(ep.out) + wbase + c0), (size_t)J * 4, o);
          else {
            uint4* og = reinterpret_cast<uint4*>(reinterpret_cast<float*>(ep.out) + rbase + c0);
#pragma unroll
            for (int v = 0; v < 8; ++v) og[v] = o[v];
          }
        }
      }
      if (EPI == EPI_DX)
        ep.ds_partial[(size_t)row * (J / 128) + (j0 / 128) + h] = fadd(fadd(grp[0], grp[1]), fadd(grp[2], grp[3]));
      }
}

template <int BN, int EPI>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
    k_igemm(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, EpiParams ep, int I, int J,
            int K, int* status) {
  constexpr int STAGE_A = BM * BK, STAGE_B = BN * BK, STAGE_BYTES = STAGE_A + STAGE_B;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  __shared__ __align__(8) uint64_t bar_full[STAGES], bar_empty[STAGES], bar_tfull[2], bar_tempty[2];
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;
  volatile int* abort_flag = &abort_s;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&bar_full[s], 1); mbar_init(&bar_empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&bar_tfull[a], 1); mbar_init(&bar_tempty[a], 4); }
    abort_s = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmA)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmB)) : "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;

  const int tiles_i = I / BM, tiles_j = J / BN;
  const int num_tiles = tiles_i * tiles_j;
  const int kblocks = K / BK;

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        int i0, j0;
        tile_origin(tile, tiles_i, tiles_j, BN, i0, j0);
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(&bar_empty[stage], phase ^ 1u, abort_flag, status)) { ok = false; break; }
          mbar_expect_tx(&bar_full[stage], STAGE_BYTES);
          uint8_t* sa = smem + stage * STAGE_BYTES;
          tma_load_2d(sa, &tmA, kb * BK, i0, &bar_full[stage]);
          tma_load_2d(sa + STAGE_A, &tmB, kb * BK, j0, &bar_full[stage]);
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // instruction descriptor: D = S32, A = B = signed 8-bit, both K-major, N = BN, M = 128
      constexpr uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
        const int acc = it & 1;
        const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
        if (!mbar_wait(&bar_tempty[acc], acc_phase ^ 1u, abort_flag, status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)(acc * BN);
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(&bar_full[stage], phase, abort_flag, status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + stage * STAGE_BYTES);
          const uint64_t da = make_smem_desc(sa), db = make_smem_desc(sa + STAGE_A);
#pragma unroll
          for (int k4 = 0; k4 < BK / 32; ++k4)
            umma_i8(tmem_d, da + (uint64_t)(k4 * 2), db + (uint64_t)(k4 * 2), idesc, (kb | k4) ? 1u : 0u);
          umma_commit(&bar_empty[stage]);
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) umma_commit(&bar_tfull[acc]);
      }
    }
  } else {
    const int q = warp & 3;  // TMEM lane quarter this warp may read
    int it = 0;
    bool ok = true;
    float cscale, inv_s, sx;
    epi_scalars<EPI>(ep, cscale, inv_s, sx);
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
      const int acc = it & 1;
      const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
      int i0, j0;
        tile_origin(tile, tiles_i, tiles_j, BN, i0, j0);
      if (!mbar_wait(&bar_tfull[acc], acc_phase, abort_flag, status)) { ok = false; break; }
      tc_fence_after();
      epi_row<BN, EPI>(ep, tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN), i0 + q * 32 + lane, J, j0, cscale, inv_s, sx);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bar_tempty[acc]);
    }
  }

  // teardown: everyone meets here; after a timeout give in-flight copies time to land first
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

// ------------------------------------------------------------------------------------------------------------
// Two-CTA variant (tcgen05 cta_group::2).  A cluster of two CTAs on neighbouring SMs computes one 256 x 256 tile:
// CTA r owns rows r*128 .. r*128+127 of the tile (its own A rows and its own 128 x 256 accumulator in TMEM) and stages
// only half of the B tile (rows r*128 .. of the 256 B rows); the MMA, issued by the leader CTA for both, reads the two
// halves of B from the two CTAs' shared memory.  Per CTA and K step that is 32 KiB staged and 32 KiB read by the tensor
// core instead of 48 + 48 KiB, which matters because TMA writes and MMA operand reads share the shared-memory port.
//   * each CTA's producer thread loads its own A / B-half tiles; the loads complete on the LEADER's full barrier
//   * the leader's MMA thread waits on that barrier, issues the MMAs, and releases the ring slot in BOTH CTAs with a
//     multicast tcgen05.commit; the same for "accumulator ready"
//   * the epilogue warps of both CTAs drain their own TMEM and arrive on the leader's "accumulator free" barrier
// No load uses cluster multicast.  All waits are bounded as in the one-CTA kernel.
// ------------------------------------------------------------------------------------------------------------
constexpr int STAGES2 = 6;
constexpr int BN2 = 256;
// warps 0 / 1 load and multiply; eight epilogue warps: warp & 3 is the TMEM lane quarter a warp may read, the two
// warps of a quarter take one half (128 columns) of the accumulator each
constexpr int GEMM2_THREADS = 64 + 8 * 32;

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t mapa_u32(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// tile load of this CTA whose completion is counted on the leader CTA's barrier (peer bit of the address cleared)
__device__ __forceinline__ void tma_load_2d_pair(void* smem_dst, const CUtensorMap* tm, int x, int y, uint64_t* bar) {
  const uint32_t leader_bar = smem_u32(bar) & 0xFEFFFFFFu;
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(
          smem_u32(smem_dst)),
      "l"(reinterpret_cast<uint64_t>(tm)), "r"(leader_bar), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void umma_i8_pair(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(da), "l"(db), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrive on the barrier at this offset in both CTAs once all MMAs issued so far have completed
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(
                   smem_u32(bar)),
               "h"(mask)
               : "memory");
}

template <int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(GEMM2_THREADS, 1)
    k_igemm2(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, EpiParams ep, int I, int J,
             int K, int* status) {
  constexpr int STAGE_A = 128 * BK, STAGE_B = 128 * BK, STAGE_BYTES = STAGE_A + STAGE_B;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  __shared__ __align__(8) uint64_t bar_full[STAGES2], bar_empty[STAGES2], bar_tfull[2], bar_tempty[2];
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;
  volatile int* abort_flag = &abort_s;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES2; ++s) { mbar_init(&bar_full[s], 1); mbar_init(&bar_empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&bar_tfull[a], 1); mbar_init(&bar_tempty[a], 16); }
    abort_s = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmA)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmB)) : "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // the peer's barriers are initialised before anything can signal them
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;

  const int tiles_i = I / 256, tiles_j = J / BN2;
  const int num_tiles = tiles_i * tiles_j;
  const int kblocks = K / BK;
  const int cluster_id = blockIdx.x >> 1, nclusters = gridDim.x >> 1;

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = cluster_id; tile < num_tiles && ok; tile += nclusters) {
        int i0, j0;
        if (tiles_j <= tiles_i) { j0 = (tile % tiles_j) * BN2; i0 = (tile / tiles_j) * 256; }
        else { i0 = (tile % tiles_i) * 256; j0 = (tile / tiles_i) * BN2; }
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(&bar_empty[stage], phase ^ 1u, abort_flag, status)) { ok = false; break; }
          if (leader) mbar_expect_tx(&bar_full[stage], 2 * STAGE_BYTES);  // both CTAs' tiles complete on this barrier
          uint8_t* sa = smem + stage * STAGE_BYTES;
          tma_load_2d_pair(sa, &tmA, kb * BK, i0 + (int)rank * 128, &bar_full[stage]);
          tma_load_2d_pair(sa + STAGE_A, &tmB, kb * BK, j0 + (int)rank * 128, &bar_full[stage]);
          if (++stage == STAGES2) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && leader) {
      // instruction descriptor: D = S32, A = B = signed 8-bit, both K-major, N = 256, M = 256 (two CTAs x 128)
      constexpr uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN2 >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      for (int tile = cluster_id; tile < num_tiles && ok; tile += nclusters, ++it) {
        const int acc = it & 1;
        const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
        if (!mbar_wait(&bar_tempty[acc], acc_phase ^ 1u, abort_flag, status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)(acc * BN2);
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(&bar_full[stage], phase, abort_flag, status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + stage * STAGE_BYTES);
          const uint64_t da = make_smem_desc(sa), db = make_smem_desc(sa + STAGE_A);
#pragma unroll
          for (int k4 = 0; k4 < BK / 32; ++k4)
            umma_i8_pair(tmem_d, da + (uint64_t)(k4 * 2), db + (uint64_t)(k4 * 2), idesc, (kb | k4) ? 1u : 0u);
          umma_commit_pair(&bar_empty[stage]);
          if (++stage == STAGES2) { stage = 0; phase ^= 1u; }
        }
        if (ok) umma_commit_pair(&bar_tfull[acc]);
      }
    }
  } else {
    const int q = warp & 3, half = (warp - 2) >> 2;
    uint8_t* stage = smem + STAGES2 * STAGE_BYTES + (warp - 2) * 4096;  // this warp's 32 x 128-byte staging tile
    int it = 0;
    bool ok = true;
    float cscale, inv_s, sx;
    epi_scalars<EPI>(ep, cscale, inv_s, sx);
    const uint32_t tempty_leader0 = mapa_u32(smem_u32(&bar_tempty[0]), 0), tempty_leader1 = mapa_u32(smem_u32(&bar_tempty[1]), 0);
    for (int tile = cluster_id; tile < num_tiles && ok; tile += nclusters, ++it) {
      const int acc = it & 1;
      const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
      int i0, j0;
      if (tiles_j <= tiles_i) { j0 = (tile % tiles_j) * BN2; i0 = (tile / tiles_j) * 256; }
      else { i0 = (tile % tiles_i) * 256; j0 = (tile / tiles_i) * BN2; }
      if (!mbar_wait(&bar_tfull[acc], acc_phase, abort_flag, status)) { ok = false; break; }
      tc_fence_after();
      epi_row<BN2 / 2, EPI>(ep, tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN2 + half * (BN2 / 2)),
                            i0 + (int)rank * 128 + q * 32 + lane, J, j0 + half * (BN2 / 2), cscale, inv_s, sx, stage);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_remote(acc ? tempty_leader1 : tempty_leader0);
    }
  }

  // teardown: both CTAs meet before either leaves (the peer may still signal this CTA's barriers or read its tiles)
  __syncthreads();
  if (abort_s) {
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000ll) { }
  }
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// ---- host side -------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = (EncodeTiledFn)p;
  }
  return fn;
}
bool make_map(CUtensorMap* tm, const int8_t* base, int rows, int K, int box_rows) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return false;
  cuuint64_t gdim[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  cuuint64_t gstr[1] = {(cuuint64_t)K};
  cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return enc(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, (void*)base, gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN, int EPI>
static int launch_one(const CUtensorMap& ta, const CUtensorMap& tb, const EpiParams& ep, int I, int J, int K, int* status,
                      cudaStream_t st) {
  constexpr size_t smem = (size_t)STAGES * (BM * BK + BN * BK) + 1024;
  static DevOnce once = {};
  if (dev_ensure_smem(once, (const void*)k_igemm<BN, EPI>, smem) != DET_OK) return DET_ERR_CUDA;
  const int sms = dev_sm_count();
  if (sms <= 0) return DET_ERR_CUDA;
  const int tiles = (I / BM) * (J / BN);
  const int grid = tiles < sms ? tiles : sms;
  k_igemm<BN, EPI><<<DET_L(grid), GEMM_THREADS, smem, st>>>(ta, tb, ep, I, J, K, status);
  if (cudaPeekAtLastError() != cudaSuccess) { cudaGetLastError(); return DET_ERR_CUDA; }
  return DET_OK;
}

template <int EPI>
static int launch_pair(const CUtensorMap& ta, const CUtensorMap& tb, const EpiParams& ep, int I, int J, int K, int* status,
                       cudaStream_t st) {
  constexpr size_t smem = (size_t)STAGES2 * (2 * 128 * BK) + 8 * 4096 + 1024;
  static DevOnce once = {};
  if (dev_ensure_smem(once, (const void*)k_igemm2<EPI>, smem) != DET_OK) return DET_ERR_CUDA;
  const int sms = dev_sm_count();
  if (sms < 2) return DET_ERR_CUDA;
  const int tiles = (I / 256) * (J / BN2);
  int clusters = sms / 2;
  if (tiles < clusters) clusters = tiles;
  k_igemm2<EPI><<<DET_L(2 * clusters), GEMM2_THREADS, smem, st>>>(ta, tb, ep, I, J, K, status);
  if (cudaPeekAtLastError() != cudaSuccess) { cudaGetLastError(); return DET_ERR_CUDA; }
  return DET_OK;
}

// Two-CTA 256 x 256 tiles when both output dimensions are multiples of 256 (unless force_one_cta), else the one-CTA kernel.
int igemm_launch(int epi, const int8_t* A, const int8_t* B, int I, int J, int K, const EpiParams& ep, int* status,
                 cudaStream_t st, int force_one_cta) {
  if (!A || !B || I <= 0 || J <= 0 || K <= 0) return DET_ERR_ARG;
  if (I % BM || J % 128 || K % BK) return DET_ERR_SHAPE;
  if (K >= (1 << 17)) return DET_ERR_RANGE;
  if (!aligned16(A) || !aligned16(B)) return DET_ERR_ALIGN;
  const int bn = (J % 256 == 0) ? 256 : 128;
  CUtensorMap ta, tb;
  if (!force_one_cta && I % 256 == 0 && J % 256 == 0) {
    if (!make_map(&ta, A, I, K, 128) || !make_map(&tb, B, J, K, 128)) return DET_ERR_CUDA;
    switch (epi) {
      case EPI_RAW: return launch_pair<EPI_RAW>(ta, tb, ep, I, J, K, status, st);
      case EPI_FWD: return launch_pair<EPI_FWD>(ta, tb, ep, I, J, K, status, st);
      case EPI_DX: return launch_pair<EPI_DX>(ta, tb, ep, I, J, K, status, st);
      case EPI_DW: return launch_pair<EPI_DW>(ta, tb, ep, I, J, K, status, st);
    }
    return DET_ERR_ARG;
  }
  if (!make_map(&ta, A, I, K, BM) || !make_map(&tb, B, J, K, bn)) return DET_ERR_CUDA;
#define DET_GEMM_CASE(E)                                                     \
  case E:                                                                    \
    return bn == 256 ? launch_one<256, E>(ta, tb, ep, I, J, K, status, st)   \
                     : launch_one<128, E>(ta, tb, ep, I, J, K, status, st);
  switch (epi) {
    DET_GEMM_CASE(EPI_RAW)
    DET_GEMM_CASE(EPI_FWD)
    DET_GEMM_CASE(EPI_DX)
    DET_GEMM_CASE(EPI_DW)
  }
#undef DET_GEMM_CASE
  return DET_ERR_ARG;
}

}  // namespace det

using namespace det;

// Self-test of the bounded wait every tensor-core kernel relies on: one warp waits on an mbarrier that nothing ever
// completes; after `limit_cycles` the wait gives up, raises DET_DEV_TIMEOUT in *status_dev and the kernel returns.
__global__ void k_selftest_wait(int* status, long long limit) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_s;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_s = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  mbar_wait(&bar, 0, &abort_s, status, limit);
}

extern "C" int det_test_wait_timeout(int* status_dev, long long limit_cycles, void* stream) {
  if (!status_dev || limit_cycles <= 0 || limit_cycles > 4000000000ll) return DET_ERR_ARG;
  k_selftest_wait<<<DET_L(1), 32, 0, (cudaStream_t)stream>>>(status_dev, limit_cycles);
  DET_CHECK_LAUNCH();
  return DET_OK;
}

extern "C" int det_test_igemm_tn(const int8_t* A, const int8_t* B, int I, int J, int K, int32_t* C, int force_one_cta,
                                 void* stream, int* status_dev) {
  if (!C) return DET_ERR_ARG;
  if (!aligned16(C)) return DET_ERR_ALIGN;
  EpiParams ep = {};
  ep.out = C;
  return igemm_launch(EPI_RAW, A, B, I, J, K, ep, status_dev, (cudaStream_t)stream, force_one_cta);
}
