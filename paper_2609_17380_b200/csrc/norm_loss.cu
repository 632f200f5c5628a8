// RMSNorm forward/backward and cross-entropy (+ z-loss) forward/backward: HBM-bound kernels whose
// reductions are the fixed pairwise tree with 256-element leaves (a lane owns 8 adjacent elements,
// a warp owns a leaf).
#include "common.cuh"
#include "internal.h"

namespace det {

template <bool BF>
__device__ __forceinline__ void load8(const void* p, size_t idx, float v[8]) {
  if (BF) {
    uint4 u = *reinterpret_cast<const uint4*>(reinterpret_cast<const uint16_t*>(p) + idx);
    v[0] = bflo(u.x); v[1] = bfhi(u.x); v[2] = bflo(u.y); v[3] = bfhi(u.y);
    v[4] = bflo(u.z); v[5] = bfhi(u.z); v[6] = bflo(u.w); v[7] = bfhi(u.w);
  } else {
    const float4* q = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(p) + idx);
    float4 a = q[0], b = q[1];
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  }
}
template <bool BF>
__device__ __forceinline__ void store8(void* p, size_t idx, const float v[8]) {
  if (BF) {
    uint4 u;
    u.x = pack_bf2(v[0], v[1]); u.y = pack_bf2(v[2], v[3]); u.z = pack_bf2(v[4], v[5]); u.w = pack_bf2(v[6], v[7]);
    *reinterpret_cast<uint4*>(reinterpret_cast<uint16_t*>(p) + idx) = u;
  } else {
    float4* q = reinterpret_cast<float4*>(reinterpret_cast<float*>(p) + idx);
    q[0] = make_float4(v[0], v[1], v[2], v[3]);
    q[1] = make_float4(v[4], v[5], v[6], v[7]);
  }
}

// ------------------------------------------------------------------------------------------------
// RMSNorm.  Rows of at most 2048 elements (8 leaves) are held in registers between the sum of squares and
// the output (k_rmsnorm_fwd8); longer rows use the two-pass variant that reads the row again.
// ------------------------------------------------------------------------------------------------
// A warp per LEAF (256 columns, 8 adjacent columns per lane), a CTA of 8 warps per block of 8 rows in two passes of four
// rows: 16 values and 8 loads in flight per lane, four CTAs per SM; the leaf sums of a row meet in shared memory (one
// barrier per pass) and every thread forms the row's tree over its leaves itself.
template <bool BF>
__global__ void __launch_bounds__(256, 4) k_rmsnorm_fwd8(const void* __restrict__ x, const void* __restrict__ gamma, int rows,
                                                         int D, float eps, float invD, void* __restrict__ y,
                                                         float* __restrict__ rstd, const float* __restrict__ s_q = nullptr,
                                                         int8_t* __restrict__ qy = nullptr) {
  __shared__ float leaf_sum[2][4][8];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int e0 = warp * 256 + lane * 8;
  const bool have = e0 < D;
  const bool full = (D & 255) == 0;
  const long long r0 = (long long)blockIdx.x * 8;
  const float inv_q = (BF && qy) ? fdiv(1.0f, s_q[0]) : 0.0f;
#pragma unroll 1
  for (int pass = 0; pass < 2; ++pass) {
    float xr[4][8];
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      const long long row = r0 + 4 * pass + a;
      if (row < rows && have) load8<BF>(x, (size_t)row * D + e0, xr[a]);
      else {
#pragma unroll
        for (int t = 0; t < 8; ++t) xr[a][t] = 0.0f;
      }
    }
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      float sq[8];
#pragma unroll
      for (int t = 0; t < 8; ++t) sq[t] = fmul(xr[a][t], xr[a][t]);
      const float t8 = tree8_full(sq);
      const float leaf = full ? warp_tree_full(t8) : warp_tree(t8, (long long)warp * 256, 8, D);
      if (lane == 0) leaf_sum[pass][a][warp] = leaf;
    }
    __syncthreads();
    float g[8];
    if (gamma && have) load8<BF>(gamma, e0, g);
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      const long long row = r0 + 4 * pass + a;
      float L[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) L[j] = leaf_sum[pass][a][j];
      const float ss = reg_tree<8>(L, 0, 256, D);          // a leaf beyond D does not exist
      const float rs = fdiv(1.0f, fsqrt(fadd(fmul(ss, invD), eps)));
      if (row >= rows) continue;
      if (threadIdx.x == a) rstd[row] = rs;
      if (!have) continue;
      float o[8];
      if (gamma) {
#pragma unroll
        for (int t = 0; t < 8; ++t) o[t] = fmul(fmul(xr[a][t], rs), g[t]);
      } else {
#pragma unroll
        for (int t = 0; t < 8; ++t) o[t] = fmul(xr[a][t], rs);
      }
      store8<BF>(y, (size_t)row * D + e0, o);
      if (BF && qy) {   // the next linear's quantiser, applied to the bf16 values just stored
#pragma unroll
        for (int t = 0; t < 8; ++t) o[t] = bf2f(f2bf(o[t]));
        *reinterpret_cast<uint2*>(qy + (size_t)row * D + e0) = quant8(o, inv_q);
      }
    }
  }
}

// Backward for rows of at most 2048 elements.  A CTA of 8 warps takes a block of 8 adjacent rows in four passes of two
// rows; warp j holds columns 256 j .. 256 j + 255 (one leaf of the fixed tree) of both rows, 8 adjacent columns per lane;
// three CTAs per SM, so that one loads or stores while another stands at its barrier (one CTA of 8 rows x 4 warps per SM
// ran 20 % slower).  A lane sees the same 8 columns of all 8 rows of the block, one pair of rows after the other, so with
// DG the column tree over the 8 rows of dy*xhat (the first three levels of the gain gradient's row-direction tree,
// written to partial8[block][D]) runs in its registers: no shared-memory copy of the products and no barrier of its own
// (0.080 ms with the products staged through shared memory by warps that each owned a quarter row, 0.070 ms now;
// 0.065-0.070 ms without the gain gradient, i.e. 0.9 of the copy bandwidth).  The row sums go through shared memory: one
// value per leaf and row, one barrier per pass.
// RPP rows per pass: 2 for f32 rows, 4 for bf16 rows (16 values and 64 bytes of loads in flight per lane and tensor either way).
template <bool BF, bool DG>
__global__ void __launch_bounds__(256, 3) k_rmsnorm_bwd8(const void* __restrict__ dy, const void* __restrict__ x,
                                                        const void* __restrict__ gamma, const float* __restrict__ rstd,
                                                        int rows, int D, float invD, void* __restrict__ dx,
                                                        float* __restrict__ partial8, int* __restrict__ tickets) {
  constexpr int RPP = BF ? 4 : 2, NPASS = 8 / RPP;
  __shared__ float leaf_sum[2][RPP][8];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int e0 = warp * 256 + lane * 8;
  const bool have = e0 < D;                       // this lane's 8 columns exist (D is a multiple of 8)
  const bool full = (D & 255) == 0;
  const long long r0 = (long long)blockIdx.x * 8;
  if (DG && blockIdx.x == 0 && (int)threadIdx.x < ((D + 255) >> 8)) tickets[threadIdx.x] = 0;   // for the kernel that follows
  if (DG) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // its blocks may start coming in; they wait for this grid
  float pair0[8], node[8];                        // column tree: a pair of rows waiting for the next pair; rows 0 .. 3
#pragma unroll
  for (int t = 0; t < 8; ++t) { pair0[t] = 0.0f; node[t] = 0.0f; }
#pragma unroll 1
  for (int pass = 0; pass < NPASS; ++pass) {
    const long long first = r0 + RPP * pass;
    float w[RPP][8], xh[RPP][8], rs[RPP];
#pragma unroll
    for (int a = 0; a < RPP; ++a) {
      const long long row = first + a;
      if (row < rows && have) {
        load8<BF>(dy, (size_t)row * D + e0, w[a]);
        load8<BF>(x, (size_t)row * D + e0, xh[a]);
      } else {
#pragma unroll
        for (int t = 0; t < 8; ++t) { w[a][t] = 0.0f; xh[a][t] = 0.0f; }
      }
      rs[a] = row < rows ? rstd[row] : 0.0f;
    }
#pragma unroll
    for (int a = 0; a < RPP; ++a)
#pragma unroll
      for (int t = 0; t < 8; ++t) xh[a][t] = fmul(xh[a][t], rs[a]);
    if (DG) {   // rows in pairs; pairs 0, 1 and 2, 3 -> nodes of four rows; those two -> the node of eight (a right node exists
                // iff its first row does, else the left one is carried up unchanged)
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        const float d0 = fmul(w[0][t], xh[0][t]), d1 = fmul(w[1][t], xh[1][t]);
        const float pa = (first + 1 < rows) ? fadd(d0, d1) : d0;
        if (RPP == 4) {
          const float d2 = fmul(w[RPP - 2][t], xh[RPP - 2][t]), d3 = fmul(w[RPP - 1][t], xh[RPP - 1][t]);
          const float pb = (first + 3 < rows) ? fadd(d2, d3) : d2;
          const float four = (first + 2 < rows) ? fadd(pa, pb) : pa;
          node[t] = (pass == 0) ? four : ((r0 + 4 < rows) ? fadd(node[t], four) : node[t]);
        } else if ((pass & 1) == 0) {
          pair0[t] = pa;
        } else {
          const float four = (first < rows) ? fadd(pair0[t], pa) : pair0[t];
          node[t] = (pass == 1) ? four : ((r0 + 4 < rows) ? fadd(node[t], four) : node[t]);
        }
      }
    }
    if (gamma && have) {
      float g[8];
      load8<BF>(gamma, e0, g);
#pragma unroll
      for (int a = 0; a < RPP; ++a)
#pragma unroll
        for (int t = 0; t < 8; ++t) w[a][t] = fmul(w[a][t], g[t]);
    }
#pragma unroll
    for (int a = 0; a < RPP; ++a) {
      float pr[8];
#pragma unroll
      for (int t = 0; t < 8; ++t) pr[t] = fmul(w[a][t], xh[a][t]);
      const float t8 = tree8_full(pr);
      const float leaf = full ? warp_tree_full(t8) : warp_tree(t8, (long long)warp * 256, 8, D);
      if (lane == 0) leaf_sum[pass & 1][a][warp] = leaf;
    }
    __syncthreads();
#pragma unroll
    for (int a = 0; a < RPP; ++a) {
      const long long row = first + a;
      float L[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) L[j] = leaf_sum[pass & 1][a][j];
      const float c = fmul(reg_tree<8>(L, 0, 256, D), invD);   // the row's tree over its leaves (a leaf beyond D does not exist)
      if (row < rows && have) {
        float o[8];
#pragma unroll
        for (int t = 0; t < 8; ++t) o[t] = fmul(rs[a], fsub(w[a][t], fmul(xh[a][t], c)));
        store8<BF>(dx, (size_t)row * D + e0, o);
      }
    }
  }
  if (DG && have) {
    float* dst = partial8 + (size_t)blockIdx.x * D + e0;
    *reinterpret_cast<float4*>(dst) = make_float4(node[0], node[1], node[2], node[3]);
    *reinterpret_cast<float4*>(dst + 4) = make_float4(node[4], node[5], node[6], node[7]);
  }
}
// partial8 [nb8][D] (node = 8 rows) -> partial256 [nb256][D]: tree over 32 adjacent 8-row nodes per column; the CTA
// that completes a block of 256 columns (a ticket counter per column block, zeroed by the kernel before, says which
// one it is) goes on to the levels above for those columns, 32 nodes at a time, and writes dgamma.  The counter
// decides only WHO evaluates those levels; operands and order are the fixed tree's.
__global__ void __launch_bounds__(256) k_colsum32(const float* __restrict__ partial8, int nb8, int rows, int D,
                                                  float* __restrict__ partial256, int nb256, int* __restrict__ tickets,
                                                  float* __restrict__ dgamma) {
  __shared__ int last_s;
  const int col = blockIdx.x * 256 + threadIdx.x;
  const int g = blockIdx.y;
  // launched as a programmatic dependent of the kernel that writes partial8: its blocks may be resident before that
  // kernel has drained; nothing of its results is read before this wait returns
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (col < D) {
    float s[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      const int b = g * 32 + i;
      s[i] = (b < nb8) ? partial8[(size_t)b * D + col] : 0.0f;
    }
    partial256[(size_t)g * D + col] = reg_tree<32>(s, (long long)g * 256, 8, rows);
  }
  __syncthreads();
  if (threadIdx.x == 0) {   // the barrier orders the CTA's stores before this thread's fence, which is cumulative
    __threadfence();
    last_s = (atomicAdd(&tickets[blockIdx.x], 1) == nb256 - 1);
    __threadfence();
  }
  __syncthreads();
  if (!last_s || col >= D) return;
  int n = nb256;
  long long stride = 256;
  while (n > 1) {
    const int groups = (n + 31) / 32;
    for (int gg = 0; gg < groups; ++gg) {
      float s[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) s[i] = (gg * 32 + i < n) ? __ldcg(&partial256[(size_t)(gg * 32 + i) * D + col]) : 0.0f;
      partial256[(size_t)gg * D + col] = reg_tree<32>(s, (long long)gg * 32 * stride, stride, rows);
    }
    n = groups;
    stride *= 32;
  }
  dgamma[col] = __ldcg(&partial256[col]);
}

// generic two-pass variants (rows longer than 2048 elements)
template <bool BF, int NL>  // NL = leaves held in registers (0: re-read)
__global__ void __launch_bounds__(256) k_rmsnorm_fwd(const void* __restrict__ x, const void* __restrict__ gamma, int rows,
                                                     int D, float eps, float invD, void* __restrict__ y,
                                                     float* __restrict__ rstd) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = blockIdx.x * 8 + warp;
  if (row >= rows) return;
  const size_t rb = (size_t)row * D;
  const int nl = (D + 255) >> 8;
  float keep[NL > 0 ? NL : 1][8];
  float mine = 0.0f;
#pragma unroll
  for (int j = 0; j < (NL > 0 ? NL : 32); ++j) {
    if (j >= nl) break;
    const int e0 = j * 256 + lane * 8;
    float v[8], sq[8];
    if (e0 < D) load8<BF>(x, rb + e0, v);
    else {
#pragma unroll
      for (int t = 0; t < 8; ++t) v[t] = 0.0f;
    }
#pragma unroll
    for (int t = 0; t < 8; ++t) sq[t] = fmul(v[t], v[t]);
    if (NL > 0) {
#pragma unroll
      for (int t = 0; t < 8; ++t) keep[j][t] = v[t];
    }
    float leaf = warp_tree(tree8_full(sq), (long long)j * 256, 8, D);
    if (lane == j) mine = leaf;
  }
  float ss = warp_tree(mine, 0, 256, D);
  float rs = fdiv(1.0f, fsqrt(fadd(fmul(ss, invD), eps)));
  if (lane == 0) rstd[row] = rs;
#pragma unroll
  for (int j = 0; j < (NL > 0 ? NL : 32); ++j) {
    if (j >= nl) break;
    const int e0 = j * 256 + lane * 8;
    if (e0 >= D) continue;
    float v[8], o[8];
    if (NL > 0) {
#pragma unroll
      for (int t = 0; t < 8; ++t) v[t] = keep[j][t];
    } else {
      load8<BF>(x, rb + e0, v);
    }
    if (gamma) {
      float g[8];
      load8<BF>(gamma, e0, g);
#pragma unroll
      for (int t = 0; t < 8; ++t) o[t] = fmul(fmul(v[t], rs), g[t]);
    } else {
#pragma unroll
      for (int t = 0; t < 8; ++t) o[t] = fmul(v[t], rs);
    }
    store8<BF>(y, rb + e0, o);
  }
}

template <bool BF, int NL>
__global__ void __launch_bounds__(256) k_rmsnorm_bwd(const void* __restrict__ dy, const void* __restrict__ x,
                                                     const void* __restrict__ gamma, const float* __restrict__ rstd,
                                                     int rows, int D, float invD, void* __restrict__ dx) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = blockIdx.x * 8 + warp;
  if (row >= rows) return;
  const size_t rb = (size_t)row * D;
  const int nl = (D + 255) >> 8;
  const float rs = rstd[row];
  float kw[NL > 0 ? NL : 1][8], kx[NL > 0 ? NL : 1][8];
  float mine = 0.0f;
#pragma unroll
  for (int j = 0; j < (NL > 0 ? NL : 32); ++j) {
    if (j >= nl) break;
    const int e0 = j * 256 + lane * 8;
    float w[8], xh[8], pr[8];
    if (e0 < D) {
      load8<BF>(dy, rb + e0, w);
      load8<BF>(x, rb + e0, xh);
      if (gamma) {
        float g[8];
        load8<BF>(gamma, e0, g);
#pragma unroll
        for (int t = 0; t < 8; ++t) w[t] = fmul(w[t], g[t]);
      }
#pragma unroll
      for (int t = 0; t < 8; ++t) xh[t] = fmul(xh[t], rs);
    } else {
#pragma unroll
      for (int t = 0; t < 8; ++t) { w[t] = 0.0f; xh[t] = 0.0f; }
    }
#pragma unroll
    for (int t = 0; t < 8; ++t) pr[t] = fmul(w[t], xh[t]);
    if (NL > 0) {
#pragma unroll
      for (int t = 0; t < 8; ++t) { kw[j][t] = w[t]; kx[j][t] = xh[t]; }
    }
    float leaf = warp_tree(tree8_full(pr), (long long)j * 256, 8, D);
    if (lane == j) mine = leaf;
  }
  const float c = fmul(warp_tree(mine, 0, 256, D), invD);
#pragma unroll
  for (int j = 0; j < (NL > 0 ? NL : 32); ++j) {
    if (j >= nl) break;
    const int e0 = j * 256 + lane * 8;
    if (e0 >= D) continue;
    float w[8], xh[8], o[8];
    if (NL > 0) {
#pragma unroll
      for (int t = 0; t < 8; ++t) { w[t] = kw[j][t]; xh[t] = kx[j][t]; }
    } else {
      load8<BF>(dy, rb + e0, w);
      load8<BF>(x, rb + e0, xh);
      if (gamma) {
        float g[8];
        load8<BF>(gamma, e0, g);
#pragma unroll
        for (int t = 0; t < 8; ++t) w[t] = fmul(w[t], g[t]);
      }
#pragma unroll
      for (int t = 0; t < 8; ++t) xh[t] = fmul(xh[t], rs);
    }
#pragma unroll
    for (int t = 0; t < 8; ++t) o[t] = fmul(rs, fsub(w[t], fmul(xh[t], c)));
    store8<BF>(dx, rb + e0, o);
  }
}

// dgamma partials: CTA = 256 rows (one leaf of the row-direction tree) x 32 columns.
template <bool BF>
__global__ void __launch_bounds__(256) k_dgamma_partial(const void* __restrict__ dy, const void* __restrict__ x,
                                                        const float* __restrict__ rstd, int rows, int D,
                                                        float* __restrict__ partial) {
  __shared__ float sm[8][33];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int col = blockIdx.x * 32 + lane;
  const long long r0 = (long long)blockIdx.y * 256 + warp * 32;
  float s[32];
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    long long r = r0 + i;
    float v = 0.0f;
    if (r < rows && col < D) {
      size_t idx = (size_t)r * D + col;
      float a, b;
      if (BF) { a = bf2f(reinterpret_cast<const uint16_t*>(dy)[idx]); b = bf2f(reinterpret_cast<const uint16_t*>(x)[idx]); }
      else { a = reinterpret_cast<const float*>(dy)[idx]; b = reinterpret_cast<const float*>(x)[idx]; }
      v = fmul(a, fmul(b, rstd[r]));
    }
    s[i] = v;
  }
  sm[warp][lane] = reg_tree<32>(s, r0, 1, rows);
  __syncthreads();
  if (warp == 0 && col < D) {
    float w[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) w[j] = sm[j][lane];
    partial[(size_t)blockIdx.y * D + col] = reg_tree<8>(w, (long long)blockIdx.y * 256, 32, rows);
  }
}
// tree over the nb row-block partials (each a node of 256 rows) of every column, 32 nodes at a time from independent
// loads; the partial buffer is reused for the intermediate levels
__global__ void k_col_tree(float* __restrict__ partial, int nb, int D, float* __restrict__ out, int rows) {
  const int col = blockIdx.x * blockDim.x + threadIdx.x;
  if (col >= D) return;
  int n = nb;
  long long stride = 256;
  while (n > 1) {
    const int groups = (n + 31) / 32;
    for (int g = 0; g < groups; ++g) {
      float s[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) s[i] = (g * 32 + i < n) ? partial[(size_t)(g * 32 + i) * D + col] : 0.0f;
      partial[(size_t)g * D + col] = reg_tree<32>(s, (long long)g * 32 * stride, stride, rows);
    }
    n = groups;
    stride *= 32;
  }
  out[col] = partial[col];
}

// ------------------------------------------------------------------------------------------------
// Cross-entropy.  One CTA (512 threads) per row: max, then exp and the leaf sums, then the tree over
// leaf sums in shared memory.
// ------------------------------------------------------------------------------------------------
constexpr int XT = 512;
__global__ void __launch_bounds__(XT) k_xent_fwd(const float* __restrict__ logits, const int32_t* __restrict__ target,
                                                 int V, float* __restrict__ loss_row, float* __restrict__ lse_out,
                                                 float* __restrict__ zsq_row, int* status) {
  extern __shared__ float leafs[];  // ceil(V/256) floats, >= 32
  __shared__ float red[XT / 32];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const float* z = logits + (size_t)blockIdx.x * V;
  float m = __int_as_float(0xff800000);
  {
    auto ld4 = [&](const float* p) { return *reinterpret_cast<const float4*>(p); };
    int i = threadIdx.x * 4;
    for (; i + 3 * XT * 4 < V; i += 4 * XT * 4) {      // four loads in flight per thread
      float4 a[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) a[u] = ld4(z + i + u * XT * 4);
#pragma unroll
      for (int u = 0; u < 4; ++u) m = fmaxf(fmaxf(m, fmaxf(a[u].x, a[u].y)), fmaxf(a[u].z, a[u].w));
    }
    for (; i < V; i += XT * 4) {
      float4 a = ld4(z + i);
      m = fmaxf(fmaxf(m, fmaxf(a.x, a.y)), fmaxf(a.z, a.w));
    }
  }
#pragma unroll
  for (int w = 16; w; w >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, w));
  if (lane == 0) red[warp] = m;
  __syncthreads();
  m = red[0];
#pragma unroll
  for (int w = 1; w < XT / 32; ++w) m = fmaxf(m, red[w]);
  const int nl = (V + 255) >> 8;
  // every argument z - m is <= 0 (or NaN), so the exponential without the overflow range applies
  const int nfull = V >> 8;  // leaves that lie wholly inside the row: no existence tests in their tree
  for (int leaf = warp; leaf < nfull; leaf += XT / 32) {
    const int e0 = leaf * 256 + lane * 8;
    // second and last read of the row: streaming loads, so that these lines leave L2 before the rows still waiting
    // between their two sweeps (the rows in flight on all SMs together fill most of L2)
    const float4 a0 = __ldcs(reinterpret_cast<const float4*>(z + e0)), a1 = __ldcs(reinterpret_cast<const float4*>(z + e0 + 4));
    float e[8];
    e[0] = det_exp_le0(fsub(a0.x, m)); e[1] = det_exp_le0(fsub(a0.y, m));          // branch-free: the chains interleave
    e[2] = det_exp_le0(fsub(a0.z, m)); e[3] = det_exp_le0(fsub(a0.w, m));
    e[4] = det_exp_le0(fsub(a1.x, m)); e[5] = det_exp_le0(fsub(a1.y, m));
    e[6] = det_exp_le0(fsub(a1.z, m)); e[7] = det_exp_le0(fsub(a1.w, m));
    const float s = warp_tree_full(tree8_full(e));
    if (lane == 0) leafs[leaf] = s;
  }
  if (nfull < nl && warp == (nfull % (XT / 32))) {  // the ragged last leaf
    const int leaf = nfull;
    const int e0 = leaf * 256 + lane * 8;
    float e[8];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      if (e0 + 4 * h < V) {
        float4 a = *reinterpret_cast<const float4*>(z + e0 + 4 * h);
        e[4 * h] = det_exp_le0(fsub(a.x, m)); e[4 * h + 1] = det_exp_le0(fsub(a.y, m));
        e[4 * h + 2] = det_exp_le0(fsub(a.z, m)); e[4 * h + 3] = det_exp_le0(fsub(a.w, m));
      } else {
        e[4 * h] = e[4 * h + 1] = e[4 * h + 2] = e[4 * h + 3] = 0.0f;
      }
    }
    float s = warp_tree(tree8(e, e0, V), (long long)leaf * 256, 8, V);
    if (lane == 0) leafs[leaf] = s;
  }
  __syncthreads();
  smem_tree(leafs, nl);
  if (threadIdx.x == 0) {
    float l = fadd(m, det_log(leafs[0]));
    lse_out[blockIdx.x] = l;
    int t = target[blockIdx.x];
    if (t < 0 || t >= V) {
      loss_row[blockIdx.x] = 0.0f;
      zsq_row[blockIdx.x] = 0.0f;
      or_status(status, DET_DEV_TARGET);
    } else {
      loss_row[blockIdx.x] = fsub(l, z[t]);
      zsq_row[blockIdx.x] = fmul(l, l);
    }
  }
}

__global__ void k_xent_finish(const float* ce_sum, const float* z_sum, float inv_rows, float z_weight,
                              float* loss_mean, float* z_mean) {
  float ce = fmul(ce_sum[0], inv_rows), zm = fmul(z_sum[0], inv_rows);
  z_mean[0] = zm;
  loss_mean[0] = (z_weight != 0.0f) ? fadd(ce, fmul(z_weight, zm)) : ce;
}

// Each thread takes two groups of four adjacent logits of a row, 1024 columns apart (every access of a warp covers whole
// lines).  The argument z - lse is at most 0 whenever lse is the row's own logsumexp, and then the exponential without the
// overflow range applies (same bits); lse is an input, though, so a thread that sees a positive argument takes the
// general form for its eight values.
__global__ void __launch_bounds__(256) k_xent_bwd(float* __restrict__ logits, const int32_t* __restrict__ target,
                                                  const float* __restrict__ lse, int rows, int V, float z_weight, float scale) {
  const int i0 = blockIdx.x * 2048 + threadIdx.x * 4;
  if (i0 >= V) return;
  const bool two = i0 + 1024 < V;
  for (int row = blockIdx.y; row < rows; row += gridDim.y) {
    float* z = logits + (size_t)row * V;
    const int t = target[row];
    const bool ok = t >= 0 && t < V;
    const float l = lse[row];
    const float zc = fmul(fmul(2.0f, z_weight), l);
    const float4 a = *reinterpret_cast<float4*>(z + i0);
    const float4 b = two ? *reinterpret_cast<float4*>(z + i0 + 1024) : make_float4(0.f, 0.f, 0.f, 0.f);
    float x[8] = {fsub(a.x, l), fsub(a.y, l), fsub(a.z, l), fsub(a.w, l), fsub(b.x, l), fsub(b.y, l), fsub(b.z, l), fsub(b.w, l)};
    bool pos = false;
#pragma unroll
    for (int k = 0; k < 8; ++k) pos |= x[k] > 0.0f;
    float p[8];
    if (!pos) {
#pragma unroll
      for (int k = 0; k < 8; ++k) p[k] = det_exp_le0(x[k]);
    } else {
#pragma unroll
      for (int k = 0; k < 8; ++k) p[k] = det_exp(x[k]);
    }
    float v[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int col = i0 + (k >> 2) * 1024 + (k & 3);
      float d = fsub(p[k], (col == t) ? 1.0f : 0.0f);
      if (z_weight != 0.0f) d = fadd(d, fmul(zc, p[k]));
      v[k] = ok ? fmul(d, scale) : 0.0f;
    }
    *reinterpret_cast<float4*>(z + i0) = make_float4(v[0], v[1], v[2], v[3]);
    if (two) *reinterpret_cast<float4*>(z + i0 + 1024) = make_float4(v[4], v[5], v[6], v[7]);
  }
}

}  // namespace det

using namespace det;

extern "C" int det_rmsnorm_fwd(int io, const void* x, const void* gamma, int rows, int D, float eps, void* y,
                               float* rstd, void* stream) {
  if (!x || !y || !rstd || rows < 0 || D <= 0 || (io != DET_F32 && io != DET_BF16)) return DET_ERR_ARG;
  if (D % 8 || D > 8192) return DET_ERR_SHAPE;
  if (!aligned16(x) || !aligned16(y) || (gamma && !aligned16(gamma))) return DET_ERR_ALIGN;
  if (rows == 0) return DET_OK;
  cudaStream_t st = (cudaStream_t)stream;
  const float invD = (float)(1.0 / (double)D);
  dim3 grid((rows + 7) / 8);
  if (io == DET_BF16) {
    if (D <= 2048) k_rmsnorm_fwd8<true><<<DET_L(grid), 256, 0, st>>>(x, gamma, rows, D, eps, invD, y, rstd);
    else k_rmsnorm_fwd<true, 0><<<DET_L(grid), 256, 0, st>>>(x, gamma, rows, D, eps, invD, y, rstd);
  } else {
    if (D <= 2048) k_rmsnorm_fwd8<false><<<DET_L(grid), 256, 0, st>>>(x, gamma, rows, D, eps, invD, y, rstd);
    else k_rmsnorm_fwd<false, 0><<<DET_L(grid), 256, 0, st>>>(x, gamma, rows, D, eps, invD, y, rstd);
  }
  DET_CHECK_LAUNCH();
  return DET_OK;
}

extern "C" int det_rmsnorm_fwd_q(const det_bf16* x, const det_bf16* gamma, int rows, int D, float eps, det_bf16* y,
                                 float* rstd, const float* s_q, int8_t* qy, void* stream) {
  if (!x || !y || !rstd || !s_q || !qy || rows < 0 || D <= 0) return DET_ERR_ARG;
  if (D % 8 || D > 2048) return DET_ERR_SHAPE;
  if (!aligned16(x) || !aligned16(y) || (gamma && !aligned16(gamma)) || (((uintptr_t)qy) & 7u)) return DET_ERR_ALIGN;
  if (rows == 0) return DET_OK;
  k_rmsnorm_fwd8<true><<<DET_L((rows + 7) / 8), 256, 0, (cudaStream_t)stream>>>(x, gamma, rows, D, eps, (float)(1.0 / (double)D), y,
                                                                              rstd, s_q, qy);
  DET_CHECK_LAUNCH();
  return DET_OK;
}

extern "C" size_t det_rmsnorm_bwd_ws_bytes(int rows, int D) {
  const size_t nb8 = (size_t)((rows + 7) / 8), nb256 = (size_t)((rows + 255) / 256);
  return align_up(nb8 * (size_t)D * sizeof(float), 256) + align_up(nb256 * (size_t)D * sizeof(float), 256) + 256;
}

template <bool BF>
static int rmsnorm_bwd8_launch(const void* dy, const void* x, const void* gamma, const float* rstd, int rows, int D,
                               float invD, void* dx, float* dgamma, float* ws, cudaStream_t st) {
  const int nb8 = (rows + 7) / 8, nb256 = (rows + 255) / 256;
  if (!dgamma) {
    k_rmsnorm_bwd8<BF, false><<<DET_L(nb8), 256, 0, st>>>(dy, x, gamma, rstd, rows, D, invD, dx, nullptr, nullptr);
    return DET_OK;
  }
  float* partial8 = ws;
  float* partial256 = ws + align_up((size_t)nb8 * D, 64);
  int* tickets = reinterpret_cast<int*>(partial256 + align_up((size_t)nb256 * D, 64));   // one per block of 256 columns (<= 8)
  k_rmsnorm_bwd8<BF, true><<<DET_L(nb8), 256, 0, st>>>(dy, x, gamma, rstd, rows, D, invD, dx, partial8, tickets);
  // the second launch overlaps its start-up with the first kernel's tail (programmatic dependent launch); the kernel
  // itself waits for the first grid to complete before it reads anything
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((D + 255) / 256, nb256);
  cfg.blockDim = dim3(256);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  note_launch();
  if (cudaLaunchKernelEx(&cfg, k_colsum32, (const float*)partial8, nb8, rows, D, partial256, nb256, tickets, dgamma) != cudaSuccess) {
    cudaGetLastError();
    return DET_ERR_CUDA;
  }
  return DET_OK;
}

extern "C" int det_rmsnorm_bwd(int io, const void* dy, const void* x, const void* gamma, const float* rstd, int rows,
                               int D, void* dx, float* dgamma, void* ws, size_t ws_bytes, void* stream) {
  if (!dy || !x || !rstd || !dx || rows < 0 || D <= 0 || (io != DET_F32 && io != DET_BF16)) return DET_ERR_ARG;
  if (D % 8 || D > 8192) return DET_ERR_SHAPE;
  if (!aligned16(x) || !aligned16(dy) || !aligned16(dx) || (gamma && !aligned16(gamma))) return DET_ERR_ALIGN;
  if (dgamma && (!ws || !aligned16(ws) || ws_bytes < det_rmsnorm_bwd_ws_bytes(rows, D))) return DET_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  if (rows == 0) {
    if (dgamma) cudaMemsetAsync(dgamma, 0, (size_t)D * sizeof(float), st);
    return DET_OK;
  }
  const float invD = (float)(1.0 / (double)D);
  if (D <= 2048) {
    int rc = (io == DET_BF16) ? rmsnorm_bwd8_launch<true>(dy, x, gamma, rstd, rows, D, invD, dx, dgamma, (float*)ws, st)
                              : rmsnorm_bwd8_launch<false>(dy, x, gamma, rstd, rows, D, invD, dx, dgamma, (float*)ws, st);
    if (rc != DET_OK) return rc;
    DET_CHECK_LAUNCH();
    return DET_OK;
  }
  dim3 grid((rows + 7) / 8);
  if (io == DET_BF16) k_rmsnorm_bwd<true, 0><<<DET_L(grid), 256, 0, st>>>(dy, x, gamma, rstd, rows, D, invD, dx);
  else k_rmsnorm_bwd<false, 0><<<DET_L(grid), 256, 0, st>>>(dy, x, gamma, rstd, rows, D, invD, dx);
  if (dgamma) {
    const int nb = (rows + 255) / 256;
    dim3 g2((D + 31) / 32, nb);
    if (io == DET_BF16) k_dgamma_partial<true><<<DET_L(g2), 256, 0, st>>>(dy, x, rstd, rows, D, (float*)ws);
    else k_dgamma_partial<false><<<DET_L(g2), 256, 0, st>>>(dy, x, rstd, rows, D, (float*)ws);
    k_col_tree<<<DET_L((D + 127) / 128), 128, 0, st>>>((float*)ws, nb, D, dgamma, rows);
  }
  DET_CHECK_LAUNCH();
  return DET_OK;
}

extern "C" size_t det_xent_ws_bytes(int rows, int V) {
  (void)V;
  size_t r = align_up((size_t)(rows > 0 ? rows : 1), 64);
  return (r + 128 + sum_ws_floats((size_t)rows)) * sizeof(float);
}

extern "C" int det_xent_fwd(const float* logits, const int32_t* target, int rows, int V, float z_weight,
                            float* loss_row, float* lse, float* loss_mean, float* z_mean, void* ws, size_t ws_bytes,
                            void* stream, int* status_dev) {
  if (!logits || !target || !loss_row || !lse || !loss_mean || !z_mean || rows <= 0 || V <= 0 || !ws) return DET_ERR_ARG;
  if (V % 4 || V > 2 * XT * 256) return DET_ERR_SHAPE;
  if (!aligned16(logits)) return DET_ERR_ALIGN;
  if (ws_bytes < det_xent_ws_bytes(rows, V)) return DET_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  float* zsq = (float*)ws;
  float* sums = zsq + align_up((size_t)rows, 64);
  float* scratch = sums + 128;
  const int nl = (V + 255) / 256;
  size_t sh = (size_t)(nl < 32 ? 32 : nl) * sizeof(float);
  k_xent_fwd<<<DET_L(rows), XT, sh, st>>>(logits, target, V, loss_row, lse, zsq, status_dev);
  sum_launch(loss_row, (size_t)rows, 0, sums, scratch, st);
  sum_launch(zsq, (size_t)rows, 0, sums + 64, scratch, st);
  k_xent_finish<<<DET_L(1), 1, 0, st>>>(sums, sums + 64, (float)(1.0 / (double)rows), z_weight, loss_mean, z_mean);
  DET_CHECK_LAUNCH();
  return DET_OK;
}

extern "C" int det_xent_bwd(float* logits_inout, const int32_t* target, const float* lse, int rows, int V,
                            float z_weight, float scale, void* stream) {
  if (!logits_inout || !target || !lse || rows <= 0 || V <= 0) return DET_ERR_ARG;
  if (V % 4) return DET_ERR_SHAPE;
  if (!aligned16(logits_inout)) return DET_ERR_ALIGN;
  dim3 grid((V + 2047) / 2048, rows < 65535 ? rows : 65535);
  k_xent_bwd<<<DET_L(grid), 256, 0, (cudaStream_t)stream>>>(logits_inout, target, lse, rows, V, z_weight, scale);
  DET_CHECK_LAUNCH();
  return DET_OK;
}
