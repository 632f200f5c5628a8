// Per-head operations of the paper's attention block (Sec. 3.1): gain-free RMS normalisation of every query and key
// head ("QK-norm", applied before the rotary embedding) and the rotary position embedding itself.  All three kernels
// work on rows of 128 values that sit inside a wider token row (the fused q|k|v projection output), one warp per
// (token, head); they are HBM-bound and touch every element once.
#include "common.cuh"
#include "internal.h"

namespace det {

constexpr int HD = 128;

// y = bf16(x * rstd), rstd = 1 / sqrt(mean(x^2) + eps); the mean is the adjacent pairwise tree over the 128 squares
// times 2^-7.  Lane l holds elements 4l .. 4l+3.
__global__ void __launch_bounds__(256) k_headnorm_fwd(const uint16_t* __restrict__ x, int ld, size_t nrows, int nh, float eps,
                                                      uint16_t* __restrict__ y, int ld_y, float* __restrict__ rstd) {
  const size_t w = (size_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (w >= nrows) return;
  const size_t t = w / nh, h = w % nh;
  const uint2 u = __ldg(reinterpret_cast<const uint2*>(x + t * ld + h * HD + lane * 4));
  const float v[4] = {bflo(u.x), bfhi(u.x), bflo(u.y), bfhi(u.y)};
  float s = fadd(fadd(fmul(v[0], v[0]), fmul(v[1], v[1])), fadd(fmul(v[2], v[2]), fmul(v[3], v[3])));
  s = warp_tree_full(s);
  const float rs = fdiv(1.0f, fsqrt(fadd(fmul(s, 0x1p-7f), eps)));
  uint2 o;
  o.x = pack_bf2(fmul(v[0], rs), fmul(v[1], rs));
  o.y = pack_bf2(fmul(v[2], rs), fmul(v[3], rs));
  *reinterpret_cast<uint2*>(y + t * ld_y + h * HD + lane * 4) = o;
  if (lane == 0) rstd[w] = rs;
}

// dx = bf16(rstd * (dy - xhat * c)), xhat = x * rstd, c = mean(dy * xhat) over the same tree
__global__ void __launch_bounds__(256) k_headnorm_bwd(const uint16_t* __restrict__ dy, int ld_dy, const uint16_t* __restrict__ x,
                                                      int ld, const float* __restrict__ rstd, size_t nrows, int nh,
                                                      uint16_t* __restrict__ dx, int ld_dx) {
  const size_t w = (size_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (w >= nrows) return;
  const size_t t = w / nh, h = w % nh;
  const uint2 ux = __ldg(reinterpret_cast<const uint2*>(x + t * ld + h * HD + lane * 4));
  const uint2 ug = __ldg(reinterpret_cast<const uint2*>(dy + t * ld_dy + h * HD + lane * 4));
  const float rs = rstd[w];
  const float g[4] = {bflo(ug.x), bfhi(ug.x), bflo(ug.y), bfhi(ug.y)};
  const float xh[4] = {fmul(bflo(ux.x), rs), fmul(bfhi(ux.x), rs), fmul(bflo(ux.y), rs), fmul(bfhi(ux.y), rs)};
  float s = fadd(fadd(fmul(g[0], xh[0]), fmul(g[1], xh[1])), fadd(fmul(g[2], xh[2]), fmul(g[3], xh[3])));
  s = warp_tree_full(s);
  const float c = fmul(s, 0x1p-7f);
  float r[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) r[e] = fmul(rs, fsub(g[e], fmul(xh[e], c)));
  uint2 o;
  o.x = pack_bf2(r[0], r[1]);
  o.y = pack_bf2(r[2], r[3]);
  *reinterpret_cast<uint2*>(dx + t * ld_dx + h * HD + lane * 4) = o;
}

// Pairs (i, i + 64): y_i = x_i c_i - x_{i+64} s_i, y_{i+64} = x_{i+64} c_i + x_i s_i with every product rounded on its own
// (scalar multiplies and adds: nothing here may be contracted).  Lane l holds i = 2l, 2l+1 and their partners.
__global__ void __launch_bounds__(256) k_rope(const uint16_t* __restrict__ x, int ld, size_t nrows, int nh, int S,
                                              const float* __restrict__ cs, const float* __restrict__ sn, int inverse,
                                              uint16_t* __restrict__ y, int ld_y) {
  const size_t w = (size_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (w >= nrows) return;
  const size_t t = w / nh, h = w % nh;
  const size_t pos = t % (size_t)S;
  const uint16_t* xr = x + t * ld + h * HD;
  const uint32_t ua = __ldg(reinterpret_cast<const uint32_t*>(xr + 2 * lane));
  const uint32_t ub = __ldg(reinterpret_cast<const uint32_t*>(xr + 64 + 2 * lane));
  const float2 c = __ldg(reinterpret_cast<const float2*>(cs + pos * 64 + 2 * lane));
  float2 s = __ldg(reinterpret_cast<const float2*>(sn + pos * 64 + 2 * lane));
  if (inverse) { s.x = -s.x; s.y = -s.y; }
  const float a0 = bflo(ua), a1 = bfhi(ua), b0 = bflo(ub), b1 = bfhi(ub);
  const float lo0 = fsub(fmul(a0, c.x), fmul(b0, s.x)), lo1 = fsub(fmul(a1, c.y), fmul(b1, s.y));
  const float hi0 = fadd(fmul(b0, c.x), fmul(a0, s.x)), hi1 = fadd(fmul(b1, c.y), fmul(a1, s.y));
  uint16_t* yr = y + t * ld_y + h * HD;
  *reinterpret_cast<uint32_t*>(yr + 2 * lane) = pack_bf2(lo0, lo1);
  *reinterpret_cast<uint32_t*>(yr + 64 + 2 * lane) = pack_bf2(hi0, hi1);
}

static inline bool head_args_ok(int ld, int T, int nh) { return T > 0 && nh > 0 && ld >= nh * HD && ld % 4 == 0; }

}  // namespace det

using namespace det;

extern "C" int det_headnorm_fwd(const det_bf16* x, int ld, int T, int nh, float eps, det_bf16* y, int ld_y, float* rstd,
                                void* stream) {
  if (!x || !y || !rstd) return DET_ERR_ARG;
  if (!head_args_ok(ld, T, nh) || !head_args_ok(ld_y, T, nh)) return DET_ERR_SHAPE;
  if ((((uintptr_t)x) | ((uintptr_t)y)) & 7u) return DET_ERR_ALIGN;
  const size_t nrows = (size_t)T * nh;
  k_headnorm_fwd<<<DET_L((unsigned)((nrows + 7) / 8)), 256, 0, (cudaStream_t)stream>>>(x, ld, nrows, nh, eps, y, ld_y, rstd);
  DET_CHECK_LAUNCH();
  return DET_OK;
}

extern "C" int det_headnorm_bwd(const det_bf16* dy, int ld_dy, const det_bf16* x, int ld, const float* rstd, int T, int nh,
                                det_bf16* dx, int ld_dx, void* stream) {
  if (!dy || !x || !rstd || !dx) return DET_ERR_ARG;
  if (!head_args_ok(ld, T, nh) || !head_args_ok(ld_dy, T, nh) || !head_args_ok(ld_dx, T, nh)) return DET_ERR_SHAPE;
  if ((((uintptr_t)x) | ((uintptr_t)dy) | ((uintptr_t)dx)) & 7u) return DET_ERR_ALIGN;
  const size_t nrows = (size_t)T * nh;
  k_headnorm_bwd<<<DET_L((unsigned)((nrows + 7) / 8)), 256, 0, (cudaStream_t)stream>>>(dy, ld_dy, x, ld, rstd, nrows, nh, dx,
                                                                                     ld_dx);
  DET_CHECK_LAUNCH();
  return DET_OK;
}

extern "C" int det_rope(const det_bf16* x, int ld, int T, int nh, int S, const float* cos_tab, const float* sin_tab,
                        int inverse, det_bf16* y, int ld_y, void* stream) {
  if (!x || !y || !cos_tab || !sin_tab || S <= 0) return DET_ERR_ARG;
  if (!head_args_ok(ld, T, nh) || !head_args_ok(ld_y, T, nh)) return DET_ERR_SHAPE;
  if (((((uintptr_t)x) | ((uintptr_t)y)) & 3u) || ((((uintptr_t)cos_tab) | ((uintptr_t)sin_tab)) & 7u)) return DET_ERR_ALIGN;
  const size_t nrows = (size_t)T * nh;
  k_rope<<<DET_L((unsigned)((nrows + 7) / 8)), 256, 0, (cudaStream_t)stream>>>(x, ld, nrows, nh, S, cos_tab, sin_tab, inverse, y,
                                                                            ld_y);
  DET_CHECK_LAUNCH();
  return DET_OK;
}
