// Order-fixed sums on CUDA cores: det_sum, global gradient norm, clip scaling, primitive test hook.
//
// A CTA reduces one aligned chunk of 16384 elements (64 leaves of 256) as a perfect subtree of the
// fixed pairwise tree: a lane reads 8 adjacent floats (two 128-bit loads) and pairs them in registers,
// a warp butterfly finishes the 256-element leaf, eight leaf sums are paired in registers, and the
// eight warp sums in shared memory.  The chunk sums are reduced by the same kernel until one value
// is left, so the tree depends on n only.
#include <atomic>
#include <mutex>

#include "common.cuh"
#include "internal.h"
#include "../../include/det_test.h"

namespace det {

static std::atomic<unsigned long long> g_launches{0};
int note_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); return 0; }

static std::mutex g_dev_mutex;

AuxStreams* aux_fork(cudaStream_t st) {
  static AuxStreams table[MAX_DEVICES] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return nullptr;
  AuxStreams* a = &table[dev];
  {
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    if (!a->ok) {
      // all or nothing: what a failed attempt created is destroyed again, so a later call starts from scratch
      AuxStreams t = {};
      int ns = 0, ne = 0;
      bool good = true, have_fork = false;
      for (int i = 0; i < 2 && good; ++i) {
        good = cudaStreamCreateWithFlags(&t.s[i], cudaStreamNonBlocking) == cudaSuccess;
        if (good) ++ns;
        if (good) { good = cudaEventCreateWithFlags(&t.join[i], cudaEventDisableTiming) == cudaSuccess; if (good) ++ne; }
      }
      if (good) { good = cudaEventCreateWithFlags(&t.fork, cudaEventDisableTiming) == cudaSuccess; have_fork = good; }
      if (!good) {
        for (int i = 0; i < ns; ++i) cudaStreamDestroy(t.s[i]);
        for (int i = 0; i < ne; ++i) cudaEventDestroy(t.join[i]);
        if (have_fork) cudaEventDestroy(t.fork);
        cudaGetLastError();
        return nullptr;
      }
      t.ok = true;
      *a = t;
    }
  }
  if (cudaEventRecord(a->fork, st) != cudaSuccess) return nullptr;
  // if the second wait fails the first auxiliary stream already depends on `st`: still hand the streams out, the
  // join below is what the caller's stream order needs
  for (int i = 0; i < 2; ++i)
    if (cudaStreamWaitEvent(a->s[i], a->fork, 0) != cudaSuccess) { cudaGetLastError(); return nullptr; }
  return a;
}
bool aux_join(cudaStream_t st, AuxStreams* a) {
  if (!a) return true;
  bool ok = true;
  for (int i = 0; i < 2; ++i)
    if (cudaEventRecord(a->join[i], a->s[i]) != cudaSuccess || cudaStreamWaitEvent(st, a->join[i], 0) != cudaSuccess) ok = false;
  return ok;
}

int dev_ensure_smem(DevOnce& once, const void* fn, size_t bytes) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return DET_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_dev_mutex);
  if (!once.done[dev]) {
    if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) {
      cudaGetLastError();
      return DET_ERR_CUDA;
    }
    once.done[dev] = true;
  }
  return DET_OK;
}
int dev_sm_count() {
  static int sms[MAX_DEVICES] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return 0;
  std::lock_guard<std::mutex> lock(g_dev_mutex);
  if (!sms[dev] && cudaDeviceGetAttribute(&sms[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) sms[dev] = 0;
  return sms[dev];
}
unsigned long long launches() { return g_launches.load(std::memory_order_relaxed); }

constexpr int SUM_CHUNK = 16384;

template <bool SQ>
__global__ void __launch_bounds__(256) k_sum_chunk(const float* __restrict__ x, long long n, float* __restrict__ partial) {
  __shared__ float wsum[8];
  const long long base = (long long)blockIdx.x * SUM_CHUNK;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float s[8];
  if (base + SUM_CHUNK <= n) {
    float4 a[8], b[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float4* p = reinterpret_cast<const float4*>(x + base + (warp * 8 + j) * 256 + lane * 8);
      a[j] = __ldg(p);
      b[j] = __ldg(p + 1);
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      float v[8] = {a[j].x, a[j].y, a[j].z, a[j].w, b[j].x, b[j].y, b[j].z, b[j].w};
      if (SQ) {
#pragma unroll
        for (int t = 0; t < 8; ++t) v[t] = fmul(v[t], v[t]);
      }
      s[j] = warp_tree_full(tree8_full(v));
    }
    float r = fadd(fadd(fadd(s[0], s[1]), fadd(s[2], s[3])), fadd(fadd(s[4], s[5]), fadd(s[6], s[7])));
    if (lane == 0) wsum[warp] = r;
    __syncthreads();
    if (threadIdx.x == 0)
      partial[blockIdx.x] = fadd(fadd(fadd(wsum[0], wsum[1]), fadd(wsum[2], wsum[3])),
                                 fadd(fadd(wsum[4], wsum[5]), fadd(wsum[6], wsum[7])));
    return;
  }
  // ragged last chunk: same tree with existence predicates
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const long long lf = base + (warp * 8 + j) * 256;
    const long long e0 = lf + lane * 8;
    float v[8];
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      float u = (e0 + t < n) ? x[e0 + t] : 0.0f;
      v[t] = SQ ? fmul(u, u) : u;
    }
    s[j] = warp_tree(tree8(v, e0, n), lf, 8, n);
  }
  float r = reg_tree<8>(s, base + (long long)warp * 2048, 256, n);
  if (lane == 0) wsum[warp] = r;
  __syncthreads();
  if (threadIdx.x == 0) {
    float w[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) w[j] = wsum[j];
    partial[blockIdx.x] = reg_tree<8>(w, base, 2048, n);
  }
}

// A lone element (n == 1) is carried by the tree without any addition; flush it explicitly, as every
// value that enters or leaves an operation is flushed.
__global__ void k_flush1(const float* x, float* out, int sq) {
  float v = x[0];
  uint32_t u = __float_as_uint(v);
  if (!(u & 0x7f800000u)) v = __uint_as_float(u & 0x80000000u);
  out[0] = sq ? fmul(v, v) : v;
}

static inline long long nchunks(long long n) { return (n + SUM_CHUNK - 1) / SUM_CHUNK; }

// runs the multi-level reduction; result lands in out[0] (device).  ws must hold sum_ws floats.
size_t sum_ws_floats(size_t n) {
  size_t tot = 0;
  long long c = nchunks((long long)n);
  while (c > 1) { tot += align_up((size_t)c, 64); c = nchunks(c); }
  return tot + 64;
}

int sum_launch(const float* x, size_t n, int squares, float* out, float* ws, cudaStream_t st) {
  if (n == 0) { cudaMemsetAsync(out, 0, sizeof(float), st); return DET_OK; }
  if (n == 1) { k_flush1<<<DET_L(1), 1, 0, st>>>(x, out, squares); return DET_OK; }
  const float* src = x;
  long long cur = (long long)n;
  bool sq = squares != 0;
  float* w = ws;
  while (true) {
    long long c = nchunks(cur);
    float* dst = (c == 1) ? out : w;
    if (sq) k_sum_chunk<true><<<DET_L((unsigned)c), 256, 0, st>>>(src, cur, dst);
    else k_sum_chunk<false><<<DET_L((unsigned)c), 256, 0, st>>>(src, cur, dst);
    if (c == 1) break;
    w += align_up((size_t)c, 64);
    src = dst;
    cur = c;
    sq = false;
  }
  return DET_OK;
}

__global__ void k_norm_finish(const float* total, float max_norm, float* norm_out, float* coef_out, int* status) {
  float nrm = fsqrt(total[0]);
  norm_out[0] = nrm;
  float coef = 1.0f;
  if (max_norm > 0.0f) coef = fminf(1.0f, fdiv(max_norm, fadd(nrm, 1e-6f)));
  coef_out[0] = coef;
  if (!(fabsf(nrm) <= 3.4028234e38f)) or_status(status, DET_DEV_NONFINITE);
}

__global__ void __launch_bounds__(256) k_scale(float* __restrict__ g, size_t n, const float* __restrict__ coef) {
  const float c = coef[0];
  size_t i = ((size_t)blockIdx.x * 256 + threadIdx.x) * 4;
  if (i + 4 <= n) {
    float4 v = *reinterpret_cast<float4*>(g + i);
    v.x = fmul(v.x, c); v.y = fmul(v.y, c); v.z = fmul(v.z, c); v.w = fmul(v.w, c);
    *reinterpret_cast<float4*>(g + i) = v;
  } else {
    for (; i < n; ++i) g[i] = fmul(g[i], c);
  }
}

__global__ void k_prim(int op, const float* a, const float* b, float* out, size_t n) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  float x = a[i], y = b ? b[i] : 0.0f, r;
  switch (op) {
    case 0: r = fadd(x, y); break;
    case 1: r = fsub(x, y); break;
    case 2: r = fmul(x, y); break;
    case 3: r = fdiv(x, y); break;
    case 4: r = fsqrt(x); break;
    case 5: r = det_exp(x); break;
    case 6: r = det_log(x); break;
    case 7: r = fmaxf(x, y); break;
    case 8: {  // narrowing is only ever applied to flushed values; flush the raw input here
      uint32_t u = __float_as_uint(x);
      if (!(u & 0x7f800000u)) x = __uint_as_float(u & 0x80000000u);
      r = bf2f(f2bf(x));
      break;
    }
    case 9: r = fadd(fmul(x, y), y); break;
    case 10: r = det_exp_le0(x); break;
    default: r = 0.0f;
  }
  out[i] = r;
}

}  // namespace det

using namespace det;

extern "C" unsigned long long det_launch_count(void) { return det::launches(); }

extern "C" int det_device_sm_count(void) {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return DET_ERR_CUDA;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return DET_ERR_CUDA;
  return sms;
}

extern "C" int det_test_prim(int op, const float* a, const float* b, float* out, size_t n, void* stream) {
  if (!a || !out || op < 0 || op > 10) return DET_ERR_ARG;
  if (n == 0) return DET_OK;
  k_prim<<<DET_L((unsigned)((n + 255) / 256)), 256, 0, (cudaStream_t)stream>>>(op, a, b, out, n);
  DET_CHECK_LAUNCH();
  return DET_OK;
}

extern "C" size_t det_sum_ws_bytes(size_t n) { return sum_ws_floats(n) * sizeof(float); }

extern "C" int det_sum(const float* x, size_t n, int squares, float* out, void* ws, size_t ws_bytes, void* stream) {
  if (!out || (n && !x)) return DET_ERR_ARG;
  if (n && !aligned16(x)) return DET_ERR_ALIGN;
  if (ws_bytes < det_sum_ws_bytes(n) || (!ws && n > (size_t)SUM_CHUNK)) return DET_ERR_WORKSPACE;
  int rc = sum_launch(x, n, squares, out, (float*)ws, (cudaStream_t)stream);
  DET_CHECK_LAUNCH();
  return rc;
}

extern "C" size_t det_grad_norm_ws_bytes(const size_t* n_elems, int ntensors) {
  size_t mx = 0;
  for (int t = 0; t < ntensors; ++t) mx = n_elems[t] > mx ? n_elems[t] : mx;
  return (align_up((size_t)(ntensors > 0 ? ntensors : 1), 64) + 64 + sum_ws_floats(mx) +
          sum_ws_floats((size_t)(ntensors > 0 ? ntensors : 1))) * sizeof(float);
}

extern "C" int det_grad_norm(const float* const* g_ptrs, const size_t* n_elems, int ntensors, float max_norm,
                             float* norm_out, float* coef_out, void* ws, size_t ws_bytes, void* stream,
                             int* status_dev) {
  if (ntensors < 0 || !norm_out || !coef_out || (ntensors && (!g_ptrs || !n_elems)) || !ws) return DET_ERR_ARG;
  if (ws_bytes < det_grad_norm_ws_bytes(n_elems, ntensors)) return DET_ERR_WORKSPACE;
  for (int t = 0; t < ntensors; ++t)
    if (n_elems[t] && (!g_ptrs[t] || !aligned16(g_ptrs[t]))) return g_ptrs[t] ? DET_ERR_ALIGN : DET_ERR_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  float* per = (float*)ws;
  float* total = per + align_up((size_t)(ntensors > 0 ? ntensors : 1), 64);
  float* scratch = total + 64;
  for (int t = 0; t < ntensors; ++t) sum_launch(g_ptrs[t], n_elems[t], 1, per + t, scratch, st);
  sum_launch(per, (size_t)ntensors, 0, total, scratch, st);
  k_norm_finish<<<DET_L(1), 1, 0, st>>>(total, max_norm, norm_out, coef_out, status_dev);
  DET_CHECK_LAUNCH();
  return DET_OK;
}

extern "C" int det_scale_inplace(float* g, size_t n, const float* coef_dev, void* stream) {
  if ((n && !g) || !coef_dev) return DET_ERR_ARG;
  if (n && !aligned16(g)) return DET_ERR_ALIGN;
  if (n == 0) return DET_OK;
  k_scale<<<DET_L((unsigned)((n + 1023) / 1024)), 256, 0, (cudaStream_t)stream>>>(g, n, coef_dev);
  DET_CHECK_LAUNCH();
  return DET_OK;
}
