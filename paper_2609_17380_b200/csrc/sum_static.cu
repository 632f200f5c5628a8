// det_sum_static: the order-fixed sum for callers that cannot bring a workspace.
//
// Some users of this library run where they may not allocate device memory at all: a plug-in inside a host
// application that owns the whole device heap and hands the plug-in nothing but its input and output
// buffers, or a control loop that must never enter cudaMalloc because that call synchronises the device.
// For them this one entry point keeps its scratch (the per-chunk partial sums of the tree) in a fixed
// array that is part of the library image, so the call allocates nothing, frees nothing and calls no
// allocating routine.  Every GPU that loads the library carries the array (256 KiB) until the process exits.
#include <mutex>

#include "common.cuh"
#include "internal.h"

namespace det {

constexpr size_t STATIC_SCRATCH_FLOATS = 65536;  // 256 KiB
// On the host this name is only a handle for the runtime, never a device address: host code must ask
// cudaGetSymbolAddress for the address and hand that to kernels.
static __device__ __align__(256) float g_sum_scratch[STATIC_SCRATCH_FLOATS];

static float* g_scratch_addr[MAX_DEVICES];  // device address of g_sum_scratch on each device, filled on first use
static std::mutex g_scratch_mutex;

// Device address of the scratch array on the CURRENT device; looked up once per device.
static int scratch_address(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return DET_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_sum_scratch) != cudaSuccess || !p) {
      cudaGetLastError();
      return DET_ERR_CUDA;
    }
    g_scratch_addr[dev] = static_cast<float*>(p);
  }
  *out = g_scratch_addr[dev];
  return DET_OK;
}

}  // namespace det

using namespace det;

extern "C" size_t det_sum_static_max_n(void) { return (size_t)DET_SUM_STATIC_MAX_N; }

extern "C" int det_sum_static(const float* x, size_t n, int squares, float* out, void* stream) {
  if (!out || (n && !x)) return DET_ERR_ARG;
  if (n > (size_t)DET_SUM_STATIC_MAX_N) return DET_ERR_SHAPE;  // the fixed scratch cannot hold more partial sums
  if (n && !aligned16(x)) return DET_ERR_ALIGN;
  if (sum_ws_floats(n) > STATIC_SCRATCH_FLOATS) return DET_ERR_SHAPE;
  float* scratch = nullptr;
  int rc = scratch_address(&scratch);
  if (rc != DET_OK) return rc;
  // Nothing in the scratch has to start at zero: every partial sum is written by one level of the tree
  // before the next level reads it, so the previous call's contents are simply overwritten.
  rc = sum_launch(x, n, squares, out, scratch, (cudaStream_t)stream);
  DET_CHECK_LAUNCH();
  return rc;
}
