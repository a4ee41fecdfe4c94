// ps_replay_sum_static: the long-queue reduce-and-apply for callers that must not allocate.
//
// The context-based path (ps_apply) keeps the partial sums of its two-stage reduction in the
// caller's arena.  Some users of this library have no arena to give and no allocator to call: a
// plugin running inside a host application that handed all device memory to its own pool at start-up,
// or a control loop that cannot afford the implicit device-wide synchronisation of an allocation.
// For them the partial sums live in a fixed array that is part of the loaded library image.
//
// This file is self-contained on purpose: it has its own kernels and touches nothing else.
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdio>
#include <mutex>

#include "kernels.h"
#include "ps.h"

namespace {

constexpr int TPB = 256;
constexpr int SPLITS = PS_STATIC_REPLAY_SPLITS;
constexpr int COL_BLOCKS = (psk::P_VEC4 + TPB - 1) / TPB;
constexpr int MAX_DEVICES = 64;

// SPLITS partial-sum vectors of PS_PARAM_STRIDE floats (about 13 MB).  Every GPU on which the
// library is loaded holds one copy until the process exits.
static __device__ __align__(256) float g_static_partials[(size_t)SPLITS * psk::P_PAD];

// In host code `g_static_partials` is only a handle.  The address kernels may use is looked up
// once per device and remembered here.
float* g_partials_addr[MAX_DEVICES] = {nullptr};
std::mutex g_setup_mutex;
thread_local char g_static_err[320] = "";

__device__ __forceinline__ void add4(float4& a, const float4& b) {
  a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
}

// Block (x, y) sums slot range y of column block x into partial vector y.  Four running sums per
// thread keep several independent 16-byte loads in flight; the order of additions is fixed.
__global__ void __launch_bounds__(TPB) static_partial(const float4* __restrict__ queue, long long K,
                                                      float4* __restrict__ partial) {
  const int col = blockIdx.x * TPB + threadIdx.x;
  if (col >= psk::P_VEC4) return;
  const int s = blockIdx.y;
  const long long per = (K + SPLITS - 1) / SPLITS;
  const long long k0 = s * per;
  const long long k1 = k0 + per < K ? k0 + per : K;
  float4 acc[4];
#pragma unroll
  for (int u = 0; u < 4; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
  const float4* q = queue + col;
  long long k = k0;
  for (; k + 4 <= k1; k += 4) {
    float4 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) v[u] = __ldcs(q + (k + u) * (long long)psk::P_VEC4);
#pragma unroll
    for (int u = 0; u < 4; ++u) add4(acc[u], v[u]);
  }
#pragma unroll
  for (int u = 0; u < 3; ++u)
    if (k + u < k1) add4(acc[u], __ldcs(q + (k + u) * (long long)psk::P_VEC4));
  add4(acc[0], acc[1]); add4(acc[2], acc[3]); add4(acc[0], acc[2]);
  // Written even when the range is empty: the array keeps the previous call's contents, and the
  // second stage reads every one of the SPLITS vectors.
  partial[(long long)s * psk::P_VEC4 + col] = acc[0];
}

__global__ void __launch_bounds__(TPB) static_finish(const float4* __restrict__ partial,
                                                     const float4* theta_in, float4* theta_out,   // may be one buffer
                                                     float coef) {
  const int col = blockIdx.x * TPB + threadIdx.x;
  if (col >= psk::P_VEC4) return;
  float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
  for (int i = 0; i < SPLITS; ++i) add4(s, partial[(long long)i * psk::P_VEC4 + col]);
  float4 t = theta_in[col];
  t.x = fmaf(-coef, s.x, t.x); t.y = fmaf(-coef, s.y, t.y);
  t.z = fmaf(-coef, s.z, t.z); t.w = fmaf(-coef, s.w, t.w);
  theta_out[col] = t;
}

int32_t static_fail(int32_t code, const char* msg, const char* detail = "") {
  snprintf(g_static_err, sizeof(g_static_err), "%s%s", msg, detail);
  return code;
}

}  // namespace

extern "C" {

const char* ps_replay_sum_static_error(void) { return g_static_err; }

int32_t ps_replay_sum_static(const float* queue_dev, int64_t K, const float* theta_in_dev,
                             float* theta_out_dev, float coef, void* stream) {
  if (!queue_dev || !theta_in_dev || !theta_out_dev) return static_fail(PS_ERR_BAD_ARG, "NULL pointer");
  if (K < 1 || K > PS_STATIC_REPLAY_MAX_GRADIENTS)
    return static_fail(PS_ERR_BAD_ARG, "K is outside 1..PS_STATIC_REPLAY_MAX_GRADIENTS (65536); "
                                       "split the queue into several calls");
  if ((((uintptr_t)queue_dev | (uintptr_t)theta_in_dev | (uintptr_t)theta_out_dev) & 15) != 0)
    return static_fail(PS_ERR_BAD_ARG, "pointers must be 16-byte aligned");
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return static_fail(PS_ERR_CUDA, "cudaGetDevice: ", cudaGetErrorString(e));
  if (dev < 0 || dev >= MAX_DEVICES) return static_fail(PS_ERR_BAD_ARG, "device ordinal above 63");
  float* partials = nullptr;
  {
    // First call on this device: resolve the device address of the static array.
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_partials_addr[dev]) {
      void* p = nullptr;
      // With lazy module loading (the CUDA 12 default) this lookup is what brings the array into being on this
      // device: the driver reserves its 13 MB now.  A device whose memory is already taken fails here, not later.
      e = cudaGetSymbolAddress(&p, g_static_partials);
      if (e == cudaErrorMemoryAllocation) {
        cudaGetLastError();
        return static_fail(PS_ERR_CUDA, "the first call on this device could not place the library's 13 MB scratch array: "
                                        "the device is out of memory.  Make one warm-up call at start-up, before the "
                                        "application's pool takes the memory");
      }
      if (e != cudaSuccess) return static_fail(PS_ERR_CUDA, "cudaGetSymbolAddress: ", cudaGetErrorString(e));
      g_partials_addr[dev] = static_cast<float*>(p);
    }
    partials = g_partials_addr[dev];
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  static_partial<<<dim3(COL_BLOCKS, SPLITS), TPB, 0, st>>>(reinterpret_cast<const float4*>(queue_dev), (long long)K,
                                                          reinterpret_cast<float4*>(partials));
  static_finish<<<COL_BLOCKS, TPB, 0, st>>>(reinterpret_cast<const float4*>(partials),
                                            reinterpret_cast<const float4*>(theta_in_dev),
                                            reinterpret_cast<float4*>(theta_out_dev), coef);
  e = cudaGetLastError();
  if (e != cudaSuccess) return static_fail(PS_ERR_CUDA, "kernel launch: ", cudaGetErrorString(e));
  return PS_OK;
}

}  // extern "C"
