// Server-side kernels: reduce the gradient queue and apply it to the weights.
//
// All three server steps of the paper are elementwise over the parameter vector and stream the
// queue exactly once, so they are bound by HBM bandwidth: per queued gradient 4*P_PAD bytes are
// read, and per step the weights are read once and written once (plus once more for the
// chain-replication mirror).  Threads own float4 columns of the parameter vector, so every load
// and store is a coalesced 16-byte access; the K loop is unrolled to keep many independent loads
// in flight per thread.
#include "kernels.h"

namespace psk {

namespace {

constexpr int TPB = 256;
constexpr int COL_BLOCKS = (P_VEC4 + TPB - 1) / TPB;   // 795

__device__ __forceinline__ float4 ld_stream(const float4* p) { return __ldcs(p); }

__device__ __forceinline__ void add4(float4& a, const float4& b) {
  a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
}

// Sum of slots [k0, k1) of one float4 column, in a fixed order: eight interleaved running sums
// (slot k goes to sum k mod 8 relative to k0), combined pairwise at the end.
__device__ __forceinline__ float4 column_sum(const float4* __restrict__ q, int64_t k0, int64_t k1) {
  float4 acc[8];
#pragma unroll
  for (int u = 0; u < 8; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
  int64_t k = k0;
  for (; k + 8 <= k1; k += 8) {
    float4 v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) v[u] = ld_stream(q + (k + u) * (int64_t)P_VEC4);
#pragma unroll
    for (int u = 0; u < 8; ++u) add4(acc[u], v[u]);
  }
#pragma unroll
  for (int u = 0; u < 7; ++u)
    if (k + u < k1) add4(acc[u], ld_stream(q + (k + u) * (int64_t)P_VEC4));
  add4(acc[0], acc[1]); add4(acc[2], acc[3]); add4(acc[4], acc[5]); add4(acc[6], acc[7]);
  add4(acc[0], acc[2]); add4(acc[4], acc[6]);
  add4(acc[0], acc[4]);
  return acc[0];
}

// theta_out = theta_in - coef * sum_k g_k, whole queue in one pass (small K).
__global__ void __launch_bounds__(TPB) sum_apply_direct(const float4* __restrict__ queue, int64_t K,
                                                        const float4* theta_in, float4* theta_out,
                                                        float4* __restrict__ replica, float coef) {
  // theta_in and theta_out may be the same buffer (a ring of depth one): each thread reads its column before it
  // writes it, and the two pointers carry no no-alias promise
  int col = blockIdx.x * TPB + threadIdx.x;
  if (col >= P_VEC4) return;
  float4 s = column_sum(queue + col, 0, K);
  float4 t = theta_in[col];
  t.x = fmaf(-coef, s.x, t.x); t.y = fmaf(-coef, s.y, t.y);
  t.z = fmaf(-coef, s.z, t.z); t.w = fmaf(-coef, s.w, t.w);
  theta_out[col] = t;
  if (replica) replica[col] = t;
}

// Stage 1 of the long-queue reduction: block (x, y) sums slot range y of column block x.
__global__ void __launch_bounds__(TPB) sum_partial(const float4* __restrict__ queue, int64_t K,
                                                   int n_split, float4* __restrict__ partial) {
  int col = blockIdx.x * TPB + threadIdx.x;
  if (col >= P_VEC4) return;
  int s = blockIdx.y;
  int64_t per = (K + n_split - 1) / n_split;
  int64_t k0 = s * per, k1 = k0 + per < K ? k0 + per : K;
  float4 acc = k0 < k1 ? column_sum(queue + col, k0, k1) : make_float4(0.f, 0.f, 0.f, 0.f);
  partial[(int64_t)s * P_VEC4 + col] = acc;
}

// Stage 2: sums the partials in slot order and applies the update.
__global__ void __launch_bounds__(TPB) sum_finish(const float4* __restrict__ partial, int n_split,
                                                  const float4* theta_in, float4* theta_out,   // may alias (see above)
                                                  float4* __restrict__ replica, float coef) {
  int col = blockIdx.x * TPB + threadIdx.x;
  if (col >= P_VEC4) return;
  float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int i = 0; i < n_split; ++i) add4(s, partial[(int64_t)i * P_VEC4 + col]);
  float4 t = theta_in[col];
  t.x = fmaf(-coef, s.x, t.x); t.y = fmaf(-coef, s.y, t.y);
  t.z = fmaf(-coef, s.z, t.z); t.w = fmaf(-coef, s.w, t.w);
  theta_out[col] = t;
  if (replica) replica[col] = t;
}

// Ordered one-by-one application: each thread keeps its float4 of the weights in registers,
// subtracts the gradients in arrival order (the same sequence of roundings as K separate
// updates), and stores only the versions that stay readable: the last ring_depth ones.
__global__ void __launch_bounds__(TPB) async_apply(AsyncApplyArgs a, AsyncOrder ord) {
  int col = blockIdx.x * TPB + threadIdx.x;
  if (col >= P_VEC4) return;
  const float4* q = reinterpret_cast<const float4*>(a.queue) + col;
  float4 t = reinterpret_cast<const float4*>(a.theta_in)[col];
  constexpr int U = 8;
  for (int k0 = 0; k0 < a.K; k0 += U) {
    float4 g[U];
#pragma unroll
    for (int u = 0; u < U; ++u)
      if (k0 + u < a.K) g[u] = ld_stream(q + (int64_t)ord.slot[k0 + u] * P_VEC4);
#pragma unroll
    for (int u = 0; u < U; ++u) {
      int k = k0 + u;
      if (k < a.K) {
        t.x = fmaf(-a.coef, g[u].x, t.x); t.y = fmaf(-a.coef, g[u].y, t.y);
        t.z = fmaf(-a.coef, g[u].z, t.z); t.w = fmaf(-a.coef, g[u].w, t.w);
        if (k >= a.first_stored) {
          int slot = (int)((a.v0 + (uint64_t)k + 1) % (uint64_t)a.ring_depth);
          reinterpret_cast<float4*>(a.ring[slot])[col] = t;
        }
        for (int m = 0; m < a.n_mirror; ++m)
          if (k == a.mirror_k[m]) reinterpret_cast<float4*>(a.replica[m])[col] = t;
      }
    }
  }
}

// Copies rows of P_PAD floats; used for the copying form of enqueue.
__global__ void __launch_bounds__(TPB) copy_rows(float4* __restrict__ dst, const float4* __restrict__ src,
                                                 int64_t n_vec) {
  int64_t i = (int64_t)blockIdx.x * TPB + threadIdx.x;
  int64_t stride = (int64_t)gridDim.x * TPB;
  for (; i < n_vec; i += stride) dst[i] = src[i];
}

}  // namespace

#define TIMED(id, launch) do { if (prof) prof->begin(id, st); launch; if (prof) prof->end(st); } while (0)

const char* kernel_name(int id) {
  static const char* names[K_COUNT] = {
      "conv1_fwd", "conv2_fwd", "fc1_fwd", "fc2_fwd_bwd", "fc1_dw", "fc1_dx", "conv2_bwd", "conv1_bwd",
      "conv_grad_reduce", "sum_apply_direct", "sum_partial", "sum_finish", "async_apply", "copy_rows",
      "dropout_mask", "conv2_dw", "prep_w1"};
  return id >= 0 && id < K_COUNT ? names[id] : "?";
}

int launch_sum_apply(const SumApplyArgs& a, cudaStream_t st, Profiler* prof) {
  const float4* q = reinterpret_cast<const float4*>(a.queue);
  const float4* tin = reinterpret_cast<const float4*>(a.theta_in);
  float4* tout = reinterpret_cast<float4*>(a.theta_out);
  float4* rep = reinterpret_cast<float4*>(a.replica);
  int n_split = 1;
  if (a.K > 160 && a.max_split > 1) {
    int64_t want = (a.K + 31) / 32;
    n_split = (int)(want < a.max_split ? want : a.max_split);
  }
  int launches = 0;
  if (n_split <= 1) {
    TIMED(K_SUM_APPLY_DIRECT, (sum_apply_direct<<<COL_BLOCKS, TPB, 0, st>>>(q, a.K, tin, tout, rep, a.coef)));
    launches = 1;
  } else {
    float4* part = reinterpret_cast<float4*>(a.partial);
    TIMED(K_SUM_PARTIAL, (sum_partial<<<dim3(COL_BLOCKS, n_split), TPB, 0, st>>>(q, a.K, n_split, part)));
    TIMED(K_SUM_FINISH, (sum_finish<<<COL_BLOCKS, TPB, 0, st>>>(part, n_split, tin, tout, rep, a.coef)));
    launches = 2;
  }
  return cudaGetLastError() == cudaSuccess ? launches : -1;
}

int launch_async_apply(const AsyncApplyArgs& a, const AsyncOrder& ord, cudaStream_t st, Profiler* prof) {
  TIMED(K_ASYNC_APPLY, (async_apply<<<COL_BLOCKS, TPB, 0, st>>>(a, ord)));
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int launch_copy_rows(float* dst, const float* src, int64_t rows, cudaStream_t st, Profiler* prof) {
  int64_t n_vec = rows * P_VEC4;
  int64_t blocks = (n_vec + TPB - 1) / TPB;
  if (blocks > 148 * 16) blocks = 148 * 16;
  TIMED(K_COPY_ROWS, (copy_rows<<<(int)blocks, TPB, 0, st>>>(reinterpret_cast<float4*>(dst),
                                                            reinterpret_cast<const float4*>(src), n_vec)));
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace psk
