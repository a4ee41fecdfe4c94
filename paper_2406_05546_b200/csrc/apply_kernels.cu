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

__device__ __forceinline__ void fma4(float c, const float4& v, float4& a) {
  a.x = fmaf(c, v.x, a.x); a.y = fmaf(c, v.y, a.y); a.z = fmaf(c, v.z, a.z); a.w = fmaf(c, v.w, a.w);
}

// Sum of slots [k0, k1) of one float4 column, in a fixed order: eight interleaved running sums
// (slot k goes to sum k mod 8 relative to k0), combined pairwise at the end.  With WEIGHTED every slot is
// multiplied by its own factor coef_k[k] (the stale-gradient treatments) as it is added.
template <bool WEIGHTED>
__device__ __forceinline__ float4 column_sum(const float4* __restrict__ q, int64_t k0, int64_t k1, const float* __restrict__ coef_k) {
  float4 acc[8];
#pragma unroll
  for (int u = 0; u < 8; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
  int64_t k = k0;
  for (; k + 8 <= k1; k += 8) {
    float4 v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) v[u] = ld_stream(q + (k + u) * (int64_t)P_VEC4);
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      if (WEIGHTED) fma4(coef_k[k + u], v[u], acc[u]);
      else add4(acc[u], v[u]);
    }
  }
#pragma unroll
  for (int u = 0; u < 7; ++u)
    if (k + u < k1) {
      const float4 v = ld_stream(q + (k + u) * (int64_t)P_VEC4);
      if (WEIGHTED) fma4(coef_k[k + u], v, acc[u]);
      else add4(acc[u], v);
    }
  add4(acc[0], acc[1]); add4(acc[2], acc[3]); add4(acc[4], acc[5]); add4(acc[6], acc[7]);
  add4(acc[0], acc[2]); add4(acc[4], acc[6]);
  add4(acc[0], acc[4]);
  return acc[0];
}

// theta_out = theta_in - coef * sum_k g_k (or - sum_k coef_k[k] g_k), whole queue in one pass (small K).
template <bool WEIGHTED>
__global__ void __launch_bounds__(TPB) sum_apply_direct(const float4* __restrict__ queue, int64_t K,
                                                        const float4* theta_in, float4* theta_out,
                                                        float4* __restrict__ replica, float coef, const float* __restrict__ coef_k) {
  // theta_in and theta_out may be the same buffer (a ring of depth one): each thread reads its column before it
  // writes it, and the two pointers carry no no-alias promise
  int col = blockIdx.x * TPB + threadIdx.x;
  if (col >= P_VEC4) return;
  float4 s = column_sum<WEIGHTED>(queue + col, 0, K, coef_k);
  float4 t = theta_in[col];
  t.x = fmaf(-coef, s.x, t.x); t.y = fmaf(-coef, s.y, t.y);
  t.z = fmaf(-coef, s.z, t.z); t.w = fmaf(-coef, s.w, t.w);
  theta_out[col] = t;
  if (replica) replica[col] = t;
}

// Stage 1 of the long-queue reduction: block (x, y) sums slot range y of column block x.
template <bool WEIGHTED>
__global__ void __launch_bounds__(TPB) sum_partial(const float4* __restrict__ queue, int64_t K,
                                                   int n_split, float4* __restrict__ partial, const float* __restrict__ coef_k) {
  int col = blockIdx.x * TPB + threadIdx.x;
  if (col >= P_VEC4) return;
  int s = blockIdx.y;
  int64_t per = (K + n_split - 1) / n_split;
  int64_t k0 = s * per, k1 = k0 + per < K ? k0 + per : K;
  float4 acc = k0 < k1 ? column_sum<WEIGHTED>(queue + col, k0, k1, coef_k) : make_float4(0.f, 0.f, 0.f, 0.f);
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
        const float c = a.coef_k ? a.coef_k[ord.slot[k]] : a.coef;
        t.x = fmaf(-c, g[u].x, t.x); t.y = fmaf(-c, g[u].y, t.y);
        t.z = fmaf(-c, g[u].z, t.z); t.w = fmaf(-c, g[u].w, t.w);
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

// ---- clipping by global norm ------------------------------------------------------------------------------------
// Block (c, k) sums the squares of chunk c of gradient k: every thread over its float4 columns in four interleaved
// sums, then lanes and warps in a fixed order.
constexpr int NORM_VEC = P_VEC4 / NORM_CHUNKS;      // 25,416 float4 columns per chunk
static_assert(NORM_VEC * NORM_CHUNKS == P_VEC4, "chunks tile the vector");
__global__ void __launch_bounds__(TPB) sq_norm_partial(const float4* __restrict__ queue, float* __restrict__ norm_part) {
  __shared__ float warp_sum[TPB / 32];
  const int64_t k = blockIdx.y;
  const float4* g = queue + k * (int64_t)P_VEC4 + (int64_t)blockIdx.x * NORM_VEC;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  int i = threadIdx.x;
  for (; i + 3 * TPB < NORM_VEC; i += 4 * TPB) {
    float4 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) v[u] = g[i + u * TPB];
#pragma unroll
    for (int u = 0; u < 4; ++u) acc[u] = fmaf(v[u].x, v[u].x, fmaf(v[u].y, v[u].y, fmaf(v[u].z, v[u].z, fmaf(v[u].w, v[u].w, acc[u]))));
  }
  for (; i < NORM_VEC; i += TPB) {
    const float4 v = g[i];
    acc[0] = fmaf(v.x, v.x, fmaf(v.y, v.y, fmaf(v.z, v.z, fmaf(v.w, v.w, acc[0]))));
  }
  float t = (acc[0] + acc[1]) + (acc[2] + acc[3]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
  if ((threadIdx.x & 31) == 0) warp_sum[threadIdx.x >> 5] = t;
  __syncthreads();
  if (threadIdx.x == 0) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < TPB / 32; ++w) s += warp_sum[w];
    norm_part[k * NORM_CHUNKS + blockIdx.x] = s;
  }
}

__global__ void __launch_bounds__(TPB) clip_coef_finish(const float* __restrict__ norm_part, int64_t K, float clip, float* __restrict__ coef_k) {
  const int64_t k = (int64_t)blockIdx.x * TPB + threadIdx.x;
  if (k >= K) return;
  float n2 = 0.f;
#pragma unroll
  for (int c = 0; c < NORM_CHUNKS; ++c) n2 += norm_part[k * NORM_CHUNKS + c];
  coef_k[k] *= fminf(1.0f, clip / sqrtf(n2));      // a zero gradient keeps its factor (clip / 0 = inf)
}

}  // namespace

#define TIMED(id, launch) do { if (prof) prof->begin(id, st); launch; if (prof) prof->end(st); } while (0)

const char* kernel_name(int id) {
  static const char* names[K_COUNT] = {
      "conv1_fwd", "conv2_fwd", "fc1_fwd", "fc2_fwd_bwd", "fc1_dw", "fc1_dx", "conv2_bwd", "conv1_bwd",
      "conv_grad_reduce", "sum_apply_direct", "sum_partial", "sum_finish", "async_apply", "copy_rows",
      "dropout_mask", "conv2_dw", "prep_w1", "sq_norm_partial", "clip_coef_finish", "eval_finish"};
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
  const float* ck = a.coef_k;
  const float coef = ck ? 1.0f : a.coef;      // the per-gradient factors already carry the learning rate
  if (n_split <= 1) {
    if (ck) TIMED(K_SUM_APPLY_DIRECT, (sum_apply_direct<true><<<COL_BLOCKS, TPB, 0, st>>>(q, a.K, tin, tout, rep, coef, ck)));
    else TIMED(K_SUM_APPLY_DIRECT, (sum_apply_direct<false><<<COL_BLOCKS, TPB, 0, st>>>(q, a.K, tin, tout, rep, coef, nullptr)));
    launches = 1;
  } else {
    float4* part = reinterpret_cast<float4*>(a.partial);
    if (ck) TIMED(K_SUM_PARTIAL, (sum_partial<true><<<dim3(COL_BLOCKS, n_split), TPB, 0, st>>>(q, a.K, n_split, part, ck)));
    else TIMED(K_SUM_PARTIAL, (sum_partial<false><<<dim3(COL_BLOCKS, n_split), TPB, 0, st>>>(q, a.K, n_split, part, nullptr)));
    TIMED(K_SUM_FINISH, (sum_finish<<<COL_BLOCKS, TPB, 0, st>>>(part, n_split, tin, tout, rep, coef)));
    launches = 2;
  }
  return cudaGetLastError() == cudaSuccess ? launches : -1;
}

int launch_clip_factors(const float* queue, int64_t K, float clip, float* coef_k, float* norm_part, cudaStream_t st, Profiler* prof) {
  TIMED(K_SQ_NORM, (sq_norm_partial<<<dim3(NORM_CHUNKS, (unsigned)K), TPB, 0, st>>>(reinterpret_cast<const float4*>(queue), norm_part)));
  TIMED(K_COEF_FINISH, (clip_coef_finish<<<(unsigned)((K + TPB - 1) / TPB), TPB, 0, st>>>(norm_part, K, clip, coef_k)));
  return cudaGetLastError() == cudaSuccess ? 2 : -1;
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
