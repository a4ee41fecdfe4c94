// Tensor-core (TF32) versions of the dense contractions of the worker gradient step: the three
// products of the 512-unit dense layer (forward, input gradient, per-worker weight gradient) and
// the second convolution as an implicit product (forward, input gradient, filter gradient).
// Operands stay fp32 in memory and are rounded to TF32 (10-bit mantissa, round to nearest) when
// the fragments are built; accumulation is fp32.  Everything else of the step (first convolution,
// output layer, softmax, pooling decisions, dropout) is shared with the FP32 path.
//
// Reductions keep a fixed order, so results are reproducible bit for bit.
#include "device_common.cuh"
#include "kernels.h"

namespace psk {

namespace {

__device__ __forceinline__ uint32_t to_tf32(float x) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
  return r;
}

// D += A(16x8, row) * B(8x8, col), TF32 inputs, fp32 accumulate.  Lane = 4*g + t:
//   a0 (g, t)  a1 (g+8, t)  a2 (g, t+4)  a3 (g+8, t+4);  b0 (k=t, n=g)  b1 (k=t+4, n=g);
//   c0 (g, 2t) c1 (g, 2t+1) c2 (g+8, 2t) c3 (g+8, 2t+1).
__device__ __forceinline__ void mma_tf32(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  asm volatile(
      "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

__device__ __forceinline__ void cp_async16(float* smem_dst, const float* gmem_src, bool valid) {
  uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
  int bytes = valid ? 16 : 0;   // src-size 0: the 16 bytes are zero-filled, nothing is read
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(gmem_src), "r"(bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N)); }

// ------------------------------------------------------------------------------------------------
// 128 x 128 x 32 tiled product, 256 threads (8 warps as 2 x 4, warp tile 64 x 32), three-stage
// cp.async pipeline.  Operand layouts in global memory:
//   A_KC: A(m,k) = A[m*lda + k]   else A(m,k) = A[k*lda + m]
//   B_KC: B(k,n) = B[n*ldb + k]   else B(k,n) = B[k*ldb + n]
// Rows m in [m0, m_end), columns n in [n0, N), k in [0, K) are valid; everything else reads as 0.
// All leading dimensions, N and (for the m-contiguous form) m_end are multiples of 4.
// ------------------------------------------------------------------------------------------------
constexpr int GM = 128, GN = 128, GK = 32, G_STAGES = 3;
constexpr int KC_STRIDE = GK + 4;     // row of 32 k-values, padded: fragment loads hit 32 distinct banks
constexpr int MC_STRIDE = GM + 8;     // row of 128 m-values, padded likewise
constexpr int OPERAND_FLOATS = GM * KC_STRIDE;   // 4608 >= 32 * 136
constexpr int GEMM_SMEM_BYTES = G_STAGES * 2 * OPERAND_FLOATS * 4;

template <bool KC>
__device__ __forceinline__ void load_operand(float* dst, const float* __restrict__ src, int ld, int r0, int r_end,
                                             int k0, int K) {
  const int tid = threadIdx.x;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int c = tid + 256 * i;
    if (KC) {
      int r = c >> 3, kc = (c & 7) * 4;
      bool ok = (r0 + r < r_end) && (k0 + kc < K);
      const float* g = ok ? src + (int64_t)(r0 + r) * ld + k0 + kc : src;
      cp_async16(dst + r * KC_STRIDE + kc, g, ok);
    } else {
      int k = c >> 5, rc = (c & 31) * 4;
      bool ok = (k0 + k < K) && (r0 + rc < r_end);
      const float* g = ok ? src + (int64_t)(k0 + k) * ld + r0 + rc : src;
      cp_async16(dst + k * MC_STRIDE + rc, g, ok);
    }
  }
}

template <bool A_KC, bool B_KC>
__device__ __forceinline__ void gemm_tile_tf32(const float* __restrict__ A, int lda, const float* __restrict__ B,
                                               int ldb, int m0, int m_end, int n0, int N, int K,
                                               float (&acc)[4][4][4]) {
  extern __shared__ __align__(16) float smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int wm = (warp >> 2) * 64, wn = (warp & 3) * 32;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int r = 0; r < 4; ++r) acc[i][j][r] = 0.f;
  const int n_k = (K + GK - 1) / GK;
  auto stage_a = [&](int s) { return smem + (s * 2) * OPERAND_FLOATS; };
  auto stage_b = [&](int s) { return smem + (s * 2 + 1) * OPERAND_FLOATS; };
#pragma unroll
  for (int s = 0; s < G_STAGES - 1; ++s) {
    if (s < n_k) {
      load_operand<A_KC>(stage_a(s), A, lda, m0, m_end, s * GK, K);
      load_operand<B_KC>(stage_b(s), B, ldb, n0, N, s * GK, K);
    }
    cp_async_commit();
  }
  for (int kt = 0; kt < n_k; ++kt) {
    cp_async_wait<G_STAGES - 2>();
    __syncthreads();
    {
      int nxt = kt + G_STAGES - 1;
      if (nxt < n_k) {
        load_operand<A_KC>(stage_a(nxt % G_STAGES), A, lda, m0, m_end, nxt * GK, K);
        load_operand<B_KC>(stage_b(nxt % G_STAGES), B, ldb, n0, N, nxt * GK, K);
      }
      cp_async_commit();
    }
    const float* As = stage_a(kt % G_STAGES);
    const float* Bs = stage_b(kt % G_STAGES);
#pragma unroll
    for (int kk = 0; kk < GK; kk += 8) {
      uint32_t af[4][4], bf[4][2];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        int m = wm + i * 16 + g;
        if (A_KC) {
          af[i][0] = to_tf32(As[m * KC_STRIDE + kk + t]);
          af[i][1] = to_tf32(As[(m + 8) * KC_STRIDE + kk + t]);
          af[i][2] = to_tf32(As[m * KC_STRIDE + kk + t + 4]);
          af[i][3] = to_tf32(As[(m + 8) * KC_STRIDE + kk + t + 4]);
        } else {
          af[i][0] = to_tf32(As[(kk + t) * MC_STRIDE + m]);
          af[i][1] = to_tf32(As[(kk + t) * MC_STRIDE + m + 8]);
          af[i][2] = to_tf32(As[(kk + t + 4) * MC_STRIDE + m]);
          af[i][3] = to_tf32(As[(kk + t + 4) * MC_STRIDE + m + 8]);
        }
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        int n = wn + j * 8 + g;
        if (B_KC) {
          bf[j][0] = to_tf32(Bs[n * KC_STRIDE + kk + t]);
          bf[j][1] = to_tf32(Bs[n * KC_STRIDE + kk + t + 4]);
        } else {
          bf[j][0] = to_tf32(Bs[(kk + t) * MC_STRIDE + n]);
          bf[j][1] = to_tf32(Bs[(kk + t + 4) * MC_STRIDE + n]);
        }
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) mma_tf32(acc[i][j], af[i], bf[j]);
    }
  }
  cp_async_wait<0>();
}

// ---- fc1 forward: d = dropout(ReLU(p2 * W1^T + b1)), one product per weight group.
__global__ void __launch_bounds__(256) fc1_fwd_tc(GradStepArgs a, WorkerTable wt, GroupTable gt, Workspace ws) {
  int grp, m0, m_end;
  if (!locate_group_tile<GM>(gt, a.b, blockIdx.y, grp, m0, m_end)) return;
  const float* theta = gt.theta[grp];
  const int n0 = blockIdx.x * GN;
  float acc[4][4][4];
  gemm_tile_tf32<true, true>(ws.p2, FLAT, theta + OFF_F1W, FLAT, m0, m_end, n0, HID, FLAT, acc);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, t = lane & 3;
  const int wm = (warp >> 2) * 64, wn = (warp & 3) * 32;
  const float scale = 1.0f / (1.0f - a.drop_p);
  const uint2 key = make_uint2((uint32_t)a.seed, (uint32_t)(a.seed >> 32));
  const uint32_t step_lo = (uint32_t)a.step, step_hi = (uint32_t)(a.step >> 32);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    // this lane draws the Philox quad of one of its two rows and trades halves with its neighbour:
    // even t covers row g (words 0,1 are its own columns), odd t covers row g+8 (words 2,3)
    const int r_lo = m0 + wm + i * 16 + g, r_hi = r_lo + 8;
    const int my_row = (t & 1) ? r_hi : r_lo;
    const bool row_ok = my_row < m_end;
    const int s = row_ok ? my_row / a.b : 0;
    const int smp = my_row - s * a.b;
    const uint32_t wid = (uint32_t)wt.wid[s];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + wn + j * 8 + 2 * t;          // this lane's two columns: n, n+1
      const int quad_col = n & ~3;
      uint4 rnd = make_uint4(0, 0, 0, 0);
      if (row_ok)
        rnd = philox4x32_10(make_uint4((uint32_t)((smp * HID + quad_col) >> 2), wid, step_lo, step_hi), key);
      // even t: keeps (x,y) for row g, sends (z,w) to t+1; odd t: keeps (z,w) for row g+8, sends (x,y) to t-1
      uint32_t send0 = (t & 1) ? rnd.x : rnd.z, send1 = (t & 1) ? rnd.y : rnd.w;
      uint32_t got0 = __shfl_xor_sync(0xffffffffu, send0, 1), got1 = __shfl_xor_sync(0xffffffffu, send1, 1);
      uint32_t lo0, lo1, hi0, hi1;   // words for (row g: cols n, n+1) and (row g+8: cols n, n+1)
      if (t & 1) { lo0 = got0; lo1 = got1; hi0 = rnd.z; hi1 = rnd.w; }
      else       { lo0 = rnd.x; lo1 = rnd.y; hi0 = got0; hi1 = got1; }
      const float2 bias = *reinterpret_cast<const float2*>(theta + OFF_F1B + n);
      if (r_lo < m_end) {
        float2 o;
        o.x = lo0 >= a.drop_thresh ? fmaxf(acc[i][j][0] + bias.x, 0.f) * scale : 0.f;
        o.y = lo1 >= a.drop_thresh ? fmaxf(acc[i][j][1] + bias.y, 0.f) * scale : 0.f;
        *reinterpret_cast<float2*>(ws.d + (int64_t)r_lo * HID + n) = o;
      }
      if (r_hi < m_end) {
        float2 o;
        o.x = hi0 >= a.drop_thresh ? fmaxf(acc[i][j][2] + bias.x, 0.f) * scale : 0.f;
        o.y = hi1 >= a.drop_thresh ? fmaxf(acc[i][j][3] + bias.y, 0.f) * scale : 0.f;
        *reinterpret_cast<float2*>(ws.d + (int64_t)r_hi * HID + n) = o;
      }
    }
  }
}

__device__ __forceinline__ void store_tile(const float (&acc)[4][4][4], float* __restrict__ C, int ldc, int m0,
                                           int m_end, int n0, int N) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, t = lane & 3;
  const int wm = (warp >> 2) * 64, wn = (warp & 3) * 32;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r_lo = m0 + wm + i * 16 + g, r_hi = r_lo + 8;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + wn + j * 8 + 2 * t;
      if (n >= N) continue;
      if (r_lo < m_end) *reinterpret_cast<float2*>(C + (int64_t)r_lo * ldc + n) = make_float2(acc[i][j][0], acc[i][j][1]);
      if (r_hi < m_end) *reinterpret_cast<float2*>(C + (int64_t)r_hi * ldc + n) = make_float2(acc[i][j][2], acc[i][j][3]);
    }
  }
}

// ---- gradient with respect to p2: dp2 [rows][1568] = da1 [rows][512] * W1 [512][1568], per group.
__global__ void __launch_bounds__(256) fc1_dx_tc(GradStepArgs a, GroupTable gt, Workspace ws) {
  int grp, m0, m_end;
  if (!locate_group_tile<GM>(gt, a.b, blockIdx.y, grp, m0, m_end)) return;
  const int n0 = blockIdx.x * GN;
  float acc[4][4][4];
  gemm_tile_tf32<true, false>(ws.da1, HID, gt.theta[grp] + OFF_F1W, FLAT, m0, m_end, n0, FLAT, HID, acc);
  store_tile(acc, ws.dp2, FLAT, m0, m_end, n0, FLAT);
}

// ---- fc1 weight gradient of one worker: dW1 [512][1568] = da1^T [512 x b] * p2 [b x 1568].
__global__ void __launch_bounds__(256) fc1_dw_tc(GradStepArgs a, WorkerTable wt, Workspace ws) {
  const int s = blockIdx.z, m0 = blockIdx.y * GM, n0 = blockIdx.x * GN;
  const float* A = ws.da1 + (int64_t)s * a.b * HID;
  const float* B = ws.p2 + (int64_t)s * a.b * FLAT;
  float acc[4][4][4];
  gemm_tile_tf32<false, false>(A, HID, B, FLAT, m0, HID, n0, FLAT, a.b, acc);
  store_tile(acc, wt.grad[s] + OFF_F1W, FLAT, m0, HID, n0, FLAT);
}

}  // namespace

#define TIMED(id, launch) do { if (prof) prof->begin(id, st); launch; if (prof) prof->end(st); } while (0)

int configure_tc_kernels() {
  cudaError_t e = cudaFuncSetAttribute(fc1_fwd_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM_BYTES);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(fc1_dx_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM_BYTES);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(fc1_dw_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM_BYTES);
  return e == cudaSuccess ? 0 : -1;
}

void launch_fc1_fwd_tc(const GradStepArgs& a, const WorkerTable& wt, const GroupTable& gt, const Workspace& ws,
                       cudaStream_t st, Profiler* prof) {
  const int mt = group_tiles(gt, a.b, GM);
  TIMED(K_FC1_FWD, (fc1_fwd_tc<<<dim3(HID / GN, mt), 256, GEMM_SMEM_BYTES, st>>>(a, wt, gt, ws)));
}

void launch_fc1_dx_tc(const GradStepArgs& a, const GroupTable& gt, const Workspace& ws, cudaStream_t st,
                      Profiler* prof) {
  const int mt = group_tiles(gt, a.b, GM);
  TIMED(K_FC1_DX, (fc1_dx_tc<<<dim3((FLAT + GN - 1) / GN, mt), 256, GEMM_SMEM_BYTES, st>>>(a, gt, ws)));
}

void launch_fc1_dw_tc(const GradStepArgs& a, const WorkerTable& wt, const Workspace& ws, cudaStream_t st,
                      Profiler* prof) {
  TIMED(K_FC1_DW, (fc1_dw_tc<<<dim3((FLAT + GN - 1) / GN, HID / GM, a.W), 256, GEMM_SMEM_BYTES, st>>>(a, wt, ws)));
}

}  // namespace psk
