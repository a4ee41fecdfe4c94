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

// ------------------------------------------------------------------------------------------------
// Second convolution (16 -> 32 channels, 3x3, pad 1) as implicit products on 14x14 maps.
// Every block handles up to TC_SPB samples of one worker and keeps the (TF32-rounded) filter bank
// in shared memory.  The reduction index is ordered tap-major: k = tap*C + channel, so that one
// 8-wide k-step covers eight channels at one filter tap and a fragment element is one shared-memory
// word of a zero-bordered image plane.
// ------------------------------------------------------------------------------------------------
constexpr int TC_SPB = 8;
constexpr int FWD_PLANE = 264;   // 16 x 16 words + 8: plane stride = 8 (mod 32 banks)

__device__ __forceinline__ float tf32f(float x) { return __uint_as_float(to_tf32(x)); }

// Forward + ReLU + 2x2 max pool.  224 threads = 7 warps; warp w owns pooled positions 8w .. 8w+7
// (49 used of 56).  The product's rows are ordered so that the four pre-pool positions of a pooled
// element are rows g and g+8 of two 16-row tiles, i.e. they all land in one thread's accumulators and
// the pooling decision needs no exchange.  Image planes are stored with even and odd columns apart
// (offset = Y*16 + (X&1)*8 + X/2), which makes the eight positions a fragment load touches consecutive.
__global__ void __launch_bounds__(224) conv2_fwd_tc(GradStepArgs a, WorkerTable wt, GroupTable gt, Workspace ws) {
  __shared__ float Wk[144 * 40];          // [k = tap*16 + ic][oc], row stride 40
  __shared__ float bias[32];
  __shared__ float img[16 * FWD_PLANE];
  const int s = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  const float* theta = group_theta(wt, gt, s);
  for (int idx = tid; idx < 4608; idx += 224) {
    int oc = idx / 144, rem = idx - oc * 144, ic = rem / 9, tap = rem - ic * 9;
    Wk[(tap * 16 + ic) * 40 + oc] = tf32f(theta[OFF_C2W + idx]);
  }
  if (tid < 32) bias[tid] = theta[OFF_C2B + tid];
  for (int idx = tid; idx < 16 * FWD_PLANE; idx += 224) img[idx] = 0.f;
  const int pp = warp * 8 + g;
  const bool valid = pp < 49;
  const int ppc = valid ? pp : 48;
  const int py = ppc / 7, px = ppc - py * 7;
  const int base = (2 * py) * 16 + px;
  const int i0 = blockIdx.x * TC_SPB, i1 = min(i0 + TC_SPB, a.b);
  for (int i = i0; i < i1; ++i) {
    const int64_t row = (int64_t)s * a.b + i;
    __syncthreads();
    for (int idx = tid; idx < P1_ELEMS; idx += 224) {
      int ic = idx / 196, p = idx - ic * 196, y = p / 14, x = p - y * 14;
      int X = x + 1, Y = y + 1;
      img[ic * FWD_PLANE + Y * 16 + (X & 1) * 8 + (X >> 1)] = tf32f(ws.p1[row * P1_ELEMS + idx]);
    }
    __syncthreads();
    float acc[2][4][4];
#pragma unroll
    for (int m = 0; m < 2; ++m)
#pragma unroll
      for (int n = 0; n < 4; ++n)
#pragma unroll
        for (int r = 0; r < 4; ++r) acc[m][n][r] = 0.f;
#pragma unroll
    for (int tap = 0; tap < 9; ++tap) {
      const int ky = tap / 3, kx = tap - ky * 3;
      int off[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int jy = j >> 1, sx = (j & 1) + kx;
        off[j] = base + (jy + ky) * 16 + (sx & 1) * 8 + (sx >> 1);
      }
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const float* pa = img + (half * 8 + t) * FWD_PLANE;
        const float* pb = pa + 4 * FWD_PLANE;
        uint32_t fa[2][4], fb[4][2];
#pragma unroll
        for (int m = 0; m < 2; ++m) {
          fa[m][0] = __float_as_uint(pa[off[2 * m]]);
          fa[m][1] = __float_as_uint(pa[off[2 * m + 1]]);
          fa[m][2] = __float_as_uint(pb[off[2 * m]]);
          fa[m][3] = __float_as_uint(pb[off[2 * m + 1]]);
        }
        const float* wk = Wk + (tap * 16 + half * 8 + t) * 40 + g;
#pragma unroll
        for (int n = 0; n < 4; ++n) {
          fb[n][0] = __float_as_uint(wk[n * 8]);
          fb[n][1] = __float_as_uint(wk[4 * 40 + n * 8]);
        }
#pragma unroll
        for (int m = 0; m < 2; ++m)
#pragma unroll
          for (int n = 0; n < 4; ++n) mma_tf32(acc[m][n], fa[m], fb[n]);
      }
    }
    if (valid) {
#pragma unroll
      for (int n = 0; n < 4; ++n)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int oc = n * 8 + 2 * t + e;
          const float bv = bias[oc];
          // window elements j = 0..3: (tile 0 row g), (tile 0 row g+8), (tile 1 row g), (tile 1 row g+8)
          const float v[4] = {acc[0][n][e] + bv, acc[0][n][2 + e] + bv, acc[1][n][e] + bv, acc[1][n][2 + e] + bv};
          float best = 0.f;
          int bi = 0;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            float r = fmaxf(v[j], 0.f);
            if (j == 0 || r > best) { best = r; bi = j; }
          }
          ws.p2[row * FLAT + oc * 49 + pp] = tf32f(best);   // its only readers are TF32 products
          ws.code2[row * FLAT + oc * 49 + pp] = best > 0.f ? (uint8_t)bi : (uint8_t)4;
        }
    }
  }
}

// Gradient with respect to the convolution's input: dp1[ic][pos] = sum_{tap,oc} g2[oc][pos - tap] * w[oc][ic][tap],
// rows = 196 positions (13 tiles of 16), 16 columns, k = tap*32 + oc (36 k-steps).  224 threads = 7 warps;
// warp w owns row tiles w and w+7.  g2 is the gradient at the convolution's output, scattered from the
// pooled gradient by the stored pooling decisions into zero-bordered 16x16 planes.
constexpr int DX_PLANE = 264;
constexpr int DX_SMEM_FLOATS = 288 * 24 + 32 * DX_PLANE;
__global__ void __launch_bounds__(224) conv2_dx_tc(GradStepArgs a, WorkerTable wt, GroupTable gt, Workspace ws) {
  extern __shared__ __align__(16) float smem[];
  float* Wk = smem;                 // [k = tap*32 + oc][ic], row stride 24
  float* g2 = smem + 288 * 24;      // [oc][Y][X]
  const int s = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  const float* theta = group_theta(wt, gt, s);
  for (int idx = tid; idx < 4608; idx += 224) {
    int oc = idx / 144, rem = idx - oc * 144, ic = rem / 9, tap = rem - ic * 9;
    Wk[(tap * 32 + oc) * 24 + ic] = tf32f(theta[OFF_C2W + idx]);
  }
  // this warp's two row tiles; positions beyond 195 are computed on clamped addresses and not stored
  int pos[2][2], offb[2][2];
  bool ok[2][2];
#pragma unroll
  for (int m = 0; m < 2; ++m)
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      int p = (warp + 7 * m) * 16 + g + 8 * h;
      ok[m][h] = p < 196;
      p = ok[m][h] ? p : 195;
      pos[m][h] = p;
      int y = p / 14, x = p - y * 14;
      offb[m][h] = (y + 2) * 16 + (x + 2);
    }
  const bool second = warp + 7 < 13;
  const int i0 = blockIdx.x * TC_SPB, i1 = min(i0 + TC_SPB, a.b);
  for (int i = i0; i < i1; ++i) {
    const int64_t row = (int64_t)s * a.b + i;
    __syncthreads();
    for (int idx = tid; idx < 32 * DX_PLANE / 4; idx += 224) reinterpret_cast<float4*>(g2)[idx] = make_float4(0.f, 0.f, 0.f, 0.f);
    __syncthreads();
    for (int o = tid; o < FLAT; o += 224) {
      int code = ws.code2[row * FLAT + o];
      if (code < 4) {
        int oc = o / 49, p = o - oc * 49, py = p / 7, px = p - py * 7;
        int y = 2 * py + (code >> 1), x = 2 * px + (code & 1);
        g2[oc * DX_PLANE + (y + 1) * 16 + x + 1] = tf32f(ws.dp2[row * FLAT + o]);
      }
    }
    __syncthreads();
    float acc[2][2][4];
#pragma unroll
    for (int m = 0; m < 2; ++m)
#pragma unroll
      for (int n = 0; n < 2; ++n)
#pragma unroll
        for (int r = 0; r < 4; ++r) acc[m][n][r] = 0.f;
#pragma unroll
    for (int tap = 0; tap < 9; ++tap) {
      const int ky = tap / 3, kx = tap - ky * 3;
      const int shift = ky * 16 + kx;        // g2 is read at (y - ky + 1, x - kx + 1) in bordered coordinates
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float* pa = g2 + (q * 8 + t) * DX_PLANE - shift;
        const float* pb = pa + 4 * DX_PLANE;
        uint32_t fa[2][4], fb[2][2];
#pragma unroll
        for (int m = 0; m < 2; ++m) {
          fa[m][0] = __float_as_uint(pa[offb[m][0]]);
          fa[m][1] = __float_as_uint(pa[offb[m][1]]);
          fa[m][2] = __float_as_uint(pb[offb[m][0]]);
          fa[m][3] = __float_as_uint(pb[offb[m][1]]);
        }
        const float* wk = Wk + (tap * 32 + q * 8 + t) * 24 + g;
#pragma unroll
        for (int n = 0; n < 2; ++n) {
          fb[n][0] = __float_as_uint(wk[n * 8]);
          fb[n][1] = __float_as_uint(wk[4 * 24 + n * 8]);
        }
#pragma unroll
        for (int n = 0; n < 2; ++n) {
          mma_tf32(acc[0][n], fa[0], fb[n]);
          if (second) mma_tf32(acc[1][n], fa[1], fb[n]);
        }
      }
    }
#pragma unroll
    for (int m = 0; m < 2; ++m) {
      if (m == 1 && !second) continue;
#pragma unroll
      for (int n = 0; n < 2; ++n) {
        const int ic = n * 8 + 2 * t;
        float* out = ws.dp1 + row * P1_ELEMS;
        if (ok[m][0]) { out[ic * 196 + pos[m][0]] = acc[m][n][0]; out[(ic + 1) * 196 + pos[m][0]] = acc[m][n][1]; }
        if (ok[m][1]) { out[ic * 196 + pos[m][1]] = acc[m][n][2]; out[(ic + 1) * 196 + pos[m][1]] = acc[m][n][3]; }
      }
    }
  }
}

// Filter gradient: dW[oc][ic][tap] = sum_{samples,pos} g2[oc][pos] * p1[ic][pos + tap]: rows = 32 output
// channels, columns = 16 input channels per tap, k = position (196 per sample, 25 k-steps, zero-padded).
// 288 threads = 9 warps, warp = filter tap; accumulators persist over the block's samples and are
// written once as the block's partial sum.  The bias gradient (sum of g2 over positions) is taken by
// eight threads per channel straight from the pooled gradient, combined in a fixed order.
constexpr int DW_G_STRIDE = 228;   // 196 positions + zeros; = 4 (mod 32 banks)
constexpr int DW_PLANE = 260;      // 16 x 16 + 4;            = 4 (mod 32 banks)
__global__ void __launch_bounds__(288) conv2_dw_tc(GradStepArgs a, WorkerTable wt, Workspace ws, int n_chunks) {
  __shared__ __align__(16) float g2[32 * DW_G_STRIDE];   // [oc][pos]
  __shared__ __align__(16) float img[16 * DW_PLANE];     // [ic][Y][X], zero border
  const int s = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  const int ky = warp / 3, kx = warp - ky * 3;
  for (int idx = tid; idx < 16 * DW_PLANE; idx += 288) img[idx] = 0.f;
  float acc[2][2][4];
#pragma unroll
  for (int m = 0; m < 2; ++m)
#pragma unroll
    for (int n = 0; n < 2; ++n)
#pragma unroll
      for (int r = 0; r < 4; ++r) acc[m][n][r] = 0.f;
  float gb = 0.f;
  const int i0 = blockIdx.x * TC_SPB, i1 = min(i0 + TC_SPB, a.b);
  for (int i = i0; i < i1; ++i) {
    const int64_t row = (int64_t)s * a.b + i;
    __syncthreads();
    for (int idx = tid; idx < 32 * DW_G_STRIDE / 4; idx += 288) reinterpret_cast<float4*>(g2)[idx] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int idx = tid; idx < P1_ELEMS; idx += 288) {
      int ic = idx / 196, p = idx - ic * 196, y = p / 14, x = p - y * 14;
      img[ic * DW_PLANE + (y + 1) * 16 + x + 1] = tf32f(ws.p1[row * P1_ELEMS + idx]);
    }
    __syncthreads();
    for (int o = tid; o < FLAT; o += 288) {
      int code = ws.code2[row * FLAT + o];
      if (code < 4) {
        int oc = o / 49, p = o - oc * 49, py = p / 7, px = p - py * 7;
        int y = 2 * py + (code >> 1), x = 2 * px + (code & 1);
        g2[oc * DW_G_STRIDE + y * 14 + x] = tf32f(ws.dp2[row * FLAT + o]);
      }
    }
    if (tid < 256) {   // bias gradient: thread (oc, l) adds pooled entries l, l+8, ...; lanes combine in a fixed order
      const int oc = tid >> 3, l = tid & 7;
      float sum = 0.f;
      for (int p = l; p < 49; p += 8) {
        int o = oc * 49 + p;
        if (ws.code2[row * FLAT + o] < 4) sum += ws.dp2[row * FLAT + o];
      }
      sum += __shfl_xor_sync(0xffffffffu, sum, 4);
      sum += __shfl_xor_sync(0xffffffffu, sum, 2);
      sum += __shfl_xor_sync(0xffffffffu, sum, 1);
      gb += sum;
    }
    __syncthreads();
#pragma unroll 5
    for (int ks = 0; ks < 25; ++ks) {
      const int p0 = ks * 8 + t, p1 = p0 + 4;
      uint32_t fa[2][4], fb[2][2];
#pragma unroll
      for (int m = 0; m < 2; ++m) {
        const float* ga = g2 + (m * 16 + g) * DW_G_STRIDE;
        fa[m][0] = __float_as_uint(ga[p0]);
        fa[m][1] = __float_as_uint(ga[8 * DW_G_STRIDE + p0]);
        fa[m][2] = __float_as_uint(ga[p1]);
        fa[m][3] = __float_as_uint(ga[8 * DW_G_STRIDE + p1]);
      }
      const int q0 = min(p0, 195), q1 = min(p1, 195);
      const int y0 = q0 / 14, x0 = q0 - y0 * 14, y1 = q1 / 14, x1 = q1 - y1 * 14;
      const int o0 = (y0 + ky) * 16 + x0 + kx, o1 = (y1 + ky) * 16 + x1 + kx;
#pragma unroll
      for (int n = 0; n < 2; ++n) {
        const float* pi = img + (n * 8 + g) * DW_PLANE;
        fb[n][0] = __float_as_uint(pi[o0]);
        fb[n][1] = __float_as_uint(pi[o1]);
      }
#pragma unroll
      for (int m = 0; m < 2; ++m)
#pragma unroll
        for (int n = 0; n < 2; ++n) mma_tf32(acc[m][n], fa[m], fb[n]);
    }
  }
  float* part = ws.part2 + ((int64_t)s * n_chunks + blockIdx.x) * C2_GRAD;
#pragma unroll
  for (int m = 0; m < 2; ++m)
#pragma unroll
    for (int n = 0; n < 2; ++n) {
      const int oc = m * 16 + g, ic = n * 8 + 2 * t;
      part[(oc * 16 + ic) * 9 + warp] = acc[m][n][0];
      part[(oc * 16 + ic + 1) * 9 + warp] = acc[m][n][1];
      part[((oc + 8) * 16 + ic) * 9 + warp] = acc[m][n][2];
      part[((oc + 8) * 16 + ic + 1) * 9 + warp] = acc[m][n][3];
    }
  if (tid < 256 && (tid & 7) == 0) part[4608 + (tid >> 3)] = gb;
}

}  // namespace

#define TIMED(id, launch) do { if (prof) prof->begin(id, st); launch; if (prof) prof->end(st); } while (0)

int configure_tc_kernels() {
  cudaError_t e = cudaFuncSetAttribute(fc1_fwd_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM_BYTES);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(fc1_dx_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM_BYTES);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(fc1_dw_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM_BYTES);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(conv2_dx_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, DX_SMEM_FLOATS * 4);
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

int tc_conv_chunks(int b) { return (b + TC_SPB - 1) / TC_SPB; }

void launch_conv2_fwd_tc(const GradStepArgs& a, const WorkerTable& wt, const GroupTable& gt, const Workspace& ws,
                         cudaStream_t st, Profiler* prof) {
  TIMED(K_CONV2_FWD, (conv2_fwd_tc<<<dim3(tc_conv_chunks(a.b), a.W), 224, 0, st>>>(a, wt, gt, ws)));
}

// Launches the input-gradient and filter-gradient kernels; returns the number of per-worker partial
// blocks the filter gradient was split into.
int launch_conv2_bwd_tc(const GradStepArgs& a, const WorkerTable& wt, const GroupTable& gt, const Workspace& ws,
                        cudaStream_t st, Profiler* prof, bool with_dx) {
  const int chunks = tc_conv_chunks(a.b);
  if (with_dx) TIMED(K_CONV2_BWD, (conv2_dx_tc<<<dim3(chunks, a.W), 224, DX_SMEM_FLOATS * 4, st>>>(a, wt, gt, ws)));
  TIMED(K_CONV2_DW, (conv2_dw_tc<<<dim3(chunks, a.W), 288, 0, st>>>(a, wt, ws, chunks)));
  return chunks;
}

}  // namespace psk
