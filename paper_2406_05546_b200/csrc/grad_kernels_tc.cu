// Filter gradient of the second convolution on the tensor cores (TF32, warp-level mma.sync): the one
// contraction of the step whose output (32 x 144 per worker) is too small for a 128-row tcgen05 tile,
// while its reduction (all positions of all samples of a worker) is long.
//
// Reductions keep a fixed order, so results are reproducible bit for bit.
#include "device_common.cuh"
#include "kernels.h"

namespace psk {

namespace {

// D += A(16x8, row) * B(8x8, col), TF32 inputs, fp32 accumulate.  Lane = 4*g + t:
//   a0 (g, t)  a1 (g+8, t)  a2 (g, t+4)  a3 (g+8, t+4);  b0 (k=t, n=g)  b1 (k=t+4, n=g);
//   c0 (g, 2t) c1 (g, 2t+1) c2 (g+8, 2t) c3 (g+8, 2t+1).
__device__ __forceinline__ void mma_tf32(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  asm volatile(
      "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

constexpr int TC_SPB = 8;
__device__ __forceinline__ float tf32f(float x) { return round_tf32(x); }

// Filter gradient: dW[oc][ic][tap] = sum_{samples,pos} g2[oc][pos] * p1[ic][pos + tap]: rows = 32 output
// channels, columns = 16 input channels per tap, k = position (196 per sample, 25 k-steps, zero-padded).
// 288 threads = 9 warps, warp = filter tap; accumulators persist over the block's samples and are
// written once as the block's partial sum.  The bias gradient (sum of g2 over positions) rides along as
// a product with a column of ones, each warp taking every ninth k-step; the nine partial sums are
// combined in a fixed order at the end.
// The next sample's inputs are fetched into registers while the current one is being multiplied, so
// that global-memory latency stays off the critical path.
constexpr int DW_G_STRIDE = 228;   // 196 positions + zeros; = 4 (mod 32 banks)
constexpr int DW_PLANE = 260;      // 16 x 16 + 4;            = 4 (mod 32 banks)
constexpr int DW_THREADS = 288;
constexpr int DW_QUADS = (4 * 196 + DW_THREADS - 1) / DW_THREADS;   // 3 four-channel positions per thread
constexpr int DW_ENTRIES = (FLAT + DW_THREADS - 1) / DW_THREADS;    // 6 pooled gradient entries per thread
__global__ void __launch_bounds__(DW_THREADS) conv2_dw_tc(GradStepArgs a, WorkerTable wt, Workspace ws, int n_chunks) {
  __shared__ __align__(16) float g2[32 * DW_G_STRIDE];   // [oc][pos]
  __shared__ __align__(16) float img[16 * DW_PLANE];     // [ic][Y][X], zero border
  __shared__ float bias_part[9][32];
  const int s = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  const int ky = warp / 3, kx = warp - ky * 3;
  for (int idx = tid; idx < 16 * DW_PLANE; idx += DW_THREADS) img[idx] = 0.f;
  for (int idx = tid; idx < 32 * DW_G_STRIDE; idx += DW_THREADS) g2[idx] = 0.f;
  float acc[2][2][4], accb[2][4];
#pragma unroll
  for (int m = 0; m < 2; ++m) {
#pragma unroll
    for (int n = 0; n < 2; ++n)
#pragma unroll
      for (int r = 0; r < 4; ++r) acc[m][n][r] = 0.f;
#pragma unroll
    for (int r = 0; r < 4; ++r) accb[m][r] = 0.f;
  }
  // the column of ones: B(k, n) = 1 for n == 0; this lane supplies column n = g
  const uint32_t one_frag[2] = {g == 0 ? __float_as_uint(1.0f) : 0u, g == 0 ? __float_as_uint(1.0f) : 0u};
  const int i0 = blockIdx.x * TC_SPB, i1 = min(i0 + TC_SPB, a.b);

  float4 pq[DW_QUADS];
  float pg[DW_ENTRIES];
  int pc[DW_ENTRIES];
  auto prefetch = [&](int i) {
    const int64_t row = (int64_t)s * a.b + i;
#pragma unroll
    for (int k = 0; k < DW_QUADS; ++k) {
      const int e = tid + k * DW_THREADS;                      // (plane q, position p)
      if (e < 4 * 196) {
        const int q = e / 196, p = e - q * 196, y = p / 14, x = p - y * 14, X = x + 1, Y = y + 1;
        pq[k] = *reinterpret_cast<const float4*>(ws.p1 + row * P1_PLANE_ELEMS + q * 1024 + (Y * 16 + (X & 1) * 8 + (X >> 1)) * 4);
      }
    }
#pragma unroll
    for (int k = 0; k < DW_ENTRIES; ++k) {
      const int o = tid + k * DW_THREADS;
      pc[k] = o < FLAT ? (int)ws.code2[row * FLAT + o] : 4;
      pg[k] = o < FLAT ? ws.dp2[row * FLAT + o] : 0.f;
    }
  };
  prefetch(i0);
  for (int i = i0; i < i1; ++i) {
    __syncthreads();                 // the previous sample's products are done with shared memory
#pragma unroll
    for (int k = 0; k < DW_QUADS; ++k) {
      const int e = tid + k * DW_THREADS;
      if (e < 4 * 196) {
        const int q = e / 196, p = e - q * 196, y = p / 14, x = p - y * 14;
        float* d = img + (4 * q) * DW_PLANE + (y + 1) * 16 + x + 1;
        d[0] = pq[k].x; d[DW_PLANE] = pq[k].y; d[2 * DW_PLANE] = pq[k].z; d[3 * DW_PLANE] = pq[k].w;
      }
    }
#pragma unroll
    for (int k = 0; k < DW_ENTRIES; ++k) {
      const int o = tid + k * DW_THREADS;
      if (o < FLAT) {
        // every pooled entry owns the four positions of its window: the gradient goes to the chosen one,
        // the others are cleared, so no separate clearing pass is needed
        const int oc = o / 49, p = o - oc * 49, py = p / 7, px = p - py * 7;
        float* d = g2 + oc * DW_G_STRIDE + (2 * py) * 14 + 2 * px;
        const float v = tf32f(pg[k]);
        d[0] = pc[k] == 0 ? v : 0.f; d[1] = pc[k] == 1 ? v : 0.f;
        d[14] = pc[k] == 2 ? v : 0.f; d[15] = pc[k] == 3 ? v : 0.f;
      }
    }
    __syncthreads();
    if (i + 1 < i1) prefetch(i + 1);
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
      if (ks % 9 == warp) {            // warp-uniform
        mma_tf32(accb[0], fa[0], one_frag);
        mma_tf32(accb[1], fa[1], one_frag);
      }
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
  // column 0 of the ones-product lives in the lanes with t == 0: rows g and g+8 of each 16-row tile
  if (t == 0) {
#pragma unroll
    for (int m = 0; m < 2; ++m) {
      bias_part[warp][m * 16 + g] = accb[m][0];
      bias_part[warp][m * 16 + g + 8] = accb[m][2];
    }
  }
  __syncthreads();
  if (tid < 32) {
    float sum = 0.f;
#pragma unroll
    for (int w = 0; w < 9; ++w) sum += bias_part[w][tid];
    part[4608 + tid] = sum;
  }
}

}  // namespace

#define TIMED(id, launch) do { if (prof) prof->begin(id, st); launch; if (prof) prof->end(st); } while (0)

int configure_tc_kernels() { return 0; }

// Returns the number of per-worker partial blocks the filter gradient was split into.
int launch_conv2_dw_tc(const GradStepArgs& a, const WorkerTable& wt, const Workspace& ws, cudaStream_t st, Profiler* prof) {
  const int chunks = (a.b + TC_SPB - 1) / TC_SPB;
  TIMED(K_CONV2_DW, (conv2_dw_tc<<<dim3(chunks, a.W), DW_THREADS, 0, st>>>(a, wt, ws, chunks)));
  return chunks;
}

}  // namespace psk
