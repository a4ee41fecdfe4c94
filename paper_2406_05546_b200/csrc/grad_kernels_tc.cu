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
      const int X = x + 1, Y = y + 1;     // p1 is stored as four-channel planes with even/odd columns apart
      img[ic * DW_PLANE + Y * 16 + X] = ws.p1[row * P1_PLANE_ELEMS + (ic >> 2) * 1024 + (Y * 16 + (X & 1) * 8 + (X >> 1)) * 4 + (ic & 3)];
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

int configure_tc_kernels() { return 0; }

// Returns the number of per-worker partial blocks the filter gradient was split into.
int launch_conv2_dw_tc(const GradStepArgs& a, const WorkerTable& wt, const Workspace& ws, cudaStream_t st, Profiler* prof) {
  const int chunks = (a.b + TC_SPB - 1) / TC_SPB;
  TIMED(K_CONV2_DW, (conv2_dw_tc<<<dim3(chunks, a.W), 288, 0, st>>>(a, wt, ws, chunks)));
  return chunks;
}

}  // namespace psk
