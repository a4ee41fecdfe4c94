// Filter gradient of the second convolution on the tensor cores (BF16 operands, warp-level mma.sync): the one
// contraction of the step whose output (32 x 144 per worker) is too small for a 128-row tcgen05 tile,
// while its reduction (all positions of all samples of a worker) is long.
//
// Reductions keep a fixed order, so results are reproducible bit for bit.
#include "device_common.cuh"
#include "kernels.h"

namespace psk {

namespace {

constexpr int TC_SPB = 8;

// Filter gradient: dW[oc][ic][tap] = sum_{samples,pos} g2[oc][pos] * p1[ic][pos + tap]: rows = 32 output
// channels, columns = 16 input channels per tap, k = position (196 per sample, 13 k-steps of 16, zero-padded).
// Both operands are rounded to BF16 here (fp32 accumulation): this product only yields gradient values, no
// ReLU or pooling decision depends on it, and at 16 positions per instruction it needs half the
// instructions and shared-memory loads of the TF32 form.
// 288 threads = 9 warps, warp = filter tap; accumulators persist over the block's samples and are
// written once as the block's partial sum.  The bias gradient (sum of g2 over positions) rides along as
// a product with a column of ones, each warp taking every ninth k-step; the nine partial sums are
// combined in a fixed order at the end.
// A BF16 fragment register holds two consecutive k = two horizontally adjacent positions (x even, x+1).
// For the taps that shift by an odd number of columns such a pair is not word-aligned in the image plane,
// so the planes are kept twice, the second copy shifted by one element.
// The next sample's inputs are fetched into registers while the current one is being multiplied.
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}
__device__ __forceinline__ uint16_t bf16_bits(float x) {
  uint16_t r;
  asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(r) : "f"(x));
  return r;
}
__device__ __forceinline__ uint32_t bf16_pair(float lo, float hi) {   // lo in the low half (lower k index)
  return (uint32_t)bf16_bits(lo) | ((uint32_t)bf16_bits(hi) << 16);
}

constexpr int DW_G_WORDS = 108;    // 216 bf16 per output channel: 196 positions + zeros; 108 = 12 (mod 32 banks)
constexpr int DW_P_WORDS = 132;    // 16 x 16 bf16 per input channel + 8; 132 = 4 (mod 32 banks)
constexpr int DW_THREADS = 288;
constexpr int DW_KSTEPS = 13;      // 208 positions / 16
constexpr int DW_QUADS = (4 * 196 + DW_THREADS - 1) / DW_THREADS;   // 3 four-channel positions per thread
constexpr int DW_ENTRIES = (FLAT + DW_THREADS - 1) / DW_THREADS;    // 6 pooled gradient entries per thread
__global__ void __launch_bounds__(DW_THREADS, 2) conv2_dw_tc(GradStepArgs a, WorkerTable wt, Workspace ws, int n_chunks) {
  __shared__ __align__(16) uint32_t g2w[32 * DW_G_WORDS];        // [oc][position pair]
  __shared__ __align__(16) uint32_t imgw[2][16 * DW_P_WORDS];    // [copy][ic][(Y*16 + X - copy) / 2], zero border
  __shared__ float bias_part[9][32];
  uint16_t* img_h[2] = {reinterpret_cast<uint16_t*>(imgw[0]), reinterpret_cast<uint16_t*>(imgw[1])};
  const int s = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  const int ky = warp / 3, kx = warp - ky * 3;
  for (int idx = tid; idx < 2 * 16 * DW_P_WORDS; idx += DW_THREADS) (&imgw[0][0])[idx] = 0u;
  for (int idx = tid; idx < 32 * DW_G_WORDS; idx += DW_THREADS) g2w[idx] = 0u;
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
  const uint32_t one_frag[2] = {g == 0 ? 0x3F803F80u : 0u, g == 0 ? 0x3F803F80u : 0u};
  // this warp's B fragments: pair index j = ks*8 + t (+4): position 2j = (y, x even); element (y+ky)*16 + x + kx
  // in the bordered plane, taken from the copy that makes it even
  const int copy = kx & 1;
  const uint32_t* plane = imgw[copy];
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
        const int el = (y + 1) * 16 + x + 1;
        const float v[4] = {pq[k].x, pq[k].y, pq[k].z, pq[k].w};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const uint16_t h = bf16_bits(v[c]);
          img_h[0][(4 * q + c) * (2 * DW_P_WORDS) + el] = h;
          img_h[1][(4 * q + c) * (2 * DW_P_WORDS) + el - 1] = h;
        }
      }
    }
#pragma unroll
    for (int k = 0; k < DW_ENTRIES; ++k) {
      const int o = tid + k * DW_THREADS;
      if (o < FLAT) {
        // every pooled entry owns the four positions of its window: the gradient goes to the chosen one,
        // the others are cleared, so no separate clearing pass is needed
        const int oc = o / 49, p = o - oc * 49, py = p / 7, px = p - py * 7;
        uint32_t* d = g2w + oc * DW_G_WORDS + (2 * py) * 7 + px;     // word of positions (2py, 2px), (2py, 2px+1)
        const float v = pg[k];
        d[0] = bf16_pair(pc[k] == 0 ? v : 0.f, pc[k] == 1 ? v : 0.f);
        d[7] = bf16_pair(pc[k] == 2 ? v : 0.f, pc[k] == 3 ? v : 0.f);
      }
    }
    __syncthreads();
    if (i + 1 < i1) prefetch(i + 1);
#pragma unroll
    for (int ks = 0; ks < DW_KSTEPS; ++ks) {
      const int j0 = ks * 8 + t, j1 = j0 + 4;                  // position pairs of this lane's k columns
      uint32_t fa[2][4], fb[2][2];
#pragma unroll
      for (int m = 0; m < 2; ++m) {
        const uint32_t* ga = g2w + (m * 16 + g) * DW_G_WORDS;
        fa[m][0] = ga[j0];
        fa[m][1] = ga[8 * DW_G_WORDS + j0];
        fa[m][2] = ga[j1];
        fa[m][3] = ga[8 * DW_G_WORDS + j1];
      }
      const int q0 = min(j0, 97), q1 = min(j1, 97);            // pairs beyond 97 meet zeros in g2
      const int y0 = q0 / 7, x0 = 2 * (q0 - y0 * 7), y1 = q1 / 7, x1 = 2 * (q1 - y1 * 7);
      const int w0 = ((y0 + ky) * 16 + x0 + kx - copy) >> 1, w1 = ((y1 + ky) * 16 + x1 + kx - copy) >> 1;
#pragma unroll
      for (int n = 0; n < 2; ++n) {
        const uint32_t* pi = plane + (n * 8 + g) * DW_P_WORDS;
        fb[n][0] = pi[w0];
        fb[n][1] = pi[w1];
      }
#pragma unroll
      for (int m = 0; m < 2; ++m)
#pragma unroll
        for (int n = 0; n < 2; ++n) mma_bf16(acc[m][n], fa[m], fb[n]);
      if (ks % 9 == warp) {            // warp-uniform
        mma_bf16(accb[0], fa[0], one_frag);
        mma_bf16(accb[1], fa[1], one_frag);
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

// ------------------------------------------------------------------------------------------------
// Filter gradient of the first convolution: dW[oc][tap] = sum_{samples,pos} da1[oc][pos] * x[pos + tap],
// rows = 16 channels, columns = 9 taps (+ one column of ones for the bias gradient), k = the 784 positions
// of a sample (49 k-steps of 16).  BF16 operands, fp32 accumulation; values only.  da1, the gradient at
// the convolution's output, is written densely from the pooled gradient and the pooling decisions (each
// pooled entry owns its 2x2 window).  The eight warps split the k-steps; their accumulators persist over
// the block's samples and are combined in a fixed order at the end.
// ------------------------------------------------------------------------------------------------
constexpr int C1B_SPB = 16;
constexpr int C1B_A_WORDS = 396;       // 392 position pairs per channel + 4: 396 = 12 (mod 32 banks)
constexpr int C1B_X_WORDS = 15 * 32;   // bordered 30 x 32 image as bf16 pairs
constexpr int C1B_ENTRIES = (P1_ELEMS + 255) / 256;   // 13 pooled entries per thread
__global__ void __launch_bounds__(256) conv1_bwd_tc(GradStepArgs a, WorkerTable wt, Workspace ws, int n_chunks) {
  __shared__ __align__(16) uint32_t da1w[16 * C1B_A_WORDS];
  __shared__ __align__(16) uint32_t xw[2][C1B_X_WORDS + 16];   // copy 1 is shifted by one element
  __shared__ float red[8][16][17];
  uint16_t* xh[2] = {reinterpret_cast<uint16_t*>(xw[0]), reinterpret_cast<uint16_t*>(xw[1])};
  const int s = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  for (int idx = tid; idx < 2 * (C1B_X_WORDS + 16); idx += 256) (&xw[0][0])[idx] = 0u;
  for (int idx = tid; idx < 16 * C1B_A_WORDS; idx += 256) da1w[idx] = 0u;
  // this lane's B columns: tile 0 column g = tap g; tile 1 column 0 = tap 8, column 1 = ones
  const int ky0 = g / 3, kx0 = g - ky0 * 3;                  // tap g (g < 8)
  const int copy0 = kx0 & 1;
  const int off0 = ky0 * 32 + kx0 - copy0;                   // element offset of tap g in its copy (even)
  const int off8 = 2 * 32 + 2;                               // tap 8 = (2, 2) in copy 0
  float acc[2][4];
#pragma unroll
  for (int n = 0; n < 2; ++n)
#pragma unroll
    for (int r = 0; r < 4; ++r) acc[n][r] = 0.f;
  const int i0 = blockIdx.x * C1B_SPB, i1 = min(i0 + C1B_SPB, a.b);

  float xr[4], gr[C1B_ENTRIES];
  int cr[C1B_ENTRIES];
  auto prefetch = [&](int i) {
    const int64_t row = (int64_t)s * a.b + i;
    const float* x = a.x + ((int64_t)wt.src[s] * a.b + i) * (IMG * IMG);
#pragma unroll
    for (int k = 0; k < 4; ++k) xr[k] = tid + 256 * k < IMG * IMG ? x[tid + 256 * k] : 0.f;
#pragma unroll
    for (int k = 0; k < C1B_ENTRIES; ++k) {
      const int o = tid + 256 * k;
      cr[k] = o < P1_ELEMS ? (int)ws.code1[row * P1_ELEMS + o] : 4;
      gr[k] = o < P1_ELEMS ? ws.dp1[row * P1_ELEMS + o] : 0.f;
    }
  };
  prefetch(i0);
  for (int i = i0; i < i1; ++i) {
    __syncthreads();                        // the previous sample's products are done with shared memory
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int e = tid + 256 * k;
      if (e < IMG * IMG) {
        const int yy = e / IMG, xx = e - yy * IMG, el = (yy + 1) * 32 + xx + 1;
        const uint16_t h = bf16_bits(xr[k]);
        xh[0][el] = h;
        xh[1][el - 1] = h;
      }
    }
#pragma unroll
    for (int k = 0; k < C1B_ENTRIES; ++k) {
      const int o = tid + 256 * k;
      if (o < P1_ELEMS) {
        const int oc = o / 196, p = o - oc * 196, py = p / 14, px = p - py * 14;
        uint32_t* d = da1w + oc * C1B_A_WORDS + py * 28 + px;     // pair of positions (2py, 2px), (2py, 2px+1)
        const float v = gr[k];
        d[0] = bf16_pair(cr[k] == 0 ? v : 0.f, cr[k] == 1 ? v : 0.f);
        d[14] = bf16_pair(cr[k] == 2 ? v : 0.f, cr[k] == 3 ? v : 0.f);
      }
    }
    __syncthreads();
    if (i + 1 < i1) prefetch(i + 1);
    for (int ks = warp; ks < 49; ks += 8) {
      const int j0 = ks * 8 + t, j1 = j0 + 4;               // position pairs of this lane's k columns
      uint32_t fa[4], fb[2][2];
      fa[0] = da1w[g * C1B_A_WORDS + j0];
      fa[1] = da1w[(g + 8) * C1B_A_WORDS + j0];
      fa[2] = da1w[g * C1B_A_WORDS + j1];
      fa[3] = da1w[(g + 8) * C1B_A_WORDS + j1];
      const int y0 = j0 / 14, x0 = 2 * (j0 - y0 * 14), y1 = j1 / 14, x1 = 2 * (j1 - y1 * 14);
      const int e0 = y0 * 32 + x0, e1 = y1 * 32 + x1;       // bordered element (y, x) of tap (0, 0)
      fb[0][0] = xw[copy0][(e0 + off0) >> 1];
      fb[0][1] = xw[copy0][(e1 + off0) >> 1];
      const uint32_t t8a = xw[0][(e0 + off8) >> 1], t8b = xw[0][(e1 + off8) >> 1];
      fb[1][0] = g == 0 ? t8a : (g == 1 ? 0x3F803F80u : 0u);
      fb[1][1] = g == 0 ? t8b : (g == 1 ? 0x3F803F80u : 0u);
      mma_bf16(acc[0], fa, fb[0]);
      mma_bf16(acc[1], fa, fb[1]);
    }
  }
  // c0 (row g, col 2t), c1 (g, 2t+1), c2 (g+8, 2t), c3 (g+8, 2t+1); columns 0..7 = taps, 8 = tap 8, 9 = bias
#pragma unroll
  for (int n = 0; n < 2; ++n) {
    red[warp][g][n * 8 + 2 * t] = acc[n][0];
    red[warp][g][n * 8 + 2 * t + 1] = acc[n][1];
    red[warp][g + 8][n * 8 + 2 * t] = acc[n][2];
    red[warp][g + 8][n * 8 + 2 * t + 1] = acc[n][3];
  }
  __syncthreads();
  if (tid < 160) {
    const int oc = tid / 10, col = tid - oc * 10;
    float sum = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) sum += red[w][oc][col];
    float* part = ws.part1 + ((int64_t)s * n_chunks + blockIdx.x) * C1_GRAD;
    part[col < 9 ? oc * 9 + col : 144 + oc] = sum;
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

int launch_conv1_bwd_tc(const GradStepArgs& a, const WorkerTable& wt, const Workspace& ws, cudaStream_t st, Profiler* prof) {
  const int chunks = (a.b + C1B_SPB - 1) / C1B_SPB;
  TIMED(K_CONV1_BWD, (conv1_bwd_tc<<<dim3(chunks, a.W), 256, 0, st>>>(a, wt, ws, chunks)));
  return chunks;
}

}  // namespace psk
