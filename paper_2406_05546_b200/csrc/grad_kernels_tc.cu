// Filter gradient of the first convolution on the tensor cores (BF16 operands, warp-level mma.sync): a 16 x 10
// output per worker with a long reduction over positions and samples.
//
// Reductions keep a fixed order, so results are reproducible bit for bit.
#include "device_common.cuh"
#include "kernels.h"
#include "tc5_common.cuh"

namespace psk {

namespace {

__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}

// ------------------------------------------------------------------------------------------------
// Filter gradient of the first convolution: dW[oc][tap] = sum_{samples,pos} da1[oc][pos] * x[pos + tap],
// rows = 16 channels, columns = 9 taps (+ one column of ones for the bias gradient), k = the 784 positions
// of a sample (49 k-steps of 16).  BF16 operands, fp32 accumulation; values only.  da1, the gradient at
// the convolution's output, is written densely from the pooled gradient and the pooling decisions (each
// pooled entry owns its 2x2 window); both arrive as [channel quad][position][4 channels], so a thread takes
// four channels of a position with one 16-byte and one 4-byte load.  The eight warps split the k-steps (a
// warp's k-steps and their shared-memory offsets are fixed, so they are worked out once); their accumulators
// persist over the block's samples and are combined in a fixed order at the end.
// ------------------------------------------------------------------------------------------------
constexpr int C1B_SPB = 8;
constexpr int C1B_A_WORDS = 396;       // 392 position pairs per channel + 4: 396 = 12 (mod 32 banks)
constexpr int C1B_ROW = 42;            // elements per row of the bordered image: 21 words, so that the three filter rows
constexpr int C1B_X_WORDS = 656;       // and the two copies (656 = 16 mod 32 words apart) fall into different banks
constexpr int C1B_ITEMS = (4 * 196 + 255) / 256;   // (channel quad, position) items per thread
constexpr int C1B_KSTEPS = 7;                       // k-steps per warp: ceil(49 / 8)
__global__ void __launch_bounds__(256) conv1_bwd_tc(GradStepArgs a, WorkerTable wt, Workspace ws, int n_chunks) {
  __shared__ __align__(16) uint32_t da1w[16 * C1B_A_WORDS];
  __shared__ __align__(16) uint32_t xw[2][C1B_X_WORDS];   // bordered 30 x 42 image as bf16 pairs; copy 1 is shifted by one element
  __shared__ float red[8][16][17];
  uint16_t* xh0 = reinterpret_cast<uint16_t*>(xw[0]);
  const int s = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
  for (int idx = tid; idx < 2 * C1B_X_WORDS; idx += 256) (&xw[0][0])[idx] = 0u;
  for (int idx = tid; idx < 16 * C1B_A_WORDS; idx += 256) da1w[idx] = 0u;
  // this lane's B columns: tile 0 column g = tap g; tile 1 column 0 = tap 8, column 1 = ones
  const int ky0 = g / 3, kx0 = g - ky0 * 3;                  // tap g (g < 8)
  const int copy0 = kx0 & 1;
  const int off0 = ky0 * C1B_ROW + kx0 - copy0;                   // element offset of tap g in its copy (even)
  const int off8 = 2 * C1B_ROW + 2;                               // tap 8 = (2, 2) in copy 0
  float acc[2][4];
#pragma unroll
  for (int n = 0; n < 2; ++n)
#pragma unroll
    for (int r = 0; r < 4; ++r) acc[n][r] = 0.f;
  const int i0 = blockIdx.x * C1B_SPB, i1 = min(i0 + C1B_SPB, a.b);
  // A fragments by ldmatrix: lane l addresses row (l & 7) + 8 * ((l >> 3) & 1) of the 16 channels, k half l >> 4;
  // k-step ks starts 32 bytes (8 position pairs) further along the row
  const uint32_t a_addr = smem_u32(da1w) + (uint32_t)(((lane & 7) + ((lane >> 3) & 1) * 8) * C1B_A_WORDS * 4 + (lane >> 4) * 16);
  // B fragments of this lane in k-step ks = warp + 8 i: position pairs j0 = 8 ks + t and j0 + 4; word offsets of tap g
  // (in its copy) and of tap 8 (copy 0) at both
  int xo[C1B_KSTEPS][4];
#pragma unroll
  for (int i7 = 0; i7 < C1B_KSTEPS; ++i7) {
    const int j0 = (warp + 8 * i7) * 8 + t, j1 = j0 + 4;
    const int y0 = j0 / 14, x0 = 2 * (j0 - y0 * 14), y1 = j1 / 14, x1 = 2 * (j1 - y1 * 14);
    const int e0 = y0 * C1B_ROW + x0, e1 = y1 * C1B_ROW + x1;         // bordered element (y, x) of tap (0, 0)
    xo[i7][0] = (e0 + off0) >> 1; xo[i7][1] = (e1 + off0) >> 1; xo[i7][2] = (e0 + off8) >> 1; xo[i7][3] = (e1 + off8) >> 1;
  }

  float4 xr = make_float4(0.f, 0.f, 0.f, 0.f), gr[C1B_ITEMS];
  uint32_t cr[C1B_ITEMS];
  auto prefetch = [&](int i) {
    const int64_t row = (int64_t)s * a.b + i;
    if (tid < 196) xr = reinterpret_cast<const float4*>(a.x + ((int64_t)wt.src[s] * a.b + i) * (IMG * IMG))[tid];
#pragma unroll
    for (int k = 0; k < C1B_ITEMS; ++k) {
      const int e = tid + 256 * k;
      cr[k] = e < 4 * 196 ? reinterpret_cast<const uint32_t*>(ws.code1 + row * P1_ELEMS)[e] : 0x04040404u;
      gr[k] = e < 4 * 196 ? reinterpret_cast<const float4*>(ws.dp1 + row * P1_ELEMS)[e] : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  };
  prefetch(i0);
  for (int i = i0; i < i1; ++i) {
    __syncthreads();                        // the previous sample's products are done with shared memory
    if (tid < 196) {
      // pixels 4 tid .. 4 tid + 3 of row yy; element (yy, xx) sits at el = (yy + 1) * C1B_ROW + xx + 1 of copy 0 and at
      // el - 1 of copy 1, so the four are two aligned words of copy 1 and half, whole, half a word of copy 0
      const int yy = tid / 7, xx = 4 * (tid - yy * 7), el = (yy + 1) * C1B_ROW + xx + 1;
      const uint32_t h01 = bf16_pair(xr.x, xr.y), h23 = bf16_pair(xr.z, xr.w);
      xw[1][(el - 1) >> 1] = h01;
      xw[1][((el - 1) >> 1) + 1] = h23;
      xh0[el] = (uint16_t)(h01 & 0xFFFFu);
      xw[0][(el + 1) >> 1] = __byte_perm(h01, h23, 0x5432);
      xh0[el + 3] = (uint16_t)(h23 >> 16);
    }
#pragma unroll
    for (int k = 0; k < C1B_ITEMS; ++k) {
      const int e = tid + 256 * k;
      if (e < 4 * 196) {
        const int cq = e / 196, pos = e - cq * 196, py = pos / 14, px = pos - py * 14;
        uint32_t* d = da1w + (4 * cq) * C1B_A_WORDS + py * 28 + px;     // pair of positions (2py, 2px), (2py, 2px+1)
        const float v[4] = {gr[k].x, gr[k].y, gr[k].z, gr[k].w};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          // the BF16 value shifted left by 16 bits per decision lands in the half-word of the window position that
          // won: low word = row 2py (even, odd column), high word = row 2py + 1; decision 4 shifts it out entirely
          const uint32_t code = (cr[k] >> (8 * c)) & 0xFFu;
          const unsigned long long slot = shl64_clamped(bf16_bits(v[c]), 16u * code);
          d[c * C1B_A_WORDS] = (uint32_t)slot;
          d[c * C1B_A_WORDS + 14] = (uint32_t)(slot >> 32);
        }
      }
    }
    __syncthreads();
    if (i + 1 < i1) prefetch(i + 1);
#pragma unroll
    for (int i7 = 0; i7 < C1B_KSTEPS; ++i7) {
      if (warp + 8 * i7 < 49) {           // warp-uniform
        uint32_t fa[4], fb[2][2];
        ldmatrix_x4(fa, a_addr + (warp + 8 * i7) * 32);
        fb[0][0] = xw[copy0][xo[i7][0]];
        fb[0][1] = xw[copy0][xo[i7][1]];
        const uint32_t t8a = xw[0][xo[i7][2]], t8b = xw[0][xo[i7][3]];
        fb[1][0] = g == 0 ? t8a : (g == 1 ? 0x3F803F80u : 0u);
        fb[1][1] = g == 0 ? t8b : (g == 1 ? 0x3F803F80u : 0u);
        mma_bf16(acc[0], fa, fb[0]);
        mma_bf16(acc[1], fa, fb[1]);
      }
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

int launch_conv1_bwd_tc(const GradStepArgs& a, const WorkerTable& wt, const Workspace& ws, cudaStream_t st, Profiler* prof) {
  const int chunks = (a.b + C1B_SPB - 1) / C1B_SPB;
  TIMED(K_CONV1_BWD, (conv1_bwd_tc<<<dim3(chunks, a.W), 256, 0, st>>>(a, wt, ws, chunks)));
  return chunks;
}

}  // namespace psk
