// First convolution (1 -> 16 channels, 3x3, pad 1) + ReLU + 2x2 max pooling of the tensor-core path.
// K = 9 is too short for the tensor cores, so the products run on the FP32 pipes; everything around
// them is arranged so that a thread does little else:
//   - the images arrive by TMA tile loads whose box starts outside the image (rows -1..28, columns
//     -4..31): the out-of-range part is filled with zeros, so the zero border of the padded
//     convolution needs no instruction;
//   - a thread owns one group of four output channels for the whole kernel and keeps its 40 weights
//     in registers as channel pairs; the multiply-adds are packed fma.rn.f32x2 over those pairs;
//   - results are collected in shared memory in exactly the layout the second convolution's kernels
//     copy from (two planes of eight BF16 channels, one 16-byte row per position of a zero-bordered
//     16x16 grid with even and odd columns apart) and leave by bulk copies, 8 KB per sample; the
//     pooling decisions leave the same way, one byte per element (1 << winner, 0 = no gradient) as
//     [channel quad][position][4 channels].
// Every wait on an mbarrier is bounded.
#include "device_common.cuh"
#include "kernels.h"
#include "tc5_common.cuh"

namespace psk {

namespace {

constexpr int C1_SPS = 1;                                // samples per step
constexpr int C1_THREADS = 112 * C1_SPS;
constexpr int C1_BLOCKS_PER_SM = 6 / C1_SPS;
constexpr int C1_SPB = 4;                                // samples per block, taken C1_SPS at a time
constexpr int C1_BOX_W = 36, C1_BOX_H = 30;              // image box: columns -4..31 (a 16-byte aligned start), rows -1..28
constexpr int C1_BOX_BYTES = C1_BOX_W * C1_BOX_H * 4;    // 4320
constexpr int C1_IMG_SLOT = 4352;                        // box padded to a multiple of 128 bytes
constexpr int C1_IN_BYTES = C1_SPS * C1_IMG_SLOT;        // the images of a step
constexpr int C1_PLANES_BYTES = P1_PLANE_ELEMS * 4;      // 8192 per sample
constexpr int C1_OUT_BYTES = C1_SPS * (C1_PLANES_BYTES + P1_ELEMS);   // a step's samples: planes, then decisions
constexpr int C1_STAGES = 2;
constexpr int C1_SMEM = C1_STAGES * C1_IN_BYTES + 2 * C1_OUT_BYTES + 64 + 128;

// Work items of a step = (sample, pooled position, group of four channels): C1_SPS * 196 * 4 = 7 per thread.
// Thread tid takes channel group tid & 3 and the pooled positions (tid >> 2) + 28 C1_SPS k of the step's samples
// laid end to end; 28 = two rows of 14, so its column is fixed and its row advances by 2 C1_SPS.  Small blocks
// (one sample per step, six blocks per SM) keep the blocks' phases apart: the barrier of a step lines up the
// multiply-add phases of all warps of a block, and with few large blocks the FMA pipe idles while all of them
// pool and store.
__global__ void __launch_bounds__(C1_THREADS, C1_BLOCKS_PER_SM) conv1_fwd_planes(const __grid_constant__ CUtensorMap xmap, GradStepArgs a,
                                                                  WorkerTable wt, GroupTable gt, Workspace ws) {
  extern __shared__ __align__(128) uint8_t sm[];
  const float* in = reinterpret_cast<const float*>(sm);
  uint8_t* outb = sm + C1_STAGES * C1_IN_BYTES;
  uint64_t* full = reinterpret_cast<uint64_t*>(sm + C1_STAGES * C1_IN_BYTES + 2 * C1_OUT_BYTES);
  const int s = blockIdx.y, tid = threadIdx.x, cg = tid & 3;
  const int i0 = blockIdx.x * C1_SPB, i1 = min(i0 + C1_SPB, a.b);
  const int n_steps = (i1 - i0 + C1_SPS - 1) / C1_SPS;
  const float* theta = group_theta(wt, gt, s);
  if (tid == 0) {
    for (int k = 0; k < C1_STAGES; ++k) mbar_init(&full[k], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // the border rows of the planes are never written below: cleared once, they leave as zeros with every sample
  for (int t = tid; t < 2 * C1_OUT_BYTES / 16; t += C1_THREADS) reinterpret_cast<uint4*>(outb)[t] = make_uint4(0u, 0u, 0u, 0u);
  u64 wp[2][10];     // wp[cp][k] = tap k of channels 4 cg + 2 cp and + 1; k = 9 is the bias
#pragma unroll
  for (int cp = 0; cp < 2; ++cp) {
    const int c0 = 4 * cg + 2 * cp;
#pragma unroll
    for (int k = 0; k < 9; ++k) wp[cp][k] = pack2(theta[OFF_C1W + c0 * 9 + k], theta[OFF_C1W + (c0 + 1) * 9 + k]);
    wp[cp][9] = pack2(theta[OFF_C1B + c0], theta[OFF_C1B + c0 + 1]);
  }
  __syncthreads();
  const int64_t src_row0 = (int64_t)wt.src[s] * a.b + i0;     // the caller's image index of the block's first sample
  auto issue = [&](int st) {     // thread 0: the images of step st
    const int n_s = min(C1_SPS, i1 - (i0 + C1_SPS * st));
    uint64_t* bar = &full[st % C1_STAGES];
    mbar_expect_tx(bar, n_s * C1_BOX_BYTES);
    for (int k = 0; k < n_s; ++k)
      tma_load_3d(sm + (st % C1_STAGES) * C1_IN_BYTES + k * C1_IMG_SLOT, &xmap, bar, -4, -1, (int)(src_row0 + C1_SPS * st + k));
  };
  if (tid == 0)
    for (int st = 0; st < C1_STAGES && st < n_steps; ++st) issue(st);
  const int px = (tid >> 2) % 14, py0 = (tid >> 2) / 14;
  const int X = px + 1, col_row = (X & 1) * 8 + (X >> 1);
  bool ok = true;
  for (int st = 0; st < n_steps && ok; ++st) {
    const int n_s = min(C1_SPS, i1 - (i0 + C1_SPS * st));
    if (!mbar_wait(&full[st % C1_STAGES], (st / C1_STAGES) & 1)) { ok = false; break; }
    const float* img = in + (st % C1_STAGES) * (C1_IN_BYTES / 4);
    uint8_t* ob = outb + (st & 1) * C1_OUT_BYTES;
#pragma unroll 1
    for (int k = 0; k < 7; ++k) {
      const int R = py0 + 2 * C1_SPS * k, sp = R / 14, py = R - 14 * sp;
      if (sp >= n_s) break;
      // image row 2 py - 1 is box row 2 py, image column 2 px - 1 is box column 2 px + 3
      const float* src = img + sp * (C1_IMG_SLOT / 4) + (2 * py) * C1_BOX_W + 2 * px + 3;
      u64 dup[4][4];   // the 4x4 input patch under the 2x2 window, every value in both halves
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const float a0 = src[r * C1_BOX_W];
        const float2 a12 = *reinterpret_cast<const float2*>(src + r * C1_BOX_W + 1);
        const float a3 = src[r * C1_BOX_W + 3];
        dup[r][0] = pack2(a0, a0); dup[r][1] = pack2(a12.x, a12.x); dup[r][2] = pack2(a12.y, a12.y); dup[r][3] = pack2(a3, a3);
      }
      u64 acc[2][4];
#pragma unroll
      for (int cp = 0; cp < 2; ++cp)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[cp][j] = wp[cp][9];
#pragma unroll
      for (int ky = 0; ky < 3; ++ky)
#pragma unroll
        for (int kx = 0; kx < 3; ++kx)
#pragma unroll
          for (int cp = 0; cp < 2; ++cp)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[cp][j] = ffma2(wp[cp][ky * 3 + kx], dup[(j >> 1) + ky][(j & 1) + kx], acc[cp][j]);
      float v[4][4];     // [channel][window element]
#pragma unroll
      for (int cp = 0; cp < 2; ++cp)
#pragma unroll
        for (int j = 0; j < 4; ++j) unpack2(acc[cp][j], v[2 * cp][j], v[2 * cp + 1][j]);
      // ReLU then max = max then ReLU; the winner is the first window element that reaches the maximum (stored as the
      // byte 1 << winner), and an element whose maximum is not positive passes no gradient (byte 0)
      float best[4];
      uint32_t codes = 0;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const float m = fmaxf(fmaxf(v[c][0], v[c][1]), fmaxf(v[c][2], v[c][3]));
        const uint32_t bi = v[c][0] == m ? 0u : (v[c][1] == m ? 1u : (v[c][2] == m ? 2u : 3u));
        best[c] = fmaxf(m, 0.f);
        codes |= (m > 0.f ? (1u << bi) : 0u) << (8 * c);      // one bit per window element: the filter-gradient kernel shifts it into a mask
      }
      const int row = (py + 1) * 16 + col_row, pos = py * 14 + px;
      *reinterpret_cast<uint2*>(ob + sp * C1_PLANES_BYTES + (cg >> 1) * (C1_PLANES_BYTES / 2) + row * 16 + (cg & 1) * 8) =
          make_uint2(bf16_pair(best[0], best[1]), bf16_pair(best[2], best[3]));
      *reinterpret_cast<uint32_t*>(ob + C1_SPS * C1_PLANES_BYTES + sp * P1_ELEMS + cg * 784 + pos * 4) = codes;
    }
    fence_proxy_async_smem();
    if (tid == 0) bulk_wait_read0();      // the previous step's copies have read their buffer, which the next step overwrites
    __syncthreads();
    if (tid == 0) {
      const int64_t row0 = (int64_t)s * a.b + i0 + C1_SPS * st;
      bulk_store(reinterpret_cast<uint8_t*>(ws.p1) + row0 * C1_PLANES_BYTES, ob, n_s * C1_PLANES_BYTES);
      bulk_store(ws.code1 + row0 * P1_ELEMS, ob + C1_SPS * C1_PLANES_BYTES, n_s * P1_ELEMS);
      bulk_commit();
      if (st + C1_STAGES < n_steps) issue(st + C1_STAGES);
    }
  }
  if (!ok && (tid & 31) == 0) atomicOr(ws.status, STATUS_WAIT_TIMEOUT);
  if (tid == 0) bulk_wait_all();          // shared memory must outlive the copies that read it
}

}  // namespace

#define TIMED(id, launch) do { if (prof) prof->begin(id, st); launch; if (prof) prof->end(st); } while (0)

int configure_conv1_kernels() {
  return cudaFuncSetAttribute(conv1_fwd_planes, cudaFuncAttributeMaxDynamicSharedMemorySize, C1_SMEM) == cudaSuccess ? 0 : -1;
}

// The caller's images [W*b][28][28] as a 3-d tensor; a.x must be 16-byte aligned.  Returns 1 (kernels launched) or -1.
int launch_conv1_fwd_planes(const GradStepArgs& a, const WorkerTable& wt, const GroupTable& gt, const Workspace& ws,
                            cudaStream_t st, Profiler* prof) {
  CUtensorMap xmap;
  const uint64_t dims[3] = {IMG, IMG, (uint64_t)a.W * a.b};
  const uint64_t strides[2] = {IMG * 4, IMG * IMG * 4};
  const uint32_t box[3] = {C1_BOX_W, C1_BOX_H, 1};
  if (!encode_tensor_map_f32(&xmap, a.x, 3, dims, strides, box)) return -1;
  const int chunks = (a.b + C1_SPB - 1) / C1_SPB;
  TIMED(K_CONV1_FWD, (conv1_fwd_planes<<<dim3(chunks, a.W), C1_THREADS, C1_SMEM, st>>>(xmap, a, wt, gt, ws)));
  return 1;
}

}  // namespace psk
