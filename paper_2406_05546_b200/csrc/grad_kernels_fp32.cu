// Worker-side gradient step on the FP32 CUDA cores: the paper's small CNN (model endnote),
// forward and backward, for W workers that may hold different weight snapshots.
//
// Rows of every activation buffer are (sorted worker s, sample i) -> s*b + i, where the sorted
// order places workers that share a snapshot next to each other, so that a group's samples form
// one contiguous row range and the dense layers can run one tiled product per group.
//
// Every reduction is taken in a fixed order (no floating-point atomics), so that two runs on the
// same inputs give the same bits.
#include "kernels.h"
#include "device_common.cuh"

namespace psk {

namespace {

// ---- conv1 (1->16, 3x3, pad 1) + ReLU + 2x2 max pool.  A block handles up to CONV1_SPB samples of one
// worker.  Thread = pooled position: it reads the 4x4 input patch under its 2x2 window once and
// evaluates all 16 channels from registers (576 multiply-adds per 8 + 48 shared-memory loads).
// (FP32 path; the tensor-core path has its own kernel, which writes the layout its convolutions copy from.)
constexpr int CONV1_SPB = 8;
__global__ void __launch_bounds__(224) conv1_fwd(GradStepArgs a, WorkerTable wt, GroupTable gt, Workspace ws) {
  __shared__ __align__(16) float xs[2][30][32];
  __shared__ __align__(16) float w[16][12];   // 9 taps + bias + padding
  const int s = blockIdx.y, tid = threadIdx.x;
  const float* theta = group_theta(wt, gt, s);
  if (tid < 160) {
    if (tid < 144) w[tid / 9][tid % 9] = theta[OFF_C1W + tid];
    else w[tid - 144][9] = theta[OFF_C1B + tid - 144];
  }
  for (int t = tid; t < 2 * 30 * 32; t += 224) (&xs[0][0][0])[t] = 0.f;
  const int i0 = blockIdx.x * CONV1_SPB, i1 = min(i0 + CONV1_SPB, a.b);
  const int py = tid / 14, px = tid - py * 14;
  const bool active = tid < 196;
  __syncthreads();
  auto stage = [&](int i, int bufi) {
    const float* x = a.x + ((int64_t)wt.src[s] * a.b + i) * (IMG * IMG);
    for (int t = tid; t < IMG * IMG; t += 224) {
      int yy = t / IMG, xx = t - yy * IMG;
      xs[bufi][yy + 1][xx + 1] = x[t];
    }
  };
  stage(i0, 0);
  for (int i = i0; i < i1; ++i) {
    const int cur = (i - i0) & 1;
    __syncthreads();                       // image `cur` is complete; image `cur^1` is no longer read
    if (i + 1 < i1) stage(i + 1, cur ^ 1);
    if (!active) continue;
    const int64_t row = (int64_t)s * a.b + i;
    float patch[4][4];
#pragma unroll
    for (int yy = 0; yy < 4; ++yy) {
      float2 lo = *reinterpret_cast<const float2*>(&xs[cur][2 * py + yy][2 * px]);
      float2 hi = *reinterpret_cast<const float2*>(&xs[cur][2 * py + yy][2 * px + 2]);
      patch[yy][0] = lo.x; patch[yy][1] = lo.y; patch[yy][2] = hi.x; patch[yy][3] = hi.y;
    }
    float outv[16];
    uint8_t outc[16];
#pragma unroll
    for (int ch = 0; ch < 16; ++ch) {
      const float4 w0 = *reinterpret_cast<const float4*>(&w[ch][0]);
      const float4 w1 = *reinterpret_cast<const float4*>(&w[ch][4]);
      const float4 w2 = *reinterpret_cast<const float4*>(&w[ch][8]);
      const float wv[9] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w, w2.x};
      const float bias = w2.y;
      float best = 0.f;
      int bi = 0;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int jy = j >> 1, jx = j & 1;
        float v = bias;
#pragma unroll
        for (int ky = 0; ky < 3; ++ky)
#pragma unroll
          for (int kx = 0; kx < 3; ++kx) v = fmaf(wv[ky * 3 + kx], patch[jy + ky][jx + kx], v);
        float r = fmaxf(v, 0.f);
        if (j == 0 || r > best) { best = r; bi = j; }
      }
      outv[ch] = best;
      outc[ch] = best > 0.f ? (uint8_t)bi : (uint8_t)4;
    }
    const int pp = tid;
#pragma unroll
    for (int ch = 0; ch < 16; ++ch) ws.code1[row * P1_ELEMS + ch * 196 + pp] = outc[ch];
#pragma unroll
    for (int ch = 0; ch < 16; ++ch) ws.p1[row * P1_ELEMS + ch * 196 + pp] = outv[ch];
  }
}

// ---- conv2 (16->32, 3x3, pad 1) + ReLU + 2x2 max pool.  A block handles up to CONV_SPB samples of
// one worker; the filter bank stays in shared memory.  Thread = (pooled position, group of 8 output
// channels): it accumulates the 2x2 pre-pool window of its 8 channels from a 4x4 input patch.
__global__ void __launch_bounds__(256) conv2_fwd(GradStepArgs a, WorkerTable wt, GroupTable gt, Workspace ws) {
  __shared__ float w[4608 + 32];
  __shared__ float in[16][16][17];
  const int s = blockIdx.y, tid = threadIdx.x;
  const float* theta = group_theta(wt, gt, s);
  for (int t = tid; t < 4640; t += 256) w[t] = theta[OFF_C2W + t];
  for (int t = tid; t < 16 * 16 * 17; t += 256) (&in[0][0][0])[t] = 0.f;
  const int i0 = blockIdx.x * CONV_SPB;
  const int i1 = min(i0 + CONV_SPB, a.b);
  for (int i = i0; i < i1; ++i) {
    const int64_t row = (int64_t)s * a.b + i;
    __syncthreads();
    for (int t = tid; t < P1_ELEMS; t += 256) {
      int ic = t / 196, pp = t % 196;
      in[ic][pp / 14 + 1][pp % 14 + 1] = ws.p1[row * P1_ELEMS + t];
    }
    __syncthreads();
    if (tid < 196) {
      const int pos = tid % 49, og = tid / 49;
      const int py = pos / 7, px = pos % 7;
      float acc[8][4];
#pragma unroll
      for (int o = 0; o < 8; ++o) {
        float bias = w[4608 + og * 8 + o];
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[o][j] = bias;
      }
      for (int ic = 0; ic < 16; ++ic) {
        float patch[4][4];
#pragma unroll
        for (int yy = 0; yy < 4; ++yy)
#pragma unroll
          for (int xx = 0; xx < 4; ++xx) patch[yy][xx] = in[ic][2 * py + yy][2 * px + xx];
#pragma unroll
        for (int o = 0; o < 8; ++o) {
          const float* wk = &w[((og * 8 + o) * 16 + ic) * 9];
#pragma unroll
          for (int ky = 0; ky < 3; ++ky)
#pragma unroll
            for (int kx = 0; kx < 3; ++kx) {
              float wv = wk[ky * 3 + kx];
              acc[o][0] = fmaf(wv, patch[ky][kx], acc[o][0]);
              acc[o][1] = fmaf(wv, patch[ky][kx + 1], acc[o][1]);
              acc[o][2] = fmaf(wv, patch[ky + 1][kx], acc[o][2]);
              acc[o][3] = fmaf(wv, patch[ky + 1][kx + 1], acc[o][3]);
            }
        }
      }
#pragma unroll
      for (int o = 0; o < 8; ++o) {
        float best = 0.f;
        int bi = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          float r = fmaxf(acc[o][j], 0.f);
          if (j == 0 || r > best) { best = r; bi = j; }
        }
        int idx = (og * 8 + o) * 49 + pos;
        ws.p2[row * FLAT + idx] = best;
        ws.code2[row * FLAT + idx] = best > 0.f ? (uint8_t)bi : (uint8_t)4;
      }
    }
  }
}

// ---- 64x64x16 tiled FP32 product, 256 threads, 4x4 outputs per thread.
// A(m,k) = A[m*lda + k] (A_KC) or A[k*lda + m]; B(k,n) = B[n*ldb + k] (B_KC) or B[k*ldb + n].
// All leading dimensions and tile origins are multiples of 4, so float4 loads stay aligned.
template <bool A_KC, bool B_KC>
__device__ __forceinline__ void gemm_tile_64(const float* __restrict__ A, int lda, const float* __restrict__ B,
                                             int ldb, int M, int N, int K, int m0, int n0,
                                             float (&acc)[4][4]) {
  __shared__ __align__(16) float As[16][68];
  __shared__ __align__(16) float Bs[16][68];
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int c = 0; c < 4; ++c) acc[r][c] = 0.f;
  for (int k0 = 0; k0 < K; k0 += 16) {
    {
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (A_KC) {
        int m = tid >> 2, k = (tid & 3) * 4;
        if (m0 + m < M && k0 + k < K) v = *reinterpret_cast<const float4*>(A + (int64_t)(m0 + m) * lda + k0 + k);
        As[k][m] = v.x; As[k + 1][m] = v.y; As[k + 2][m] = v.z; As[k + 3][m] = v.w;
      } else {
        int k = tid >> 4, m = (tid & 15) * 4;
        if (k0 + k < K && m0 + m < M) v = *reinterpret_cast<const float4*>(A + (int64_t)(k0 + k) * lda + m0 + m);
        *reinterpret_cast<float4*>(&As[k][m]) = v;
      }
    }
    {
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (B_KC) {
        int n = tid >> 2, k = (tid & 3) * 4;
        if (n0 + n < N && k0 + k < K) v = *reinterpret_cast<const float4*>(B + (int64_t)(n0 + n) * ldb + k0 + k);
        Bs[k][n] = v.x; Bs[k + 1][n] = v.y; Bs[k + 2][n] = v.z; Bs[k + 3][n] = v.w;
      } else {
        int k = tid >> 4, n = (tid & 15) * 4;
        if (k0 + k < K && n0 + n < N) v = *reinterpret_cast<const float4*>(B + (int64_t)(k0 + k) * ldb + n0 + n);
        *reinterpret_cast<float4*>(&Bs[k][n]) = v;
      }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      float4 av = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
      float4 bv = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
      float ar[4] = {av.x, av.y, av.z, av.w}, br[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[r][c] = fmaf(ar[r], br[c], acc[r][c]);
    }
    __syncthreads();
  }
}

// ---- fc1 forward: d = dropout(ReLU(p2 * W1^T + b1)), one product per weight group.
__global__ void __launch_bounds__(256) fc1_fwd(GradStepArgs a, WorkerTable wt, GroupTable gt, Workspace ws) {
  int g, m0, m_end;
  if (!locate_group_tile<64>(gt, a.b, blockIdx.y, g, m0, m_end)) return;
  const float* theta = gt.theta[g];
  const int n0 = blockIdx.x * 64;
  float acc[4][4];
  gemm_tile_64<true, true>(ws.p2, FLAT, theta + OFF_F1W, FLAT, m_end, HID, FLAT, m0, n0, acc);
  const int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
  const int n = n0 + tx * 4;
  const float4 bias = *reinterpret_cast<const float4*>(theta + OFF_F1B + n);
  const float scale = 1.0f / (1.0f - a.drop_p);
  const uint2 key = make_uint2((uint32_t)a.seed, (uint32_t)(a.seed >> 32));
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    int m = m0 + ty * 4 + r;
    if (m >= m_end) continue;
    int s = m / a.b, i = m - s * a.b;
    uint32_t q = (uint32_t)((i * HID + n) >> 2);
    uint4 rnd = philox4x32_10(make_uint4(q, (uint32_t)wt.wid[s], (uint32_t)a.step, (uint32_t)(a.step >> 32)), key);
    float4 o;
    o.x = rnd.x >= a.drop_thresh ? fmaxf(acc[r][0] + bias.x, 0.f) * scale : 0.f;
    o.y = rnd.y >= a.drop_thresh ? fmaxf(acc[r][1] + bias.y, 0.f) * scale : 0.f;
    o.z = rnd.z >= a.drop_thresh ? fmaxf(acc[r][2] + bias.z, 0.f) * scale : 0.f;
    o.w = rnd.w >= a.drop_thresh ? fmaxf(acc[r][3] + bias.w, 0.f) * scale : 0.f;
    *reinterpret_cast<float4*>(ws.d + (int64_t)m * HID + n) = o;
  }
}

// ---- fc2 forward, softmax cross-entropy, argmax, and the backward pass down to the gradient with
// respect to fc1's pre-activation; then the worker's fc2 weight/bias and fc1 bias gradients.
// FC2_SPLIT blocks of 16 warps per worker, each with its share of the worker's samples: first four samples per
// warp at a time; then thread = hidden unit sums its outputs over the block's samples in sample order, many
// loads in flight.  The block's sums (and its share of the loss) are partial results added later in block order.
constexpr int FC2_THREADS = 512;
constexpr int FC2_NS = 4;          // samples per warp and pass
constexpr int DZ_CHUNK = 128;      // samples whose logits gradients are held in shared memory at a time
constexpr int W2T_PITCH = 12;      // 48-byte rows: 16-byte loads of consecutive rows fall on distinct banks
__global__ void __launch_bounds__(FC2_THREADS, 1) fc2_fwd_bwd(GradStepArgs a, WorkerTable wt, GroupTable gt, Workspace ws) {
  __shared__ __align__(16) float w2t[HID][W2T_PITCH];     // w2t[j][c] = W2[c][j]; the two pad columns are zero
  __shared__ __align__(16) float dzs[DZ_CHUNK][W2T_PITCH];   // logits gradients of a chunk of samples
  __shared__ float b2[NCLS];
  __shared__ float warp_loss[FC2_THREADS / 32];
  const int s = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* theta = group_theta(wt, gt, s);
  const int src = wt.src[s];
  const int per = ((a.b + FC2_SPLIT - 1) / FC2_SPLIT + 1) & ~1;          // samples per block, even
  const int i_lo = min(a.b, (int)blockIdx.y * per), i_hi = min(a.b, i_lo + per);
  for (int t = tid; t < NCLS * HID; t += FC2_THREADS) w2t[t % HID][t / HID] = theta[OFF_F2W + t];
  w2t[tid][NCLS] = w2t[tid][NCLS + 1] = 0.f;
  if (tid < NCLS) b2[tid] = theta[OFF_F2B + tid];
  __syncthreads();
  const float scale = 1.0f / (1.0f - a.drop_p);
  const float inv_b = 1.0f / (float)a.b;
  float loss_acc = 0.f;
  // Four samples per warp and pass, so that every weight read from shared memory is used four times.  A lane owns
  // the 16 hidden units lane + 32 t.
  const bool hi16 = lane & 16, hi8 = lane & 8, hi4 = lane & 4;
  const int my_u = lane >> 3, sub = lane & 7;          // after the reduction a lane works for sample my_u of the pass
  for (int i0 = i_lo + FC2_NS * warp; i0 < i_hi; i0 += FC2_NS * (FC2_THREADS / 32)) {
    const int n_s = min(FC2_NS, i_hi - i0);              // warp-uniform
    const bool mine = my_u < n_s;
    // the weights are re-read from shared memory on every pass: 160 of them per lane would not fit in the
    // registers of a 512-thread block, so their address is made to look pass-dependent
    uint32_t opaque_zero;
    asm volatile("mov.u32 %0, 0;" : "=r"(opaque_zero));
    const float4* w2p = reinterpret_cast<const float4*>(&w2t[0][0] + opaque_zero);
    const int64_t row0 = (int64_t)s * a.b + i0;
    // the label is asked for now: by the time the softmax needs it, it has arrived
    int label = a.y[(int64_t)src * a.b + i0 + (mine ? my_u : 0)];
    // classes in pairs, one packed multiply-add per pair: zp[u][k] = logits 2k and 2k + 1 of sample u
    u64 zp[FC2_NS][NCLS / 2];
    uint32_t live[FC2_NS];                               // which of the lane's 16 units passed ReLU and dropout
#pragma unroll
    for (int u = 0; u < FC2_NS; ++u) {
      live[u] = 0u;
#pragma unroll
      for (int k = 0; k < NCLS / 2; ++k) zp[u][k] = 0ull;
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {                        // the units in two halves, to bound the registers
      float dv[FC2_NS][8];
#pragma unroll
      for (int u = 0; u < FC2_NS; ++u)
#pragma unroll
        for (int t = 0; t < 8; ++t) dv[u][t] = ws.d[(row0 + (u < n_s ? u : 0)) * HID + lane + 32 * (8 * h + t)];
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        const float4* wr = w2p + (lane + 32 * (8 * h + t)) * (W2T_PITCH / 4);
        const float4 q0 = wr[0], q1 = wr[1], q2 = wr[2];
        const u64 wk[NCLS / 2] = {pack2(q0.x, q0.y), pack2(q0.z, q0.w), pack2(q1.x, q1.y), pack2(q1.z, q1.w), pack2(q2.x, q2.y)};
#pragma unroll
        for (int u = 0; u < FC2_NS; ++u) {
          live[u] |= (dv[u][t] > 0.f ? 1u : 0u) << (8 * h + t);
          const u64 du = pack2(dv[u][t], dv[u][t]);
#pragma unroll
          for (int k = 0; k < NCLS / 2; ++k) zp[u][k] = ffma2(wk[k], du, zp[u][k]);
        }
      }
    }
    // Sum over the lanes.  Each exchange halves what a lane goes on with: after the first two a lane holds the ten
    // partial logits of sample lane / 8 only, after the third five of them; two plain exchanges finish the sums and a
    // last one brings the two halves of the classes together.
    float v[FC2_NS * NCLS];
#pragma unroll
    for (int u = 0; u < FC2_NS; ++u)
#pragma unroll
      for (int k = 0; k < NCLS / 2; ++k) unpack2(zp[u][k], v[u * NCLS + 2 * k], v[u * NCLS + 2 * k + 1]);
    float w20[2 * NCLS], x10[NCLS], y5[NCLS / 2], z[NCLS];
#pragma unroll
    for (int k = 0; k < 2 * NCLS; ++k) {
      const float keep = hi16 ? v[2 * NCLS + k] : v[k], send = hi16 ? v[k] : v[2 * NCLS + k];
      w20[k] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
    }
#pragma unroll
    for (int k = 0; k < NCLS; ++k) {
      const float keep = hi8 ? w20[NCLS + k] : w20[k], send = hi8 ? w20[k] : w20[NCLS + k];
      x10[k] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
    }
#pragma unroll
    for (int k = 0; k < NCLS / 2; ++k) {
      const float keep = hi4 ? x10[NCLS / 2 + k] : x10[k], send = hi4 ? x10[k] : x10[NCLS / 2 + k];
      y5[k] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
      y5[k] += __shfl_xor_sync(0xffffffffu, y5[k], 2);
      y5[k] += __shfl_xor_sync(0xffffffffu, y5[k], 1);
    }
#pragma unroll
    for (int k = 0; k < NCLS / 2; ++k) {
      const float other = __shfl_xor_sync(0xffffffffu, y5[k], 4);
      z[k] = (hi4 ? other : y5[k]) + b2[k];
      z[NCLS / 2 + k] = (hi4 ? y5[k] : other) + b2[NCLS / 2 + k];
    }
    // softmax, loss and logits gradient of the lane's sample (the eight lanes of a sample do the same work)
    float dzl[NCLS];
    {
      float zmax = z[0];
      int am = 0;
#pragma unroll
      for (int c = 1; c < NCLS; ++c)
        if (z[c] > zmax) { zmax = z[c]; am = c; }
      float ez[NCLS], se = 0.f;
#pragma unroll
      for (int c = 0; c < NCLS; ++c) { ez[c] = expf(z[c] - zmax); se += ez[c]; }
      const float lse = zmax + logf(se), inv_se = 1.0f / se;
      if (label < 0 || label >= NCLS) {
        if (mine && sub == 0) atomicOr(ws.status, STATUS_BAD_LABEL);
        label = 0;
      }
      float zy = 0.f;
#pragma unroll
      for (int c = 0; c < NCLS; ++c) {
        if (c == label) zy = z[c];
        const float g = (ez[c] * inv_se - (c == label ? 1.f : 0.f)) * inv_b;     // softmax from the exponentials already taken
        dzl[c] = mine ? g : 0.f;
      }
      if (mine) {
        loss_acc += lse - zy;
        if (sub == 0) a.argmax[(int64_t)src * a.b + i0 + my_u] = am;
        float e0 = 0.f, e1 = 0.f;                          // lane sub of a sample stores elements 2 sub and 2 sub + 1 of its padded row
#pragma unroll
        for (int m = 0; m < NCLS / 2; ++m)
          if (sub == m) { e0 = dzl[2 * m]; e1 = dzl[2 * m + 1]; }
        *reinterpret_cast<float2*>(ws.dz + (row0 + my_u) * DZ_STRIDE + 2 * sub) = make_float2(e0, e1);
      }
    }
    // every lane needs the logits gradients of all four samples, as class pairs
    u64 dzk[FC2_NS][NCLS / 2];
#pragma unroll
    for (int u = 0; u < FC2_NS; ++u)
#pragma unroll
      for (int k = 0; k < NCLS / 2; ++k)
        dzk[u][k] = pack2(__shfl_sync(0xffffffffu, dzl[2 * k], 8 * u), __shfl_sync(0xffffffffu, dzl[2 * k + 1], 8 * u));
    asm volatile("mov.u32 %0, 0;" : "=r"(opaque_zero));    // second read of the weights, as above
    w2p = reinterpret_cast<const float4*>(&w2t[0][0] + opaque_zero);
#pragma unroll 2
    for (int t = 0; t < 16; ++t) {
      const int j = lane + 32 * t;
      const float4* wr = w2p + j * (W2T_PITCH / 4);
      const float4 q0 = wr[0], q1 = wr[1], q2 = wr[2];
      const u64 wk[NCLS / 2] = {pack2(q0.x, q0.y), pack2(q0.z, q0.w), pack2(q1.x, q1.y), pack2(q1.z, q1.w), pack2(q2.x, q2.y)};
#pragma unroll
      for (int u = 0; u < FC2_NS; ++u) {
        // even classes accumulate in the low half, odd classes in the high half; the halves are added at the end
        u64 e = 0ull;
#pragma unroll
        for (int k = 0; k < NCLS / 2; ++k) e = ffma2(wk[k], dzk[u][k], e);
        float lo, hi;
        unpack2(e, lo, hi);
        float o = (live[u] >> t) & 1u ? (lo + hi) * scale : 0.f;
        if (a.precision != 0) o = round_tf32(o);             // it feeds tensor-core products only
        if (u < n_s) ws.da1[(row0 + u) * HID + j] = o;
      }
    }
  }
  {
    // the eight lanes of a sample hold the same loss: one of each, in lane order
    const float l0 = __shfl_sync(0xffffffffu, loss_acc, 0), l1 = __shfl_sync(0xffffffffu, loss_acc, 8);
    const float l2 = __shfl_sync(0xffffffffu, loss_acc, 16), l3 = __shfl_sync(0xffffffffu, loss_acc, 24);
    loss_acc = (l0 + l1) + (l2 + l3);
  }
  if (lane == 0) warp_loss[warp] = loss_acc;
  __syncthreads();   // also makes this block's dz / da1 stores visible to all of its threads
  float* part = ws.partf + ((int64_t)s * FC2_SPLIT + blockIdx.y) * FC_PART;
  if (tid == 0) {
    float t = 0.f;
    for (int w = 0; w < FC2_THREADS / 32; ++w) t += warp_loss[w];
    part[NCLS * HID + HID + NCLS] = t;
  }
  const int j = tid;                                  // hidden unit (FC2_THREADS == HID)
  float gw[NCLS], gb1 = 0.f, gb2 = 0.f;
#pragma unroll
  for (int c = 0; c < NCLS; ++c) gw[c] = 0.f;
  const float* dzp = ws.dz + (int64_t)s * a.b * DZ_STRIDE;
  const float* dp = ws.d + (int64_t)s * a.b * HID + j;
  const float* da1p = ws.da1 + (int64_t)s * a.b * HID + j;
  u64 gwk[NCLS / 2];
#pragma unroll
  for (int k = 0; k < NCLS / 2; ++k) gwk[k] = 0ull;
  // The logits gradients of DZ_CHUNK samples at a time are brought into shared memory, where every thread reads
  // them as broadcasts; what is left per sample is two loads from global memory, many of them in flight.
  for (int c0 = i_lo; c0 < i_hi; c0 += DZ_CHUNK) {
    const int n = min(DZ_CHUNK, i_hi - c0);
    __syncthreads();
    for (int t = tid; t < n * (W2T_PITCH / 4); t += FC2_THREADS) {
      const int i = t / (W2T_PITCH / 4), q = t - i * (W2T_PITCH / 4);
      reinterpret_cast<float4*>(&dzs[i][0])[q] = *reinterpret_cast<const float4*>(dzp + (c0 + i) * DZ_STRIDE + 4 * q);
    }
    __syncthreads();
#pragma unroll 16
    for (int i = 0; i < n; ++i) {
      const float dval = dp[(int64_t)(c0 + i) * HID];
      const float4* zr = reinterpret_cast<const float4*>(&dzs[i][0]);
      const float4 z0 = zr[0], z1 = zr[1], z2 = zr[2];
      const u64 dzk[NCLS / 2] = {pack2(z0.x, z0.y), pack2(z0.z, z0.w), pack2(z1.x, z1.y), pack2(z1.z, z1.w), pack2(z2.x, z2.y)};
      const u64 dd = pack2(dval, dval);
#pragma unroll
      for (int k = 0; k < NCLS / 2; ++k) gwk[k] = ffma2(dzk[k], dd, gwk[k]);
      gb1 += da1p[(int64_t)(c0 + i) * HID];
    }
    if (j < NCLS)
      for (int i = 0; i < n; ++i) gb2 += dzs[i][j];
  }
#pragma unroll
  for (int k = 0; k < NCLS / 2; ++k) unpack2(gwk[k], gw[2 * k], gw[2 * k + 1]);
#pragma unroll
  for (int c = 0; c < NCLS; ++c) part[c * HID + j] = gw[c];
  part[NCLS * HID + j] = gb1;
  if (j < NCLS) part[NCLS * HID + HID + j] = gb2;
}

// ---- fc1 weight gradient of one worker: dW1 [512][1568] = da1^T [512 x b] * p2 [b x 1568].
__global__ void __launch_bounds__(256) fc1_dw(GradStepArgs a, WorkerTable wt, Workspace ws) {
  const int s = blockIdx.z, m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  const float* A = ws.da1 + (int64_t)s * a.b * HID;
  const float* B = ws.p2 + (int64_t)s * a.b * FLAT;
  float acc[4][4];
  gemm_tile_64<false, false>(A, HID, B, FLAT, HID, FLAT, a.b, m0, n0, acc);
  const int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
  const int n = n0 + tx * 4;
  if (n >= FLAT) return;
  float* out = wt.grad[s] + OFF_F1W;
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    int m = m0 + ty * 4 + r;
    *reinterpret_cast<float4*>(out + (int64_t)m * FLAT + n) = make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]);
  }
}

// ---- gradient with respect to p2: dp2 [rows][1568] = da1 [rows][512] * W1 [512][1568], per group.
__global__ void __launch_bounds__(256) fc1_dx(GradStepArgs a, GroupTable gt, Workspace ws) {
  int g, m0, m_end;
  if (!locate_group_tile<64>(gt, a.b, blockIdx.y, g, m0, m_end)) return;
  const int n0 = blockIdx.x * 64;
  float acc[4][4];
  gemm_tile_64<true, false>(ws.da1, HID, gt.theta[g] + OFF_F1W, FLAT, m_end, FLAT, HID, m0, n0, acc);
  const int ty = threadIdx.x >> 4, tx = threadIdx.x & 15;
  const int n = n0 + tx * 4;
  if (n >= FLAT) return;
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    int m = m0 + ty * 4 + r;
    if (m >= m_end) continue;
    *reinterpret_cast<float4*>(ws.dp2 + (int64_t)m * FLAT + n) = make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]);
  }
}

// ---- backward through pool2, ReLU and conv2 for up to CONV_SPB samples of one worker:
// writes dp1 per sample and the block's partial filter / bias gradients.
constexpr int C2B_SMEM_FLOATS = 4608 + 32 * 16 * 17 + 16 * 16 * 17;
__global__ void __launch_bounds__(256) conv2_bwd(GradStepArgs a, WorkerTable wt, GroupTable gt, Workspace ws, int n_chunks) {
  extern __shared__ float smem[];
  float* w = smem;                                                        // [32][16][9]
  float (*g2)[16][17] = reinterpret_cast<float (*)[16][17]>(smem + 4608); // [32] padded gradient at conv2 output
  float (*in)[16][17] = reinterpret_cast<float (*)[16][17]>(smem + 4608 + 32 * 16 * 17);  // [16] padded p1
  const int s = blockIdx.y, tid = threadIdx.x;
  const float* theta = group_theta(wt, gt, s);
  for (int t = tid; t < 4608; t += 256) w[t] = theta[OFF_C2W + t];
  for (int t = tid; t < 16 * 16 * 17; t += 256) (&in[0][0][0])[t] = 0.f;
  const int oc_w = tid >> 3, ic_w = (tid & 7) * 2;   // filter-gradient ownership: (oc, two input channels)
  float gw[2][9], gb = 0.f;
#pragma unroll
  for (int h = 0; h < 2; ++h)
#pragma unroll
    for (int k = 0; k < 9; ++k) gw[h][k] = 0.f;
  const int i0 = blockIdx.x * CONV_SPB;
  const int i1 = min(i0 + CONV_SPB, a.b);
  for (int i = i0; i < i1; ++i) {
    const int64_t row = (int64_t)s * a.b + i;
    __syncthreads();
    for (int t = tid; t < 32 * 16 * 17; t += 256) (&g2[0][0][0])[t] = 0.f;
    for (int t = tid; t < P1_ELEMS; t += 256) {
      int ic = t / 196, pp = t % 196;
      in[ic][pp / 14 + 1][pp % 14 + 1] = ws.p1[row * P1_ELEMS + t];
    }
    __syncthreads();
    for (int t = tid; t < FLAT; t += 256) {
      int code = ws.code2[row * FLAT + t];
      if (code < 4) {
        int oc = t / 49, pp = t % 49;
        int y = 2 * (pp / 7) + (code >> 1), x = 2 * (pp % 7) + (code & 1);
        g2[oc][y + 1][x + 1] = ws.dp2[row * FLAT + t];
      }
    }
    __syncthreads();
    // gradient with respect to the conv2 input (p1)
    if (tid < 196) {
      const int y = tid / 14, x = tid % 14;
      float acc[16];
#pragma unroll
      for (int ic = 0; ic < 16; ++ic) acc[ic] = 0.f;
      for (int oc = 0; oc < 32; ++oc) {
#pragma unroll
        for (int ky = 0; ky < 3; ++ky)
#pragma unroll
          for (int kx = 0; kx < 3; ++kx) {
            float g = g2[oc][y - ky + 2][x - kx + 2];
            if (g != 0.f) {
#pragma unroll
              for (int ic = 0; ic < 16; ++ic) acc[ic] = fmaf(g, w[(oc * 16 + ic) * 9 + ky * 3 + kx], acc[ic]);
            }
          }
      }
#pragma unroll
      for (int ic = 0; ic < 16; ++ic) ws.dp1[row * P1_ELEMS + ic * 196 + tid] = acc[ic];
    }
    // filter and bias gradients
    for (int y = 0; y < 14; ++y)
      for (int x = 0; x < 14; ++x) {
        float g = g2[oc_w][y + 1][x + 1];
        if (g != 0.f) {
          if ((tid & 7) == 0) gb += g;
#pragma unroll
          for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int ky = 0; ky < 3; ++ky)
#pragma unroll
              for (int kx = 0; kx < 3; ++kx) gw[h][ky * 3 + kx] = fmaf(g, in[ic_w + h][y + ky][x + kx], gw[h][ky * 3 + kx]);
        }
      }
  }
  float* part = ws.part2 + ((int64_t)s * n_chunks + blockIdx.x) * C2_GRAD;
#pragma unroll
  for (int h = 0; h < 2; ++h)
#pragma unroll
    for (int k = 0; k < 9; ++k) part[(oc_w * 16 + ic_w + h) * 9 + k] = gw[h][k];
  if ((tid & 7) == 0) part[4608 + oc_w] = gb;
}

// ---- backward through pool1, ReLU and conv1 (filter / bias gradients only: the input needs none).
// Thread (channel, lane of 16) owns 13 pooled positions of its channel.  The image, the pooling decisions
// and the pooled gradients of the NEXT sample are fetched into registers while the current one is
// accumulated, so that no global-memory latency sits between the multiply-adds.
constexpr int CONV1B_SPB = 16;
__global__ void __launch_bounds__(256) conv1_bwd(GradStepArgs a, WorkerTable wt, Workspace ws, int n_chunks) {
  __shared__ float xs[30][31];
  constexpr int PER = 13;                   // ceil(196 / 16)
  const int s = blockIdx.y, tid = threadIdx.x;
  const int oc = tid >> 4, l = tid & 15;
  float gw[9], gb = 0.f;
#pragma unroll
  for (int k = 0; k < 9; ++k) gw[k] = 0.f;
  for (int t = tid; t < 30 * 31; t += 256) (&xs[0][0])[t] = 0.f;
  const int i0 = blockIdx.x * CONV1B_SPB;
  const int i1 = min(i0 + CONV1B_SPB, a.b);
  float xr[4], gr[PER];
  int cr[PER];
  auto prefetch = [&](int i) {
    const int64_t row = (int64_t)s * a.b + i;
    const float* x = a.x + ((int64_t)wt.src[s] * a.b + i) * (IMG * IMG);
#pragma unroll
    for (int k = 0; k < 4; ++k) xr[k] = tid + 256 * k < IMG * IMG ? x[tid + 256 * k] : 0.f;
#pragma unroll
    for (int k = 0; k < PER; ++k) {
      const int pp = l + 16 * k;
      cr[k] = pp < 196 ? (int)ws.code1[row * P1_ELEMS + oc * 196 + pp] : 4;
      gr[k] = pp < 196 ? ws.dp1[row * P1_ELEMS + oc * 196 + pp] : 0.f;
    }
  };
  prefetch(i0);
  for (int i = i0; i < i1; ++i) {
    __syncthreads();                        // the previous sample's image is no longer read
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int t = tid + 256 * k;
      if (t < IMG * IMG) xs[t / IMG + 1][t % IMG + 1] = xr[k];
    }
    float g_cur[PER];
    int c_cur[PER];
#pragma unroll
    for (int k = 0; k < PER; ++k) { g_cur[k] = gr[k]; c_cur[k] = cr[k]; }
    __syncthreads();
    if (i + 1 < i1) prefetch(i + 1);
#pragma unroll
    for (int k = 0; k < PER; ++k) {
      if (c_cur[k] < 4) {
        const int pp = l + 16 * k;
        const float g = g_cur[k];
        const int y = 2 * (pp / 14) + (c_cur[k] >> 1), xq = 2 * (pp % 14) + (c_cur[k] & 1);
        gb += g;
#pragma unroll
        for (int ky = 0; ky < 3; ++ky)
#pragma unroll
          for (int kx = 0; kx < 3; ++kx) gw[ky * 3 + kx] = fmaf(g, xs[y + ky][xq + kx], gw[ky * 3 + kx]);
      }
    }
  }
  // fixed-order reduction over the 16 lanes that share an output channel
#pragma unroll
  for (int o = 8; o > 0; o >>= 1) {
    gb += __shfl_xor_sync(0xffffffffu, gb, o);
#pragma unroll
    for (int k = 0; k < 9; ++k) gw[k] += __shfl_xor_sync(0xffffffffu, gw[k], o);
  }
  if (l == 0) {
    float* part = ws.part1 + ((int64_t)s * n_chunks + blockIdx.x) * C1_GRAD;
#pragma unroll
    for (int k = 0; k < 9; ++k) part[oc * 9 + k] = gw[k];
    part[144 + oc] = gb;
  }
}

// ---- sums the per-block partial gradients in block order, finishes the loss and zeroes the padding.
// part2 holds n_chunks2 slots per worker; all of them are summed when seg_len == 0, otherwise one for every
// range of seg_len rows that meets the worker's b rows (the tensor-core filter-gradient kernel's layout).
// A worker's outputs are numbered conv2 (4640), conv1 (160), output layer (5642), loss, padding; a block takes
// RED_PER_BLOCK of them.
constexpr int RED_PER_BLOCK = 1024;
constexpr int RED_OUTPUTS = C2_GRAD + C1_GRAD + (NCLS * HID + HID + NCLS) + 1 + (P_PAD - P);
constexpr int RED_BLOCKS = (RED_OUTPUTS + RED_PER_BLOCK - 1) / RED_PER_BLOCK;
__global__ void __launch_bounds__(256) conv_grad_reduce(GradStepArgs a, WorkerTable wt, Workspace ws, int n_chunks, int seg_len1,
                                                        int n_chunks2, int seg_len) {
  const int s = blockIdx.x, b = a.b;
  float* grad = wt.grad[s];
  const int used2 = seg_len > 0 ? (s * b + b - 1) / seg_len - (s * b) / seg_len + 1 : n_chunks2;
  // part1 likewise: all n_chunks slots, or eight (sample of a pair x window element) for every range of seg_len1 rows
  const int used1 = seg_len1 > 0 ? 8 * ((s * b + b - 1) / seg_len1 - (s * b) / seg_len1 + 1) : n_chunks;
  for (int v = blockIdx.y * RED_PER_BLOCK + threadIdx.x; v < min(RED_OUTPUTS, ((int)blockIdx.y + 1) * RED_PER_BLOCK); v += 256) {
    int o = v;
    if (o < C2_GRAD) {
      float t = 0.f;
      for (int c = 0; c < used2; ++c) t += ws.part2[((int64_t)s * n_chunks2 + c) * C2_GRAD + o];
      grad[OFF_C2W + o] = t;
      continue;
    }
    o -= C2_GRAD;
    if (o < C1_GRAD) {
      float t = 0.f;
      for (int c = 0; c < used1; ++c) t += ws.part1[((int64_t)s * n_chunks + c) * C1_GRAD + o];
      grad[OFF_C1W + o] = t;
      continue;
    }
    o -= C1_GRAD;
    if (o <= NCLS * HID + HID + NCLS) {
      float t = 0.f;
#pragma unroll
      for (int c = 0; c < FC2_SPLIT; ++c) t += ws.partf[((int64_t)s * FC2_SPLIT + c) * FC_PART + o];
      if (o < NCLS * HID) grad[OFF_F2W + o] = t;
      else if (o < NCLS * HID + HID) grad[OFF_F1B + o - NCLS * HID] = t;
      else if (o < NCLS * HID + HID + NCLS) grad[OFF_F2B + o - NCLS * HID - HID] = t;
      else a.loss[wt.src[s]] = t * (1.0f / (float)b);
      continue;
    }
    o -= NCLS * HID + HID + NCLS + 1;
    grad[P + o] = 0.f;
  }
}

// ---- the summed step's final reduction: ONE gradient vector, the sum over all workers (who share one weight
// snapshot).  The 512-unit layer's weight gradient arrives as n_super partial vectors (one per group of workers whose
// samples went through one product), every other tensor as the per-worker, per-block partial sums the per-worker
// reduction also reads; everything is added in a fixed order (group after group, worker after worker, block after
// block).  Blocks 0 .. FUSED_W1_BLOCKS - 1 take the float4 columns of the big tensor, the rest the small outputs.
constexpr int FUSED_W1_VEC = HID * FLAT / 4;                                 // 200,704 float4
constexpr int FUSED_W1_BLOCKS = (FUSED_W1_VEC + 255) / 256;                  // 784
constexpr int FUSED_SMALL = C2_GRAD + C1_GRAD + (NCLS * HID + HID + NCLS) + (P_PAD - P);
constexpr int FUSED_SMALL_BLOCKS = (FUSED_SMALL + 7) / 8;                    // one warp per small output
__global__ void __launch_bounds__(256) fused_finish(GradStepArgs a, WorkerTable wt, Workspace ws, const float* __restrict__ super_part,
                                                    int n_super, float* __restrict__ grad_sum, int n_chunks, int seg_len1,
                                                    int n_chunks2, int seg_len) {
  const int b = a.b;
  if (blockIdx.x < FUSED_W1_BLOCKS) {
    const int i = blockIdx.x * 256 + threadIdx.x;
    if (i >= FUSED_W1_VEC) return;
    float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int g = 0; g < n_super; ++g) {
      const float4 v = reinterpret_cast<const float4*>(super_part + (int64_t)g * P_PAD + OFF_F1W)[i];
      t.x += v.x; t.y += v.y; t.z += v.z; t.w += v.w;
    }
    reinterpret_cast<float4*>(grad_sum + OFF_F1W)[i] = t;
    return;
  }
  // A small output is summed by one warp: lane l adds the partial sums of workers l, l + 32, ... in order, then the
  // lanes are combined by a butterfly, which is the same sequence of additions on every run.
  const int lane = threadIdx.x & 31;
  int o = (blockIdx.x - FUSED_W1_BLOCKS) * 8 + (threadIdx.x >> 5);
  if (blockIdx.x == FUSED_W1_BLOCKS && threadIdx.x < a.W) {      // the per-worker losses ride along (W <= 256)
    float t = 0.f;
#pragma unroll
    for (int c = 0; c < FC2_SPLIT; ++c) t += ws.partf[((int64_t)threadIdx.x * FC2_SPLIT + c) * FC_PART + NCLS * HID + HID + NCLS];
    a.loss[wt.src[threadIdx.x]] = t * (1.0f / (float)b);
  }
  if (o >= FUSED_SMALL) return;
  float t = 0.f;
  float* dst;
  if (o < C2_GRAD) {
    for (int s = lane; s < a.W; s += 32) {
      const int used2 = seg_len > 0 ? (s * b + b - 1) / seg_len - (s * b) / seg_len + 1 : n_chunks2;
      for (int c = 0; c < used2; ++c) t += ws.part2[((int64_t)s * n_chunks2 + c) * C2_GRAD + o];
    }
    dst = grad_sum + OFF_C2W + o;
  } else if (o < C2_GRAD + C1_GRAD) {
    const int oo = o - C2_GRAD;
    for (int s = lane; s < a.W; s += 32) {
      const int used1 = seg_len1 > 0 ? 8 * ((s * b + b - 1) / seg_len1 - (s * b) / seg_len1 + 1) : n_chunks;
      for (int c = 0; c < used1; ++c) t += ws.part1[((int64_t)s * n_chunks + c) * C1_GRAD + oo];
    }
    dst = grad_sum + OFF_C1W + oo;
  } else if (o < C2_GRAD + C1_GRAD + NCLS * HID + HID + NCLS) {
    const int oo = o - C2_GRAD - C1_GRAD;
    for (int s = lane; s < a.W; s += 32)
#pragma unroll
      for (int c = 0; c < FC2_SPLIT; ++c) t += ws.partf[((int64_t)s * FC2_SPLIT + c) * FC_PART + oo];
    dst = oo < NCLS * HID ? grad_sum + OFF_F2W + oo : (oo < NCLS * HID + HID ? grad_sum + OFF_F1B + oo - NCLS * HID : grad_sum + OFF_F2B + oo - NCLS * HID - HID);
  } else {
    dst = grad_sum + P + (o - C2_GRAD - C1_GRAD - NCLS * HID - HID - NCLS);      // padding: zero
  }
#pragma unroll
  for (int sh = 16; sh > 0; sh >>= 1) t += __shfl_xor_sync(0xffffffffu, t, sh);
  if (lane == 0) *dst = t;
}

// ---- evaluation: per worker, the mean loss from the output-layer kernel's partial sums and the number of samples
// whose predicted label equals the given one (an integer count, summed in a fixed order).
__global__ void __launch_bounds__(128) eval_finish(GradStepArgs a, WorkerTable wt, Workspace ws, int32_t* __restrict__ correct) {
  __shared__ int warp_hits[4];
  const int s = blockIdx.x, src = wt.src[s];
  int hits = 0;
  for (int i = threadIdx.x; i < a.b; i += 128) {
    const int64_t r = (int64_t)src * a.b + i;
    hits += a.argmax[r] == a.y[r] ? 1 : 0;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) hits += __shfl_xor_sync(0xffffffffu, hits, o);
  if ((threadIdx.x & 31) == 0) warp_hits[threadIdx.x >> 5] = hits;
  __syncthreads();
  if (threadIdx.x == 0) {
    correct[src] = warp_hits[0] + warp_hits[1] + warp_hits[2] + warp_hits[3];
    float t = 0.f;
#pragma unroll
    for (int c = 0; c < FC2_SPLIT; ++c) t += ws.partf[((int64_t)s * FC2_SPLIT + c) * FC_PART + NCLS * HID + HID + NCLS];
    a.loss[src] = t * (1.0f / (float)a.b);
  }
}

// ---- the keep mask on its own: thread e/4 draws the four words of elements 4*(e/4) .. +3.
__global__ void __launch_bounds__(256) dropout_mask(uint64_t seed, uint32_t worker, uint64_t step, int n_quads,
                                                    uint32_t thresh, uchar4* __restrict__ keep) {
  int q = blockIdx.x * 256 + threadIdx.x;
  if (q >= n_quads) return;
  uint4 r = philox4x32_10(make_uint4((uint32_t)q, worker, (uint32_t)step, (uint32_t)(step >> 32)),
                          make_uint2((uint32_t)seed, (uint32_t)(seed >> 32)));
  keep[q] = make_uchar4(r.x >= thresh, r.y >= thresh, r.z >= thresh, r.w >= thresh);
}

}  // namespace

#define TIMED(id, launch) do { if (prof) prof->begin(id, st); launch; if (prof) prof->end(st); } while (0)

int launch_dropout_mask(uint64_t seed, uint32_t worker, uint64_t step, int b, uint32_t thresh,
                        uint8_t* keep, cudaStream_t st, Profiler* prof) {
  int n_quads = b * HID / 4;
  TIMED(K_DROPOUT_MASK, (dropout_mask<<<(n_quads + 255) / 256, 256, 0, st>>>(seed, worker, step, n_quads, thresh,
                                                                            reinterpret_cast<uchar4*>(keep))));
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int configure_grad_kernels() {
  cudaError_t e = cudaFuncSetAttribute(conv2_bwd, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)(C2B_SMEM_FLOATS * sizeof(float)));
  return e == cudaSuccess ? 0 : -1;
}

// Evaluation pass: the forward kernels of the grad step with the dropout switched off (the output-layer kernel also
// produces backward quantities into the workspace; nothing reads them), then the per-worker loss and hit count.
int launch_eval(const GradStepArgs& a, const WorkerTable& wt, const GroupTable& gt, const Workspace& ws, int32_t* correct,
                cudaStream_t st, Profiler* prof) {
  const int n_chunks = (a.b + CONV_SPB - 1) / CONV_SPB;
  const int mt = group_tiles(gt, a.b, 64);
  int launches = 0;
  if (a.precision != 0) {
    if (!a.skip_prep_w1) launches += launch_prep_w1(gt, ws, st, prof);
    if (launch_conv1_fwd_planes(a, wt, gt, ws, st, prof) < 0) return -1;
    launch_conv2_fwd_tc5(a, wt, gt, ws, st, prof);
    const int n = launch_fc1_fwd_tc5(a, wt, gt, ws, st, prof);
    if (n < 0) return -1;
    launches += 2 + n;
  } else {
    const int n_chunks1 = (a.b + CONV1_SPB - 1) / CONV1_SPB;
    TIMED(K_CONV1_FWD, (conv1_fwd<<<dim3(n_chunks1, a.W), 224, 0, st>>>(a, wt, gt, ws)));
    TIMED(K_CONV2_FWD, (conv2_fwd<<<dim3(n_chunks, a.W), 256, 0, st>>>(a, wt, gt, ws)));
    TIMED(K_FC1_FWD, (fc1_fwd<<<dim3(HID / 64, mt), 256, 0, st>>>(a, wt, gt, ws)));
    launches += 3;
  }
  TIMED(K_FC2_FWD_BWD, (fc2_fwd_bwd<<<dim3(a.W, FC2_SPLIT), FC2_THREADS, 0, st>>>(a, wt, gt, ws)));
  TIMED(K_EVAL_FINISH, (eval_finish<<<a.W, 128, 0, st>>>(a, wt, ws, correct)));
  launches += 2;
  return cudaGetLastError() == cudaSuccess ? launches : -1;
}

// Launch order of one grad step.  On the tensor-core path the copies of the dense layer's weights are made on a
// side stream while the convolutions run, and the backward pass forks: once the output
// layer's backward has produced da1, the dense layer's per-worker weight gradient (bound by its 3.2 MB
// per worker of writes) runs on a side stream next to the input-gradient chain, and once dp2 exists the
// second convolution's filter gradient runs on another side stream next to its input gradient and the
// first convolution's backward.  Everything joins before the final reduction.
int launch_grad_step(const GradStepArgs& a, const WorkerTable& wt, const GroupTable& gt, const Workspace& ws,
                     cudaStream_t st, const SideStreams& side, Profiler* prof, const SummedStep* sum) {
  const int n_chunks = (a.b + CONV_SPB - 1) / CONV_SPB;
  const int mt = group_tiles(gt, a.b, 64);
  const bool tc = a.precision != 0;
  const int n_chunks1 = (a.b + CONV1_SPB - 1) / CONV1_SPB;
  const int n_chunks1b = (a.b + CONV1B_SPB - 1) / CONV1B_SPB;
  int launches = 0, n_chunks2 = n_chunks, seg_len = 0;
  // Summed step: the 512-unit layer's weight gradient is taken over groups of workers at once ("super-workers" of
  // W / n_super workers: their samples are consecutive rows, so the product only sees a longer batch) and written to
  // n_super partial vectors instead of one vector per worker.
  GradStepArgs a_dw = a;
  WorkerTable wt_dw = wt;
  if (sum) {
    a_dw.W = sum->n_super;
    a_dw.b = a.b * (a.W / sum->n_super);
    for (int g = 0; g < sum->n_super; ++g) wt_dw.grad[g] = sum->super_part + (int64_t)g * P_PAD;
  }
  if (tc) {
    cudaStream_t s1 = side.s1 ? side.s1 : st, s2 = side.s2 ? side.s2 : st;
    // the copies of W1 are not needed before the dense layer: they are made next to the convolutions
    if (!a.skip_prep_w1) {
      if (side.s1) { cudaEventRecord(side.fork1, st); cudaStreamWaitEvent(s1, side.fork1, 0); }
      launches += launch_prep_w1(gt, ws, s1, prof);
      if (side.s1) cudaEventRecord(side.join1, s1);
    }
    if (launch_conv1_fwd_planes(a, wt, gt, ws, st, prof) < 0) return -1;
    launch_conv2_fwd_tc5(a, wt, gt, ws, st, prof);
    if (!a.skip_prep_w1 && side.s1) cudaStreamWaitEvent(st, side.join1, 0);
    int n = launch_fc1_fwd_tc5(a, wt, gt, ws, st, prof);
    if (n < 0) return -1;
    launches += 2 + n;
    TIMED(K_FC2_FWD_BWD, (fc2_fwd_bwd<<<dim3(a.W, FC2_SPLIT), FC2_THREADS, 0, st>>>(a, wt, gt, ws)));
    launches += 1;
    if (side.s1) { cudaEventRecord(side.fork1, st); cudaStreamWaitEvent(s1, side.fork1, 0); }
    n = sum ? launch_fc1_dw_tc5(a_dw, wt_dw, gt, ws, s1, prof) : launch_fc1_dw_tc5(a, wt, gt, ws, s1, prof);
    if (n < 0) return -1;
    launches += n;
    if (side.s1) cudaEventRecord(side.join1, s1);
    n = launch_fc1_dx_tc5(a, wt, gt, ws, st, prof);
    if (n < 0) return -1;
    launches += n;
    if (side.s2) { cudaEventRecord(side.fork2, st); cudaStreamWaitEvent(s2, side.fork2, 0); }
    n_chunks2 = launch_conv2_dw_tc5(a, wt, ws, s2, prof, &seg_len);
    if (side.s2) cudaEventRecord(side.join2, s2);
    launch_conv2_dx_tc5(a, wt, gt, ws, st, prof);
    int seg_len1 = 0;
    const int n_chunks1t = launch_conv1_dw_tc5(a, wt, ws, st, prof, &seg_len1);
    if (n_chunks1t < 0) return -1;
    if (side.s1) cudaStreamWaitEvent(st, side.join1, 0);
    if (side.s2) cudaStreamWaitEvent(st, side.join2, 0);
    if (sum) TIMED(K_CONV_GRAD_REDUCE, (fused_finish<<<FUSED_W1_BLOCKS + FUSED_SMALL_BLOCKS, 256, 0, st>>>(a, wt, ws, sum->super_part, sum->n_super, sum->grad_sum, n_chunks1t, seg_len1, n_chunks2, seg_len)));
    else TIMED(K_CONV_GRAD_REDUCE, (conv_grad_reduce<<<dim3(a.W, RED_BLOCKS), 256, 0, st>>>(a, wt, ws, n_chunks1t, seg_len1, n_chunks2, seg_len)));
    launches += 4;
  } else {
    TIMED(K_CONV1_FWD, (conv1_fwd<<<dim3(n_chunks1, a.W), 224, 0, st>>>(a, wt, gt, ws)));
    TIMED(K_CONV2_FWD, (conv2_fwd<<<dim3(n_chunks, a.W), 256, 0, st>>>(a, wt, gt, ws)));
    TIMED(K_FC1_FWD, (fc1_fwd<<<dim3(HID / 64, mt), 256, 0, st>>>(a, wt, gt, ws)));
    TIMED(K_FC2_FWD_BWD, (fc2_fwd_bwd<<<dim3(a.W, FC2_SPLIT), FC2_THREADS, 0, st>>>(a, wt, gt, ws)));
    if (sum) TIMED(K_FC1_DW, (fc1_dw<<<dim3((FLAT + 63) / 64, HID / 64, a_dw.W), 256, 0, st>>>(a_dw, wt_dw, ws)));
    else TIMED(K_FC1_DW, (fc1_dw<<<dim3((FLAT + 63) / 64, HID / 64, a.W), 256, 0, st>>>(a, wt, ws)));
    TIMED(K_FC1_DX, (fc1_dx<<<dim3((FLAT + 63) / 64, mt), 256, 0, st>>>(a, gt, ws)));
    TIMED(K_CONV2_BWD, (conv2_bwd<<<dim3(n_chunks, a.W), 256, C2B_SMEM_FLOATS * sizeof(float), st>>>(a, wt, gt, ws, n_chunks)));
    TIMED(K_CONV1_BWD, (conv1_bwd<<<dim3(n_chunks1b, a.W), 256, 0, st>>>(a, wt, ws, n_chunks1b)));
    if (sum) TIMED(K_CONV_GRAD_REDUCE, (fused_finish<<<FUSED_W1_BLOCKS + FUSED_SMALL_BLOCKS, 256, 0, st>>>(a, wt, ws, sum->super_part, sum->n_super, sum->grad_sum, n_chunks1b, 0, n_chunks2, 0)));
    else TIMED(K_CONV_GRAD_REDUCE, (conv_grad_reduce<<<dim3(a.W, RED_BLOCKS), 256, 0, st>>>(a, wt, ws, n_chunks1b, 0, n_chunks2, 0)));
    launches = 9;
  }
  return cudaGetLastError() == cudaSuccess ? launches : -1;
}

}  // namespace psk
