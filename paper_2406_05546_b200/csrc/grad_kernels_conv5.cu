// Second convolution (16 -> 32 channels, 3x3, pad 1, 14x14 maps) on the fifth-generation tensor cores:
// forward with fused ReLU + 2x2 max pooling, and the gradient with respect to the input.  BF16 operands,
// fp32 accumulation in tensor memory.
//
// Both are implicit products with k = (filter tap, channel).  The trick that makes them fit
// tcgen05.mma without an im2col copy: an un-swizzled k-contiguous shared-memory operand is a stack of
// "core matrices" of 8 rows x 16 bytes, so if the image is stored as planes of EIGHT BF16 channels
// (one position = one 16-byte row), then for a fixed filter tap the operand "all positions x 8 channels"
// is just that plane read from a shifted start address.  One MMA (K = 16) takes two such planes.
//
// Forward: rows are POOLED positions and the four pre-pool window elements go to four accumulators
// (four column ranges of tensor memory), so that a thread of the epilogue holds the whole 2x2 window
// and pools without exchanging data.  For that the planes keep even and odd columns apart
// (position (Y, X) at row Y*16 + (X&1)*8 + X/2): consecutive pooled columns are then consecutive rows.
//
// The stages of each kernel (staging, MMA issue, epilogue) run in different warps and overlap through
// mbarriers; every wait is bounded.
#include "device_common.cuh"
#include "kernels.h"
#include "tc5_common.cuh"

namespace psk {

namespace {

constexpr int THREADS = 448;           // input-gradient kernel: 1 MMA warp, 8 staging warps, 4 epilogue warps, 1 copy warp
constexpr int LOADERS = 256;

__host__ __device__ constexpr uint32_t idesc_bf16(int m, int n) {     // fp32 accumulate, BF16 x BF16, k-contiguous
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

constexpr int RAW_SLOTS = 8;          // raw input slots of the input-gradient kernel
constexpr int F_NBUF = 4;             // shared-memory tile buffers of the forward kernel (copies run four tiles ahead)
struct Pipe {
  uint64_t a_full[F_NBUF], a_empty[F_NBUF], acc_full[2], acc_empty[2], raw_full[RAW_SLOTS], raw_empty[RAW_SLOTS];
  uint32_t tmem_base;
  volatile uint32_t abort_flag;
};

__device__ __forceinline__ void pipe_init(Pipe* p, int a_full_arrivals, int acc_empty_arrivals) {
  for (int i = 0; i < F_NBUF; ++i) {
    mbar_init(&p->a_full[i], a_full_arrivals);
    mbar_init(&p->a_empty[i], 1);
  }
  for (int i = 0; i < 2; ++i) {
    mbar_init(&p->acc_full[i], 1);
    mbar_init(&p->acc_empty[i], acc_empty_arrivals);
  }
  for (int i = 0; i < RAW_SLOTS; ++i) {
    mbar_init(&p->raw_full[i], 1);
    mbar_init(&p->raw_empty[i], LOADERS / 64);
  }
  p->abort_flag = 0;
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

// ------------------------------------------------------------------------------------------------
// Forward.  Tile = two samples = 128 rows: row 8*g + i is pooled position (py = g mod 8, px = i) of
// sample g / 8 (py = 7 and px = 7 are padding rows whose results are dropped).  The first convolution
// already wrote its output in the plane layout, borders included, so staging a tile is four plain
// bulk copies of 4 KB issued by one thread.
// Warps: 0 = MMA issuer and tensor-memory owner, 1 = copy producer, 2..9 = epilogue (warp w reads the
// accumulator lanes of quarter w mod 4 and the output channels of half (w-2)/4).
// ------------------------------------------------------------------------------------------------
constexpr int F_THREADS = 320;
constexpr int F_PLANE_ROWS = 2 * 256 + 32;                 // two stacked 16x16 images + overrun of the padding rows
constexpr int F_PLANE_BYTES = F_PLANE_ROWS * 16;           // 8704
constexpr int F_BUF_BYTES = 2 * F_PLANE_BYTES;             // two planes of eight channels
// One MMA per input SHIFT instead of one per (window element, tap).  Window element (jy, jx) and tap (ky, kx) read the
// input plane shifted by (sy, sx) = (jy + ky, jx + kx), sixteen shifts in all, and a shift serves every (window
// element, tap) pair that adds up to it: the products of one shifted plane with the filters of all those taps land
// side by side in the accumulator columns [window element][channel] when the weight operand stacks the taps' filters
// in that column order.  Where a shift's two window elements are not neighbours in the column order, the 32 columns
// between them get a block of zero filters, so a tile costs 16 MMAs (four each of N = 128, 96, 64 and 32) instead of
// 36 of N = 32: the tensor core spends about as long on an MMA of M = 128, K = 16 with N = 32 as with N = 96.  The
// host lists the MMAs (FoldTable).
constexpr int F_OPS = 16;
constexpr int F_W_BLOCKS = 40;                             // 32-row blocks of the stacked weight operand (1,280 rows)
constexpr int F_W_ROWS = 32 * F_W_BLOCKS;
constexpr int F_W_BYTES = 2 * F_W_ROWS * 16;               // [channel octet][row][8 bf16]
constexpr int F_SMEM = F_NBUF * F_BUF_BYTES + F_W_BYTES + 32 * 4 + sizeof(Pipe) + 128;
static_assert(2 * F_SMEM <= 227 * 1024, "two CTAs per SM");

constexpr uint8_t F_ZERO_BLOCK = 255;
struct FoldTable {
  int32_t a_off[F_OPS];        // start of the shifted plane, in 16-byte rows
  int32_t d_col[F_OPS];        // first accumulator column
  int32_t b_row[F_OPS];        // first row of the op's block of the weight operand
  uint32_t idesc[F_OPS];       // instruction descriptor (M = 128, the op's N)
  uint8_t tap_of_block[F_W_BLOCKS];   // filter tap ky * 3 + kx whose 32 filters fill a 32-row block; F_ZERO_BLOCK: 32 rows of zeros
};

FoldTable make_fold_table() {
  FoldTable t;
  int n_ops = 0, row = 0;
  // one op: the plane shifted by (sy, sx) against the filters of the column blocks [first, first + n_blocks); block c
  // belongs to window element c = 2 jy + jx, whose tap for this shift is (sy - jy, sx - jx), or is a block of zeros
  auto add = [&](int sy, int sx, int first, int n_blocks, unsigned used) {
    t.a_off[n_ops] = sy * 16 + (sx & 1) * 8 + (sx >> 1);
    t.d_col[n_ops] = first * 32;
    t.b_row[n_ops] = row;
    t.idesc[n_ops] = idesc_bf16(128, 32 * n_blocks);
    for (int c = first; c < first + n_blocks; ++c, row += 32)
      t.tap_of_block[row / 32] = (used >> c) & 1u ? (uint8_t)((sy - (c >> 1)) * 3 + (sx - (c & 1))) : F_ZERO_BLOCK;
    ++n_ops;
  };
  for (int pass = 0; pass < 2; ++pass)          // the op that covers all 128 columns comes first: it starts the sums
    for (int sy = 0; sy < 4; ++sy)
      for (int sx = 0; sx < 4; ++sx) {
        if ((pass == 0) != (sy == 1 && sx == 1)) continue;
        const int jy0 = sy == 3 ? 1 : 0, ny = (sy == 0 || sy == 3) ? 1 : 2;
        const int jx0 = sx == 3 ? 1 : 0, nx = (sx == 0 || sx == 3) ? 1 : 2;
        unsigned used = 0;
        for (int jy = jy0; jy < jy0 + ny; ++jy)
          for (int jx = jx0; jx < jx0 + nx; ++jx) used |= 1u << (2 * jy + jx);
        // the window elements of a shift are the blocks from its first to its last one; where two of them are not
        // neighbours (same column of the window, both rows) the block between them is zeros: one MMA of N = 96 costs
        // less than two of N = 32
        const int first = 2 * jy0 + jx0, last = 2 * (jy0 + ny - 1) + (jx0 + nx - 1);
        add(sy, sx, first, last - first + 1, used);
      }
  return t;      // n_ops == F_OPS and row == F_W_ROWS by construction
}

__global__ void __launch_bounds__(F_THREADS, 2) conv2_fwd_tc5(GradStepArgs a, GroupTable gt, Workspace ws, int range_len, const __grid_constant__ FoldTable fold) {
  extern __shared__ __align__(128) uint8_t smem[];
  uint16_t* Wk = reinterpret_cast<uint16_t*>(smem + F_NBUF * F_BUF_BYTES);
  float* bias = reinterpret_cast<float*>(smem + F_NBUF * F_BUF_BYTES + F_W_BYTES);
  Pipe* pipe = reinterpret_cast<Pipe*>(smem + F_NBUF * F_BUF_BYTES + F_W_BYTES + 128);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // a CTA walks over a contiguous range of rows (worker-major samples) that share one weight snapshot
  int grp, r_begin, r_end;
  if (!locate_row_range(gt, a.b, range_len, blockIdx.x, grp, r_begin, r_end)) return;
  const float* theta = gt.theta[grp];
  const int n_tiles = (r_end - r_begin + 1) / 2;

  // the filter bank comes in once with coalesced 16-byte loads (into the tile buffers, which are cleared afterwards) ...
  float* wtmp = reinterpret_cast<float*>(smem);
  for (int idx = tid; idx < 4608 / 4; idx += F_THREADS) reinterpret_cast<float4*>(wtmp)[idx] = reinterpret_cast<const float4*>(theta + OFF_C2W)[idx];
  if (tid < 32) bias[tid] = theta[OFF_C2B + tid];
  __syncthreads();
  // ... and is laid out as the stacked weight operand: block rb holds the 32 filters of tap fold.tap_of_block[rb], one
  // row per output channel
  for (int idx = tid; idx < F_W_BLOCKS * 512; idx += F_THREADS) {
    const int rb = idx >> 9, oc = (idx >> 4) & 31, ic = idx & 15;
    const uint32_t tap = fold.tap_of_block[rb];
    Wk[((ic >> 3) * F_W_ROWS + rb * 32 + oc) * 8 + (ic & 7)] = tap == F_ZERO_BLOCK ? (uint16_t)0 : bf16_bits(wtmp[(oc * 16 + ic) * 9 + tap]);
  }
  __syncthreads();
  // rows never written by a copy (the overrun of the padding rows, a missing second sample) only feed
  // results that are dropped; they are cleared once so that those results stay finite
  for (int idx = tid; idx < F_NBUF * F_BUF_BYTES / 16; idx += F_THREADS) reinterpret_cast<float4*>(smem)[idx] = make_float4(0.f, 0.f, 0.f, 0.f);
  if (tid == 0) pipe_init(pipe, 1, 8);
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&pipe->tmem_base)), "r"(256) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_proxy_async_smem();      // the filter bank and the cleared rows are read by the tensor core
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = pipe->tmem_base;

  if (warp == 0) {
    if (lane == 0) {
      const uint32_t w_lo = plain_desc_lo(smem_u32(Wk), F_W_ROWS * 16);
      // one pass of the outer loop takes the four tile buffers in turn (unrolled: buffer, accumulator and the parity of
      // the accumulator's barrier are constants of each copy of the body, and the backward branch comes once per four tiles)
      static_assert(F_NBUF == 4, "the accumulator parities below assume four tile buffers");
      const uint32_t a_lo0 = plain_desc_lo(smem_u32(smem), F_PLANE_BYTES);
      bool go_on = true;
      uint32_t parity = 0;
      for (int t = 0; go_on && t < n_tiles; parity ^= 1) {
#pragma unroll
        for (int buf = 0; buf < F_NBUF; ++buf, ++t) {
          const int ab = buf & 1;
          if (t >= n_tiles) { go_on = false; break; }
          if (!mbar_wait(&pipe->a_full[buf], parity)) { pipe->abort_flag = 1; go_on = false; break; }
          // tile t = 4 k + buf is the (2 k + buf / 2)-th user of its accumulator: it waits for the phase of the user before
          if (t >= 2 && !mbar_wait(&pipe->acc_empty[ab], ((buf >> 1) ^ 1) & 1)) { pipe->abort_flag = 1; go_on = false; break; }
          if (pipe->abort_flag) { go_on = false; break; }
          tc_fence_after();
          // 16 MMAs, one per input shift (K = 16 channels); every descriptor is a per-tile base plus a table entry
          const uint32_t a_lo = a_lo0 + buf * (F_BUF_BYTES / 16);
          const uint32_t d_tmem = tmem + ab * 128;
#pragma unroll
          for (int op = 0; op < F_OPS; ++op)
            umma_f16_split(d_tmem + fold.d_col[op], a_lo + fold.a_off[op], plain_desc_hi(512), w_lo + fold.b_row[op],
                           plain_desc_hi(128), fold.idesc[op], op ? 1u : 0u);
          umma_commit(&pipe->a_empty[buf]);
          umma_commit(&pipe->acc_full[ab]);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      for (int t = 0; t < n_tiles; ++t) {
        const int buf = t % F_NBUF;
        if (t >= F_NBUF && !mbar_wait(&pipe->a_empty[buf], ((t / F_NBUF) - 1) & 1)) { pipe->abort_flag = 1; break; }
        if (pipe->abort_flag) break;
        const int n_s = min(2, r_end - (r_begin + 2 * t));
        mbar_expect_tx(&pipe->a_full[buf], (uint32_t)n_s * 2 * 4096u);
        for (int sp = 0; sp < n_s; ++sp) {
          const float* src = ws.p1 + (int64_t)(r_begin + 2 * t + sp) * P1_PLANE_ELEMS;
#pragma unroll
          for (int q = 0; q < 2; ++q)
            bulk_load(smem + buf * F_BUF_BYTES + q * F_PLANE_BYTES + sp * 4096, src + q * 1024, 4096, &pipe->a_full[buf]);
        }
      }
    }
  } else {
    const int quarter = warp & 3, ch = (warp - 2) >> 2;
    const int r = quarter * 32 + lane, g = r >> 3, px = r & 7, sp = g >> 3, py = g & 7;
    for (int t = 0; t < n_tiles; ++t) {
      const int buf = t & 1;
      if (!mbar_wait(&pipe->acc_full[buf], (t >> 1) & 1) || pipe->abort_flag) { pipe->abort_flag = 1; break; }
      tc_fence_after();
      const int64_t row = r_begin + 2 * t + sp;
      const bool valid = py < 7 && px < 7 && row < r_end;
      const int pp = py * 7 + px;
      uint32_t v[4][16];
#pragma unroll
      for (int j = 0; j < 4; ++j)
        tmem_ld16(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * 128 + j * 32 + ch * 16), v[j]);
      tmem_ld_wait();
      // the accumulators are in registers: hand the buffer back before the pooling arithmetic
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&pipe->acc_empty[buf]);
      if (valid) {
        // the bias is the same for the four window elements, so the winner is taken on the raw sums:
        // ReLU then max = max then ReLU, first element that reaches the maximum wins
        uint32_t codes[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int o = 0; o < 16; ++o) {
          const int oc = ch * 16 + o;
          const float v0 = __uint_as_float(v[0][o]), v1 = __uint_as_float(v[1][o]), v2 = __uint_as_float(v[2][o]), v3 = __uint_as_float(v[3][o]);
          const float m = fmaxf(fmaxf(v0, v1), fmaxf(v2, v3));
          const uint32_t bi = v0 == m ? 0u : (v1 == m ? 1u : (v2 == m ? 2u : 3u));
          const float best = fmaxf(m + bias[oc], 0.f);
          ws.p2[row * FLAT + oc * 49 + pp] = round_tf32(best);   // its only readers are TF32 products
          codes[o >> 2] |= (best > 0.f ? bi : 4u) << (8 * (o & 3));
        }
        // decisions as [channel quad][position][4 channels] bytes
        uint32_t* c2 = reinterpret_cast<uint32_t*>(ws.code2 + row * FLAT);
#pragma unroll
        for (int q = 0; q < 4; ++q) c2[(ch * 4 + q) * 49 + pp] = codes[q];
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(256) : "memory");
  }
  if (tid == 0 && pipe->abort_flag) {
    atomicOr(ws.status, STATUS_WAIT_TIMEOUT);
    for (int k = 0; k < 1000; ++k) __nanosleep(1000);   // let copies already issued land before the CTA ends
  }
}

// ------------------------------------------------------------------------------------------------
// Gradient with respect to the convolution's input.  Tile = one sample = two 128-row blocks of the
// 16-wide position grid (row = y*16 + x; y, x >= 14 are padding rows).  g2, the gradient at the
// convolution's output, is written from the pooled gradient and the stored pooling decisions into
// zero-bordered planes of EIGHT output channels in BF16 (one position = one 16-byte row); tap (ky, kx)
// reads them shifted by (2-ky)*16 + (2-kx) rows.  BF16 operands, fp32 accumulation: this product only
// yields gradient values, and at K = 16 per instruction it needs half the MMAs and half the operand bytes.
// ------------------------------------------------------------------------------------------------
constexpr int X_PLANE_ROWS = 256 + 51;                     // 34 rows of tap overrun (+ 17: a plane pitch of 3 rows mod 8 spreads the
constexpr int X_PLANE_BYTES = X_PLANE_ROWS * 16;           // staging stores of the four planes over all shared-memory banks)
constexpr int X_BUF_BYTES = 4 * X_PLANE_BYTES;             // four planes of eight output channels
constexpr int X_W_BYTES = 12 * 48 * 16;                    // [filter row ky][k chunk oc/8][column = kx*16 + ic][8 bf16]
constexpr int X_RAW_BYTES = FLAT * 2 + FLAT;                // one sample's pooled gradients (BF16) and pooling decisions (bytes)
constexpr int X_RAW_SLOTS = RAW_SLOTS;
constexpr int X_SMEM = 2 * X_BUF_BYTES + X_W_BYTES + X_RAW_SLOTS * X_RAW_BYTES + sizeof(Pipe) + 128;

__global__ void __launch_bounds__(THREADS, 2) conv2_dx_tc5(GradStepArgs a, GroupTable gt, Workspace ws, int range_len) {
  extern __shared__ __align__(128) uint8_t smem[];
  uint16_t* bufs = reinterpret_cast<uint16_t*>(smem);
  uint16_t* Wk = reinterpret_cast<uint16_t*>(smem + 2 * X_BUF_BYTES);
  uint8_t* raw = smem + 2 * X_BUF_BYTES + X_W_BYTES;        // raw slots filled by bulk copies
  Pipe* pipe = reinterpret_cast<Pipe*>(smem + 2 * X_BUF_BYTES + X_W_BYTES + X_RAW_SLOTS * X_RAW_BYTES);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int grp, r_begin, r_end;
  if (!locate_row_range(gt, a.b, range_len, blockIdx.x, grp, r_begin, r_end)) return;
  const float* theta = gt.theta[grp];
  const int n_tiles = r_end - r_begin;

  for (int idx = tid; idx < 4608; idx += THREADS) {
    int oc = idx / 144, rem = idx - oc * 144, ic = rem / 9, tap = rem - ic * 9;
    Wk[(((tap / 3) * 4 + (oc >> 3)) * 48 + (tap % 3) * 16 + ic) * 8 + (oc & 7)] = bf16_bits(theta[OFF_C2W + idx]);
  }
  for (int idx = tid; idx < 2 * X_BUF_BYTES / 16; idx += THREADS) reinterpret_cast<float4*>(smem)[idx] = make_float4(0.f, 0.f, 0.f, 0.f);
  if (tid == 0) pipe_init(pipe, LOADERS / 64, 4);
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&pipe->tmem_base)), "r"(256) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_proxy_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = pipe->tmem_base;

  if (warp == 0) {
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_bf16(128, 48);
      const uint32_t w_lo = plain_desc_lo(smem_u32(Wk), 48 * 16);
      // one pass of the outer loop takes the two plane buffers in turn (unrolled: the buffer's addresses are constants
      // of its copy of the body, and the backward branch comes once per two tiles)
      const uint32_t a_lo0 = plain_desc_lo(smem_u32(smem), X_PLANE_BYTES);
      bool go_on = true;
      uint32_t parity = 0;
      for (int t = 0; go_on && t < n_tiles; parity ^= 1) {
#pragma unroll
        for (int buf = 0; buf < 2; ++buf, ++t) {
          if (t >= n_tiles) { go_on = false; break; }
          if (!mbar_wait(&pipe->a_full[buf], parity)) { pipe->abort_flag = 1; go_on = false; break; }
          if (t >= 2 && !mbar_wait(&pipe->acc_empty[buf], parity ^ 1)) { pipe->abort_flag = 1; go_on = false; break; }
          if (pipe->abort_flag) { go_on = false; break; }
          tc_fence_after();
          const uint32_t a_lo = a_lo0 + buf * (X_BUF_BYTES / 16);
          const uint32_t d_tmem = tmem + buf * 128;
          // 12 MMAs: per block of 128 positions and filter row ky, the products with the three taps of that row sit
          // side by side in the 48 accumulator columns (kx, ic); the rows read are shifted by the filter row only
#pragma unroll
          for (int ky = 0; ky < 3; ++ky)
#pragma unroll
            for (int q = 0; q < 2; ++q)                                        // 16 output channels per MMA
#pragma unroll
              for (int m = 0; m < 2; ++m)
                umma_f16_split(d_tmem + m * 48, a_lo + (2 * q) * (X_PLANE_BYTES / 16) + m * 128 + (2 - ky) * 16 + 1, plain_desc_hi(128),
                               w_lo + ((ky * 4 + 2 * q) * 48), plain_desc_hi(128), idesc, (ky | q) ? 1u : 0u);
          umma_commit(&pipe->a_empty[buf]);
          umma_commit(&pipe->acc_full[buf]);
        }
      }
    }
  } else if (warp <= LOADERS / 32) {
    // Two groups of four staging warps: group g builds the tiles t = g, g + 2, ... into plane buffer g, so two
    // tiles are being staged at any time (a tile's staging is a chain of dependent shared-memory accesses, bound
    // by latency rather than by throughput).  The pooled gradients and decisions of a sample arrive in one of
    // eight raw slots by two bulk copies that a warp of its own issues (a staging thread that issued them held its
    // whole group up for hundreds of cycles per tile).
    const int grp_w = (warp - 1) >> 2, lt = (tid - 32) & 127;
    constexpr int X_ITEMS = (4 * 49 + 127) / 128;                  // (channel octet, position) items per thread
    for (int t = grp_w; t < n_tiles; t += 2) {
      const int buf = t & 1, slot_i = t & (X_RAW_SLOTS - 1);
      // every staging warp waits and reports on its own (no block-level barrier among them)
      bool ok = mbar_wait(&pipe->raw_full[slot_i], (t >> 3) & 1);
      if (ok && t >= 2) ok = mbar_wait(&pipe->a_empty[buf], ((t >> 1) - 1) & 1);
      if (!__all_sync(0xffffffffu, ok) || pipe->abort_flag) { pipe->abort_flag = 1; break; }
      uint16_t* dst = bufs + buf * (X_BUF_BYTES / 2);
      const uint2* rg = reinterpret_cast<const uint2*>(raw + slot_i * X_RAW_BYTES);      // four BF16 channels of a position
      const uint8_t* rc = raw + slot_i * X_RAW_BYTES + FLAT * 2;
      // Item e = lt + 128 k is (octet of output channels e / 49, pooled position e % 49).  The raw slot holds
      // the gradients and the decisions as [channel quad][position][4 channels], so an item is two 8-byte and
      // two 4-byte loads.  Its eight gradients arrive as four BF16 pairs; for each of the four positions of
      // the window the pairs are masked by "this position won" and stored as the position's 16-byte row, which
      // also clears the losers.
#pragma unroll
      for (int k = 0; k < X_ITEMS; ++k) {
        const int e = lt + k * 128;
        if (e < 4 * 49) {
          const int o8 = e / 49, p = e - o8 * 49, py = p / 7, px = p - py * 7;
          const uint2 va = rg[(2 * o8) * 49 + p], vb = rg[(2 * o8 + 1) * 49 + p];
          const uint32_t ca = reinterpret_cast<const uint32_t*>(rc)[(2 * o8) * 49 + p], cb = reinterpret_cast<const uint32_t*>(rc)[(2 * o8 + 1) * 49 + p];
          const uint32_t h0 = va.x, h1 = va.y, h2 = vb.x, h3 = vb.y;
          uint4* d = reinterpret_cast<uint4*>(dst) + o8 * (X_PLANE_BYTES / 16) + (2 * py + 1) * 16 + 2 * px + 1;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            // a decision byte is 0..4, so (byte xor j) + 0x7F has its top bit set exactly when the byte differs from j;
            // byte permutes that replicate the top bit turn the four flags into two pairs of half-word masks
            const uint32_t ea = ~((ca ^ (0x01010101u * j)) + 0x7F7F7F7Fu) & 0x80808080u;
            const uint32_t eb = ~((cb ^ (0x01010101u * j)) + 0x7F7F7F7Fu) & 0x80808080u;
            d[(j >> 1) * 16 + (j & 1)] = make_uint4(h0 & prmt(ea, 0u, 0x9988u), h1 & prmt(ea, 0u, 0xBBAAu),
                                                    h2 & prmt(eb, 0u, 0x9988u), h3 & prmt(eb, 0u, 0xBBAAu));
          }
        }
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) { mbar_arrive(&pipe->a_full[buf]); mbar_arrive(&pipe->raw_empty[slot_i]); }
    }
  } else if (warp == THREADS / 32 - 1) {
    // ---------------- copies: one thread brings every sample's pooled gradients (BF16) and decisions into the raw slots
    // in turn, up to eight samples ahead; a slot is refilled once the four warps that staged its last sample have read it
    if (lane == 0)
      for (int t = 0; t < n_tiles; ++t) {
        const int slot_i = t & (X_RAW_SLOTS - 1);
        if (t >= X_RAW_SLOTS && (!mbar_wait(&pipe->raw_empty[slot_i], ((t >> 3) - 1) & 1) || pipe->abort_flag)) { pipe->abort_flag = 1; break; }
        const int64_t row = r_begin + t;
        uint8_t* slot = raw + slot_i * X_RAW_BYTES;
        mbar_expect_tx(&pipe->raw_full[slot_i], X_RAW_BYTES);
        bulk_load(slot, ws.dp2 + row * FLAT, FLAT * 2, &pipe->raw_full[slot_i]);      // BF16 in the first half of the row
        bulk_load(slot + FLAT * 2, ws.code2 + row * FLAT, FLAT, &pipe->raw_full[slot_i]);
      }
  } else {
    const int quarter = warp & 3;
    for (int t = 0; t < n_tiles; ++t) {
      const int buf = t & 1;
      if (!mbar_wait(&pipe->acc_full[buf], (t >> 1) & 1) || pipe->abort_flag) { pipe->abort_flag = 1; break; }
      tc_fence_after();
      const int64_t row = r_begin + t;
#pragma unroll
      for (int m = 0; m < 2; ++m) {
        // the thread's position holds, per filter column kx, the sum over filter rows of what the gradient AT this
        // position sends through tap (ky, kx); the input gradient here collects kx = 0 from the position to the
        // right, kx = 1 from itself and kx = 2 from the position to the left (zero borders make the rows' ends right)
        uint32_t e0[16], e1[16], e2[16];
        const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * 128 + m * 48);
        tmem_ld16(taddr, e0);
        tmem_ld16(taddr + 16, e1);
        tmem_ld16(taddr + 32, e2);
        tmem_ld_wait();
        const int r = m * 128 + quarter * 32 + lane, y = r >> 4, x = r & 15;
        float v[16];
#pragma unroll
        for (int ic = 0; ic < 16; ++ic) {
          const float right = __shfl_down_sync(0xffffffffu, __uint_as_float(e0[ic]), 1);
          const float left = __shfl_up_sync(0xffffffffu, __uint_as_float(e2[ic]), 1);
          v[ic] = (__uint_as_float(e1[ic]) + right) + (x == 0 ? 0.f : left);
        }
        if (y < 14 && x < 14) {      // dp1 of a sample is [channel quad][position][4 channels] in BF16 (its only reader
          // multiplies in BF16): a warp writes 224 contiguous bytes per quad; a row keeps its fp32-sized pitch
          uint2* out = reinterpret_cast<uint2*>(ws.dp1 + row * P1_ELEMS) + (y * 14 + x);
#pragma unroll
          for (int q = 0; q < 4; ++q) out[q * 196] = make_uint2(bf16_pair(v[4 * q], v[4 * q + 1]), bf16_pair(v[4 * q + 2], v[4 * q + 3]));
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&pipe->acc_empty[buf]);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(256) : "memory");
  }
  if (tid == 0 && pipe->abort_flag) {
    atomicOr(ws.status, STATUS_WAIT_TIMEOUT);
    for (int k = 0; k < 1000; ++k) __nanosleep(1000);   // let copies already issued land before the CTA ends
  }
}

}  // namespace

#define TIMED(id, launch) do { if (prof) prof->begin(id, st); launch; if (prof) prof->end(st); } while (0)

int configure_conv5_kernels() {
  cudaError_t e = cudaFuncSetAttribute(conv2_fwd_tc5, cudaFuncAttributeMaxDynamicSharedMemorySize, F_SMEM);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(conv2_dx_tc5, cudaFuncAttributeMaxDynamicSharedMemorySize, X_SMEM);
  return e == cudaSuccess ? 0 : -1;
}

void launch_conv2_fwd_tc5(const GradStepArgs& a, const WorkerTable& wt, const GroupTable& gt, const Workspace& ws,
                          cudaStream_t st, Profiler* prof) {
  static const FoldTable fold = make_fold_table();
  int len;
  const int n = plan_row_ranges(gt, a.b, 2 * g_sm_count, 2, &len);      // two CTAs per SM, tiles of two samples
  TIMED(K_CONV2_FWD, (conv2_fwd_tc5<<<n, F_THREADS, F_SMEM, st>>>(a, gt, ws, len, fold)));
}

void launch_conv2_dx_tc5(const GradStepArgs& a, const WorkerTable& wt, const GroupTable& gt, const Workspace& ws,
                         cudaStream_t st, Profiler* prof) {
  int len;
  const int n = plan_row_ranges(gt, a.b, 2 * g_sm_count, 1, &len);
  TIMED(K_CONV2_BWD, (conv2_dx_tc5<<<n, THREADS, X_SMEM, st>>>(a, gt, ws, len)));
}

}  // namespace psk
