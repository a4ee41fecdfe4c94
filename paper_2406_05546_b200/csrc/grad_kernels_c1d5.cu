// Filter and bias gradient of the first convolution on the fifth-generation tensor cores, in pooled form (BF16
// operands, fp32 accumulation in tensor memory; values only, no decision depends on them).
//
// The gradient at the convolution's output is the pooled gradient dp1 put back at the pooling winners: of the four
// positions of a 2x2 window at most one is non-zero.  Instead of scattering it into a dense 28x28 map (three
// quarters zeros) the contraction runs over the 196 POOLED positions, with the window element w = (wy, wx) that won
// as part of the row index:
//
//   T[(w, oc)][(sy, sx)] = sum over pooled positions p = (py, px) of  G_w[oc][p] * Xs[(sy, sx)][p]
//       G_w[oc][p]      = dp1[oc][p] if the winner of window p in channel oc is w, else 0
//       Xs[(sy, sx)][p] = x[2 py + sy - 1][2 px + sx - 1]   (sy, sx = 0..3: the sixteen stride-2 shifts of the image)
//   dW[oc][ky][kx]      = sum over w of T[(w, oc)][(wy + ky, wx + kx)],    db[oc] = sum over w, p of G_w[oc][p]
//
// i.e. per sample one product of M = 64, N = 24 (sixteen shifts, a row of ones whose products are the bias gradient,
// seven rows of zeros), K = 208 (196 positions, padded): thirteen tcgen05 MMAs of K = 16, accumulated in tensor
// memory over all samples of a worker.  Both operands have the position index contiguous (core matrices of 8 rows x
// 8 positions); the 128-byte core matrices of a row group lie 144 bytes apart, so that threads that fill consecutive
// core matrices store to different shared-memory banks.
// One CTA per SM walks over a contiguous range of rows (sorted worker, sample); where the range passes from one
// worker to the next, and at its end, the accumulator is written out as a partial sum that a later kernel adds in a
// fixed order.  The images arrive by TMA tile loads whose box starts outside the image (zero border for free), the
// pooled gradients (BF16, as the second convolution's input-gradient kernel stores them) and the decisions by bulk
// copies, two samples ahead.  Every mbarrier wait is bounded.
#include "device_common.cuh"
#include "kernels.h"
#include "tc5_common.cuh"

namespace psk {

namespace {

constexpr int D1_LOAD_WARPS = 16;                        // two groups: group g stages samples n = g, g + 2, ...
constexpr int D1_GW = D1_LOAD_WARPS / 2;                 // warps per group
constexpr int D1_GT = 32 * D1_GW;                        // threads per group
constexpr int D1_THREADS = 32 * (1 + D1_LOAD_WARPS + 4); // warp 0: MMA issue and tensor memory; the last four warps write out
constexpr int D1_CHUNKS = 26;                            // 8-position chunks of the 208 contraction indices of a sample
constexpr int D1_CHUNK_PITCH = 144;                      // bytes from one core matrix of a row group to the next
constexpr int D1_GROUP_BYTES = D1_CHUNKS * D1_CHUNK_PITCH;   // 3,744: one group of 8 operand rows
constexpr int D1_A_GROUPS = 8;                           // (window element, channel octet)
constexpr int D1_B_GROUPS = 3;                           // shifts 0..7, shifts 8..15, ones row + zero rows
constexpr int D1_A_BYTES = D1_A_GROUPS * D1_GROUP_BYTES;
constexpr int D1_STAGE_BYTES = ((D1_A_GROUPS + D1_B_GROUPS) * D1_GROUP_BYTES + 127) / 128 * 128;    // 41,216
constexpr int D1_BOX_W = 36, D1_BOX_H = 30;              // image box: columns -4..31 (a 16-byte aligned start), rows -1..28
constexpr int D1_BOX_BYTES = D1_BOX_W * D1_BOX_H * 4;    // 4,320
constexpr int D1_RAW_X = 4352;                           // box padded to a multiple of 128 bytes
constexpr int D1_RAW_G = P1_ELEMS * 2, D1_RAW_CODE = P1_ELEMS;
constexpr int D1_RAW_SLOT = (D1_RAW_X + D1_RAW_G + D1_RAW_CODE + 127) / 128 * 128;     // 13,824
constexpr int D1_NRAW = 4;                               // raw input slots: each group's copies run two of its samples ahead
constexpr int D1_SMEM = 2 * D1_STAGE_BYTES + D1_NRAW * D1_RAW_SLOT + 256 + 128;
constexpr int D1_NACC = 4;                               // accumulators used in turn: an MMA that adds to the sum of the one before
                                                         // it waits for that one to finish, and these MMAs are short
constexpr int D1_TMEM_COLS = 32 * D1_NACC;               // 24 accumulator columns each, 32 apart
constexpr int D1_KSTEPS = D1_CHUNKS / 2;                 // 13
static_assert(D1_SMEM <= 227 * 1024, "shared memory");
static_assert(D1_GT == 256, "the item split below assumes 256 threads per group");

__host__ __device__ constexpr uint32_t d1_idesc(int m, int n) {     // fp32 accumulate, BF16 x BF16, both k-contiguous
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

struct D1Bars {
  uint64_t op_full[2], op_empty[2], raw_full[D1_NRAW], raw_empty[D1_NRAW], acc_full, acc_empty;
  uint32_t tmem_base;
  volatile uint32_t abort_flag;
};

// The decisions arrive as one byte per (channel, position) holding 1 << winner (0 = no gradient).  Shifting a word of
// four such bytes left by 7 - w brings "the winner is w" into the top bit of every byte, which is the only bit the
// sign-replicating byte permute below looks at.
__device__ __forceinline__ uint32_t win_flags(uint32_t onehot, int w) { return onehot << (7 - w); }

// Rows (sorted worker, sample) are split into gridDim.x contiguous ranges of seg_len.  Partial sums of worker s go
// to part1[s][4 (range index - first range of s) + window element].
__global__ void __launch_bounds__(D1_THREADS, 1) conv1_dw_tc5(const __grid_constant__ CUtensorMap xmap, GradStepArgs a, WorkerTable wt,
                                                              Workspace ws, int seg_len, int slots) {
  extern __shared__ __align__(1024) uint8_t sm[];
  uint8_t* raw = sm + 2 * D1_STAGE_BYTES;
  D1Bars* bars = reinterpret_cast<D1Bars*>(raw + D1_NRAW * D1_RAW_SLOT);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int total = a.W * a.b;
  const int r0 = blockIdx.x * seg_len, r1 = min(r0 + seg_len, total), n_samples = r1 - r0;

  // Operand stages start as zeros: positions 196..207, the zero rows of B, and every entry of A that no sample's
  // staging writes.  The ones row of B (row 0 of its third group) is written once.
  for (int i = tid; i < 2 * D1_STAGE_BYTES / 16; i += D1_THREADS) reinterpret_cast<uint4*>(sm)[i] = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
  for (int i = tid; i < 2 * D1_CHUNKS; i += D1_THREADS)
    *reinterpret_cast<uint4*>(sm + (i / D1_CHUNKS) * D1_STAGE_BYTES + D1_A_BYTES + 2 * D1_GROUP_BYTES + (i % D1_CHUNKS) * D1_CHUNK_PITCH) =
        make_uint4(0x3F803F80u, 0x3F803F80u, 0x3F803F80u, 0x3F803F80u);
  if (tid == 0) {
    for (int i = 0; i < 2; ++i) { mbar_init(&bars->op_full[i], D1_GW); mbar_init(&bars->op_empty[i], 1); }
    for (int i = 0; i < D1_NRAW; ++i) { mbar_init(&bars->raw_full[i], 1); mbar_init(&bars->raw_empty[i], D1_GW); }
    mbar_init(&bars->acc_full, 1);
    mbar_init(&bars->acc_empty, 4);
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)), "r"(D1_TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_proxy_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;

  if (warp == 0) {
    // ---------------- MMA issue
    if (lane == 0) {
      constexpr uint32_t idesc = d1_idesc(64, 24);
      int writes = 0;
      bool fresh = true;                       // the next MMA starts a new sum
      for (int n = 0; n < n_samples; ++n) {
        const int st = n & 1;
        if (!mbar_wait(&bars->op_full[st], (n >> 1) & 1) || bars->abort_flag) { bars->abort_flag = 1; break; }
        tc_fence_after();
        const uint32_t a_lo = plain_desc_lo(smem_u32(sm) + st * D1_STAGE_BYTES, D1_CHUNK_PITCH);
        const uint32_t b_lo = plain_desc_lo(smem_u32(sm) + st * D1_STAGE_BYTES + D1_A_BYTES, D1_CHUNK_PITCH);
        // contraction indices 16 ks .. 16 ks + 15: two core matrices, 2 x 144 bytes further along every row group
#pragma unroll
        for (int ks = 0; ks < D1_KSTEPS; ++ks)
          umma_f16_split(tmem + (ks % D1_NACC) * 32, a_lo + ks * (2 * D1_CHUNK_PITCH / 16), plain_desc_hi(D1_GROUP_BYTES),
                         b_lo + ks * (2 * D1_CHUNK_PITCH / 16), plain_desc_hi(D1_GROUP_BYTES), idesc, (ks < D1_NACC && fresh) ? 0u : 1u);
        fresh = false;
        umma_commit(&bars->op_empty[st]);
        const int row = r0 + n;
        if (row + 1 == r1 || (row + 1) % a.b == 0) {
          // last row of the range or of a worker: hand the sum to the write-out warps and wait until they have read it
          umma_commit(&bars->acc_full);
          if (!mbar_wait(&bars->acc_empty, writes & 1)) { bars->abort_flag = 1; break; }
          tc_fence_after();
          ++writes;
          fresh = true;
        }
      }
    }
  } else if (warp <= D1_LOAD_WARPS) {
    // ---------------- staging: group g (D1_GW warps) builds the operands of samples n = g, g + 2, ... in stage g
    const int grp = (warp - 1) / D1_GW, gt_ = (warp - 1 - grp * D1_GW) * 32 + lane;      // thread index inside the group
    auto issue = [&](int n) {            // one thread: the three inputs of sample r0 + n
      const int row = r0 + n, s = row / a.b, i = row - s * a.b;
      uint8_t* dst = raw + (n & 3) * D1_RAW_SLOT;
      uint64_t* bar = &bars->raw_full[n & 3];
      mbar_expect_tx(bar, D1_BOX_BYTES + D1_RAW_G + D1_RAW_CODE);
      tma_load_3d(dst, &xmap, bar, -4, -1, wt.src[s] * a.b + i);
      bulk_load(dst + D1_RAW_X, reinterpret_cast<const uint8_t*>(ws.dp1) + (int64_t)row * (P1_ELEMS * 4), D1_RAW_G, bar);
      bulk_load(dst + D1_RAW_X + D1_RAW_G, ws.code1 + (int64_t)row * P1_ELEMS, D1_RAW_CODE, bar);
    };
    // A item of this thread: (channel quad aq, chunk ac, half ah) = four pooled positions of four channels.
    // 4 quads x (24 chunks x 2 halves + the first half of chunk 24) = 196 items; the other threads have none.
    const int aq = gt_ / 49, arem = gt_ - aq * 49, ac = arem >> 1, ah = arem & 1;
    const bool a_item = gt_ < 196;
    const int a_src = (aq * 196 + 8 * ac + 4 * ah);                       // (quad, first position) in units of one position's 4 channels
    const int a_dst = ((aq >> 1)) * D1_GROUP_BYTES + ac * D1_CHUNK_PITCH + ((aq & 1) * 4) * 16 + ah * 8;   // window element 0, channel 0 of the quad
    // B items of this thread: shift bn = (sy, sx) and chunks bc0 = gt_ / 16 and bc0 + 16 (the latter for bc0 < 9;
    // chunk 24 holds positions 192..195 only).  The word offsets of the sixteen elements in the image box are fixed
    // for the whole kernel (box row 2 py + sy is image row 2 py + sy - 1, box column 2 px + sx + 3 is image column
    // 2 px + sx - 1) and are worked out once.
    const int bn = gt_ & 15, sy = bn >> 2, sx = bn & 3, bc0 = gt_ >> 4;
    const int b_dst = (bn >> 3) * D1_GROUP_BYTES + (bn & 7) * 16;
    int b_off[2][8];                     // word 0 of the box is outside the image (always zero): positions past 195 read it
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int p = 8 * (bc0 + 16 * h) + j, py = p / 14, px = p - 14 * py;
        b_off[h][j] = p < 196 ? sy * D1_BOX_W + sx + 3 + 2 * py * D1_BOX_W + 2 * px : 0;
      }

    if (gt_ == 0) { if (grp < n_samples) issue(grp); if (grp + 2 < n_samples) issue(grp + 2); }
    for (int n = grp; n < n_samples; n += 2) {
      const int slot = n & 3;
      bool ok = mbar_wait(&bars->raw_full[slot], (n >> 2) & 1);
      if (ok && n >= 2) ok = mbar_wait(&bars->op_empty[grp], ((n >> 1) - 1) & 1);
      if (!__all_sync(0xffffffffu, ok) || bars->abort_flag) { bars->abort_flag = 1; break; }
      const uint8_t* rslot = raw + slot * D1_RAW_SLOT;
      const float* img = reinterpret_cast<const float*>(rslot);
      uint8_t* stage = sm + grp * D1_STAGE_BYTES;
      if (a_item) {
        // four positions of four channels: the gradients as two 16-byte loads ([position][4 channels] BF16), the
        // decisions as one ([position][4 channels] bytes)
        const uint4 g01 = reinterpret_cast<const uint4*>(rslot + D1_RAW_X)[a_src >> 1];          // positions 0, 1: {c0c1, c2c3, c0c1, c2c3}
        const uint4 g23 = reinterpret_cast<const uint4*>(rslot + D1_RAW_X)[(a_src >> 1) + 1];
        const uint4 cd = reinterpret_cast<const uint4*>(rslot + D1_RAW_X + D1_RAW_G)[a_src >> 2];
        // per channel, the position pairs (0, 1) and (2, 3) as one word each
        const uint32_t v[4][2] = {{prmt(g01.x, g01.z, 0x5410u), prmt(g23.x, g23.z, 0x5410u)},
                                  {prmt(g01.x, g01.z, 0x7632u), prmt(g23.x, g23.z, 0x7632u)},
                                  {prmt(g01.y, g01.w, 0x5410u), prmt(g23.y, g23.w, 0x5410u)},
                                  {prmt(g01.y, g01.w, 0x7632u), prmt(g23.y, g23.w, 0x7632u)}};
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          const uint32_t e0 = win_flags(cd.x, w), e1 = win_flags(cd.y, w), e2 = win_flags(cd.z, w), e3 = win_flags(cd.w, w);
          uint8_t* d = stage + a_dst + w * (2 * D1_GROUP_BYTES);
          // channel c: half-word masks from the top bits of byte c of the two positions' flags
          *reinterpret_cast<uint2*>(d) = make_uint2(v[0][0] & prmt(e0, e1, 0xCC88u), v[0][1] & prmt(e2, e3, 0xCC88u));
          *reinterpret_cast<uint2*>(d + 16) = make_uint2(v[1][0] & prmt(e0, e1, 0xDD99u), v[1][1] & prmt(e2, e3, 0xDD99u));
          *reinterpret_cast<uint2*>(d + 32) = make_uint2(v[2][0] & prmt(e0, e1, 0xEEAAu), v[2][1] & prmt(e2, e3, 0xEEAAu));
          *reinterpret_cast<uint2*>(d + 48) = make_uint2(v[3][0] & prmt(e0, e1, 0xFFBBu), v[3][1] & prmt(e2, e3, 0xFFBBu));
        }
      }
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int bc = bc0 + 16 * h;
        if (bc < 25) {
          float xv[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) xv[j] = img[b_off[h][j]];
          *reinterpret_cast<uint4*>(stage + D1_A_BYTES + b_dst + bc * D1_CHUNK_PITCH) =
              make_uint4(bf16_pair(xv[0], xv[1]), bf16_pair(xv[2], xv[3]), bf16_pair(xv[4], xv[5]), bf16_pair(xv[6], xv[7]));
        }
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) { mbar_arrive(&bars->op_full[grp]); mbar_arrive(&bars->raw_empty[slot]); }
      if (gt_ == 0 && n + 4 < n_samples) {
        if (!mbar_wait(&bars->raw_empty[slot], (n >> 2) & 1)) { bars->abort_flag = 1; break; }
        issue(n + 4);
      }
    }
  } else {
    // ---------------- write-out: a warp reads the accumulator lanes 32 (warp % 4) .. + 31.  An accumulator of 64 rows
    // keeps rows 16 q .. 16 q + 15 in the first sixteen lanes of quarter q, so warp q holds window element q = (wy, wx)
    // and lane oc < 16 one output channel.  Each warp writes its window element's share of the 160 sums to a partial
    // slot of its own (the final reduction adds the four in a fixed order), so the warps exchange nothing.
    const int quarter = warp & 3;
    int writes = 0;
    for (int row = r0; row < r1; ++row) {
      if (!(row + 1 == r1 || (row + 1) % a.b == 0)) continue;
      if (!mbar_wait(&bars->acc_full, writes & 1) || bars->abort_flag) { bars->abort_flag = 1; break; }
      tc_fence_after();
      float v0[16], vb = 0.f;
#pragma unroll
      for (int j = 0; j < 16; ++j) v0[j] = 0.f;
#pragma unroll
      for (int acc = 0; acc < D1_NACC; ++acc) {      // the accumulators are added in a fixed order
        uint32_t t0[16], t1[16];
        tmem_ld16(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * 32), t0);
        tmem_ld16(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * 32 + 16), t1);      // column 16 = bias, 17..23 zero rows, 24..31 unused
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 16; ++j) v0[j] += __uint_as_float(t0[j]);
        vb += __uint_as_float(t1[0]);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->acc_empty);
      const int s = row / a.b;
      float* part = ws.part1 + (((int64_t)s * slots + (blockIdx.x - (s * a.b) / seg_len)) * 4 + quarter) * C1_GRAD;
      if (lane < 16) {
        // dW[oc][ky][kx] takes shift (wy + ky, wx + kx) of this window element
#pragma unroll
        for (int w = 0; w < 4; ++w)
          if (w == quarter) {
#pragma unroll
            for (int tap = 0; tap < 9; ++tap) part[lane * 9 + tap] = v0[((w >> 1) + tap / 3) * 4 + (w & 1) + tap % 3];
          }
        part[144 + lane] = vb;
      }
      ++writes;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(D1_TMEM_COLS) : "memory");
  }
  if (tid == 0 && bars->abort_flag) {
    atomicOr(ws.status, STATUS_WAIT_TIMEOUT);
    for (int k = 0; k < 1000; ++k) __nanosleep(1000);   // let copies already issued land before the CTA ends
  }
}

}  // namespace

#define TIMED(id, launch) do { if (prof) prof->begin(id, st); launch; if (prof) prof->end(st); } while (0)

int configure_c1d5_kernels() {
  return cudaFuncSetAttribute(conv1_dw_tc5, cudaFuncAttributeMaxDynamicSharedMemorySize, D1_SMEM) == cudaSuccess ? 0 : -1;
}

// Returns the number of partial-sum slots reserved per worker (the stride of part1: four per range), or -1;
// *seg_len receives the length of a CTA's range of rows: worker s owns four partial sums per range that meets its rows.
int launch_conv1_dw_tc5(const GradStepArgs& a, const WorkerTable& wt, const Workspace& ws, cudaStream_t st, Profiler* prof,
                        int* seg_len) {
  CUtensorMap xmap;
  const uint64_t dims[3] = {IMG, IMG, (uint64_t)a.W * a.b};
  const uint64_t strides[2] = {IMG * 4, IMG * IMG * 4};
  const uint32_t box[3] = {D1_BOX_W, D1_BOX_H, 1};
  if (!encode_tensor_map_f32(&xmap, a.x, 3, dims, strides, box)) return -1;
  const int total = a.W * a.b;
  int grid = total / 16;                  // a range is at least 16 rows long (bounds the partial sums per worker)
  if (grid > g_sm_count) grid = g_sm_count;
  if (grid < 1) grid = 1;
  const int len = (total + grid - 1) / grid;
  grid = (total + len - 1) / len;
  const int slots = (a.b - 1) / len + 2;
  TIMED(K_CONV1_BWD, (conv1_dw_tc5<<<grid, D1_THREADS, D1_SMEM, st>>>(xmap, a, wt, ws, len, slots)));
  *seg_len = len;
  return 4 * slots;
}

}  // namespace psk
