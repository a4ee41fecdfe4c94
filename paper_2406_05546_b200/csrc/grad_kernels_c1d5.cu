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
// Per sample that is a product of 64 x 24 (sixteen shifts, a row of ones whose products are the bias gradient, seven
// rows of zeros) over K = 208 (196 positions, padded).  A tcgen05 MMA costs some forty to sixty cycles however small
// it is, so two samples of a worker share every MMA: their row blocks are stacked (M = 128) and their shift blocks
// too (N = 48); the two diagonal blocks of the 128 x 48 product are the two samples' sums, the off-diagonal blocks
// are never read.  Thirteen MMAs of K = 16 per pair, accumulated in tensor memory over all pairs of a worker; a
// worker's odd last sample runs as a pair whose second shift block is zero.
// Both operands have the position index contiguous (core matrices of 8 rows x 8 positions); the 128-byte core
// matrices of a row group lie 144 bytes apart, so that threads that fill consecutive core matrices store to
// different shared-memory banks.
// One CTA per SM walks over a contiguous range of rows (sorted worker, sample); where the range passes from one
// worker to the next, and at its end, the accumulator is written out as partial sums that a later kernel adds in a
// fixed order.  Two groups of eight warps build the operands, one sample of the pair each; a sample's inputs (image,
// pooled gradients in BF16 as the second convolution's input-gradient kernel stores them, pooling decisions) arrive
// by bulk copies issued by a warp of their own into five raw slots used in turn, i.e. two to three pairs ahead.
// What bounds the kernel is shared-memory traffic: per pair the tensor core reads 73 KB of operands (three quarters
// of the row operand are the zeros of the window elements that did not win), the staging warps write 66 KB and the
// copies 25 KB.  Every mbarrier wait is bounded.
#include "device_common.cuh"
#include "kernels.h"
#include "tc5_common.cuh"

namespace psk {

namespace {

constexpr int D1_LOAD_WARPS = 16;                        // two groups: group h stages sample h of every pair
constexpr int D1_GW = D1_LOAD_WARPS / 2;                 // warps per group
constexpr int D1_GT = 32 * D1_GW;                        // threads per group
constexpr int D1_THREADS = 32 * (1 + D1_LOAD_WARPS + 4 + 1); // warp 0: MMA issue and tensor memory; then the staging warps, four
                                                            // write-out warps, and the warp that issues the loads
constexpr int D1_CHUNKS = 26;                            // 8-position chunks of the 208 contraction indices of a sample
constexpr int D1_CHUNK_PITCH = 144;                      // bytes from one core matrix of a row group to the next
constexpr int D1_GROUP_BYTES = D1_CHUNKS * D1_CHUNK_PITCH;   // 3,744: one group of 8 operand rows
constexpr int D1_A_GROUPS = 16;                          // (sample of the pair, window element, channel octet)
constexpr int D1_B_GROUPS = 6;                           // per sample: shifts 0..7, shifts 8..15, ones row + zero rows
constexpr int D1_A_BYTES = D1_A_GROUPS * D1_GROUP_BYTES;
constexpr int D1_STAGE_BYTES = ((D1_A_GROUPS + D1_B_GROUPS) * D1_GROUP_BYTES + 127) / 128 * 128;    // 82,432
constexpr int D1_NSTAGE = 2;                             // operand stages (pair u -> stage u % 2)
constexpr int D1_RAW_ZERO = 16;                          // a zero word at the start of a raw slot: what elements outside the image read
constexpr int D1_RAW_X = IMG * IMG * 4;                  // 3,136: the image as it lies in memory
constexpr int D1_RAW_G = P1_ELEMS * 2, D1_RAW_CODE = P1_ELEMS;
constexpr int D1_RAW_BYTES = D1_RAW_X + D1_RAW_G + D1_RAW_CODE;                        // 12,544 copied per sample
constexpr int D1_RAW_SLOT = (D1_RAW_ZERO + D1_RAW_BYTES + 127) / 128 * 128;            // 12,672
constexpr int D1_NRAW = 5;                               // raw input slots: the q-th sample of the range -> slot q % 5
constexpr int D1_SMEM = D1_NSTAGE * D1_STAGE_BYTES + D1_NRAW * D1_RAW_SLOT + 256 + 128;
constexpr int D1_TMEM_COLS = 64;                         // 48 accumulator columns
constexpr int D1_KSTEPS = D1_CHUNKS / 2;                 // 13
constexpr int D1_SUBSLOTS = 8;                           // partial sums per range: (sample of the pair, window element)
static_assert(D1_SMEM <= 227 * 1024, "shared memory");
static_assert(D1_GT == 256, "the item split below assumes 256 threads per group");

__host__ __device__ constexpr uint32_t d1_idesc(int m, int n) {     // fp32 accumulate, BF16 x BF16, both k-contiguous
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

struct D1Bars {
  uint64_t op_full[D1_NSTAGE], op_empty[D1_NSTAGE], raw_full[D1_NRAW], raw_empty[D1_NRAW], acc_full, acc_empty;
  uint32_t tmem_base;
  volatile uint32_t abort_flag;
};

// The decisions arrive as one byte per (channel, position) holding 1 << winner (0 = no gradient).  Shifting a word of
// four such bytes left by 7 - w brings "the winner is w" into the top bit of every byte, which is the only bit the
// sign-replicating byte permute below looks at.
__device__ __forceinline__ uint32_t win_flags(uint32_t onehot, int w) { return onehot << (7 - w); }

// The rows [row, r1) of a CTA are taken in units of two consecutive samples of one worker, or of one sample where a
// worker's (or the range's) last sample has no partner.  After a unit with `flush` the accumulator is written out.
// The walk carries the worker's index and the first row of the next worker along: every role's loop is a serial
// instruction stream, in which an integer division per unit costs hundreds of cycles.
struct D1Unit { int row, n, s; bool flush; };       // first row, rows, sorted worker of those rows
struct D1Walk { int row, wend, s; };                // next row, first row of the next worker, worker of `row`
__device__ __forceinline__ D1Walk d1_begin(int r0, int b) {
  const int s = r0 / b;
  return {r0, (s + 1) * b, s};
}
__device__ __forceinline__ bool d1_next_unit(D1Walk& w, int r1, int b, D1Unit& u) {
  if (w.row >= r1) return false;
  u.row = w.row;
  u.s = w.s;
  u.n = (w.row + 1 < r1 && w.row + 1 < w.wend) ? 2 : 1;
  w.row += u.n;
  u.flush = w.row == r1 || w.row == w.wend;
  if (w.row == w.wend) { w.wend += b; ++w.s; }
  return true;
}

// Rows (sorted worker, sample) are split into gridDim.x contiguous ranges of seg_len.  Partial sums of worker s go
// to part1[s][8 (range index - first range of s) + 4 (sample of the pair) + window element].
__global__ void __launch_bounds__(D1_THREADS, 1) conv1_dw_tc5(GradStepArgs a, WorkerTable wt, Workspace ws, int seg_len, int slots) {
  extern __shared__ __align__(1024) uint8_t sm[];
  uint8_t* raw = sm + D1_NSTAGE * D1_STAGE_BYTES;
  D1Bars* bars = reinterpret_cast<D1Bars*>(raw + D1_NRAW * D1_RAW_SLOT);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int total = a.W * a.b;
  const int r0 = blockIdx.x * seg_len, r1 = min(r0 + seg_len, total);

  // Operand stages start as zeros: positions 196..207, the zero rows of B, and every entry that no staging writes.
  for (int i = tid; i < D1_NSTAGE * D1_STAGE_BYTES / 16; i += D1_THREADS) reinterpret_cast<uint4*>(sm)[i] = make_uint4(0u, 0u, 0u, 0u);
  if (tid < D1_NRAW) *reinterpret_cast<uint4*>(raw + tid * D1_RAW_SLOT) = make_uint4(0u, 0u, 0u, 0u);
  if (tid == 0) {
    for (int i = 0; i < D1_NSTAGE; ++i) { mbar_init(&bars->op_full[i], D1_LOAD_WARPS); mbar_init(&bars->op_empty[i], 1); }
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
      constexpr uint32_t idesc = d1_idesc(128, 48);
      int writes = 0;
      D1Walk walk = d1_begin(r0, a.b);
      bool fresh = true;                       // the next MMA starts a new sum
      D1Unit un;
      // One pass of the outer loop takes the two stages in turn (unrolled: a stage's addresses are constants of its
      // copy of the body, and the backward branch comes once per two units).
      const uint32_t a_lo0 = plain_desc_lo(smem_u32(sm), D1_CHUNK_PITCH), b_lo0 = plain_desc_lo(smem_u32(sm) + D1_A_BYTES, D1_CHUNK_PITCH);
      const uint32_t full0 = smem_u32(&bars->op_full[0]), empty0 = smem_u32(&bars->op_empty[0]);
      bool go_on = true;
      for (uint32_t parity = 0; go_on; parity ^= 1) {
#pragma unroll
        for (int st = 0; st < D1_NSTAGE; ++st) {
          if (!d1_next_unit(walk, r1, a.b, un)) { go_on = false; break; }
          if (!mbar_wait_addr(full0 + 8 * st, parity) || bars->abort_flag) { bars->abort_flag = 1; go_on = false; break; }
          tc_fence_after();
          const uint32_t a_lo = a_lo0 + st * (D1_STAGE_BYTES / 16), b_lo = b_lo0 + st * (D1_STAGE_BYTES / 16);
          // contraction indices 16 ks .. 16 ks + 15: two core matrices, 2 x 144 bytes further along every row group
#pragma unroll
          for (int ks = 0; ks < D1_KSTEPS; ++ks)
            umma_f16_split(tmem, a_lo + ks * (2 * D1_CHUNK_PITCH / 16), plain_desc_hi(D1_GROUP_BYTES), b_lo + ks * (2 * D1_CHUNK_PITCH / 16),
                           plain_desc_hi(D1_GROUP_BYTES), idesc, (ks == 0 && fresh) ? 0u : 1u);
          fresh = false;
          umma_commit_addr(empty0 + 8 * st);
          if (un.flush) {
            // last rows of the range or of a worker: hand the sums to the write-out warps and wait until they have read them
            umma_commit(&bars->acc_full);
            if (!mbar_wait(&bars->acc_empty, writes & 1)) { bars->abort_flag = 1; go_on = false; break; }
            tc_fence_after();
            ++writes;
            fresh = true;
          }
        }
      }
    }
  } else if (warp <= D1_LOAD_WARPS) {
    // ---------------- staging: group h (D1_GW warps) builds the operands of sample h of every pair
    const int h = (warp - 1) / D1_GW, gt_ = (warp - 1 - h * D1_GW) * 32 + lane;      // thread index inside the group
    // A item of this thread: (channel quad aq, chunk ac, half ah) = four pooled positions of four channels.
    // 4 quads x (24 chunks x 2 halves + the first half of chunk 24) = 196 items; the other threads have none.
    const int aq = gt_ / 49, arem = gt_ - aq * 49, ac = arem >> 1, ah = arem & 1;
    const bool a_item = gt_ < 196;
    const int a_src = (aq * 196 + 8 * ac + 4 * ah);                       // (quad, first position) in units of one position's 4 channels
    const int a_dst = (8 * h + (aq >> 1)) * D1_GROUP_BYTES + ac * D1_CHUNK_PITCH + ((aq & 1) * 4) * 16 + ah * 8;   // window element 0, channel 0 of the quad
    // B items of this thread: shift bn = (sy, sx) and chunks bc0 = gt_ / 16 and bc0 + 16 (the latter for bc0 < 9;
    // chunk 24 holds positions 192..195 only); threads 0..24 also write the ones row's chunk gt_.  Where the sixteen
    // elements lie in the raw slot is fixed for the whole kernel and worked out once: element (sy, sx) of pooled
    // position (py, px) is image pixel (2 py + sy - 1, 2 px + sx - 1); a pixel outside the image, and a position past
    // 195, reads the slot's zero word.
    const int bn = gt_ & 15, sy = bn >> 2, sx = bn & 3, bc0 = gt_ >> 4;
    const int b_dst = D1_A_BYTES + (3 * h + (bn >> 3)) * D1_GROUP_BYTES + (bn & 7) * 16;
    const int ones_dst = D1_A_BYTES + (3 * h + 2) * D1_GROUP_BYTES + gt_ * D1_CHUNK_PITCH;
    int b_off[2][8];
#pragma unroll
    for (int hh = 0; hh < 2; ++hh)
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int p = 8 * (bc0 + 16 * hh) + j, py = p / 14, px = p - 14 * py;
        const int iy = 2 * py + sy - 1, ix = 2 * px + sx - 1;
        b_off[hh][j] = (p < 196 && iy >= 0 && iy < IMG && ix >= 0 && ix < IMG) ? D1_RAW_ZERO / 4 + iy * IMG + ix : 0;
      }

    // The range's q-th sample uses raw slot q % 5 for the (q / 5)-th time; slot0 / use0 are those of the unit's first
    // sample, kept as counters.
    D1Walk walk = d1_begin(r0, a.b);
    int slot0 = 0;
    uint32_t use0 = 0;
    D1Unit un;
    for (int u = 0; d1_next_unit(walk, r1, a.b, un); ++u) {
      const int st = u & 1;
      int slot = slot0 + h;                          // this group's sample is the unit's h-th
      uint32_t use = use0;
      if (slot >= D1_NRAW) { slot -= D1_NRAW; ++use; }
      slot0 += un.n;
      if (slot0 >= D1_NRAW) { slot0 -= D1_NRAW; ++use0; }
      const bool mine = h < un.n;                    // an odd last sample: group 1 only clears its shift block
      bool ok = true;
      if (mine) ok = mbar_wait(&bars->raw_full[slot], use & 1);
      if (ok && u >= 2) ok = mbar_wait(&bars->op_empty[st], ((u >> 1) - 1) & 1);      // the MMAs of unit u - 2 have read the stage
      if (!__all_sync(0xffffffffu, ok) || bars->abort_flag) { bars->abort_flag = 1; break; }
      const uint8_t* rslot = raw + slot * D1_RAW_SLOT;
      const float* img = reinterpret_cast<const float*>(rslot);
      const uint8_t* rg = rslot + D1_RAW_ZERO + D1_RAW_X;
      uint8_t* stage = sm + st * D1_STAGE_BYTES;
      if (mine && a_item) {
        // four positions of four channels: the gradients as two 16-byte loads ([position][4 channels] BF16), the
        // decisions as one ([position][4 channels] bytes)
        const uint4 g01 = reinterpret_cast<const uint4*>(rg)[a_src >> 1];          // positions 0, 1: {c0c1, c2c3, c0c1, c2c3}
        const uint4 g23 = reinterpret_cast<const uint4*>(rg)[(a_src >> 1) + 1];
        const uint4 cd = reinterpret_cast<const uint4*>(rg + D1_RAW_G)[a_src >> 2];
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
      for (int hh = 0; hh < 2; ++hh) {
        const int bc = bc0 + 16 * hh;
        if (bc < 25) {
          uint4 o = make_uint4(0u, 0u, 0u, 0u);        // no second sample: its shift block is zero, so whatever its row block
          if (mine) {                                  // still holds from an earlier pair adds nothing
            float xv[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) xv[j] = img[b_off[hh][j]];
            o = make_uint4(bf16_pair(xv[0], xv[1]), bf16_pair(xv[2], xv[3]), bf16_pair(xv[4], xv[5]), bf16_pair(xv[6], xv[7]));
          }
          *reinterpret_cast<uint4*>(stage + b_dst + bc * D1_CHUNK_PITCH) = o;
        }
      }
      if (gt_ < 25) {
        const uint32_t one2 = mine ? 0x3F803F80u : 0u;                       // the ones row (bias gradient), zero likewise
        *reinterpret_cast<uint4*>(stage + ones_dst) = gt_ < 24 ? make_uint4(one2, one2, one2, one2) : make_uint4(one2, one2, 0u, 0u);
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) { mbar_arrive(&bars->op_full[st]); if (mine) mbar_arrive(&bars->raw_empty[slot]); }
    }
  } else if (warp == D1_LOAD_WARPS + 5) {
    // ---------------- loads: one thread issues every sample's three bulk copies into the raw slots in turn; before a
    // slot's k-th reuse it waits until the eight warps that staged the slot's previous sample have read it
    if (lane == 0) {
      D1Walk walk = d1_begin(r0, a.b);
      int slot = 0, use = 0;
      D1Unit un;
      bool ok = true;
      while (ok && d1_next_unit(walk, r1, a.b, un))
        for (int h = 0; h < un.n; ++h) {
          if (use > 0 && (!mbar_wait(&bars->raw_empty[slot], (use - 1) & 1) || bars->abort_flag)) { bars->abort_flag = 1; ok = false; break; }
          const int r = un.row + h, s = un.s, i = r - s * a.b;
          uint8_t* dst = raw + slot * D1_RAW_SLOT + D1_RAW_ZERO;
          uint64_t* bar = &bars->raw_full[slot];
          mbar_expect_tx(bar, D1_RAW_BYTES);
          bulk_load(dst, a.x + ((int64_t)wt.src[s] * a.b + i) * (IMG * IMG), D1_RAW_X, bar);
          bulk_load(dst + D1_RAW_X, reinterpret_cast<const uint8_t*>(ws.dp1) + (int64_t)r * (P1_ELEMS * 4), D1_RAW_G, bar);
          bulk_load(dst + D1_RAW_X + D1_RAW_G, ws.code1 + (int64_t)r * P1_ELEMS, D1_RAW_CODE, bar);
          if (++slot == D1_NRAW) { slot = 0; ++use; }
        }
    }
  } else {
    // ---------------- write-out: warp q reads the accumulator lanes 32 q .. 32 q + 31 = rows (sample q / 2 of the pair,
    // window elements 2 (q % 2) and 2 (q % 2) + 1, 16 channels each); a sample's sums are in its own 24 columns.  Every
    // (sample, window element) writes its share of the 160 sums to a partial slot of its own (the final reduction adds
    // them in a fixed order), so the warps exchange nothing.
    const int quarter = warp & 3, half = quarter >> 1, my_w = 2 * (quarter & 1) + (lane >> 4), oc = lane & 15;
    int writes = 0;
    D1Walk walk = d1_begin(r0, a.b);
    D1Unit un;
    while (d1_next_unit(walk, r1, a.b, un)) {
      if (!un.flush) continue;
      if (!mbar_wait(&bars->acc_full, writes & 1) || bars->abort_flag) { bars->abort_flag = 1; break; }
      tc_fence_after();
      uint32_t v0[16], v1[16];
      tmem_ld16(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(24 * half), v0);
      tmem_ld16(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(24 * half + 16), v1);      // first column: the bias gradient
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->acc_empty);
      const int s = un.s;
      float* part = ws.part1 + (((int64_t)s * slots + (blockIdx.x - (s * a.b) / seg_len)) * D1_SUBSLOTS + 4 * half + my_w) * C1_GRAD;
      // dW[oc][ky][kx] takes shift (wy + ky, wx + kx) of this window element
#pragma unroll
      for (int w = 0; w < 4; ++w)
        if (w == my_w) {
#pragma unroll
          for (int tap = 0; tap < 9; ++tap) part[oc * 9 + tap] = __uint_as_float(v0[((w >> 1) + tap / 3) * 4 + (w & 1) + tap % 3]);
        }
      part[144 + oc] = __uint_as_float(v1[0]);
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

// Returns the number of partial-sum slots reserved per worker (the stride of part1: eight per range), or -1;
// *seg_len receives the length of a CTA's range of rows: worker s owns eight partial sums per range that meets its rows.
int launch_conv1_dw_tc5(const GradStepArgs& a, const WorkerTable& wt, const Workspace& ws, cudaStream_t st, Profiler* prof,
                        int* seg_len) {
  const int total = a.W * a.b;
  int grid = total / 16;                  // a range is at least 16 rows long (bounds the partial sums per worker)
  if (grid > g_sm_count) grid = g_sm_count;
  if (grid < 1) grid = 1;
  const int len = (total + grid - 1) / grid;
  grid = (total + len - 1) / len;
  const int slots = (a.b - 1) / len + 2;
  TIMED(K_CONV1_BWD, (conv1_dw_tc5<<<grid, D1_THREADS, D1_SMEM, st>>>(a, wt, ws, len, slots)));
  *seg_len = len;
  return D1_SUBSLOTS * slots;
}

}  // namespace psk
