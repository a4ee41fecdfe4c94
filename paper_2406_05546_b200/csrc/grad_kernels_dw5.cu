// Filter and bias gradient of the second convolution on the fifth-generation tensor cores (BF16 operands,
// fp32 accumulation in tensor memory; values only, no decision depends on them).
//
//   dW[oc][ic][ky][kx] = sum over samples and positions of g2[oc][y][x] * p1pad[ic][y + ky][x + kx]
//
// with g2 the gradient at the convolution's output (the pooled gradient put back at the pooling winners) and
// p1pad the zero-bordered 16x16 input.  The contraction runs over positions, so both operands are needed with
// the position index contiguous ("k-major": core matrices of 8 rows x 8 positions).  With q = (y + ky) * 16 + x
// as the contraction index, one MMA per image row q / 16 computes
//
//   D[(kx, ic)][(ky, oc)] += A[(kx, ic)][q] * B[(ky, oc)][q],   A[(kx, ic)][q] = p1pad[ic][q + kx],
//                                                                B[(ky, oc)][q] = g2[oc][q - 16 ky]
//                                                                (at the k-step of image row ks: row ks - ky of g2)
//
// i.e. M = 48 (+ one row of ones, whose products are the bias gradient; the tile is M = 64, the other rows
// are never read), N = 96, K = 16: fourteen MMAs per sample (the input's two border rows contribute nothing),
// accumulated over all samples of a worker.
// The staging warps build both operands: A by transposing 8 x 8 blocks of the BF16 input planes (one
// ldmatrix.trans + stmatrix pair per four blocks; the three kx copies differ in the rows addressed), B from the
// pooled gradient and the pooling decisions.  B is stored ONCE: its three ky copies are the same rows of g2 one
// image row apart, and with the image rows stored in descending order, 512 bytes apart, and the four channel octets
// of a row 128 bytes apart, row group (ky, octet) of the operand is simply 128 (4 ky + octet) bytes after the start
// address of the k-step: a uniform stride, which is all a shared-memory descriptor can express.
// One CTA per SM walks over a contiguous range of rows (sorted worker, sample); where the range passes from one
// worker to the next, and at its end, the accumulator is written out as a partial sum that a later kernel adds
// in a fixed order.  Two groups of staging warps take alternate samples; three operand stages are used in turn, so
// that a group's next sample does not wait for the MMAs of its previous one.  Every mbarrier wait is bounded.
#include "device_common.cuh"
#include "kernels.h"
#include "tc5_common.cuh"

namespace psk {

namespace {

constexpr int W5_LOAD_WARPS = 16;                       // two groups: group g stages samples n = g, g + 2, ...
constexpr int W5_GW = W5_LOAD_WARPS / 2;                // warps per group
constexpr int W5_THREADS = 32 * (1 + W5_LOAD_WARPS + 4 + 1);   // warp 0: MMA issue and tensor memory; then the staging warps, four
                                                               // write-out warps, and the warp that issues the loads
constexpr int W5_CHUNKS = 32;                           // 8-position chunks of the 256 contraction indices of a sample
constexpr int W5_GROUP_BYTES = W5_CHUNKS * 128;         // one group of 8 operand rows: 32 core matrices of 128 bytes
constexpr int W5_A_GROUPS = 7;                          // (kx, channel octet) x 6, then the group whose first row is all ones
constexpr int W5_A_BYTES = W5_A_GROUPS * W5_GROUP_BYTES;     // 28,672
// B: [column parity (x & 1)][image row, descending: y = 14 .. -1][channel octet][8 channels x 8 places (x / 2)];
// rows y = 14 and y = -1 are never written (zeros): the k-steps next to the border read them
constexpr int W5_B_ROW = 4 * 128, W5_B_HALF = 16 * W5_B_ROW;      // 512 bytes per image row, 8,192 per half
constexpr int W5_B_BYTES = 2 * W5_B_HALF;               // 16,384
constexpr int W5_STAGE_BYTES = W5_A_BYTES + W5_B_BYTES; // 45,056; the A descriptor of M = 64 spans 8 groups from the stage's
                                                        // start (the eighth is B's first 4 KB: rows never read)
constexpr int W5_NSTAGE = 3;                            // operand stages, used in turn (sample n -> stage n % 3)
constexpr int W5_RAW_P1 = P1_PLANE_ELEMS * 4, W5_RAW_DP2 = FLAT * 2, W5_RAW_CODE = FLAT;      // dp2 arrives as BF16
constexpr int W5_RAW_BYTES = W5_RAW_P1 + W5_RAW_DP2 + W5_RAW_CODE;          // 12,896
constexpr int W5_RAW_SLOT = (W5_RAW_BYTES + 127) / 128 * 128;
constexpr int W5_NRAW = 6;                              // raw input slots (sample n -> slot n % 6): the copies, issued by a warp of their
                                                        // own (issuing them costs a staging thread hundreds of cycles per sample, which
                                                        // its whole group then waits for), run up to six samples ahead
constexpr int W5_SMEM = W5_NSTAGE * W5_STAGE_BYTES + W5_NRAW * W5_RAW_SLOT + 256 + 128;
constexpr int W5_NACC = 1;                              // accumulators used in turn and added up at write-out (measured: four instead of one
                                                        // change nothing, so consecutive MMAs into one accumulator do not wait for each other)
constexpr int W5_TMEM_COLS = 128;                       // W5_NACC x 96 accumulator columns, rounded up to a power of two
static_assert(8 * W5_GROUP_BYTES <= W5_STAGE_BYTES, "the 64-row A operand must stay inside its stage");
static_assert(W5_SMEM <= 227 * 1024, "shared memory");

__host__ __device__ constexpr uint32_t w5_idesc(int m, int n) {     // fp32 accumulate, BF16 x BF16, both k-contiguous
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void stmatrix_x4(uint32_t addr, const uint32_t (&r)[4]) {
  asm volatile("stmatrix.sync.aligned.m8n8.x4.shared.b16 [%0], {%1,%2,%3,%4};"
               ::"r"(addr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
}

struct W5Bars {
  uint64_t op_full[W5_NSTAGE], op_empty[W5_NSTAGE], raw_full[W5_NRAW], raw_empty[W5_NRAW], acc_full, acc_empty;
  uint32_t tmem_base;
  volatile uint32_t abort_flag;
};

// Rows (sorted worker, sample) are split into gridDim.x contiguous ranges of seg_len.  Partial sums of worker s go
// to part2[s][range index - first range of s].
__global__ void __launch_bounds__(W5_THREADS, 1) conv2_dw_tc5(GradStepArgs a, WorkerTable wt, Workspace ws, int seg_len, int slots) {
  extern __shared__ __align__(1024) uint8_t sm[];
  uint8_t* raw = sm + W5_NSTAGE * W5_STAGE_BYTES;
  W5Bars* bars = reinterpret_cast<W5Bars*>(raw + W5_NRAW * W5_RAW_SLOT);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int total = a.W * a.b;
  const int r0 = blockIdx.x * seg_len, r1 = min(r0 + seg_len, total), n_samples = r1 - r0;

  // operand stages start as zeros (B: borders and rows that a ky copy never reaches); the ones row of A is
  // written once: row 0 of group 6, i.e. the first 16 bytes of each of its core matrices
  for (int i = tid; i < W5_NSTAGE * W5_STAGE_BYTES / 16; i += W5_THREADS) reinterpret_cast<uint4*>(sm)[i] = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
  for (int i = tid; i < W5_NSTAGE * W5_CHUNKS; i += W5_THREADS)
    *reinterpret_cast<uint4*>(sm + (i / W5_CHUNKS) * W5_STAGE_BYTES + 6 * W5_GROUP_BYTES + (i % W5_CHUNKS) * 128) =
        make_uint4(0x3F803F80u, 0x3F803F80u, 0x3F803F80u, 0x3F803F80u);
  if (tid == 0) {
    for (int i = 0; i < W5_NSTAGE; ++i) { mbar_init(&bars->op_full[i], W5_LOAD_WARPS / 2); mbar_init(&bars->op_empty[i], 1); }
    for (int i = 0; i < W5_NRAW; ++i) { mbar_init(&bars->raw_full[i], 1); mbar_init(&bars->raw_empty[i], W5_LOAD_WARPS / 2); }
    mbar_init(&bars->acc_full, 1);
    mbar_init(&bars->acc_empty, 4);
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)), "r"(W5_TMEM_COLS) : "memory");
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
      // This loop is one thread's serial instruction stream, with nothing to hide its latencies: an integer division
      // or modulo here costs hundreds of cycles per sample, so stage, parity, descriptors and the next write-out row are
      // all carried along as counters.
      constexpr uint32_t idesc = w5_idesc(64, 96);
      constexpr uint32_t stage_step = W5_STAGE_BYTES / 16;
      const uint32_t a_lo0 = plain_desc_lo(smem_u32(sm), 128);
      // B at k-step ks starts at the stored row of y = ks (14 - ks rows in); its two k-chunks are the halves of a row
      const uint32_t b_lo0 = plain_desc_lo(smem_u32(sm) + W5_A_BYTES + 14 * W5_B_ROW, W5_B_HALF);
      const uint32_t full0 = smem_u32(&bars->op_full[0]), empty0 = smem_u32(&bars->op_empty[0]);
      uint32_t parity = 0, writes = 0;
      int flush_at = min(r1, (r0 / a.b + 1) * a.b) - 1 - r0;     // index in the range of the next row that ends a worker or the range
      bool fresh = true;                       // the next MMA starts a new sum
      bool go_on = true;
      // One pass of the outer loop takes the stages in turn (unrolled: a stage's addresses are constants of its copy
      // of the body, and the backward branch, after which the instruction fetch starts afresh, comes once per three samples).
      for (int n = 0; go_on && n < n_samples; parity ^= 1) {
#pragma unroll
        for (int st = 0; st < W5_NSTAGE; ++st, ++n) {
          if (n >= n_samples) { go_on = false; break; }
          const uint32_t a_lo = a_lo0 + st * stage_step, b_lo = b_lo0 + st * stage_step;
          if (!mbar_wait_addr(full0 + 8 * st, parity) || bars->abort_flag) { bars->abort_flag = 1; go_on = false; break; }
          tc_fence_after();
          // contraction indices 16 ks .. 16 ks + 15 (image row ks of the bordered input): two chunks of 128 bytes.
          // Rows 0 and 15 are the input's zero border, so their products vanish and are not issued.
#pragma unroll
          for (int ks = 1; ks < 15; ++ks)
            umma_f16_split(tmem, a_lo + ks * 16, plain_desc_hi(W5_GROUP_BYTES), b_lo - ks * (W5_B_ROW / 16), plain_desc_hi(128), idesc,
                           (ks == 1 && fresh) ? 0u : 1u);
          fresh = false;
          umma_commit_addr(empty0 + 8 * st);
          if (n == flush_at) {
            // last row of the range or of a worker: hand the sum to the write-out warps and wait until they have read it
            umma_commit(&bars->acc_full);
            if (!mbar_wait(&bars->acc_empty, writes & 1)) { bars->abort_flag = 1; go_on = false; break; }
            tc_fence_after();
            ++writes;
            fresh = true;
            flush_at = min(flush_at + a.b, n_samples - 1);
          }
        }
      }
    }
  } else if (warp <= W5_LOAD_WARPS) {
    // ---------------- staging: group g (W5_GW warps) builds the operands of samples n = g, g + 2, ... in stage n % 3
    const int grp = (warp - 1) / W5_GW, gw = (warp - 1) - grp * W5_GW;      // group, and warp inside the group
    // sample n uses raw slot n % 6 for the (n / 6)-th time and operand stage n % 3 for the (n / 3)-th: kept as counters
    int slot = grp, st = grp;
    uint32_t slot_use = 0, st_use = 0;
    for (int n = grp; n < n_samples; n += 2) {
      bool ok = mbar_wait(&bars->raw_full[slot], slot_use & 1);
      if (ok && st_use > 0) ok = mbar_wait(&bars->op_empty[st], (st_use - 1) & 1);      // the MMAs of sample n - 3 have read the stage
      if (!__all_sync(0xffffffffu, ok) || bars->abort_flag) { bars->abort_flag = 1; break; }
      const uint8_t* rp1 = raw + slot * W5_RAW_SLOT;
      const uint16_t* rdp2h = reinterpret_cast<const uint16_t*>(rp1 + W5_RAW_P1);
      const uint8_t* rcode8 = rp1 + W5_RAW_P1 + W5_RAW_DP2;
      uint8_t* stage = sm + st * W5_STAGE_BYTES;
      // Inside an image row the sixteen positions are taken in the order of the input planes' rows, even columns then
      // odd columns (contraction index 16 y + 8 (x & 1) + x / 2 for both operands: a sum does not care about its order),
      // so that the eight positions of a chunk are eight CONSECUTIVE plane rows and a transposing load meets no bank twice.
      // A: 6 groups x 32 chunks = 192 blocks of 8 positions x 8 channels, transposed four at a time.  Operation o of
      // the 48 covers chunks 4 (o % 8) .. + 3 of group o / 8 = (kx, channel octet).  Lane l addresses row l % 8 of
      // block l / 8: on the way in the plane row of the position kx columns to the right of the chunk's (l % 8)-th
      // (positions past the end read the all-zero row 0), on the way out the core matrix's row.
#pragma unroll
      for (int o = gw; o < 48; o += W5_GW) {
        const int g = o >> 3, kx = g >> 1, oct = g & 1, chunk = 4 * (o & 7) + (lane >> 3);
        const int i = 16 * (chunk >> 1) + 2 * (lane & 7) + (chunk & 1) + kx;       // position y * 16 + x
        const int prow = i < 256 ? (i & ~15) + ((i & 1) << 3) + ((i & 15) >> 1) : 0;
        uint32_t r[4];
        ldmatrix_x4_trans(r, smem_u32(rp1 + oct * 4096 + prow * 16));
        stmatrix_x4(smem_u32(stage + g * W5_GROUP_BYTES + chunk * 128 + (lane & 7) * 16), r);
      }
      // B: a warp takes (octet of output channels, pooled row py) and a lane one channel of the octet and the pooled
      // columns 2j, 2j + 1: its words then fall into 32 different banks.  Every pooled entry owns the four positions of
      // its window: shifted left by 16 bits per decision, the BF16 gradient lands in the half-word of the winner (low
      // word: image row 2py, high word: row 2py + 1; in each, low half: column 2px, high half: column 2px + 1; decision
      // 4 shifts it out), the other three are cleared.  Column x of an image row sits in chunk x & 1 at place x / 2, so
      // the two entries' half-words of equal (row, column parity) make one word; image row y is stored 14 - y rows into
      // its half.
      for (int wi = gw; wi < 28; wi += W5_GW) {
        const int oct = wi / 7, py = wi - oct * 7;
        const int rr = lane >> 2, j = lane & 3, oc = 8 * oct + rr;
        const int e = ((oc >> 2) * 49 + py * 7 + 2 * j) * 4 + (oc & 3);
        const uint32_t code0 = rcode8[e], code1 = j < 3 ? rcode8[e + 4] : 4u;      // pooled column 7 does not exist
        const unsigned long long s0 = shl64_clamped(rdp2h[e], 16u * code0), s1 = shl64_clamped(j < 3 ? rdp2h[e + 4] : (uint16_t)0, 16u * code1);
        const uint32_t lo0 = (uint32_t)s0, hi0 = (uint32_t)(s0 >> 32), lo1 = (uint32_t)s1, hi1 = (uint32_t)(s1 >> 32);
        uint32_t* d = reinterpret_cast<uint32_t*>(stage + W5_A_BYTES + (14 - 2 * py) * W5_B_ROW + oct * 128 + rr * 16) + j;
        d[0] = prmt(lo0, lo1, 0x5410u);                                   // image row 2py, even columns
        d[W5_B_HALF / 4] = prmt(lo0, lo1, 0x7632u);                       // image row 2py, odd columns
        d[-(W5_B_ROW / 4)] = prmt(hi0, hi1, 0x5410u);                     // image row 2py + 1, even columns
        d[W5_B_HALF / 4 - W5_B_ROW / 4] = prmt(hi0, hi1, 0x7632u);        // image row 2py + 1, odd columns
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) { mbar_arrive(&bars->op_full[st]); mbar_arrive(&bars->raw_empty[slot]); }
      slot += 2;
      if (slot >= W5_NRAW) { slot -= W5_NRAW; ++slot_use; }
      st += 2;
      if (st >= W5_NSTAGE) { st -= W5_NSTAGE; ++st_use; }
    }
  } else if (warp == W5_LOAD_WARPS + 5) {
    // ---------------- loads: one thread issues every sample's three bulk copies into the raw slots in turn; before a
    // slot's reuse it waits until the eight warps that staged the slot's previous sample have read it
    if (lane == 0) {
      int slot = 0, use = 0;
      for (int n = 0; n < n_samples; ++n) {
        if (use > 0 && (!mbar_wait(&bars->raw_empty[slot], (use - 1) & 1) || bars->abort_flag)) { bars->abort_flag = 1; break; }
        const int64_t row = r0 + n;
        uint8_t* dst = raw + slot * W5_RAW_SLOT;
        uint64_t* bar = &bars->raw_full[slot];
        mbar_expect_tx(bar, W5_RAW_BYTES);
        bulk_load(dst, ws.p1 + row * P1_PLANE_ELEMS, W5_RAW_P1, bar);
        bulk_load(dst + W5_RAW_P1, ws.dp2 + row * FLAT, W5_RAW_DP2, bar);
        bulk_load(dst + W5_RAW_P1 + W5_RAW_DP2, ws.code2 + row * FLAT, W5_RAW_CODE, bar);
        if (++slot == W5_NRAW) { slot = 0; ++use; }
      }
    }
  } else {
    // ---------------- write-out: a warp reads the accumulator lanes 32 (warp % 4) .. + 31.  An accumulator of 64 rows
    // keeps rows 16 w .. 16 w + 15 in the first sixteen lanes of quarter w.
    const int quarter = warp & 3;
    int writes = 0;
    int s = r0 / a.b;                                    // sorted worker of the rows being summed
    // the rows after which the sum is written out: the last of every worker in the range, and the range's last
    for (int row = min(r1, (s + 1) * a.b) - 1; row < r1; row = (row + 1 == r1) ? r1 : min(row + a.b, r1 - 1), ++s) {
      if (!mbar_wait(&bars->acc_full, writes & 1) || bars->abort_flag) { bars->abort_flag = 1; break; }
      tc_fence_after();
      float* part = ws.part2 + ((int64_t)s * slots + (blockIdx.x - (s * a.b) / seg_len)) * C2_GRAD;
      const int rr = lane < 16 ? quarter * 16 + lane : 64;   // accumulator row: (kx, ic) for rr < 48, the ones row at 48
#pragma unroll
      for (int cb = 0; cb < 6; ++cb) {                 // 16 columns at a time: ky = cb / 2, oc = 16 (cb % 2) + j
        float v[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) v[j] = 0.f;
#pragma unroll
        for (int acc = 0; acc < W5_NACC; ++acc) {       // fixed order
          uint32_t t[16];
          tmem_ld16(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * 96 + cb * 16), t);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 16; ++j) v[j] += __uint_as_float(t[j]);
        }
        const int ky = cb >> 1;
        if (rr < 48) {
          const int kx = rr >> 4, ic = rr & 15;
#pragma unroll
          for (int j = 0; j < 16; ++j) part[((16 * (cb & 1) + j) * 16 + ic) * 9 + ky * 3 + kx] = v[j];
        } else if (rr == 48 && ky == 1) {     // the ones row against the ky = 1 copy, whose rows 1..14 are all issued
#pragma unroll
          for (int j = 0; j < 16; ++j) part[4608 + 16 * (cb & 1) + j] = v[j];
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->acc_empty);
      ++writes;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(W5_TMEM_COLS) : "memory");
  }
  if (tid == 0 && bars->abort_flag) {
    atomicOr(ws.status, STATUS_WAIT_TIMEOUT);
    for (int k = 0; k < 1000; ++k) __nanosleep(1000);   // let copies already issued land before the CTA ends
  }
}

}  // namespace

#define TIMED(id, launch) do { if (prof) prof->begin(id, st); launch; if (prof) prof->end(st); } while (0)

int configure_dw5_kernels() {
  return cudaFuncSetAttribute(conv2_dw_tc5, cudaFuncAttributeMaxDynamicSharedMemorySize, W5_SMEM) == cudaSuccess ? 0 : -1;
}

// Returns the number of partial-sum slots reserved per worker (the stride of part2) and, in *seg_len, the length
// of a CTA's range of rows: worker s owns one partial sum per range that meets its rows.
int launch_conv2_dw_tc5(const GradStepArgs& a, const WorkerTable& wt, const Workspace& ws, cudaStream_t st, Profiler* prof,
                        int* seg_len) {
  const int total = a.W * a.b;
  int grid = total / 16;                  // a range is at least 16 rows long (bounds the partial sums per worker)
  if (grid > g_sm_count) grid = g_sm_count;
  if (grid < 1) grid = 1;
  const int len = (total + grid - 1) / grid;
  grid = (total + len - 1) / len;
  const int slots = (a.b - 1) / len + 2;
  TIMED(K_CONV2_DW, (conv2_dw_tc5<<<grid, W5_THREADS, W5_SMEM, st>>>(a, wt, ws, len, slots)));
  *seg_len = len;
  return slots;
}

}  // namespace psk
