// Filter gradient of the second convolution on the tensor cores (BF16 operands, warp-level mma.sync): the one
// contraction of the step whose output (32 x 144 per worker) is too small for a 128-row tcgen05 tile,
// while its reduction (all positions of all samples of a worker) is long.
//
// Reductions keep a fixed order, so results are reproducible bit for bit.
#include "device_common.cuh"
#include "kernels.h"
#include "tc5_common.cuh"

namespace psk {

namespace {

// Filter gradient: dW[oc][ic][tap] = sum_{samples,pos} g2[oc][pos] * p1[ic][pos + tap]: rows = 32 output
// channels, columns = 16 input channels per tap, k = position (196 per sample, 13 k-steps of 16, zero-padded).
// Both operands are rounded to BF16 here (fp32 accumulation): this product only yields gradient values, no
// ReLU or pooling decision depends on it, and at 16 positions per instruction it needs half the
// instructions and shared-memory loads of the TF32 form.
// 512 threads: twelve MMA warps and four loader warps, one CTA per SM walking over a contiguous range of samples.
// The loaders fetch a sample's pooled gradient, pooling decisions and input planes one sample ahead, write
// them as BF16 operands into one of two shared-memory buffers and signal an mbarrier; the MMA warps never
// wait for staging.  MMA warp = (share of the 13 k-steps, filter row): it multiplies one set of g2 fragments
// (ldmatrix) with the image fragments of the three taps of its filter row, twelve independent MMAs per
// k-step; accumulators persist over the range and are written as partial sums at its end (and where the
// range passes from one worker to the next); a later kernel adds the partial sums in a fixed order.  The bias
// gradient (sum of g2 over positions) rides along as a product with a column of ones in the warps of
// filter row 0.
// A BF16 fragment register holds two consecutive k = two horizontally adjacent positions (x even, x+1) of
// the flattened 14-wide image, so a tap is a constant word offset (7 words per filter row).  The image
// is kept three times, once per filter column: the copy of the left (right) taps is shifted by one element
// so that its pairs are word-aligned, and leaves out column 13 (0), whose shifted slot is the neighbouring
// row's out-of-image column and must read zero.
// Every mbarrier wait is bounded; on a timeout the kernel raises a status flag and all warps leave.
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

constexpr int DW_G_WORDS = 108;    // 216 bf16 per output channel: 196 positions + zeros; 108 = 12 (mod 32 banks)
constexpr int DW_P_WORDS = 132;    // plane of one input channel: 16 rows x 14 bf16 (rows 0 and 15 stay zero) = 112
                                   // words, + the words the zero-padded k tail reaches; 132 = 4 (mod 32 banks)
constexpr int DW_MMA_WARPS = 12, DW_LOAD_WARPS = 8;
constexpr int DW_THREADS = 32 * (DW_MMA_WARPS + DW_LOAD_WARPS);
constexpr int DW_LOADERS = 32 * DW_LOAD_WARPS;
constexpr int DW_BUF_WORDS = 32 * DW_G_WORDS + 3 * 16 * DW_P_WORDS;   // one sample: g2 and three image copies
constexpr int DW_RAW_P1 = P1_PLANE_ELEMS * 4, DW_RAW_DP2 = FLAT * 4, DW_RAW_CODE = FLAT;   // bytes of one sample's inputs
constexpr int DW_RAW_BYTES = DW_RAW_P1 + DW_RAW_DP2 + DW_RAW_CODE;
constexpr int DW_RAW_WORDS = (DW_RAW_BYTES + 127) / 128 * 32;          // raw buffer, padded to 128 bytes
constexpr int DW_NRAW = 3;         // raw input buffers: copies run three samples ahead of the MMAs
constexpr int DW_SMEM_BYTES = (2 * DW_BUF_WORDS + DW_NRAW * DW_RAW_WORDS) * 4 + 128;
static_assert(DW_RAW_P1 % 16 == 0 && DW_RAW_DP2 % 16 == 0 && DW_RAW_CODE % 16 == 0, "bulk copies move multiples of 16 bytes");
constexpr int DW_MIN_SEG = 16;     // a CTA's range is at least this long (bounds the partial sums per worker)
constexpr int DW_PAIRS = (2 * 98 + DW_LOADERS - 1) / DW_LOADERS;      // (plane, position pair) items per loader thread
constexpr int DW_ENTRIES = (8 * 49 + DW_LOADERS - 1) / DW_LOADERS;    // (channel quad, position) items per loader thread

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}

// The k-steps K0..K1-1 of one sample for one warp: two ldmatrix for g2, twelve word loads for the three taps of the
// warp's filter row, twelve MMAs (+ two for the bias in the warps of filter row 0).
template <int K0, int K1>
__device__ __forceinline__ void dw_ksteps(uint32_t a_addr, const uint32_t* b_base, float (&acc)[3][2][2][4],
                                          float (&accb)[2][4], bool with_bias, const uint32_t (&one_frag)[2]) {
#pragma unroll
  for (int ks = K0; ks < K1; ++ks) {
    uint32_t fa[2][4], fb[3][2][2];
    ldmatrix_x4(fa[0], a_addr + ks * 32);
    ldmatrix_x4(fa[1], a_addr + 16 * DW_G_WORDS * 4 + ks * 32);
#pragma unroll
    for (int kx = 0; kx < 3; ++kx)
#pragma unroll
      for (int n = 0; n < 2; ++n) {
        fb[kx][n][0] = b_base[(kx * 16 + n * 8) * DW_P_WORDS + ks * 8];
        fb[kx][n][1] = b_base[(kx * 16 + n * 8) * DW_P_WORDS + ks * 8 + 4];
      }
#pragma unroll
    for (int kx = 0; kx < 3; ++kx)
#pragma unroll
      for (int m = 0; m < 2; ++m)
#pragma unroll
        for (int n = 0; n < 2; ++n) mma_bf16(acc[kx][m][n], fa[m], fb[kx][n]);
    if (with_bias) {                   // warp-uniform
      mma_bf16(accb[0], fa[0], one_frag);
      mma_bf16(accb[1], fa[1], one_frag);
    }
  }
}

// Rows (sorted worker, sample) are split into gridDim.x contiguous ranges of seg_len; a range may cross from one
// worker into the next, where the accumulators are written out and cleared.  Partial sums of worker s go to
// part2[s][4 * (range index - first range of s) + k-share].
__global__ void __launch_bounds__(DW_THREADS, 1) conv2_dw_tc(GradStepArgs a, WorkerTable wt, Workspace ws, int seg_len, int slots) {
  extern __shared__ __align__(128) uint32_t dw_smem[];
  uint32_t* raw = dw_smem + 2 * DW_BUF_WORDS;                                   // [DW_NRAW][DW_RAW_WORDS]
  uint64_t* full = reinterpret_cast<uint64_t*>(raw + DW_NRAW * DW_RAW_WORDS);   // [2] loaders -> MMA warps
  uint64_t* empty = full + 2;                                                    // [2] MMA warps -> loaders
  uint64_t* raw_full = full + 4;                                                 // [DW_NRAW] bulk copies -> loaders
  uint64_t* raw_empty = raw_full + DW_NRAW;                                      // [DW_NRAW] loaders -> copy issuer
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(raw_empty + DW_NRAW);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int total = a.W * a.b;
  const int r0 = blockIdx.x * seg_len, r1 = min(r0 + seg_len, total);
  for (int idx = tid; idx < 2 * DW_BUF_WORDS; idx += DW_THREADS) dw_smem[idx] = 0u;
  if (tid == 0) {
    mbar_init(&full[0], DW_LOADERS); mbar_init(&full[1], DW_LOADERS);
    mbar_init(&empty[0], 32 * DW_MMA_WARPS); mbar_init(&empty[1], 32 * DW_MMA_WARPS);
    for (int i = 0; i < DW_NRAW; ++i) { mbar_init(&raw_full[i], 1); mbar_init(&raw_empty[i], DW_LOADERS); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  if (warp >= DW_MMA_WARPS) {
    // ---------------- loaders: bulk copies global -> raw buffers (three samples ahead), then BF16 operands
    const int lt = tid - 32 * DW_MMA_WARPS;
    auto issue = [&](int n) {            // one thread: the three input rows of sample r0 + n
      const int64_t row = r0 + n;
      uint8_t* dst = reinterpret_cast<uint8_t*>(raw + (n % DW_NRAW) * DW_RAW_WORDS);
      uint64_t* bar = &raw_full[n % DW_NRAW];
      mbar_expect_tx(bar, DW_RAW_BYTES);
      bulk_load(dst, ws.p1 + row * P1_PLANE_ELEMS, DW_RAW_P1, bar);
      bulk_load(dst + DW_RAW_P1, ws.dp2 + row * FLAT, DW_RAW_DP2, bar);
      bulk_load(dst + DW_RAW_P1 + DW_RAW_DP2, ws.code2 + row * FLAT, DW_RAW_CODE, bar);
    };
    if (lt == 0)
      for (int n = 0; n < DW_NRAW && r0 + n < r1; ++n) issue(n);
    for (int row = r0, n = 0; row < r1; ++row, ++n) {
      const int buf = n & 1, rb = n % DW_NRAW;
      bool ok = mbar_wait(&raw_full[rb], (n / DW_NRAW) & 1);
      if (ok && n >= 2) ok = mbar_wait(&empty[buf], ((n >> 1) - 1) & 1);
      if (!ok) { *abort_flag = 1; atomicOr(ws.status, STATUS_WAIT_TIMEOUT); }
      if (*abort_flag) break;
      const float* rp1 = reinterpret_cast<const float*>(raw + rb * DW_RAW_WORDS);
      const float* rdp2 = rp1 + P1_PLANE_ELEMS;
      const uint8_t* rcode = reinterpret_cast<const uint8_t*>(rdp2 + FLAT);
      uint32_t* g2w = dw_smem + buf * DW_BUF_WORDS;
      // Item = (plane q of eight channels, pair w of horizontally adjacent positions 2w, 2w+1 of the flattened
      // 14-wide image).  Word w + 7 of a channel's plane holds positions (x, x+1) in the middle copy,
      // (x-1, x) in the copy of the left taps and (x+1, x+2) in the copy of the right taps; x-1 = -1 and
      // x+2 = 14 read the zero border of the source plane.  The source is already BF16 (one position =
      // eight channels = 16 bytes), so a pair is two half-words picked out of two rows.
#pragma unroll
      for (int k = 0; k < DW_PAIRS; ++k) {
        const int e = lt + k * DW_LOADERS;
        if (e < 2 * 98) {
          const int q = e / 98, w = e - q * 98, y = w / 7, x = 2 * (w - y * 7);
          const uint4* src = reinterpret_cast<const uint4*>(rp1) + q * 256 + (y + 1) * 16;   // row Y = y + 1: even X in rows 0..7, odd X in 8..15
          // X = x + 1 + j for j = -1..2: X = x (even), x + 1 (odd), x + 2 (even), x + 3 (odd)
          const uint4 v0 = src[x >> 1], v1 = src[8 + (x >> 1)], v2 = src[(x >> 1) + 1], v3 = src[8 + (x >> 1) + 1];
          const uint32_t a0[4] = {v0.x, v0.y, v0.z, v0.w}, a1[4] = {v1.x, v1.y, v1.z, v1.w};
          const uint32_t a2[4] = {v2.x, v2.y, v2.z, v2.w}, a3[4] = {v3.x, v3.y, v3.z, v3.w};
          uint32_t* d = g2w + 32 * DW_G_WORDS + (8 * q) * DW_P_WORDS + w + 7;
#pragma unroll
          for (int j = 0; j < 4; ++j) {      // word j of a row holds channels 2j (low half) and 2j + 1 (high half)
            d[(2 * j) * DW_P_WORDS] = __byte_perm(a0[j], a1[j], 0x5410);
            d[(2 * j + 1) * DW_P_WORDS] = __byte_perm(a0[j], a1[j], 0x7632);
            d[(16 + 2 * j) * DW_P_WORDS] = __byte_perm(a1[j], a2[j], 0x5410);
            d[(16 + 2 * j + 1) * DW_P_WORDS] = __byte_perm(a1[j], a2[j], 0x7632);
            d[(32 + 2 * j) * DW_P_WORDS] = __byte_perm(a2[j], a3[j], 0x5410);
            d[(32 + 2 * j + 1) * DW_P_WORDS] = __byte_perm(a2[j], a3[j], 0x7632);
          }
        }
      }
      // Item = (quad of output channels, pooled position): the raw buffer holds gradients and decisions as
      // [channel quad][position][4 channels].  Every pooled entry owns the four positions of its window: its
      // gradient goes to the chosen one, the others are cleared, so no separate clearing pass is needed.
#pragma unroll
      for (int k = 0; k < DW_ENTRIES; ++k) {
        const int e = lt + k * DW_LOADERS;
        if (e < 8 * 49) {
          const int q = e / 49, p = e - q * 49, py = p / 7, px = p - py * 7;
          const float4 v4 = reinterpret_cast<const float4*>(rdp2)[e];
          const uint32_t c4 = reinterpret_cast<const uint32_t*>(rcode)[e];
          const float v[4] = {v4.x, v4.y, v4.z, v4.w};
          uint32_t* d = g2w + (4 * q) * DW_G_WORDS + (2 * py) * 7 + px;    // word of positions (2py, 2px), (2py, 2px+1)
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            // shifted left by 16 bits per decision, the BF16 value lands in the half-word of the winning window position
            // (low word: row 2py, high word: row 2py + 1); decision 4 shifts it out entirely
            const uint32_t code = (c4 >> (8 * c)) & 0xFFu;
            const unsigned long long slot = shl64_clamped(bf16_bits(v[c]), 16u * code);
            d[c * DW_G_WORDS] = (uint32_t)slot;
            d[c * DW_G_WORDS + 7] = (uint32_t)(slot >> 32);
          }
        }
      }
      mbar_arrive(&full[buf]);
      mbar_arrive(&raw_empty[rb]);
      if (lt == 0 && row + DW_NRAW < r1) {
        // every loader has read this raw buffer: refill it with the sample three ahead
        if (!mbar_wait(&raw_empty[rb], (n / DW_NRAW) & 1)) { *abort_flag = 1; atomicOr(ws.status, STATUS_WAIT_TIMEOUT); break; }
        issue(n + DW_NRAW);
      }
    }
  } else {
    // ---------------- MMA warps: warp = (k-share, filter row); the k-shares are 4, 3, 3, 3 of the 13 k-steps
    const int g = lane >> 2, t = lane & 3;
    const int kpart = warp / 3, ky = warp - kpart * 3;
    float acc[3][2][2][4], accb[2][4];
    auto clear = [&]() {
#pragma unroll
      for (int m = 0; m < 2; ++m) {
#pragma unroll
        for (int kx = 0; kx < 3; ++kx)
#pragma unroll
          for (int n = 0; n < 2; ++n)
#pragma unroll
            for (int r = 0; r < 4; ++r) acc[kx][m][n][r] = 0.f;
#pragma unroll
        for (int r = 0; r < 4; ++r) accb[m][r] = 0.f;
      }
    };
    clear();
    // the column of ones: B(k, n) = 1 for n == 0; this lane supplies column n = g
    const uint32_t one_frag[2] = {g == 0 ? 0x3F803F80u : 0u, g == 0 ? 0x3F803F80u : 0u};
    // A fragments by ldmatrix: lane l addresses row (l & 7) + 8 * ((l >> 3) & 1) of the 16-row tile, k half l >> 4
    const uint32_t a_off = (uint32_t)(((lane & 7) + ((lane >> 3) & 1) * 8) * DW_G_WORDS * 4 + (lane >> 4) * 16);
    // B fragments: column n = input channel g (+8), k pair ks*8 + t (+4) -> word ks*8 + t + 7*ky of the tap's copy
    const int b_off = 32 * DW_G_WORDS + g * DW_P_WORDS + t + 7 * ky;
    for (int row = r0, n = 0; row < r1; ++row, ++n) {
      const int buf = n & 1;
      // the products below are warp-wide instructions: the decision to go on must be the same in all lanes
      const bool ready = mbar_wait(&full[buf], (n >> 1) & 1) && *abort_flag == 0;
      if (!__all_sync(0xffffffffu, ready)) {
        if (lane == 0) { *abort_flag = 1; atomicOr(ws.status, STATUS_WAIT_TIMEOUT); }
        break;
      }
      const uint32_t a_addr = smem_u32(dw_smem + buf * DW_BUF_WORDS) + a_off;
      const uint32_t* b_base = dw_smem + buf * DW_BUF_WORDS + b_off;
      if (kpart == 0) dw_ksteps<0, 4>(a_addr, b_base, acc, accb, ky == 0, one_frag);
      else if (kpart == 1) dw_ksteps<4, 7>(a_addr, b_base, acc, accb, ky == 0, one_frag);
      else if (kpart == 2) dw_ksteps<7, 10>(a_addr, b_base, acc, accb, ky == 0, one_frag);
      else dw_ksteps<10, 13>(a_addr, b_base, acc, accb, ky == 0, one_frag);
      mbar_arrive(&empty[buf]);
      const int s = row / a.b;
      if (row + 1 == r1 || (row + 1) % a.b == 0) {
        // last row of the range or of worker s: write this warp's partial sums and start over
        const int sub = 4 * (blockIdx.x - (s * a.b) / seg_len) + kpart;
        float* part = ws.part2 + ((int64_t)s * slots + sub) * C2_GRAD;
#pragma unroll
        for (int kx = 0; kx < 3; ++kx)
#pragma unroll
          for (int m = 0; m < 2; ++m)
#pragma unroll
            for (int nn = 0; nn < 2; ++nn) {
              const int oc = m * 16 + g, ic = nn * 8 + 2 * t, tap = ky * 3 + kx;
              part[(oc * 16 + ic) * 9 + tap] = acc[kx][m][nn][0];
              part[(oc * 16 + ic + 1) * 9 + tap] = acc[kx][m][nn][1];
              part[((oc + 8) * 16 + ic) * 9 + tap] = acc[kx][m][nn][2];
              part[((oc + 8) * 16 + ic + 1) * 9 + tap] = acc[kx][m][nn][3];
            }
        // column 0 of the ones-product lives in the lanes with t == 0: rows g and g+8 of each 16-row tile
        if (ky == 0 && t == 0) {
#pragma unroll
          for (int m = 0; m < 2; ++m) {
            part[4608 + m * 16 + g] = accb[m][0];
            part[4608 + m * 16 + g + 8] = accb[m][2];
          }
        }
        clear();
      }
    }
  }
  // after a timeout, give bulk copies that are still in flight time to land before the CTA's shared memory is released
  if (tid == 32 * DW_MMA_WARPS && *abort_flag)
    for (int i = 0; i < 1000; ++i) __nanosleep(1000);
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
constexpr int C1B_SPB = 16;
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

int configure_tc_kernels() {
  return cudaFuncSetAttribute(conv2_dw_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, DW_SMEM_BYTES) == cudaSuccess ? 0 : -1;
}

// Returns the number of partial-sum slots reserved per worker (the stride of part2) and, in *seg_len, the length
// of a CTA's range of rows: worker s owns 4 x (ranges that meet its rows) partial sums.
int launch_conv2_dw_tc(const GradStepArgs& a, const WorkerTable& wt, const Workspace& ws, cudaStream_t st, Profiler* prof,
                       int* seg_len) {
  const int total = a.W * a.b;
  int grid = total / DW_MIN_SEG;
  if (grid > g_sm_count) grid = g_sm_count;
  if (grid < 1) grid = 1;
  const int len = (total + grid - 1) / grid;
  grid = (total + len - 1) / len;
  const int slots = 4 * ((a.b - 1) / len + 2);
  TIMED(K_CONV2_DW, (conv2_dw_tc<<<grid, DW_THREADS, DW_SMEM_BYTES, st>>>(a, wt, ws, len, slots)));
  *seg_len = len;
  return slots;
}

int launch_conv1_bwd_tc(const GradStepArgs& a, const WorkerTable& wt, const Workspace& ws, cudaStream_t st, Profiler* prof) {
  const int chunks = (a.b + C1B_SPB - 1) / C1B_SPB;
  TIMED(K_CONV1_BWD, (conv1_bwd_tc<<<dim3(chunks, a.W), 256, 0, st>>>(a, wt, ws, chunks)));
  return chunks;
}

}  // namespace psk
