// The three products of the 512-unit dense layer on the fifth-generation tensor cores:
// tcgen05.mma (kind::tf32) issued by one thread, operands brought into 128-byte-swizzled shared
// memory by TMA (cp.async.bulk.tensor, each CTA loading its own tiles), accumulators in tensor memory, read back with
// tcgen05.ld for the epilogue.
//
// Two are "both operands k-contiguous" products C[m][n] = sum_k A[m][k] * B[n][k]:
//   forward          A = p2 [rows][1568]            B = W1 [512][1568]           (per weight group)
//   input gradient   A = dA1 [rows][512]            B = W1^T [1568][512]         (per weight group)
// The weight gradient of a worker, C[m][n] = sum_k dA1[k][m] * p2[k][n] over the worker's samples k, reads
// both operands as they lie in memory (m and n contiguous, one row per sample): the tensor core takes them
// "MN-major", so no transposed copy is made.
// Every operand is rounded to TF32 by its producer, so the tensor core's own handling of the low mantissa
// bits cannot change a result.
//
// Every wait on an mbarrier is bounded: when a bound is exceeded the kernel raises a status flag,
// stops issuing work, frees its tensor memory and returns.
#include <cuda.h>

#include "device_common.cuh"
#include "kernels.h"
#include "tc5_common.cuh"

namespace psk {

namespace {

constexpr int BM = 128, BK = 32;                    // CTA tile rows; BK floats = one 128-byte swizzle row
constexpr int A_BYTES = BM * BK * 4;
constexpr int MAX_STAGES = 4;
constexpr int EPI_ROW_FLOATS = 36;                       // 32 columns + 4 of padding: conflict-free both ways
constexpr int EPI_WARP_BYTES = 32 * EPI_ROW_FLOATS * 4;  // per epilogue warp: a 32 x 32 block being transposed
__host__ __device__ constexpr int stage_bytes(int bn) { return A_BYTES + bn * BK * 4; }
__host__ __device__ constexpr int gemm_smem_bytes(int bn, int stages, int epi_warps) {
  return stages * stage_bytes(bn) + 1024 /* alignment slack */ + 256 /* barriers */ + epi_warps * EPI_WARP_BYTES;
}

// Shared-memory matrix descriptor, k-contiguous operand, 128-byte swizzle: rows are 128 bytes apart,
// groups of eight rows 1024 bytes apart (stride byte offset), descriptor version 1.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFF) >> 4);
  d |= (uint64_t)1 << 16;                // leading byte offset (unused for swizzled k-contiguous operands)
  d |= (uint64_t)(1024 >> 4) << 32;      // stride byte offset
  d |= (uint64_t)1 << 46;                // version
  d |= (uint64_t)2 << 61;                // layout type: 128-byte swizzle
  return d;
}

// Shared-memory matrix descriptor of a 32-bit operand whose m (or n) index is contiguous.  The only layout the
// tensor core takes for it is the 128-byte swizzle with 32-byte atoms (layout type 1): the tile is a row of
// blocks of 32 columns; inside a block the k-th row (one sample) is 128 bytes, and the four 32-byte pieces of
// a row are permuted by the row index modulo 4.  Blocks are `block_bytes` apart (leading byte offset),
// groups of four rows 512 bytes apart (stride byte offset).  TMA writes the same pattern with
// CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B.
__device__ __forceinline__ uint64_t smem_desc_mn_sw128(uint32_t addr, uint32_t block_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFF) >> 4);
  d |= (uint64_t)(block_bytes >> 4) << 16;
  d |= (uint64_t)(512 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)1 << 61;
  return d;
}

// Instruction descriptor: fp32 accumulate, TF32 x TF32, tile M x N; bits 15 / 16 say that A / B are stored
// with their m / n index contiguous instead of k.
__host__ __device__ constexpr uint32_t instr_desc_tf32(int m, int n, bool mn_major = false) {
  return (1u << 4) | (2u << 7) | (2u << 10) | (mn_major ? (3u << 15) : 0u) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(m >> 4) << 24);
}

// Tensor maps of one launch, passed by value in the kernel's parameter space.
struct GemmMaps {
  CUtensorMap a;
  CUtensorMap b[MAX_GROUPS];
};

enum { EPI_FC1_FWD = 0, EPI_STORE = 1, EPI_STORE_BF16 = 2 };   // the last: the output rounded to BF16 (its readers multiply in BF16)
// Epilogue warps: the plain-store products are bound by getting the accumulator out to global memory, so two warps
// share each quarter of the accumulator rows and take alternate 32-column blocks; the forward product's epilogue
// keeps one warp per quarter (its registers and shared memory leave no room for more).
__host__ __device__ constexpr int epi_warps(int epi) { return epi == EPI_FC1_FWD ? 4 : 8; }
__host__ __device__ constexpr int gemm_threads(int epi) { return 64 + 32 * epi_warps(epi); }

struct GemmArgs {
  int K;            // reduction length (columns beyond it are zero-filled by TMA)
  int N;            // valid output columns
  int ldc;
  int per_worker;   // 1: one 512-row output per sorted worker (tensor-map slab z); 0: grouped rows
  float* c;         // output base when !per_worker
  int n_tiles_n;    // tiles along the columns
  int n_tiles;      // all tiles of the launch
};

// Persistent kernel: one CTA per SM walks over output tiles (columns fastest, so that neighbouring CTAs
// share their A rows in L2).  Warp 0 = TMA producer, warp 1 = tensor-memory owner and MMA issuer, warps 2.. =
// epilogue (each reads the 32 accumulator lanes of its quarter, quarter = warp index mod 4).  The accumulator is double-buffered in tensor memory (2 x BN columns), so the epilogue of one
// tile (tensor memory -> registers -> global) overlaps the loads and MMAs of the next.
// BN = tile columns: 256 for the 512-wide forward product, 224 = 1568/7 for the other two.
struct TileCoord { int grp, m0, m_end, n0, z; };

// A CTA's tiles are t = blockIdx.x, + gridDim.x, ...; their (column tile, row-tile index) pair is carried along by
// additions: the role loops below are serial instruction streams in which a division per tile is dead time.
struct TileWalk { int nt, rest, d_nt, d_rest; };
__device__ __forceinline__ TileWalk tile_walk_begin(const GemmArgs& ga) {
  TileWalk w;
  w.nt = (int)blockIdx.x % ga.n_tiles_n;
  w.rest = (int)blockIdx.x / ga.n_tiles_n;
  w.d_nt = (int)gridDim.x % ga.n_tiles_n;
  w.d_rest = (int)gridDim.x / ga.n_tiles_n;
  return w;
}
__device__ __forceinline__ void tile_walk_next(TileWalk& w, const GemmArgs& ga) {
  w.nt += w.d_nt;
  w.rest += w.d_rest;
  if (w.nt >= ga.n_tiles_n) { w.nt -= ga.n_tiles_n; ++w.rest; }
}
template <int BN>
__device__ __forceinline__ bool decode_tile(const TileWalk& w, const GemmArgs& ga, const GroupTable& gt, int b, TileCoord& c) {
  c.n0 = w.nt * BN;
  c.grp = 0;
  if (ga.per_worker) {
    c.z = w.rest / (HID / BM);
    c.m0 = (w.rest % (HID / BM)) * BM;
    c.m_end = HID;
    return true;
  }
  c.z = 0;
  return locate_group_tile<BM>(gt, b, w.rest, c.grp, c.m0, c.m_end);
}

template <int EPI, int BN, bool MN = false>
__global__ void __launch_bounds__(gemm_threads(EPI), 1) tc5_gemm(const __grid_constant__ GemmMaps maps, GemmArgs ga, GradStepArgs a,
                                                   WorkerTable wt, GroupTable gt, Workspace ws) {
  constexpr int STAGES = MAX_STAGES;
  constexpr int B_BYTES = BN * BK * 4, STAGE_BYTES = A_BYTES + B_BYTES;
  static_assert(STAGE_BYTES % 1024 == 0 && BN % 32 == 0 && 2 * BN <= 512, "tile shape");
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* tiles = smem_raw + (base - smem_u32(smem_raw));
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + STAGES * STAGE_BYTES);
  uint64_t* full = bars;                     // [STAGES] TMA -> MMA
  uint64_t* empty = bars + STAGES;           // [STAGES] MMA -> TMA
  uint64_t* acc_full = bars + 2 * STAGES;    // [2] MMA -> epilogue
  uint64_t* acc_empty = bars + 2 * STAGES + 2;   // [2] epilogue -> MMA
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  float* epi_stage = reinterpret_cast<float*>(tiles + STAGES * STAGE_BYTES + 256);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_k = (ga.K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], epi_warps(EPI)); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_acc = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      int it = 0;                            // k-blocks issued so far, over all tiles
      bool ok = true;
      TileWalk tw = tile_walk_begin(ga);
      for (int t = blockIdx.x; t < ga.n_tiles && ok; t += gridDim.x, tile_walk_next(tw, ga)) {
        TileCoord c;
        if (!decode_tile<BN>(tw, ga, gt, a.b, c)) continue;
        const CUtensorMap* map_a = &maps.a;
        const CUtensorMap* map_b = &maps.b[c.grp];
        for (int kb = 0; kb < n_k; ++kb, ++it) {
          const int s = it % STAGES;
          if (it >= STAGES && !mbar_wait(&empty[s], ((it / STAGES) - 1) & 1)) { *abort_flag = 1; ok = false; break; }
          if (*abort_flag) { ok = false; break; }
          mbar_expect_tx(&full[s], STAGE_BYTES);
          if (MN) {      // boxes of {32 columns, BK samples, BM/32 or BN/32 column blocks} of worker z
            tma_load_4d(tiles + s * STAGE_BYTES, map_a, &full[s], 0, kb * BK, c.m0 / 32, c.z);
            tma_load_4d(tiles + s * STAGE_BYTES + A_BYTES, map_b, &full[s], 0, kb * BK, c.n0 / 32, c.z);
          } else {
            tma_load_3d(tiles + s * STAGE_BYTES, map_a, &full[s], kb * BK, c.m0, c.z);
            tma_load_3d(tiles + s * STAGE_BYTES + A_BYTES, map_b, &full[s], kb * BK, c.n0, c.z);
          }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc_tf32(BM, BN, MN);
      const uint32_t desc_hi = (uint32_t)((MN ? smem_desc_mn_sw128(0, 0) : smem_desc_sw128(0)) >> 32);
      int it = 0, tile_i = 0;
      bool ok = true;
      TileWalk tw = tile_walk_begin(ga);
      for (int t = blockIdx.x; t < ga.n_tiles && ok; t += gridDim.x, tile_walk_next(tw, ga)) {
        TileCoord c;
        if (!decode_tile<BN>(tw, ga, gt, a.b, c)) continue;
        const int ab = tile_i & 1;
        if (tile_i >= 2 && !mbar_wait(&acc_empty[ab], ((tile_i >> 1) - 1) & 1)) { *abort_flag = 1; break; }
        tc_fence_after();
        for (int kb = 0; kb < n_k; ++kb, ++it) {
          const int s = it % STAGES;
          if (!mbar_wait(&full[s], (it / STAGES) & 1) || *abort_flag) { *abort_flag = 1; ok = false; break; }
          tc_fence_after();
          // k-contiguous operands: eight k = 32 bytes along the swizzled row; m/n-contiguous operands: eight k
          // = eight 128-byte rows.  (Descriptor addresses count 16-byte units.)
          const uint32_t a_lo = MN ? (uint32_t)smem_desc_mn_sw128(base + s * STAGE_BYTES, BK * 128)
                                   : (uint32_t)smem_desc_sw128(base + s * STAGE_BYTES);
          const uint32_t b_lo = MN ? (uint32_t)smem_desc_mn_sw128(base + s * STAGE_BYTES + A_BYTES, BK * 128)
                                   : (uint32_t)smem_desc_sw128(base + s * STAGE_BYTES + A_BYTES);
          constexpr uint32_t K_STEP = MN ? 1024 / 16 : 32 / 16;
#pragma unroll
          for (int k = 0; k < BK / 8; ++k)
            umma_tf32_split(tmem_acc + ab * BN, a_lo + k * K_STEP, desc_hi, b_lo + k * K_STEP, desc_hi, idesc, (kb | k) ? 1u : 0u);
          umma_commit(&empty[s]);            // the stage may be refilled once these MMAs have read it
        }
        if (ok) umma_commit(&acc_full[ab]);
        ++tile_i;
      }
    }
  } else {
    const int quarter = warp & 3;
    int tile_i = 0;
    const float scale = 1.0f / (1.0f - a.drop_p);
    const uint2 key = make_uint2((uint32_t)a.seed, (uint32_t)(a.seed >> 32));
    TileWalk tw = tile_walk_begin(ga);
    for (int t = blockIdx.x; t < ga.n_tiles; t += gridDim.x, tile_walk_next(tw, ga)) {
      TileCoord c;
      if (!decode_tile<BN>(tw, ga, gt, a.b, c)) continue;
      const int ab = tile_i & 1;
      if (!mbar_wait(&acc_full[ab], (tile_i >> 1) & 1) || *abort_flag) {
        if (lane == 0) { *abort_flag = 1; atomicOr(ws.status, STATUS_WAIT_TIMEOUT); }
        break;
      }
      tc_fence_after();
      // Each lane reads one accumulator row (32 columns at a time); the 32 x 32 block then goes through a
      // padded shared-memory buffer so that one store instruction writes four full 128-byte row segments
      // instead of 32 scattered 16-byte pieces.
      const int m_lane = c.m0 + quarter * 32 + lane;
      const bool row_ok = m_lane < c.m_end;
      float* stage = epi_stage + (warp - 2) * (EPI_WARP_BYTES / 4);
      float* cbase = ga.per_worker ? wt.grad[c.z] + OFF_F1W : ga.c;
      int s_w = 0, smp = 0;
      if (EPI == EPI_FC1_FWD && row_ok) { s_w = m_lane / a.b; smp = m_lane - s_w * a.b; }
      const float* bias = gt.theta[c.grp] + OFF_F1B;
#pragma unroll 1
      for (int ch = (warp - 2) >> 2; ch < BN / 32; ch += epi_warps(EPI) / 4) {
        const int n = c.n0 + ch * 32;
        if (n >= ga.N) break;                    // warp-uniform
        uint32_t r[32];
        tmem_ld32(tmem_acc + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(ab * BN + ch * 32), r);
        if (EPI == EPI_FC1_FWD && row_ok) {
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const int nq = n + q * 4;
            uint4 rnd = philox4x32_10(make_uint4((uint32_t)((smp * HID + nq) >> 2), (uint32_t)wt.wid[s_w],
                                                 (uint32_t)a.step, (uint32_t)(a.step >> 32)), key);
            const float4 bv = *reinterpret_cast<const float4*>(bias + nq);
            r[q * 4 + 0] = __float_as_uint(rnd.x >= a.drop_thresh ? fmaxf(__uint_as_float(r[q * 4 + 0]) + bv.x, 0.f) * scale : 0.f);
            r[q * 4 + 1] = __float_as_uint(rnd.y >= a.drop_thresh ? fmaxf(__uint_as_float(r[q * 4 + 1]) + bv.y, 0.f) * scale : 0.f);
            r[q * 4 + 2] = __float_as_uint(rnd.z >= a.drop_thresh ? fmaxf(__uint_as_float(r[q * 4 + 2]) + bv.z, 0.f) * scale : 0.f);
            r[q * 4 + 3] = __float_as_uint(rnd.w >= a.drop_thresh ? fmaxf(__uint_as_float(r[q * 4 + 3]) + bv.w, 0.f) * scale : 0.f);
          }
        }
        __syncwarp();                            // the previous block has been read out of the buffer
#pragma unroll
        for (int q = 0; q < 8; ++q)
          *reinterpret_cast<uint4*>(stage + lane * EPI_ROW_FLOATS + q * 4) = make_uint4(r[q * 4], r[q * 4 + 1], r[q * 4 + 2], r[q * 4 + 3]);
        __syncwarp();
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int rr = i * 4 + (lane >> 3), cc = (lane & 7) * 4;
          const int m = c.m0 + quarter * 32 + rr;
          const uint4 v = *reinterpret_cast<const uint4*>(stage + rr * EPI_ROW_FLOATS + cc);
          if (EPI == EPI_STORE_BF16) {     // ga.ldc counts BF16 elements here
            if (m < c.m_end)
              *reinterpret_cast<uint2*>(reinterpret_cast<uint16_t*>(cbase) + (int64_t)m * ga.ldc + n + cc) =
                  make_uint2(bf16_pair(__uint_as_float(v.x), __uint_as_float(v.y)), bf16_pair(__uint_as_float(v.z), __uint_as_float(v.w)));
          } else if (m < c.m_end) {
            *reinterpret_cast<uint4*>(cbase + (int64_t)m * ga.ldc + n + cc) = v;
          }
        }
      }
      // all of this warp's tensor-memory reads of the buffer are complete (tmem_ld32 waits): hand it back
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[ab]);
      ++tile_i;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(512) : "memory");
  }
  if (threadIdx.x == 0 && *abort_flag) {
    atomicOr(ws.status, STATUS_WAIT_TIMEOUT);
    // give copies that were already issued time to land in this CTA's shared memory before it is released
    for (int i = 0; i < 1000; ++i) __nanosleep(1000);
  }
}

// ---- operand preparation ----------------------------------------------------------------------
__device__ __forceinline__ float rna_tf32(float x) { return round_tf32(x); }

// W1 of every weight group: a TF32-rounded copy [512][1568] and its transpose [1568][512] (rows permuted, below).
__global__ void __launch_bounds__(256) prep_w1(GroupTable gt, float* __restrict__ w1r, float* __restrict__ w1tr) {
  __shared__ float tile[32][33];
  const float* src = gt.theta[blockIdx.z] + OFF_F1W;
  float* dr = w1r + (int64_t)blockIdx.z * HID * FLAT;
  float* dt = w1tr + (int64_t)blockIdx.z * HID * FLAT;
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;      // c: 0..1567 (49 tiles), r: 0..511 (16 tiles)
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  for (int i = ty; i < 32; i += 8) {
    float v = rna_tf32(src[(int64_t)(r0 + i) * FLAT + c0 + tx]);
    dr[(int64_t)(r0 + i) * FLAT + c0 + tx] = v;
    tile[i][tx] = v;
  }
  __syncthreads();
  // row of the transpose = column of W1 in the order the convolution's backward kernels read dp2:
  // [channel quad][position][4 channels] instead of channel * 49 + position
  for (int i = ty; i < 32; i += 8) dt[(int64_t)dp2_column(c0 + i) * HID + r0 + tx] = tile[tx][i];
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

// fp32 tensor [d2][d1][d0] (d0 contiguous, row pitch pitch1 floats, slab pitch pitch2 floats), box {32, rows, 1}.
bool make_map(CUtensorMap* m, const float* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t pitch1, uint64_t pitch2,
              uint32_t box_rows) {
  cuuint64_t dims[3] = {d0, d1, d2};
  cuuint64_t strides[2] = {pitch1 * 4, pitch2 * 4};
  cuuint32_t box[3] = {BK, box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = g_encode(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// One worker's [b][F] rows as {32 columns, b samples, F/32 column blocks, W workers}; box {32, BK, blocks, 1}.
// Samples beyond b are out of bounds in their own dimension and arrive as zeros.
bool make_map_mn(CUtensorMap* m, const float* base, uint64_t F, uint64_t b, uint64_t W, uint32_t box_blocks) {
  cuuint64_t dims[4] = {32, b, F / 32, W};
  cuuint64_t strides[3] = {F * 4, 128, b * F * 4};
  cuuint32_t box[4] = {32, BK, box_blocks, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = g_encode(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<float*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace

bool encode_tensor_map_f32(CUtensorMap* m, const float* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                           const uint32_t* box) {
  if (!g_encode || rank < 1 || rank > 5) return false;
  cuuint64_t d[5], sb[4];
  cuuint32_t bx[5], es[5];
  for (int i = 0; i < rank; ++i) { d[i] = dims[i]; bx[i] = box[i]; es[i] = 1; }
  for (int i = 0; i + 1 < rank; ++i) sb[i] = strides_bytes[i];
  return g_encode(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, (cuuint32_t)rank, const_cast<float*>(base), d, sb, bx, es,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

#define TIMED(id, launch) do { if (prof) prof->begin(id, st); launch; if (prof) prof->end(st); } while (0)

int g_sm_count = 0;

int configure_tc5_kernels() {
  if (!g_encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn) return -1;
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  }
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&g_sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || g_sm_count <= 0) return -1;
  cudaError_t e = cudaFuncSetAttribute(tc5_gemm<EPI_FC1_FWD, 256>, cudaFuncAttributeMaxDynamicSharedMemorySize, gemm_smem_bytes(256, MAX_STAGES, epi_warps(EPI_FC1_FWD)));
  if (e == cudaSuccess) e = cudaFuncSetAttribute(tc5_gemm<EPI_STORE_BF16, 224>, cudaFuncAttributeMaxDynamicSharedMemorySize, gemm_smem_bytes(224, MAX_STAGES, epi_warps(EPI_STORE_BF16)));
  if (e == cudaSuccess) e = cudaFuncSetAttribute(tc5_gemm<EPI_STORE, 224, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, gemm_smem_bytes(224, MAX_STAGES, epi_warps(EPI_STORE)));
  return e == cudaSuccess ? 0 : -1;
}

// Rounded / transposed copies of W1 for every weight group of this call.
int launch_prep_w1(const GroupTable& gt, const Workspace& ws, cudaStream_t st, Profiler* prof) {
  TIMED(K_PREP_W1, (prep_w1<<<dim3(FLAT / 32, HID / 32, gt.n_groups), 256, 0, st>>>(gt, ws.w1r, ws.w1tr)));
  return 1;
}

// The forward product; the copies of W1 must be in place.
int launch_fc1_fwd_tc5(const GradStepArgs& a, const WorkerTable& wt, const GroupTable& gt, const Workspace& ws,
                       cudaStream_t st, Profiler* prof) {
  GemmMaps maps;
  const uint64_t rows = (uint64_t)a.W * a.b;
  if (!make_map(&maps.a, ws.p2, FLAT, rows, 1, FLAT, rows * FLAT, BM)) return -1;
  for (int g = 0; g < gt.n_groups; ++g)
    if (!make_map(&maps.b[g], ws.w1r + (int64_t)g * HID * FLAT, FLAT, HID, 1, FLAT, (uint64_t)HID * FLAT, 256)) return -1;
  const int mt = group_tiles(gt, a.b, BM);
  GemmArgs ga{FLAT, HID, HID, 0, ws.d, HID / 256, (HID / 256) * mt};
  const int grid = ga.n_tiles < g_sm_count ? ga.n_tiles : g_sm_count;
  TIMED(K_FC1_FWD, (tc5_gemm<EPI_FC1_FWD, 256><<<grid, gemm_threads(EPI_FC1_FWD), gemm_smem_bytes(256, MAX_STAGES, epi_warps(EPI_FC1_FWD)), st>>>(maps, ga, a, wt, gt, ws)));
  return 1;
}

int launch_fc1_dx_tc5(const GradStepArgs& a, const WorkerTable& wt, const GroupTable& gt, const Workspace& ws,
                      cudaStream_t st, Profiler* prof) {
  GemmMaps maps;
  const uint64_t rows = (uint64_t)a.W * a.b;
  if (!make_map(&maps.a, ws.da1, HID, rows, 1, HID, rows * HID, BM)) return -1;
  for (int g = 0; g < gt.n_groups; ++g)
    if (!make_map(&maps.b[g], ws.w1tr + (int64_t)g * HID * FLAT, HID, FLAT, 1, HID, (uint64_t)HID * FLAT, 224)) return -1;
  const int mt = group_tiles(gt, a.b, BM);
  // dp2 leaves as BF16, in the first half of each row of the fp32-sized buffer (row pitch 2 FLAT half-words): the
  // convolution's two backward kernels multiply it in BF16, so rounding it here once changes no result
  GemmArgs ga{HID, FLAT, 2 * FLAT, 0, ws.dp2, FLAT / 224, (FLAT / 224) * mt};
  const int grid = ga.n_tiles < g_sm_count ? ga.n_tiles : g_sm_count;
  TIMED(K_FC1_DX, (tc5_gemm<EPI_STORE_BF16, 224><<<grid, gemm_threads(EPI_STORE_BF16), gemm_smem_bytes(224, MAX_STAGES, epi_warps(EPI_STORE_BF16)), st>>>(maps, ga, a, wt, gt, ws)));
  return 1;
}

int launch_fc1_dw_tc5(const GradStepArgs& a, const WorkerTable& wt, const GroupTable& gt, const Workspace& ws,
                      cudaStream_t st, Profiler* prof) {
  GemmMaps maps;
  if (!make_map_mn(&maps.a, ws.da1, HID, a.b, a.W, BM / 32)) return -1;
  if (!make_map_mn(&maps.b[0], ws.p2, FLAT, a.b, a.W, 224 / 32)) return -1;
  GemmArgs ga{a.b, FLAT, FLAT, 1, nullptr, FLAT / 224, (FLAT / 224) * (HID / BM) * a.W};
  const int grid = ga.n_tiles < g_sm_count ? ga.n_tiles : g_sm_count;
  TIMED(K_FC1_DW, (tc5_gemm<EPI_STORE, 224, true><<<grid, gemm_threads(EPI_STORE), gemm_smem_bytes(224, MAX_STAGES, epi_warps(EPI_STORE)), st>>>(maps, ga, a, wt, gt, ws)));
  return 1;
}

}  // namespace psk
