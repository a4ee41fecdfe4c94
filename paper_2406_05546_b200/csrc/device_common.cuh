// Device helpers shared by the grad-step kernel files.
#pragma once
#include "kernels.h"

namespace psk {

// ---- Philox4x32-10 (Salmon et al., SC'11): ten rounds of two 32x32->64 multiplications; the high
// halves are xored with the neighbouring counter words and the key; the key advances by two Weyl
// constants per round.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
  constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    uint32_t hi0 = __umulhi(M0, c.x), lo0 = M0 * c.x;
    uint32_t hi1 = __umulhi(M1, c.z), lo1 = M1 * c.z;
    c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
    k.x += W0; k.y += W1;
  }
  return c;
}

// Pairs of fp32 values in one 64-bit register, for the packed multiply-add.
typedef unsigned long long u64;
__device__ __forceinline__ u64 pack2(float lo, float hi) {
  u64 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(u64 v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
// Two independent single-rounded fp32 multiply-adds in one instruction.
__device__ __forceinline__ u64 ffma2(u64 a, u64 b, u64 c) {
  u64 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}

// Rounds to TF32 (10-bit mantissa, nearest, ties away from zero); the result is still an fp32 value.
__device__ __forceinline__ float round_tf32(float x) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
  return __uint_as_float(r);
}

// fp32 -> BF16, round to nearest even.
__device__ __forceinline__ uint16_t bf16_bits(float x) {
  uint16_t r;
  asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(r) : "f"(x));
  return r;
}
__device__ __forceinline__ uint32_t bf16_pair(float lo, float hi) {   // lo in the low half
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// prmt.b32 in its default mode: selector nibble n picks byte (n & 7) of {b, a}; with bit 3 of the nibble set, the
// picked byte's top bit is replicated over the whole output byte instead.
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t selector) {
  uint32_t r;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(selector));
  return r;
}
// x << n for a 64-bit x, with n >= 64 giving 0 (PTX clamps the shift amount; C++ leaves it undefined).
__device__ __forceinline__ unsigned long long shl64_clamped(unsigned long long x, uint32_t n) {
  unsigned long long r;
  asm("shl.b64 %0, %1, %2;" : "=l"(r) : "l"(x), "r"(n));
  return r;
}

// Where element (channel oc, pooled position p) of a sample's pooled gradient dp2 and of its pooling decisions
// sits on the tensor-core path: [channel quad][position][4 channels], so that a thread of the backward
// kernels takes four channels of a position with one vector load.  `canonical` = oc * 49 + p.
__host__ __device__ __forceinline__ int dp2_column(int canonical) {
  const int oc = canonical / 49, p = canonical - oc * 49;
  return (oc >> 2) * 196 + p * 4 + (oc & 3);
}

__device__ __forceinline__ const float* group_theta(const WorkerTable& wt, const GroupTable& gt, int s) {
  return gt.theta[wt.group[s]];
}


// Maps a tile index to (group, first row of the tile, end row of the group) for TM-row tiles laid
// out group after group.
template <int TM>
__device__ __forceinline__ bool locate_group_tile(const GroupTable& gt, int b, int tile, int& g, int& m0, int& m_end) {
  for (g = 0; g < gt.n_groups; ++g) {
    int rows = (gt.first[g + 1] - gt.first[g]) * b;
    int tiles = (rows + TM - 1) / TM;
    if (tile < tiles) {
      m0 = gt.first[g] * b + tile * TM;
      m_end = gt.first[g + 1] * b;
      return true;
    }
    tile -= tiles;
  }
  return false;
}

// Same with a run-time range length: range `index` covers rows [r0, r1) of weight group g (ranges never cross
// from one weight group into the next).  False past the last range.
__device__ __forceinline__ bool locate_row_range(const GroupTable& gt, int b, int len, int index, int& g, int& r0, int& r1) {
  for (g = 0; g < gt.n_groups; ++g) {
    const int first = gt.first[g] * b, end = gt.first[g + 1] * b;
    const int n = (end - first + len - 1) / len;
    if (index < n) {
      r0 = first + index * len;
      r1 = min(r0 + len, end);
      return true;
    }
    index -= n;
  }
  return false;
}

// Host: a range length (a multiple of `unit` rows) that gives about `slots` ranges over all rows, and the number
// of ranges it makes when no range crosses a weight-group boundary.
inline int plan_row_ranges(const GroupTable& gt, int b, int slots, int unit, int* len_out) {
  const int total = gt.first[gt.n_groups] * b;
  int len = (total + slots - 1) / slots;
  len = (len + unit - 1) / unit * unit;
  if (len < unit) len = unit;
  int n = 0;
  for (int g = 0; g < gt.n_groups; ++g) n += ((gt.first[g + 1] - gt.first[g]) * b + len - 1) / len;
  *len_out = len;
  return n;
}

inline int group_tiles(const GroupTable& gt, int b, int tm) {
  int t = 0;
  for (int g = 0; g < gt.n_groups; ++g) t += ((gt.first[g + 1] - gt.first[g]) * b + tm - 1) / tm;
  return t;
}

}  // namespace psk
