// Softmax arithmetic of the tensor-core score (Eq. 4, Section 2.2) on accumulator pieces read back from tensor
// memory: the row-wise running (max, sum) of the first sweep and the per-key sums of the second.  Shared by the
// stand-alone score kernels and the fused prune kernel.
#pragma once

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace fastav {
namespace widemath {

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// 2^x for a pair of x <= ~0, computed on the FMA and integer pipes so that it can run next to the
// exponentials the special-function unit is busy with: x = n + f with n the nearest integer (read off
// the mantissa after adding 1.5 * 2^23), a cubic for 2^f on [-1/2, 1/2] (relative error below 7.5e-5),
// and n added into the exponent field.  Inputs below -126 (including -inf) give about 2^-126.
__device__ __forceinline__ float2 exp2_pair_fma(float2 x) {
  const float kMagic = 12582912.f;
  x.x = fmaxf(x.x, -126.f);
  x.y = fmaxf(x.y, -126.f);
  const float2 t = __fadd2_rn(x, make_float2(kMagic, kMagic));
  const float2 n = __fadd2_rn(t, make_float2(-kMagic, -kMagic));
  const float2 f = __ffma2_rn(n, make_float2(-1.f, -1.f), x);
  float2 p = __ffma2_rn(f, make_float2(0.055171460f, 0.055171460f), make_float2(0.24261086f, 0.24261086f));
  p = __ffma2_rn(p, f, make_float2(0.69326097f, 0.69326097f));
  p = __ffma2_rn(p, f, make_float2(0.99992812f, 0.99992812f));
  return make_float2(__int_as_float(__float_as_int(p.x) + (__float_as_int(t.x) << 23)),
                     __int_as_float(__float_as_int(p.y) + (__float_as_int(t.y) << 23)));
}

// The softmax is bound by exponentials, so they are split over two pipes: of the 8 column pairs of every
// 16-column block, the pairs in kFmaPairs go through exp2_pair_fma, the others through the special-function unit.
#ifndef FASTAV_FMA_PAIRS
#define FASTAV_FMA_PAIRS 0x88  // pairs 3 and 7: two of eight (three or four of eight measured no faster)
#endif
constexpr unsigned kFmaPairs = FASTAV_FMA_PAIRS;

__device__ __forceinline__ float2 exp2_pair(float2 x, int pair) {
  if ((kFmaPairs >> (pair & 7)) & 1u) return exp2_pair_fma(x);
  return make_float2(ptx::ex2_approx(x.x), ptx::ex2_approx(x.y));
}

using ptx::tmem_ld_wait_for;

// Sweep 1, one 32-key piece of a row: fold it into the row's running (max, sum).  Under MASKED,
// columns above `bound` (relative to the piece's first column) are hidden from this row.  Branch-free:
// a row that has seen nothing yet carries zmax = -inf and sum 0, and stays that way until a key shows up.
template <bool MASKED>
__device__ __forceinline__ void fold_row_piece(const uint32_t (&v)[32], int bound, float scale, float& zmax, float2& sum2) {
  float z[32];
#pragma unroll
  for (int j = 0; j < 32; ++j) z[j] = (!MASKED || j <= bound) ? __uint_as_float(v[j]) : -INFINITY;
  float m0 = max3(z[0], z[1], z[2]), m1 = max3(z[3], z[4], z[5]);
#pragma unroll
  for (int j = 6; j + 3 < 32; j += 4) {
    m0 = max3(m0, z[j], z[j + 1]);
    m1 = max3(m1, z[j + 2], z[j + 3]);
  }
  const float newmax = fmaxf(zmax, max3(m0, m1, fmaxf(z[30], z[31])));
  const float ref = newmax == -INFINITY ? 0.f : newmax;      // keeps the differences below free of inf - inf
  const float corr = ptx::ex2_approx((zmax - ref) * scale);  // 1 when the maximum did not move, 0 on the first keys
  sum2.x *= corr;
  sum2.y *= corr;
  zmax = newmax;
  const float shift = -ref * scale;
  const float2 sc = make_float2(scale, scale), sh = make_float2(shift, shift);
#pragma unroll
  for (int j = 0; j < 32; j += 2)
    sum2 = __fadd2_rn(sum2, exp2_pair(__ffma2_rn(make_float2(z[j], z[j + 1]), sc, sh), j / 2));
}

__device__ __forceinline__ void fold_row_piece_any(const uint32_t (&v)[32], int bound, float scale, float& zmax, float2& sum2) {
  if (bound >= 31) fold_row_piece<false>(v, bound, scale, zmax, sum2);
  else fold_row_piece<true>(v, bound, scale, zmax, sum2);
  __syncwarp();  // rows of one warp may differ in `bound`; the tcgen05 instructions that follow need the whole warp
}

// Sweep 2, 32 query-row columns of one key: add 2^(z - lse).  `key` is the sequence-local key index;
// under MASKED, a column whose row may not see the key adds nothing.
template <bool MASKED>
__device__ __forceinline__ void add_key_piece(const uint32_t (&v)[32], const float* neg_lse, const int* limit, int key,
                                              float scale, float2& sum2) {
  const float2 sc = make_float2(scale, scale);
#pragma unroll
  for (int j = 0; j < 32; j += 4) {
    const float4 nl = *reinterpret_cast<const float4*>(neg_lse + j);
    float2 p0 = exp2_pair(__ffma2_rn(make_float2(__uint_as_float(v[j]), __uint_as_float(v[j + 1])), sc, make_float2(nl.x, nl.y)), j / 2);
    float2 p1 = exp2_pair(__ffma2_rn(make_float2(__uint_as_float(v[j + 2]), __uint_as_float(v[j + 3])), sc, make_float2(nl.z, nl.w)), j / 2 + 1);
    if (MASKED) {
      const int4 lim = *reinterpret_cast<const int4*>(limit + j);
      p0.x = key <= lim.x ? p0.x : 0.f;
      p0.y = key <= lim.y ? p0.y : 0.f;
      p1.x = key <= lim.z ? p1.x : 0.f;
      p1.y = key <= lim.w ? p1.y : 0.f;
    }
    sum2 = __fadd2_rn(sum2, p0);
    sum2 = __fadd2_rn(sum2, p1);
  }
}

// Sweep 2, the (at most 64) query-row columns of one key that belong to this warpgroup.
template <bool MASKED>
__device__ __forceinline__ float sum_key_columns(uint32_t taddr, int pieces, const float* neg_lse, const int* limit, int key,
                                                 float scale) {
  float2 sum2 = make_float2(0.f, 0.f);
  uint32_t v[32];
  ptx::tmem_ld32(taddr, v);
  tmem_ld_wait_for(v);
  add_key_piece<MASKED>(v, neg_lse, limit, key, scale, sum2);
  if (pieces > 1) {  // the other warps of the scheduler cover this load's latency
    ptx::tmem_ld32(taddr + 32, v);
    tmem_ld_wait_for(v);
    add_key_piece<MASKED>(v, neg_lse + 32, limit + 32, key, scale, sum2);
  }
  return sum2.x + sum2.y;
}

}  // namespace widemath
}  // namespace fastav
