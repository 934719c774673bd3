// Attention rollout (Section 2.1, "Analysis of audio-visual token importance via attention rollout", Eq. 2-3).
//
// Per layer: the head-mean attention map A^l of one sequence (tensor cores: S = Q_h K_h^T tile by tile, softmax
// weights from per-row log-sum-exp statistics that a first kernel computes or the caller hands in), Eq. 2
// (A~ = alpha A + (1 - alpha) I), and Eq. 3 as one n x n x n product R <- A~ R, again on the tensor cores.
//
// Precision.  The product runs in bf16 operands with fp32 accumulation, but both factors are kept as a PAIR of
// bf16 planes (x = hi + lo, hi = bf16(x), lo = bf16(x - hi): about 16 mantissa bits), and each product is the
// three leading terms hi*hi + lo*hi + hi*lo accumulated into the same TMEM tile, so that a chain of a dozen
// layers stays within about 1e-4 relative of the double-precision definition instead of drifting by 2^-9 per
// layer.
//
// Layout.  R is kept TRANSPOSED, RT[j][i] = R[i][j], row-major with the rows padded to n_pad = ceil(n / 128) *
// 128: then RT_new = RT_old * A~^T has both operands K-major (RT_old rows as the M side, A~ rows as the N
// side), which is what TMA tiles with the 128-byte swizzle feed to tcgen05.mma without any transpose.  Under
// the causal mask RT is upper and A~ lower triangular: tiles above the diagonal are written as zeros and the
// K loop of tile (m, n) only covers the blocks m..n.
//
// One CTA per 128 x 128 output tile: warp 0 issues the TMA loads, warp 1 the MMAs, warps 2..17 are the epilogue
// (thread <-> accumulator row, four warps per 32-lane quarter of TMEM, 32 columns each: the epilogue, one
// exponential per element, is what a tile costs, so it gets four warps per scheduler).  All waits are bounded.
#include <cuda.h>
#include <cuda_bf16.h>
#include <limits.h>
#include <math.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace fastav {
namespace {

constexpr int kTile = 128;
constexpr int kThreads = 576;
constexpr int kEpilogueThreads = 512;
constexpr int kColGroups = 4;  // epilogue warps per TMEM quarter; each takes 32 of the 128 columns
constexpr int kTmemCols = 256;  // two 128-column accumulators
constexpr int kMaxStages = 6;
constexpr int kSubTileBytes = kTile * 128;  // 128 rows of one 64-element (128-byte) column block

struct alignas(16) PipeControl {
  uint64_t full[kMaxStages], empty[kMaxStages], tmem_full[2], tmem_empty[2];
  uint32_t tmem_base;
  int abort;
  float2 part[kColGroups - 1][kTile];  // statistics kernel: (max, sum) per row of column groups 1..3
};

__device__ __forceinline__ void split_bf16(float x, __nv_bfloat16& hi, __nv_bfloat16& lo) {
  hi = __float2bfloat16_rn(x);
  lo = __float2bfloat16_rn(x - __bfloat162float(hi));
}

// 32 consecutive values of one row as hi / lo planes: 4 stores of 16 bytes each.
__device__ __forceinline__ void store_split_row(const float (&x)[32], __nv_bfloat16* hi_row, __nv_bfloat16* lo_row) {
#pragma unroll
  for (int c0 = 0; c0 < 32; c0 += 8) {
    alignas(16) __nv_bfloat16 h[8], l[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) split_bf16(x[c0 + c], h[c], l[c]);
    *reinterpret_cast<uint4*>(hi_row + c0) = *reinterpret_cast<const uint4*>(h);
    *reinterpret_cast<uint4*>(lo_row + c0) = *reinterpret_cast<const uint4*>(l);
  }
}

__device__ __forceinline__ void pipe_setup(PipeControl& ctl, int stages, int warp, const void* map_a, const void* map_b) {
  if (threadIdx.x == 0) {
    for (int i = 0; i < stages; ++i) {
      ptx::mbar_init(ptx::smem_u32(&ctl.full[i]), 1);
      ptx::mbar_init(ptx::smem_u32(&ctl.empty[i]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      ptx::mbar_init(ptx::smem_u32(&ctl.tmem_full[i]), 1);
      ptx::mbar_init(ptx::smem_u32(&ctl.tmem_empty[i]), kEpilogueThreads);
    }
    ctl.abort = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(map_a);
    ptx::prefetch_tensormap(map_b);
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(&ctl.tmem_base), kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
}

__device__ __forceinline__ void pipe_teardown(PipeControl& ctl, int warp, int32_t* device_status) {
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(ctl.tmem_base, kTmemCols);
  }
  if (threadIdx.x == 0 && ctl.abort && device_status) atomicOr(device_status, FASTAV_DEV_WAIT_EXPIRED);
}

// After giving up: copies already issued still write into this block's shared memory, so wait (bounded once
// more) for each of them before the block may exit.
__device__ __forceinline__ void drain_loads(PipeControl& ctl, int issued, int stages) {
  int never = 0;
  for (int t = max(0, issued - stages); t < issued; ++t)
    ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.full[t % stages]), (t / stages) & 1, &never);
}

// ---- the attention map ---------------------------------------------------------------------------
template <int DIM, int MODE>
struct AttnSmem {
  static constexpr int kOperandBytes = (DIM / 64) * kSubTileBytes;
  static constexpr int kSlots = MODE == 0 ? 1 : 3;
  static constexpr int kStages = 6 - kSlots;  // six tiles in all: 192 KB at head_dim 128
  static constexpr size_t kBytes = (size_t)6 * kOperandBytes + sizeof(PipeControl) + 1024;
};

// MODE 0: grid (row blocks, heads); the block walks the key blocks its rows may see and leaves, per row, the
//         log2-sum-exp2 of the scaled logits of head blockIdx.y in lse2_out[head][row].
// MODE 1: grid (row blocks, key blocks); the block walks the heads and accumulates the softmax weights of its
//         128 x 128 tile, then applies Eq. 2 and stores the hi / lo planes (and, if asked, A itself in fp32).
template <int DIM, int MODE>
__global__ void __launch_bounds__(kThreads, 1)
rollout_attn_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map, int n, int n_pad,
                    int hq, int group, float scale_log2, int causal, float* __restrict__ lse2_out,
                    const float* __restrict__ lse, long long lse_row, long long lse_head, float lse_mult, float alpha,
                    __nv_bfloat16* __restrict__ a_hi, __nv_bfloat16* __restrict__ a_lo, float* __restrict__ map_out,
                    int32_t* device_status) {
  // Shared memory: a ring of tiles of the operand that changes every iteration (MODE 0: the K tile of the key
  // block; MODE 1: the Q tile of the head) and a few slots for the one that changes rarely (MODE 0: the Q tile,
  // loaded once; MODE 1: the K tile, loaded once per KV head and shared by the G heads of its group -- three
  // slots used in turn, so that a slot is overwritten no sooner than three iterations after its last use,
  // which is the distance the ring's own barriers already guarantee).
  using Cfg = AttnSmem<DIM, MODE>;
  constexpr int kStages = Cfg::kStages, kSlots = Cfg::kSlots;
  constexpr int kSubTiles = DIM / 64;
  constexpr int kOperandBytes = Cfg::kOperandBytes;  // one 128 x DIM tile
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t slots = base + kStages * kOperandBytes;
  PipeControl& ctl = *reinterpret_cast<PipeControl*>(smem_raw + (base - ptx::smem_u32(smem_raw)) + (kStages + kSlots) * kOperandBytes);
  volatile int* abort = &ctl.abort;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int blocks = n_pad / kTile;
  // Under the causal mask the last row block has the most key blocks to walk: the statistics kernel starts those first.
  const int rb = (MODE == 0 && causal) ? blocks - 1 - (int)blockIdx.x : (int)blockIdx.x;

  if (MODE == 1 && causal && (int)blockIdx.y > rb) {
    // a tile no row may see: zeros (uniform for the block, before anything is set up)
    for (int i = threadIdx.x; i < kTile * (kTile / 8); i += kThreads) {
      const int r = i / (kTile / 8), c = (i % (kTile / 8)) * 8;
      const long long at = (long long)(rb * kTile + r) * n_pad + blockIdx.y * kTile + c;
      *reinterpret_cast<uint4*>(a_hi + at) = make_uint4(0, 0, 0, 0);
      *reinterpret_cast<uint4*>(a_lo + at) = make_uint4(0, 0, 0, 0);
    }
    if (map_out)
      for (int i = threadIdx.x; i < kTile * kTile; i += kThreads) {
        const int r = rb * kTile + i / kTile, c = blockIdx.y * kTile + i % kTile;
        if (r < n && c < n) map_out[(long long)r * n + c] = 0.f;
      }
    return;
  }
  const int iters = MODE == 0 ? (causal ? rb + 1 : blocks) : hq;

  pipe_setup(ctl, kStages, warp, &q_map, &k_map);
  const uint32_t tmem = ctl.tmem_base;

  if (warp == 0) {
    if (lane == 0) {
      int it = 0;
      for (; it < iters; ++it) {
        const int stage = it % kStages;
        if (!ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.empty[stage]), ((it / kStages) & 1) ^ 1u, abort)) break;
        const int head = MODE == 0 ? (int)blockIdx.y : it, jb = MODE == 0 ? it : (int)blockIdx.y;
        const uint32_t bar = ptx::smem_u32(&ctl.full[stage]);
        const bool load_q = MODE == 1 || it == 0, load_k = MODE == 0 || it % group == 0;
        const uint32_t ring = base + stage * kOperandBytes;
        const uint32_t q_dst = MODE == 0 ? slots : ring;
        const uint32_t k_dst = MODE == 0 ? ring : slots + ((it / group) % kSlots) * kOperandBytes;
        ptx::mbar_arrive_expect_tx(bar, (load_q ? kOperandBytes : 0) + (load_k ? kOperandBytes : 0));
#pragma unroll
        for (int sub = 0; sub < kSubTiles; ++sub) {
          if (load_q) ptx::tma_load_3d(q_dst + sub * kSubTileBytes, &q_map, sub * 64, head, rb * kTile, bar);
          if (load_k) ptx::tma_load_3d(k_dst + sub * kSubTileBytes, &k_map, sub * 64, head / group, jb * kTile, bar);
        }
      }
      if (*abort) drain_loads(ctl, it, kStages);
    }
  } else if (warp == 1) {
    if (lane == 0) {
      for (int it = 0; it < iters; ++it) {
        const int stage = it % kStages, buf = it & 1;
        if (!ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.full[stage]), (it / kStages) & 1, abort)) break;
        if (!ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.tmem_empty[buf]), ((it >> 1) & 1) ^ 1u, abort)) break;
        ptx::tc_fence_after_sync();
        const uint32_t ring = base + stage * kOperandBytes;
        const uint32_t q_tile = MODE == 0 ? slots : ring;
        const uint32_t k_tile = MODE == 0 ? ring : slots + ((it / group) % kSlots) * kOperandBytes;
#pragma unroll
        for (int ks = 0; ks < DIM / 16; ++ks) {
          const uint32_t sub = ks / 4, off = (ks % 4) * 32;
          ptx::umma_bf16(tmem + buf * kTile, ptx::umma_desc_sw128(q_tile + sub * kSubTileBytes, off),
                         ptx::umma_desc_sw128(k_tile + sub * kSubTileBytes, off), ptx::umma_idesc_bf16(kTile, kTile), ks > 0);
        }
        ptx::umma_commit(ptx::smem_u32(&ctl.empty[stage]));
        ptx::umma_commit(ptx::smem_u32(&ctl.tmem_full[buf]));
      }
    }
  } else {
    const int quarter = warp & 3, cg = (warp - 2) >> 2;  // TMEM lanes 32 quarter .., columns 32 cg ..
    const int row_in = quarter * 32 + lane, row = rb * kTile + row_in;
    const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
    const int last_visible = min(n - 1, causal ? row : INT_MAX);
    float zmax = -INFINITY, sum = 0.f;  // MODE 0, in scaled log2 units
    float acc[32];                      // MODE 1
#pragma unroll
    for (int c = 0; c < 32; ++c) acc[c] = 0.f;
    bool ok = true;
    // MODE 1: the row's statistic of the NEXT head is fetched while this head's tile is worked on
    float lse_next = (MODE == 1 && row < n) ? lse[row * lse_row] : 0.f;
    for (int it = 0; it < iters; ++it) {
      const int buf = it & 1;
      const float lse_here = lse_next;
      if (MODE == 1 && row < n && it + 1 < iters) lse_next = lse[row * lse_row + (it + 1) * lse_head];
      ok = ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.tmem_full[buf]), (it >> 1) & 1, abort);
      if (!ok) break;
      ptx::tc_fence_after_sync();
      const int jb = MODE == 0 ? it : (int)blockIdx.y;
      uint32_t v[32];
      ptx::tmem_ld32(lane_addr + buf * kTile + cg * 32, v);
      ptx::tmem_ld_wait_for(v);
      ptx::tc_fence_before_sync();
      ptx::mbar_arrive(ptx::smem_u32(&ctl.tmem_empty[buf]));  // the accumulator may be overwritten
      const int limit = last_visible - (jb * kTile + cg * 32);  // columns 0..limit of this group are visible
      if (limit < 0) continue;
      const bool whole = limit >= 31;  // the usual case; only tiles on the diagonal or at the end of the sequence are cut
      if constexpr (MODE == 0) {
        float tile_max = -INFINITY;
        if (whole) {
#pragma unroll
          for (int c = 0; c < 32; ++c) tile_max = fmaxf(tile_max, __uint_as_float(v[c]));
        } else {
#pragma unroll
          for (int c = 0; c < 32; ++c)
            if (c <= limit) tile_max = fmaxf(tile_max, __uint_as_float(v[c]));
        }
        const float new_max = fmaxf(zmax, tile_max * scale_log2);
        float add0 = 0.f, add1 = 0.f;
        if (whole) {
#pragma unroll
          for (int c = 0; c < 32; c += 2) {
            add0 += ptx::ex2_approx(fmaf(__uint_as_float(v[c]), scale_log2, -new_max));
            add1 += ptx::ex2_approx(fmaf(__uint_as_float(v[c + 1]), scale_log2, -new_max));
          }
        } else {
#pragma unroll
          for (int c = 0; c < 32; ++c)
            if (c <= limit) add0 += ptx::ex2_approx(fmaf(__uint_as_float(v[c]), scale_log2, -new_max));
        }
        sum = sum * ptx::ex2_approx(zmax - new_max) + (add0 + add1);  // zmax = -inf the first time: the factor is 0
        zmax = new_max;
      } else {
        const float neg_lse2 = -lse_here * lse_mult;
        if (whole) {
#pragma unroll
          for (int c = 0; c < 32; ++c) acc[c] += ptx::ex2_approx(fmaf(__uint_as_float(v[c]), scale_log2, neg_lse2));
        } else {
#pragma unroll
          for (int c = 0; c < 32; ++c)
            if (c <= limit) acc[c] += ptx::ex2_approx(fmaf(__uint_as_float(v[c]), scale_log2, neg_lse2));
        }
      }
    }
    if constexpr (MODE == 0) {
      // the four column groups of a row meet in shared memory; group 0 writes the result
      if (cg > 0) ctl.part[cg - 1][row_in] = make_float2(zmax, sum);
      asm volatile("bar.sync 1, %0;" ::"n"(kEpilogueThreads) : "memory");
      if (cg == 0 && ok && !*abort) {
        float m = zmax;
#pragma unroll
        for (int g = 0; g < kColGroups - 1; ++g) m = fmaxf(m, ctl.part[g][row_in].x);
        float total = zmax > -INFINITY ? sum * ptx::ex2_approx(zmax - m) : 0.f;
#pragma unroll
        for (int g = 0; g < kColGroups - 1; ++g) {
          const float2 other = ctl.part[g][row_in];
          if (other.x > -INFINITY) total += other.y * ptx::ex2_approx(other.x - m);
        }
        lse2_out[(long long)blockIdx.y * n_pad + row] = total > 0.f ? m + log2f(total) : INFINITY;  // a row that sees nothing adds 0
      }
    } else if (ok) {
      const int col0 = blockIdx.y * kTile + cg * 32;
      const float inv_heads = 1.0f / (float)hq;
      float x[32];
#pragma unroll
      for (int c = 0; c < 32; ++c) {
        const float a = row < n ? acc[c] * inv_heads : 0.f;
        if (map_out && row < n && col0 + c < n) map_out[(long long)row * n + col0 + c] = a;
        x[c] = alpha * a + ((row < n && col0 + c == row) ? 1.0f - alpha : 0.f);  // Eq. 2
      }
      const long long at = (long long)row * n_pad + col0;
      store_split_row(x, a_hi + at, a_lo + at);
    }
  }
  pipe_teardown(ctl, warp, device_status);
}

// ---- Eq. 3: RT_new = RT_old * A~^T ------------------------------------------------------------------
// Grid (n_pad / 128, n_pad / 128): one block per 128 x 128 tile of RT_new.  Per 64-wide K block the four
// operand tiles (RT hi, RT lo, A~ hi, A~ lo) are loaded once and used for the three products
// RT hi * A~ hi, RT lo * A~ hi, RT hi * A~ lo, all accumulated into the same TMEM tile.
__global__ void __launch_bounds__(kThreads, 1)
rollout_gemm_kernel(const __grid_constant__ CUtensorMap rt_hi_map, const __grid_constant__ CUtensorMap rt_lo_map,
                    const __grid_constant__ CUtensorMap a_hi_map, const __grid_constant__ CUtensorMap a_lo_map, int n_pad,
                    int causal, __nv_bfloat16* __restrict__ out_hi, __nv_bfloat16* __restrict__ out_lo, int32_t* device_status) {
  constexpr int kStages = 3;
  constexpr int kStageBytes = 4 * kSubTileBytes;  // 128 x 64 each of RT hi, RT lo, A~ hi, A~ lo
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  PipeControl& ctl = *reinterpret_cast<PipeControl*>(smem_raw + (base - ptx::smem_u32(smem_raw)) + kStages * kStageBytes);
  volatile int* abort = &ctl.abort;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Tile of this block.  Under the causal mask tile (m, nn) has a K loop of nn - m + 1 blocks: the blocks are handed
  // out by decreasing nn - m (longest first, so that the short ones fill the tail), the all-zero tiles last.
  int mb = blockIdx.x, nb = blockIdx.y;
  if (causal) {
    const int blocks = gridDim.x;
    int id = blockIdx.y * blocks + blockIdx.x, diag = blocks - 1;  // diag = nn - m, from blocks - 1 down to -(blocks - 1)
    while (id >= blocks - abs(diag)) {
      id -= blocks - abs(diag);
      --diag;
    }
    mb = diag >= 0 ? id : id - diag;
    nb = mb + diag;
  }

  if (causal && mb > nb) {  // RT is upper triangular: nothing but zeros here
    for (int i = threadIdx.x; i < kTile * (kTile / 8); i += kThreads) {
      const int r = i / (kTile / 8), c = (i % (kTile / 8)) * 8;
      const long long at = (long long)(mb * kTile + r) * n_pad + nb * kTile + c;
      *reinterpret_cast<uint4*>(out_hi + at) = make_uint4(0, 0, 0, 0);
      *reinterpret_cast<uint4*>(out_lo + at) = make_uint4(0, 0, 0, 0);
    }
    return;
  }
  // 64-wide K blocks: RT[m][k] is zero for k < m, A~[nn][k] for k > nn
  const int kb_lo = causal ? mb * 2 : 0, kb_hi = causal ? (nb + 1) * 2 : n_pad / 64;
  const int iters = kb_hi - kb_lo;

  pipe_setup(ctl, kStages, warp, &rt_hi_map, &a_hi_map);
  const uint32_t tmem = ctl.tmem_base;

  if (warp == 0) {
    if (lane == 0) {
      int it = 0;
      for (; it < iters; ++it) {
        const int stage = it % kStages;
        if (!ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.empty[stage]), ((it / kStages) & 1) ^ 1u, abort)) break;
        const int kb = kb_lo + it;
        const uint32_t bar = ptx::smem_u32(&ctl.full[stage]);
        const uint32_t dst = base + stage * kStageBytes;
        ptx::mbar_arrive_expect_tx(bar, kStageBytes);
        ptx::tma_load_2d(dst, &rt_hi_map, kb * 64, mb * kTile, bar);
        ptx::tma_load_2d(dst + kSubTileBytes, &rt_lo_map, kb * 64, mb * kTile, bar);
        ptx::tma_load_2d(dst + 2 * kSubTileBytes, &a_hi_map, kb * 64, nb * kTile, bar);
        ptx::tma_load_2d(dst + 3 * kSubTileBytes, &a_lo_map, kb * 64, nb * kTile, bar);
      }
      if (*abort) drain_loads(ctl, it, kStages);
    }
  } else if (warp == 1) {
    if (lane == 0) {
      bool ok = true;
      for (int it = 0; it < iters && ok; ++it) {
        const int stage = it % kStages;
        ok = ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.full[stage]), (it / kStages) & 1, abort);
        if (!ok) break;
        ptx::tc_fence_after_sync();
        const uint32_t rt_hi = base + stage * kStageBytes, rt_lo = rt_hi + kSubTileBytes, a_hi = rt_hi + 2 * kSubTileBytes,
                       a_lo = rt_hi + 3 * kSubTileBytes;
#pragma unroll
        for (int term = 0; term < 3; ++term) {
          const uint32_t rt_tile = term == 1 ? rt_lo : rt_hi, a_tile = term == 2 ? a_lo : a_hi;
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)
            ptx::umma_bf16(tmem, ptx::umma_desc_sw128(rt_tile, ks * 32), ptx::umma_desc_sw128(a_tile, ks * 32),
                           ptx::umma_idesc_bf16(kTile, kTile), (it > 0 || term > 0 || ks > 0) ? 1u : 0u);
        }
        ptx::umma_commit(ptx::smem_u32(&ctl.empty[stage]));
      }
      if (ok) ptx::umma_commit(ptx::smem_u32(&ctl.tmem_full[0]));
    }
  } else {
    const int quarter = warp & 3, cg = (warp - 2) >> 2;
    const int row = mb * kTile + quarter * 32 + lane;
    if (ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.tmem_full[0]), 0, abort)) {
      ptx::tc_fence_after_sync();
      uint32_t v[32];
      ptx::tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + cg * 32, v);
      ptx::tmem_ld_wait_for(v);
      float x[32];
#pragma unroll
      for (int c = 0; c < 32; ++c) x[c] = __uint_as_float(v[c]);
      const long long at = (long long)row * n_pad + nb * kTile + cg * 32;
      store_split_row(x, out_hi + at, out_lo + at);
    }
  }
  pipe_teardown(ctl, warp, device_status);
}

// ---- small kernels ----------------------------------------------------------------------------------
// RT <- I on the first n rows (the padding stays zero): 8 elements per thread.
__global__ void rollout_identity_kernel(int n, int n_pad, __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo) {
  const long long i = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * 8;
  if (i >= (long long)n_pad * n_pad) return;
  const int r = (int)(i / n_pad), c = (int)(i % n_pad);
  alignas(16) __nv_bfloat16 h[8];
#pragma unroll
  for (int u = 0; u < 8; ++u) h[u] = __float2bfloat16_rn((r < n && c + u == r) ? 1.f : 0.f);
  *reinterpret_cast<uint4*>(hi + i) = *reinterpret_cast<const uint4*>(h);
  *reinterpret_cast<uint4*>(lo + i) = make_uint4(0, 0, 0, 0);
}

// importance[j] = (1 / n) sum_i R[i][j] = mean of row j of RT: one warp per row, a fixed summation order.
__global__ void __launch_bounds__(256) rollout_importance_kernel(int n, int n_pad, const __nv_bfloat16* __restrict__ hi,
                                                                  const __nv_bfloat16* __restrict__ lo,
                                                                  float* __restrict__ importance) {
  const int j = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (j >= n) return;
  const __nv_bfloat16 *h = hi + (long long)j * n_pad, *l = lo + (long long)j * n_pad;
  float total = 0.f;
  for (int i = lane; i < n; i += 32) total += __bfloat162float(h[i]) + __bfloat162float(l[i]);
#pragma unroll
  for (int d = 16; d; d >>= 1) total += __shfl_xor_sync(0xFFFFFFFFu, total, d);
  if (lane == 0) importance[j] = total / (float)n;
}

// R[i][j] = RT[j][i] in fp32: 32 x 32 tiles through shared memory.
__global__ void __launch_bounds__(256) rollout_export_kernel(int n, int n_pad, const __nv_bfloat16* __restrict__ hi,
                                                              const __nv_bfloat16* __restrict__ lo, float* __restrict__ out) {
  __shared__ float tile[32][33];
  const int j0 = blockIdx.y * 32, i0 = blockIdx.x * 32, tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  for (int r = ty; r < 32; r += 8) {
    const int j = j0 + r, i = i0 + tx;
    const long long at = (long long)j * n_pad + i;
    tile[r][tx] = (j < n && i < n) ? __bfloat162float(hi[at]) + __bfloat162float(lo[at]) : 0.f;
  }
  __syncthreads();
  for (int r = ty; r < 32; r += 8) {
    const int i = i0 + r, j = j0 + tx;
    if (i < n && j < n) out[(long long)i * n + j] = tile[tx][r];
  }
}

// keep mask and cut position from the importance: one block.
__global__ void __launch_bounds__(1024) rollout_threshold_kernel(int n, const float* __restrict__ importance, float threshold,
                                                                  const uint8_t* __restrict__ protect,
                                                                  uint8_t* __restrict__ keep_mask, int32_t* __restrict__ cut) {
  __shared__ int warp_last[32];
  int last = 0;  // one past the last unprotected token that reaches the threshold
  for (int j = threadIdx.x; j < n; j += blockDim.x) {
    const bool reaches = importance[j] >= threshold, prot = protect && protect[j];
    keep_mask[j] = (reaches || prot) ? 1 : 0;
    if (reaches && !prot) last = j + 1;
  }
  last = __reduce_max_sync(0xFFFFFFFFu, last);
  if ((threadIdx.x & 31) == 0) warp_last[threadIdx.x >> 5] = last;
  __syncthreads();
  if (threadIdx.x < 32) {
    last = __reduce_max_sync(0xFFFFFFFFu, warp_last[threadIdx.x]);
    if (threadIdx.x == 0) *cut = last;
  }
}

// ---- host side ----------------------------------------------------------------------------------------
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                   const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// [n_pad, n_pad] bf16 row-major plane; a box is 128 rows of one 64-element column block.
bool plane_map(const void* ptr, int n_pad, CUtensorMap* map) {
  auto encode = reinterpret_cast<EncodeTiledFn>(tensor_map_encode_entry());
  if (!encode) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)n_pad, (cuuint64_t)n_pad};
  const cuuint64_t strides[1] = {(cuuint64_t)n_pad * 2};
  const cuuint32_t box[2] = {64, kTile};
  const cuuint32_t elem[2] = {1, 1};
  return encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, elem,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// [tokens, heads, d] bf16 with element strides (st, sh, 1) as (d, heads, tokens); a box is 128 tokens of one
// head's 64-element column block.  Tokens past the end read as zeros.
bool qk_map(const void* ptr, int dim, int heads, int tokens, long long st, long long sh, CUtensorMap* map) {
  auto encode = reinterpret_cast<EncodeTiledFn>(tensor_map_encode_entry());
  if (!encode) return false;
  const cuuint64_t dims[3] = {(cuuint64_t)dim, (cuuint64_t)heads, (cuuint64_t)tokens};
  const cuuint64_t strides[2] = {(cuuint64_t)sh * 2, (cuuint64_t)st * 2};
  const cuuint32_t box[3] = {64, 1, kTile};
  const cuuint32_t elem[3] = {1, 1, 1};
  return encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, elem,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int pad_of(int n) { return (n + kTile - 1) / kTile * kTile; }
size_t plane_bytes(int n) { return (size_t)pad_of(n) * pad_of(n) * sizeof(__nv_bfloat16); }

// The state: copy 0 (hi, lo), copy 1 (hi, lo).
__nv_bfloat16* state_plane(void* state, int n, int copy, int lo) {
  return reinterpret_cast<__nv_bfloat16*>(static_cast<unsigned char*>(state) + (size_t)(copy * 2 + lo) * plane_bytes(n));
}

template <int DIM>
cudaError_t run_layer(const fastav_params& p, const CUtensorMap& q_map, const CUtensorMap& k_map, const float* lse_opt,
                      float alpha, float* lse2, __nv_bfloat16* a_hi, __nv_bfloat16* a_lo, float* map_out,
                      int32_t* device_status, cudaStream_t stream) {
  constexpr size_t smem = AttnSmem<DIM, 0>::kBytes;
  static_assert(AttnSmem<DIM, 0>::kBytes == AttnSmem<DIM, 1>::kBytes, "both kernels are launched with the same size");
  const int n = p.total_tokens, n_pad = pad_of(n), blocks = n_pad / kTile;
  const int causal = (p.flags & FASTAV_CAUSAL) ? 1 : 0;
  const float scale = p.softmax_scale > 0.f ? p.softmax_scale : 1.0f / sqrtf((float)p.head_dim);
  const float scale_log2 = scale * kLog2e;
  const int group = p.num_q_heads / p.num_kv_heads;
  cudaError_t e;
  if (!lse_opt) {
    e = cudaFuncSetAttribute(rollout_attn_kernel<DIM, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    rollout_attn_kernel<DIM, 0><<<dim3(blocks, p.num_q_heads), kThreads, smem, stream>>>(
        q_map, k_map, n, n_pad, p.num_q_heads, group, scale_log2, causal, lse2, nullptr, 0, 0, 0.f, 0.f, nullptr, nullptr,
        nullptr, device_status);
    count_launches(1);
  }
  e = cudaFuncSetAttribute(rollout_attn_kernel<DIM, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  // statistics: ours are [head][row] in log2 units; the caller's are [row][head] natural logarithms
  const float* lse = lse_opt ? lse_opt : lse2;
  const long long lse_row = lse_opt ? p.num_q_heads : 1, lse_head = lse_opt ? 1 : n_pad;
  rollout_attn_kernel<DIM, 1><<<dim3(blocks, blocks), kThreads, smem, stream>>>(
      q_map, k_map, n, n_pad, p.num_q_heads, group, scale_log2, causal, nullptr, lse, lse_row, lse_head,
      lse_opt ? kLog2e : 1.0f, alpha, a_hi, a_lo, map_out, device_status);
  count_launches(1);
  return cudaGetLastError();
}

bool aligned256(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }

}  // namespace
}  // namespace fastav

using namespace fastav;

extern "C" int32_t fastav_rollout_state_bytes(int32_t n, size_t* out_bytes) {
  if (!out_bytes || n < 1) return FASTAV_ERR_INVALID_ARG;
  if (n > FASTAV_ROLLOUT_MAX_TOKENS) return FASTAV_ERR_UNSUPPORTED;
  *out_bytes = 4 * plane_bytes(n);
  return FASTAV_OK;
}

extern "C" int32_t fastav_rollout_workspace_bytes(const fastav_params* p, size_t* out_bytes) {
  if (!p || !out_bytes || p->total_tokens < 1 || p->num_q_heads < 1) return FASTAV_ERR_INVALID_ARG;
  if (p->total_tokens > FASTAV_ROLLOUT_MAX_TOKENS) return FASTAV_ERR_UNSUPPORTED;
  *out_bytes = 2 * plane_bytes(p->total_tokens) + align_up((size_t)p->num_q_heads * pad_of(p->total_tokens) * sizeof(float), 256);
  return FASTAV_OK;
}

extern "C" int32_t fastav_rollout_begin(int32_t n, void* state, size_t state_bytes, void* stream) {
  size_t need = 0;
  const int32_t rc = fastav_rollout_state_bytes(n, &need);
  if (rc != FASTAV_OK) return rc;
  if (!state || !aligned256(state) || state_bytes < need) return FASTAV_ERR_WORKSPACE;
  const int n_pad = pad_of(n);
  const long long threads = (long long)n_pad * n_pad / 8;
  rollout_identity_kernel<<<(unsigned)((threads + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      n, n_pad, state_plane(state, n, 0, 0), state_plane(state, n, 0, 1));
  count_launches(1);
  return cudaGetLastError() == cudaSuccess ? FASTAV_OK : FASTAV_ERR_CUDA;
}

extern "C" int32_t fastav_rollout_layer(const fastav_params* p, const void* q, const void* k, const float* lse_opt, float alpha,
                                        int32_t layer_index, void* state, size_t state_bytes, float* map_out_opt, void* workspace,
                                        size_t workspace_bytes, int32_t* device_status, void* stream) {
  if (!p || !q || !k || layer_index < 0 || !(alpha >= 0.f && alpha <= 1.f)) return FASTAV_ERR_INVALID_ARG;
  const int n = p->total_tokens;
  if (p->batch != 1 || n < 1 || p->total_q != n || p->max_seqlen != n || p->max_qlen != n) return FASTAV_ERR_INVALID_ARG;
  if (p->num_q_heads < 1 || p->num_kv_heads < 1 || p->num_q_heads % p->num_kv_heads != 0) return FASTAV_ERR_INVALID_ARG;
  if (p->head_dim != 64 && p->head_dim != 128) return FASTAV_ERR_UNSUPPORTED;
  if (n > FASTAV_ROLLOUT_MAX_TOKENS) return FASTAV_ERR_UNSUPPORTED;
  if (p->q_stride_head < p->head_dim || p->q_stride_tok < p->head_dim || p->k_stride_head < p->head_dim ||
      p->k_stride_tok < p->head_dim)
    return FASTAV_ERR_INVALID_ARG;
  if (p->q_stride_tok % 8 || p->q_stride_head % 8 || p->k_stride_tok % 8 || p->k_stride_head % 8 ||
      (reinterpret_cast<uintptr_t>(q) & 15u) || (reinterpret_cast<uintptr_t>(k) & 15u))
    return FASTAV_ERR_UNSUPPORTED;
  size_t need_state = 0, need_ws = 0;
  fastav_rollout_state_bytes(n, &need_state);
  fastav_rollout_workspace_bytes(p, &need_ws);
  if (!state || !aligned256(state) || state_bytes < need_state) return FASTAV_ERR_WORKSPACE;
  if (!workspace || !aligned256(workspace) || workspace_bytes < need_ws) return FASTAV_ERR_WORKSPACE;

  const int n_pad = pad_of(n);
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  __nv_bfloat16* a_hi = reinterpret_cast<__nv_bfloat16*>(ws);
  __nv_bfloat16* a_lo = reinterpret_cast<__nv_bfloat16*>(ws + plane_bytes(n));
  float* lse2 = reinterpret_cast<float*>(ws + 2 * plane_bytes(n));
  const int src = layer_index & 1, dst = src ^ 1;
  CUtensorMap q_map, k_map, rt_hi_map, rt_lo_map, a_hi_map, a_lo_map;
  if (!qk_map(q, p->head_dim, p->num_q_heads, n, p->q_stride_tok, p->q_stride_head, &q_map) ||
      !qk_map(k, p->head_dim, p->num_kv_heads, n, p->k_stride_tok, p->k_stride_head, &k_map) ||
      !plane_map(state_plane(state, n, src, 0), n_pad, &rt_hi_map) || !plane_map(state_plane(state, n, src, 1), n_pad, &rt_lo_map) ||
      !plane_map(a_hi, n_pad, &a_hi_map) || !plane_map(a_lo, n_pad, &a_lo_map))
    return FASTAV_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e = p->head_dim == 128
                      ? run_layer<128>(*p, q_map, k_map, lse_opt, alpha, lse2, a_hi, a_lo, map_out_opt, device_status, st)
                      : run_layer<64>(*p, q_map, k_map, lse_opt, alpha, lse2, a_hi, a_lo, map_out_opt, device_status, st);
  if (e != cudaSuccess) return FASTAV_ERR_CUDA;
  constexpr size_t gemm_smem = 3 * 4 * kSubTileBytes + sizeof(PipeControl) + 1024;
  e = cudaFuncSetAttribute(rollout_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemm_smem);
  if (e != cudaSuccess) return FASTAV_ERR_CUDA;
  rollout_gemm_kernel<<<dim3(n_pad / kTile, n_pad / kTile), kThreads, gemm_smem, st>>>(
      rt_hi_map, rt_lo_map, a_hi_map, a_lo_map, n_pad, (p->flags & FASTAV_CAUSAL) ? 1 : 0, state_plane(state, n, dst, 0),
      state_plane(state, n, dst, 1), device_status);
  count_launches(1);
  return cudaGetLastError() == cudaSuccess ? FASTAV_OK : FASTAV_ERR_CUDA;
}

extern "C" int32_t fastav_rollout_read(int32_t n, int32_t layers_applied, const void* state, size_t state_bytes,
                                       float* importance_out, float* rollout_out_opt, void* stream) {
  size_t need = 0;
  const int32_t rc = fastav_rollout_state_bytes(n, &need);
  if (rc != FASTAV_OK) return rc;
  if (layers_applied < 0 || !importance_out) return FASTAV_ERR_INVALID_ARG;
  if (!state || !aligned256(state) || state_bytes < need) return FASTAV_ERR_WORKSPACE;
  const int n_pad = pad_of(n), cur = layers_applied & 1;
  const __nv_bfloat16* hi = state_plane(const_cast<void*>(state), n, cur, 0);
  const __nv_bfloat16* lo = state_plane(const_cast<void*>(state), n, cur, 1);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  rollout_importance_kernel<<<(n + 7) / 8, 256, 0, st>>>(n, n_pad, hi, lo, importance_out);
  count_launches(1);
  if (rollout_out_opt) {
    rollout_export_kernel<<<dim3((n + 31) / 32, (n + 31) / 32), 256, 0, st>>>(n, n_pad, hi, lo, rollout_out_opt);
    count_launches(1);
  }
  return cudaGetLastError() == cudaSuccess ? FASTAV_OK : FASTAV_ERR_CUDA;
}

extern "C" int32_t fastav_rollout_threshold(int32_t n, const float* importance, float threshold, const uint8_t* protect_opt,
                                            uint8_t* keep_mask_out, int32_t* cut_out, void* stream) {
  if (n < 1 || !importance || !keep_mask_out || !cut_out) return FASTAV_ERR_INVALID_ARG;
  rollout_threshold_kernel<<<1, 1024, 0, static_cast<cudaStream_t>(stream)>>>(n, importance, threshold, protect_opt,
                                                                              keep_mask_out, cut_out);
  count_launches(1);
  return cudaGetLastError() == cudaSuccess ? FASTAV_OK : FASTAV_ERR_CUDA;
}
