// Importance score, Eq. 4 (Section 2.2), for MANY scored rows per sequence -- the tensor-core path.
//
// With R scored rows and G query heads per KV head, the logits of one KV head are a dense
// [R G, d] x [d, n] contraction: every K byte is reused by R G query rows, so it runs on the 5th-gen
// tensor cores (tcgen05.mma, operands in shared memory, fp32 accumulators in tensor memory) and is
// bound by the exponentials of the softmax, not by HBM.  The [R G, n] logits are never stored; two
// sweeps over K recompute them:
//
//   sweep 1 (S = Q K^T, TMEM lanes = query rows): each thread owns one row and keeps a running
//            (max, sum 2^(z - max)) over the key chunk of its block -> stats, merged into a
//            log2-sum-exp2 per (row, head);
//   sweep 2 (S^T = K Q^T, TMEM lanes = keys): each thread owns one key and adds 2^(z - lse) over the
//            block's query rows in a fixed column order -> partial[KV head, row chunk][token];
//   finalize: scores = (sum of the partials in a fixed order) / (Hq R).
//
// One block = one (sequence, KV head, chunk of 256 query rows, chunk of key tiles).  Warp 0 streams
// 128-key K tiles with TMA (128-byte swizzle) through a 4-stage mbarrier ring, warp 1 issues the MMAs
// into a double-buffered accumulator, warps 2-9 (two warpgroups) read the accumulators back with
// tcgen05.ld and do the softmax arithmetic.  The per-key arithmetic does not depend on the key's
// position, so equal keys get bit-equal scores; all sums have a fixed order, so runs are reproducible.
// Every wait is bounded: a wait that expires makes the block give up, wait for its own copies, free its
// tensor memory and set FASTAV_DEV_WAIT_EXPIRED.
#include <cuda.h>

#include <limits.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace fastav {
namespace {

constexpr int kTileKeys = 128;    // keys per K tile
constexpr int kRowsPerCta = 256;  // query rows (flat over scored row x head of the KV group) per block
constexpr int kStages = 4;        // K tiles in flight
constexpr int kThreads = 320;     // warp 0: TMA, warp 1: MMA, warps 2-9: softmax
constexpr int kEpiThreads = 256;
constexpr int kTmemCols = 512;
constexpr int kMaxChunkTiles = 16;

template <int DIM>
struct Layout {
  static constexpr int kSubTiles = DIM / 64;                      // 128-byte-wide column blocks of a row
  static constexpr int kQSubBytes = kRowsPerCta * 128;            // one column block of the Q tile
  static constexpr int kKSubBytes = kTileKeys * 128;              // one column block of a K tile
  static constexpr int kQBytes = kSubTiles * kQSubBytes;
  static constexpr int kKTileBytes = kSubTiles * kKSubBytes;
  static constexpr int kQOff = 0;
  static constexpr int kKOff = kQOff + kQBytes;
  static constexpr int kCtrlOff = kKOff + kStages * kKTileBytes;  // barriers and small arrays
  static constexpr int kTotal = kCtrlOff + 4096 + 1024;           // + slack to align the base to 1024 bytes
};

struct Control {
  uint64_t full_k[kStages], empty_k[kStages];
  uint64_t q_ready;
  uint64_t tmem_full[4], tmem_empty[4];
  uint32_t tmem_base;
  int abort;
  int min_limit;
  int pad;
  alignas(16) float neg_lse[kRowsPerCta];  // sweep 2: -lse of each query-row column (-inf for padding)
  alignas(16) int limit[kRowsPerCta];      // sweep 2: last key each column's row may see
};
static_assert(sizeof(Control) <= 4096, "control block must fit its slot");

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

// tcgen05.wait::ld, tied to the registers of the load it completes so that no use can move above it.
__device__ __forceinline__ void tmem_ld_wait_for(uint32_t (&v)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]), "+r"(v[8]),
                 "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15]), "+r"(v[16]),
                 "+r"(v[17]), "+r"(v[18]), "+r"(v[19]), "+r"(v[20]), "+r"(v[21]), "+r"(v[22]), "+r"(v[23]), "+r"(v[24]),
                 "+r"(v[25]), "+r"(v[26]), "+r"(v[27]), "+r"(v[28]), "+r"(v[29]), "+r"(v[30]), "+r"(v[31])
               :
               : "memory");
}

__device__ __forceinline__ void epilogue_barrier() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// Sweep 1, one 32-key piece of a row: fold it into the row's running (max, sum).  Columns above
// `bound` (relative to the piece's first column) are hidden from this row.
__device__ __forceinline__ void fold_row_piece(const uint32_t (&v)[32], int bound, float scale, float& zmax, float2& sum2) {
  if (bound < 0) return;
  float z[32];
  if (bound >= 31) {
#pragma unroll
    for (int j = 0; j < 32; ++j) z[j] = __uint_as_float(v[j]);
  } else {
#pragma unroll
    for (int j = 0; j < 32; ++j) z[j] = j <= bound ? __uint_as_float(v[j]) : -INFINITY;
  }
  float m = max3(z[0], z[1], z[2]);
#pragma unroll
  for (int j = 3; j + 1 < 32; j += 2) m = max3(m, z[j], z[j + 1]);
  m = fmaxf(m, z[31]);
  const float newmax = fmaxf(zmax, m);
  if (newmax == -INFINITY) return;  // nothing visible so far
  if (newmax != zmax) {             // rescale what has been summed under the old maximum
    const float corr = ptx::ex2_approx((zmax - newmax) * scale);
    sum2.x *= corr;
    sum2.y *= corr;
    zmax = newmax;
  }
  const float shift = -newmax * scale;
  const float2 sc = make_float2(scale, scale), sh = make_float2(shift, shift);
#pragma unroll
  for (int j = 0; j < 32; j += 2) {
    const float2 x = __ffma2_rn(make_float2(z[j], z[j + 1]), sc, sh);
    sum2 = __fadd2_rn(sum2, make_float2(ptx::ex2_approx(x.x), ptx::ex2_approx(x.y)));
  }
}

// Sweep 2, 32 query-row columns of one key: add 2^(z - lse).  `key` is the sequence-local key index;
// under `masked`, a column whose row may not see the key adds nothing.
__device__ __forceinline__ void add_key_piece(const uint32_t (&v)[32], const float* neg_lse, const int* limit, bool masked,
                                              int key, float scale, float2& sum2) {
  const float2 sc = make_float2(scale, scale);
#pragma unroll
  for (int j = 0; j < 32; j += 4) {
    const float4 nl = *reinterpret_cast<const float4*>(neg_lse + j);
    const float2 x0 = __ffma2_rn(make_float2(__uint_as_float(v[j]), __uint_as_float(v[j + 1])), sc, make_float2(nl.x, nl.y));
    const float2 x1 = __ffma2_rn(make_float2(__uint_as_float(v[j + 2]), __uint_as_float(v[j + 3])), sc, make_float2(nl.z, nl.w));
    float p0 = ptx::ex2_approx(x0.x), p1 = ptx::ex2_approx(x0.y), p2 = ptx::ex2_approx(x1.x), p3 = ptx::ex2_approx(x1.y);
    if (masked) {
      const int4 lim = *reinterpret_cast<const int4*>(limit + j);
      p0 = key <= lim.x ? p0 : 0.f;
      p1 = key <= lim.y ? p1 : 0.f;
      p2 = key <= lim.z ? p2 : 0.f;
      p3 = key <= lim.w ? p3 : 0.f;
    }
    sum2 = __fadd2_rn(sum2, make_float2(p0, p1));
    sum2 = __fadd2_rn(sum2, make_float2(p2, p3));
  }
}

template <int DIM, int SWEEP>
__global__ void __launch_bounds__(kThreads, 1)
score_wide_kernel(const __grid_constant__ CUtensorMap k_map, Shapes s, const uint16_t* __restrict__ q,
                  const int32_t* __restrict__ q_idx, const int32_t* __restrict__ cu_qlens,
                  const int32_t* __restrict__ cu_seqlens, int chunk_tiles, int stat_chunks, int rc_max,
                  float2* __restrict__ stats, const float* __restrict__ lse, float* __restrict__ partial,
                  int32_t* device_status) {
  using L = Layout<DIM>;
  extern __shared__ unsigned char smem_raw[];

  // ---- which piece of work is this block? (uniform per block; empty pieces leave before any set-up)
  const int b = blockIdx.z, g = blockIdx.y / rc_max, rc = blockIdx.y % rc_max, kc = blockIdx.x;
  const int tok0 = cu_seqlens[b], n = cu_seqlens[b + 1] - tok0;
  const int row0 = cu_qlens[b], flat_rows = (cu_qlens[b + 1] - row0) * s.group;
  const int key_begin = kc * chunk_tiles * kTileKeys;
  if (key_begin >= n || rc * kRowsPerCta >= flat_rows) return;
  const int rows_here = min(kRowsPerCta, flat_rows - rc * kRowsPerCta);
  const int tiles = (min(n - key_begin, chunk_tiles * kTileKeys) + kTileKeys - 1) / kTileKeys;
  const int mtiles = (rows_here + 127) / 128;         // sweep 1: 128-row MMA tiles in use
  const int n_cols = (rows_here + 31) / 32 * 32;      // sweep 2: MMA N (query rows as columns)
  const bool causal = (s.flags & FASTAV_CAUSAL) != 0;

  const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_raw + (base - ptx::smem_u32(smem_raw));
  Control& ctl = *reinterpret_cast<Control*>(base_ptr + L::kCtrlOff);
  const uint32_t q_smem = base + L::kQOff, k_smem = base + L::kKOff;
  volatile int* abort = &ctl.abort;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int i = 0; i < kStages; ++i) {
      ptx::mbar_init(ptx::smem_u32(&ctl.full_k[i]), 1);
      ptx::mbar_init(ptx::smem_u32(&ctl.empty_k[i]), 1);
    }
    ptx::mbar_init(ptx::smem_u32(&ctl.q_ready), kEpiThreads);
    for (int i = 0; i < 4; ++i) {
      ptx::mbar_init(ptx::smem_u32(&ctl.tmem_full[i]), 1);
      ptx::mbar_init(ptx::smem_u32(&ctl.tmem_empty[i]), 128);
    }
    ctl.abort = 0;
    ctl.min_limit = INT_MAX;
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(&k_map);
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(&ctl.tmem_base), kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem = ctl.tmem_base;

  if (warp == 0) {
    // ---- TMA producer: one elected lane streams the K tiles of this block's key chunk ----------
    if (lane == 0) {
      int issued = 0;
      for (int t = 0; t < tiles; ++t) {
        const int stage = t % kStages;
        const uint32_t parity = (t / kStages) & 1;
        if (!ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.empty_k[stage]), parity ^ 1u, abort)) break;
        const uint32_t bar = ptx::smem_u32(&ctl.full_k[stage]);
        ptx::mbar_arrive_expect_tx(bar, L::kKTileBytes);
#pragma unroll
        for (int sub = 0; sub < L::kSubTiles; ++sub)
          ptx::tma_load_3d(k_smem + stage * L::kKTileBytes + sub * L::kKSubBytes, &k_map, sub * 64, g,
                           tok0 + key_begin + t * kTileKeys, bar);
        issued = t + 1;
      }
      if (*abort) {
        // Giving up: the copies already issued still write into this block's shared memory, so wait
        // (bounded once more) for each of them before the block may exit.
        int never = 0;
        for (int t = max(0, issued - kStages); t < issued; ++t)
          ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.full_k[t % kStages]), (t / kStages) & 1, &never);
      }
    }
  } else if (warp == 1) {
    // ---- MMA issuer: one elected lane ----------------------------------------------------------
    if (lane == 0 && ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.q_ready), 0, abort)) {
      ptx::tc_fence_after_sync();
      for (int t = 0; t < tiles; ++t) {
        const int stage = t % kStages, buf = t & 1;
        const uint32_t parity = (t / kStages) & 1, buf_parity = (t >> 1) & 1;
        if (!ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.full_k[stage]), parity, abort)) break;
        const uint32_t k_tile = k_smem + stage * L::kKTileBytes;
        if constexpr (SWEEP == 1) {
          // S = Q K^T: A = 128 query rows, B = 128 keys; accumulator (buf, e) at columns buf*256 + e*128.
          bool ok = true;
          for (int e = 0; e < mtiles && ok; ++e) {
            ok = ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.tmem_empty[buf * 2 + e]), buf_parity ^ 1u, abort);
            if (!ok) break;
            ptx::tc_fence_after_sync();
#pragma unroll
            for (int ks = 0; ks < DIM / 16; ++ks) {
              const uint32_t sub = ks / 4, off = (ks % 4) * 32;
              ptx::umma_bf16(tmem + buf * 256 + e * 128, ptx::umma_desc_sw128(q_smem + sub * L::kQSubBytes + e * 128 * 128, off),
                             ptx::umma_desc_sw128(k_tile + sub * L::kKSubBytes, off), ptx::umma_idesc_bf16(128, kTileKeys),
                             ks > 0);
            }
            ptx::umma_commit(ptx::smem_u32(&ctl.tmem_full[buf * 2 + e]));
          }
          if (!ok) break;
          ptx::umma_commit(ptx::smem_u32(&ctl.empty_k[stage]));
        } else {
          // S^T = K Q^T: A = 128 keys, B = n_cols query rows; accumulator buf at columns buf*256.
          if (!ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.tmem_empty[buf]), buf_parity ^ 1u, abort)) break;
          ptx::tc_fence_after_sync();
          const uint32_t idesc = ptx::umma_idesc_bf16(kTileKeys, n_cols);
#pragma unroll
          for (int ks = 0; ks < DIM / 16; ++ks) {
            const uint32_t sub = ks / 4, off = (ks % 4) * 32;
            ptx::umma_bf16(tmem + buf * 256, ptx::umma_desc_sw128(k_tile + sub * L::kKSubBytes, off),
                           ptx::umma_desc_sw128(q_smem + sub * L::kQSubBytes, off), idesc, ks > 0);
          }
          ptx::umma_commit(ptx::smem_u32(&ctl.empty_k[stage]));
          ptx::umma_commit(ptx::smem_u32(&ctl.tmem_full[buf]));
        }
      }
    }
  } else {
    // ---- softmax warps ---------------------------------------------------------------------------
    const int et = threadIdx.x - 64;          // 0..255
    const int wg = (warp - 2) >> 2;           // warpgroup 0 / 1
    const int quarter = warp & 3;             // the 32 TMEM lanes this warp may read
    const int my_lane = quarter * 32 + lane;  // row (sweep 1) or key (sweep 2) inside the tile
    const long long q_row_base = (long long)row0 * s.q_st + (long long)g * s.group * s.q_sh;

    // Query tile -> shared memory, in the 128-byte-swizzled K-major layout the MMA descriptors describe.
    // Flat row f of the KV group is (scored row f / G, head f % G); rows past the end are zero.
    constexpr int kPieces = DIM / 8;  // 16-byte pieces per row
    for (int idx = et; idx < kRowsPerCta * kPieces; idx += kEpiThreads) {
      const int row = idx / kPieces, piece = idx % kPieces;
      uint4 val = make_uint4(0, 0, 0, 0);
      if (row < rows_here) {
        const int f = rc * kRowsPerCta + row;
        val = __ldg(reinterpret_cast<const uint4*>(q + q_row_base + (long long)(f / s.group) * s.q_st +
                                                   (long long)(f % s.group) * s.q_sh + piece * 8));
      }
      const uint32_t dst = q_smem + (piece / 8) * L::kQSubBytes + row * 128 + (((piece % 8) ^ (row & 7)) << 4);
      asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(val.x), "r"(val.y), "r"(val.z), "r"(val.w) : "memory");
    }
    if constexpr (SWEEP == 2) {
      // Per column (query row): -lse and the last key the row may see.
      const int f = rc * kRowsPerCta + et;
      float nl = -INFINITY;
      int lim = -1;
      if (et < rows_here) {
        const int r = f / s.group;
        nl = -lse[(long long)(row0 + r) * s.hq + g * s.group + f % s.group];
        lim = causal ? q_idx[row0 + r] : INT_MAX;
        atomicMin(&ctl.min_limit, lim);
      }
      ctl.neg_lse[et] = nl;
      ctl.limit[et] = lim;
    }
    ptx::fence_proxy_async_smem();  // the MMA reads the tile through the async proxy
    ptx::mbar_arrive(ptx::smem_u32(&ctl.q_ready));
    epilogue_barrier();

    const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
    if constexpr (SWEEP == 1) {
      // Warpgroup e owns the rows of 128-row tile e: thread <-> row.
      const int e = wg;
      const int f = rc * kRowsPerCta + e * 128 + my_lane;
      const bool row_valid = e * 128 + my_lane < rows_here;
      const int r = row_valid ? f / s.group : 0;
      const int last_visible = min(n - 1, (causal && row_valid) ? q_idx[row0 + r] : INT_MAX);
      float zmax = -INFINITY;
      float2 sum2 = make_float2(0.f, 0.f);
      if (e < mtiles) {
        for (int t = 0; t < tiles; ++t) {
          const int buf = t & 1;
          if (!ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.tmem_full[buf * 2 + e]), (t >> 1) & 1, abort)) break;
          ptx::tc_fence_after_sync();
          const int bound = last_visible - (key_begin + t * kTileKeys);  // columns 0..bound of this tile are visible
          const uint32_t taddr = lane_addr + buf * 256 + e * 128;
          uint32_t va[32], vb[32];
          ptx::tmem_ld32(taddr, va);
          tmem_ld_wait_for(va);
          ptx::tmem_ld32(taddr + 32, vb);
          fold_row_piece(va, bound, s.scale_log2, zmax, sum2);
          __syncwarp();  // the rows of a warp may have taken different branches; tcgen05.ld needs them together
          tmem_ld_wait_for(vb);
          ptx::tmem_ld32(taddr + 64, va);
          fold_row_piece(vb, bound - 32, s.scale_log2, zmax, sum2);
          __syncwarp();
          tmem_ld_wait_for(va);
          ptx::tmem_ld32(taddr + 96, vb);
          fold_row_piece(va, bound - 64, s.scale_log2, zmax, sum2);
          __syncwarp();
          tmem_ld_wait_for(vb);
          ptx::tc_fence_before_sync();
          ptx::mbar_arrive(ptx::smem_u32(&ctl.tmem_empty[buf * 2 + e]));  // the accumulator may be overwritten
          fold_row_piece(vb, bound - 96, s.scale_log2, zmax, sum2);
          __syncwarp();
        }
        if (row_valid) {
          const long long rh = (long long)(row0 + r) * s.hq + g * s.group + f % s.group;
          stats[rh * stat_chunks + kc] = make_float2(zmax * s.scale_log2, sum2.x + sum2.y);
        }
      }
    } else {
      // Warpgroup w owns the K tiles of parity w: thread <-> key, all query-row columns.
      float* out = partial + (long long)(g * rc_max + rc) * s.total_tokens + tok0;
      const int pieces = n_cols / 32;
      for (int t = wg; t < tiles; t += 2) {
        const int buf = t & 1;  // == wg
        if (!ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.tmem_full[buf]), (t >> 1) & 1, abort)) break;
        ptx::tc_fence_after_sync();
        const int key = key_begin + t * kTileKeys + my_lane;
        const bool masked = causal && (key_begin + t * kTileKeys + kTileKeys - 1 > ctl.min_limit);
        const uint32_t taddr = lane_addr + buf * 256;
        float2 sum2 = make_float2(0.f, 0.f);
        uint32_t va[32], vb[32];
        ptx::tmem_ld32(taddr, va);
        tmem_ld_wait_for(va);
        for (int c = 0; c < pieces; c += 2) {
          if (c + 1 < pieces) ptx::tmem_ld32(taddr + (c + 1) * 32, vb);
          add_key_piece(va, ctl.neg_lse + c * 32, ctl.limit + c * 32, masked, key, s.scale_log2, sum2);
          if (c + 1 < pieces) {
            tmem_ld_wait_for(vb);
            if (c + 2 < pieces) ptx::tmem_ld32(taddr + (c + 2) * 32, va);
            add_key_piece(vb, ctl.neg_lse + (c + 1) * 32, ctl.limit + (c + 1) * 32, masked, key, s.scale_log2, sum2);
            if (c + 2 < pieces) tmem_ld_wait_for(va);
          }
        }
        ptx::tc_fence_before_sync();
        ptx::mbar_arrive(ptx::smem_u32(&ctl.tmem_empty[buf]));
        if (key < n) out[key] = sum2.x + sum2.y;
      }
    }
  }

  // ---- teardown: everybody meets here, whatever happened above ------------------------------------
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem, kTmemCols);
  }
  if (threadIdx.x == 0 && ctl.abort && device_status) atomicOr(device_status, FASTAV_DEV_WAIT_EXPIRED);
}

// One warp per (scored row, head): fold the per-chunk (max, sum) pairs into log2-sum-exp2.
__global__ void __launch_bounds__(256) score_wide_merge_kernel(Shapes s, const int32_t* __restrict__ cu_qlens,
                                                               const int32_t* __restrict__ cu_seqlens,
                                                               const float2* __restrict__ stats, int stat_chunks,
                                                               int chunk_keys, float* __restrict__ lse) {
  const int w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (w >= s.total_q * s.hq) return;
  const int row = w / s.hq;
  int lo = 0, hi = s.batch;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (cu_qlens[mid] <= row) lo = mid; else hi = mid;
  }
  const int n = cu_seqlens[lo + 1] - cu_seqlens[lo];
  const int chunks = (n + chunk_keys - 1) / chunk_keys;
  const float2* mine = stats + (long long)w * stat_chunks;
  float m = -INFINITY;
  for (int t = lane; t < chunks; t += 32) m = fmaxf(m, mine[t].x);
#pragma unroll
  for (int d = 16; d; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, d));
  float l = 0.f;
  if (m > -INFINITY)
    for (int t = lane; t < chunks; t += 32) {
      const float2 v = mine[t];
      if (v.x > -INFINITY) l += v.y * exp2f(v.x - m);
    }
#pragma unroll
  for (int d = 16; d; d >>= 1) l += __shfl_xor_sync(0xFFFFFFFFu, l, d);
  if (lane == 0) lse[w] = (l > 0.f) ? m + log2f(l) : INFINITY;  // a row that sees no key contributes 0
}

__global__ void __launch_bounds__(256) score_wide_finalize_kernel(Shapes s, const int32_t* __restrict__ cu_seqlens,
                                                                  const int32_t* __restrict__ cu_qlens, int rc_max,
                                                                  const float* __restrict__ partial,
                                                                  float* __restrict__ scores) {
  const int b = blockIdx.y;
  const int tok0 = cu_seqlens[b], n = cu_seqlens[b + 1] - tok0;
  const int rows = cu_qlens[b + 1] - cu_qlens[b];
  const int row_chunks = (rows * s.group + kRowsPerCta - 1) / kRowsPerCta;
  const float inv = rows > 0 ? 1.0f / ((float)s.hq * (float)rows) : 0.f;
  for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < n; j += gridDim.x * blockDim.x) {
    float total = 0.f;
    for (int g = 0; g < s.hkv; ++g)
      for (int rc = 0; rc < row_chunks; ++rc) total += partial[(long long)(g * rc_max + rc) * s.total_tokens + tok0 + j];
    scores[tok0 + j] = total * inv;
  }
}

// ---- host side -----------------------------------------------------------------------------------

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                   const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult res;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &res) != cudaSuccess ||
        res != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// K [N, Hkv, d] bf16 with element strides (k_st, k_sh, 1) as a rank-3 tensor (d, Hkv, N); one box is a
// 64-element (128-byte) column block of 128 consecutive tokens of one KV head.
bool make_k_map(const Shapes& s, const void* k, CUtensorMap* map) {
  EncodeTiledFn encode = encode_tiled_fn();
  if (!encode) return false;
  const cuuint64_t dims[3] = {(cuuint64_t)s.dim, (cuuint64_t)s.hkv, (cuuint64_t)s.total_tokens};
  const cuuint64_t strides[2] = {(cuuint64_t)s.k_sh * 2, (cuuint64_t)s.k_st * 2};
  const cuuint32_t box[3] = {64, 1, (cuuint32_t)kTileKeys};
  const cuuint32_t elem[3] = {1, 1, 1};
  return encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(k), dims, strides, box, elem,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int DIM>
cudaError_t run(const Shapes& s, const Workspace& w, const CUtensorMap& map, const uint16_t* q, const int32_t* q_idx,
                const int32_t* cu_qlens, const int32_t* cu_seqlens, float* scores_out, unsigned char* ws,
                int32_t* device_status, cudaStream_t stream) {
  float2* stats = reinterpret_cast<float2*>(ws + w.stats_off);
  float* lse = reinterpret_cast<float*>(ws + w.lse_off);
  float* partial = reinterpret_cast<float*>(ws + w.partial_off);
  const int rc_max = wide_row_chunks(s.max_qlen, s.group);
  // Key chunk per block: enough blocks for several waves of the 148 SMs, at most 16 tiles each.
  const long long tiles_total = (long long)s.total_tokens / kTileKeys + s.batch;
  long long chunk_tiles = tiles_total * s.hkv * rc_max / (kNumSMs * 6);
  chunk_tiles = chunk_tiles < 1 ? 1 : (chunk_tiles > kMaxChunkTiles ? kMaxChunkTiles : chunk_tiles);
  const int chunk_keys = (int)chunk_tiles * kTileKeys;
  const int stat_chunks = (s.max_seqlen + chunk_keys - 1) / chunk_keys;
  const int smem = Layout<DIM>::kTotal;
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(score_wide_kernel<DIM, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(score_wide_kernel<DIM, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)) != cudaSuccess) return e;
  const dim3 grid(stat_chunks, s.hkv * rc_max, s.batch);
  score_wide_kernel<DIM, 1><<<grid, kThreads, smem, stream>>>(map, s, q, q_idx, cu_qlens, cu_seqlens, (int)chunk_tiles, stat_chunks,
                                                              rc_max, stats, nullptr, nullptr, device_status);
  const int warps = s.total_q * s.hq;
  score_wide_merge_kernel<<<(warps + 7) / 8, 256, 0, stream>>>(s, cu_qlens, cu_seqlens, stats, stat_chunks, chunk_keys, lse);
  score_wide_kernel<DIM, 2><<<grid, kThreads, smem, stream>>>(map, s, q, q_idx, cu_qlens, cu_seqlens, (int)chunk_tiles, stat_chunks,
                                                              rc_max, nullptr, lse, partial, device_status);
  score_wide_finalize_kernel<<<dim3((s.max_seqlen + 255) / 256, s.batch), 256, 0, stream>>>(s, cu_seqlens, cu_qlens, rc_max, partial,
                                                                                          scores_out);
  count_launches(4);
  return cudaGetLastError();
}

}  // namespace

int wide_row_chunks(int max_qlen, int group) {
  const int c = (max_qlen * group + kRowsPerCta - 1) / kRowsPerCta;
  return c < 1 ? 1 : c;
}

bool score_wide_applies(const Shapes& s) {
  return s.max_qlen >= 1 && s.total_q >= 1 && s.max_seqlen >= 1 && (s.dim == 64 || s.dim == 128) && s.k_st % 8 == 0 &&
         s.k_sh % 8 == 0 && s.k_st > 0 && s.k_sh > 0 && (s.k_st >> 36) == 0 && (s.k_sh >> 36) == 0;
}

cudaError_t launch_score_wide(const Shapes& s, const Workspace& w, const void* q, const int32_t* q_idx,
                              const int32_t* cu_qlens, const void* k, const int32_t* cu_seqlens, float* scores_out,
                              unsigned char* ws, int32_t* device_status, cudaStream_t stream, bool* used) {
  CUtensorMap map;
  *used = make_k_map(s, k, &map);
  if (!*used) return cudaSuccess;  // the caller falls back to the CUDA-core path
  const uint16_t* qq = static_cast<const uint16_t*>(q);
  if (s.dim == 128) return run<128>(s, w, map, qq, q_idx, cu_qlens, cu_seqlens, scores_out, ws, device_status, stream);
  return run<64>(s, w, map, qq, q_idx, cu_qlens, cu_seqlens, scores_out, ws, device_status, stream);
}

}  // namespace fastav
