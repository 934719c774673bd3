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
//   sweep 2 (S^T = K Q^T, TMEM lanes = keys): each thread owns one key and adds 2^(z - lse) over 64 of
//            the block's query rows in a fixed column order; four such sums -> partial[KV head, row chunk][token];
//   finalize: scores = (sum of the partials in a fixed order) / (Hq R).
//
// One persistent block per SM works through its share of the units (sequence, KV head, chunk of up to 256
// query rows, chunk of key tiles); the share is computed on the device from cu_seqlens.  Warp 0 streams
// 128-key K tiles and the query tile with TMA (128-byte swizzle) through a 4-stage mbarrier ring, warp 1
// issues the MMAs into double-buffered accumulators, warps 2-17 (four warpgroups) read the accumulators
// back with tcgen05.ld and do the softmax arithmetic, part of the exponentials on the FMA pipe.  A third
// mode of the same kernel only writes the scaled, masked logits (few scored rows: see score_narrow.cu).
// The per-key arithmetic does not depend on the key's position, so equal keys get bit-equal scores; all
// sums have a fixed order, so runs are reproducible.  Every wait is bounded: a wait that expires makes the
// block give up, wait for its own copies, free its tensor memory and set FASTAV_DEV_WAIT_EXPIRED.
#include <cuda.h>

#include <limits.h>

#include "common.cuh"
#include "sm100_ptx.cuh"
#include "score_wide_math.cuh"

namespace fastav {
namespace {

constexpr int kTileKeys = 128;    // keys per K tile
constexpr int kRowsPerCta = 256;  // query rows (flat over scored row x head of the KV group) per block
constexpr int kStages = 4;        // K tiles in flight
constexpr int kGroups = 4;        // softmax warpgroups: four warps per scheduler hide each other's latencies
constexpr int kThreads = 64 + 128 * kGroups;  // warp 0: TMA, warp 1: MMA, warps 2-17: softmax
constexpr int kTmemCols = 512;
#ifndef FASTAV_UNITS_PER_BLOCK
#define FASTAV_UNITS_PER_BLOCK 7
#endif
constexpr int kUnitsPerBlock = FASTAV_UNITS_PER_BLOCK;  // aimed-at number of work units per block
constexpr int kMaxUnits = 48;       // work units one block may be given (the host sizes key chunks accordingly)
constexpr int kCtrlBytes = 18 * 1024;

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
  static constexpr int kTotal = kCtrlOff + kCtrlBytes + 1024;     // + slack to align the base to 1024 bytes
};

using namespace widemath;
using ptx::tmem_ld_wait_for;

// What one block works on at a time: a run of K tiles of one (sequence, KV head, chunk of query rows).
struct Unit {
  int tok0, n;         // the sequence: first token in the packed batch, length
  int row0;            // first scored row of the sequence in q / q_idx
  int g, rc, kc;       // KV head, query-row chunk, key chunk
  int rows_here;       // query rows of the chunk that exist (a multiple of G)
  int new_q;           // the query tile differs from the previous unit's
};

struct Control {
  uint64_t full_k[kStages], empty_k[kStages];
  uint64_t q_ready, q_free;
  uint64_t tmem_full[4], tmem_empty[4];
  uint64_t sums_ready[2];  // sweep 2: warpgroups 1-3 have published their partial sums of accumulator i
  uint32_t tmem_base;
  int abort;
  int n_units;
  int start_b, start_off;
  int warp_sums[kThreads / 32];
  int seq_first_unit[kThreads + 1];            // batch <= kThreads: first unit of every sequence, then the total
  alignas(16) float neg_lse[4 * kGroups][64];  // sweep 2, per softmax warp: -lse of its query-row columns (-inf: padding)
  alignas(16) int limit[4 * kGroups][64];      // sweep 2, per softmax warp: last key each column's row may see
  float sums[2][kGroups - 1][kTileKeys];       // sweep 2: per accumulator, the partial sums of warpgroups 1-3
  Unit units[kMaxUnits];
};
static_assert(sizeof(Control) <= kCtrlBytes, "control block must fit its slot");

// Number of work units of sequence b: KV heads x query-row chunks x key chunks (0 for an empty sequence
// or one without scored rows).
__device__ __forceinline__ int units_of_sequence(const Shapes& s, const int32_t* cu_seqlens, const int32_t* cu_qlens, int b,
                                                 int rows_per_chunk, int chunk_keys) {
  const int n = seq_span(s, cu_seqlens, b).count;
  const int flat_rows = row_span(s, cu_qlens, b).count * s.group;
  if (n <= 0 || flat_rows <= 0) return 0;
  return s.hkv * ((flat_rows + rows_per_chunk - 1) / rows_per_chunk) * ((n + chunk_keys - 1) / chunk_keys);
}

// Block-wide sum of one int per thread (all threads get the result).
__device__ __forceinline__ int block_sum(int v, int* warp_sums) {
#pragma unroll
  for (int d = 16; d; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) warp_sums[threadIdx.x >> 5] = v;
  __syncthreads();
  int total = 0;
#pragma unroll
  for (int w = 0; w < kThreads / 32; ++w) total += warp_sums[w];
  return total;
}

template <int DIM, int SWEEP>
__global__ void __launch_bounds__(kThreads, 1)
score_wide_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap q_map, Shapes s,
                  const int32_t* __restrict__ q_idx, const int32_t* __restrict__ cu_qlens,
                  const int32_t* __restrict__ cu_seqlens, int chunk_tiles, int stat_chunks, int rc_max, int rows_per_chunk,
                  float2* __restrict__ stats, const float* __restrict__ lse, float* __restrict__ partial,
                  float* __restrict__ logits, int rq, int32_t* device_status) {
  using L = Layout<DIM>;
  extern __shared__ unsigned char smem_raw[];
  pdl_trigger();
  const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_raw + (base - ptx::smem_u32(smem_raw));
  Control& ctl = *reinterpret_cast<Control*>(base_ptr + L::kCtrlOff);
  const uint32_t q_smem = base + L::kQOff, k_smem = base + L::kKOff;
  volatile int* abort = &ctl.abort;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int chunk_keys = chunk_tiles * kTileKeys;
  const bool causal = (s.flags & FASTAV_CAUSAL) != 0;
  const int scored_per_chunk = rows_per_chunk / s.group;  // scored rows per query-row chunk (a multiple of 8)

  // ---- this block's share of the work: units [u0, u1) of the list ordered by (sequence, KV head,
  //      row chunk, key chunk), so that consecutive units mostly share their query tile -------------
  const bool table = s.batch <= kThreads;  // one sequence per thread: the unit table can be built in parallel
  int total_units = 0, my_units = 0, my_excl = 0;
  if (table) {
    const int b = threadIdx.x;
    my_units = b < s.batch ? units_of_sequence(s, cu_seqlens, cu_qlens, b, rows_per_chunk, chunk_keys) : 0;
    int incl = my_units;  // inclusive scan inside the warp, then across warps through shared memory
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int t = __shfl_up_sync(0xFFFFFFFFu, incl, d);
      if (lane >= d) incl += t;
    }
    if (lane == 31) ctl.warp_sums[warp] = incl;
    __syncthreads();
    int warp_base = 0;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) {
      if (w < warp) warp_base += ctl.warp_sums[w];
      total_units += ctl.warp_sums[w];
    }
    my_excl = warp_base + incl - my_units;
    ctl.seq_first_unit[b] = my_excl;  // first unit of sequence b in the global order
    if (b == 0) ctl.seq_first_unit[kThreads] = total_units;
  } else {
    for (int b0 = 0; b0 < s.batch; b0 += kThreads) {
      const int b = b0 + threadIdx.x;
      total_units += block_sum(b < s.batch ? units_of_sequence(s, cu_seqlens, cu_qlens, b, rows_per_chunk, chunk_keys) : 0,
                               ctl.warp_sums);
    }
  }
  const int u0 = (int)((long long)total_units * blockIdx.x / gridDim.x);
  const int u1 = (int)((long long)total_units * (blockIdx.x + 1) / gridDim.x);
  if (u1 <= u0) {  // uniform: nothing for this block
    pdl_wait();
    return;
  }
  // The host sized the key chunks so that a block's share fits its table; a longer share means the device's
  // cu_seqlens describe more work than the host's total_tokens / batch did: the excess is left out and reported.
  const int n_mine = min(u1 - u0, kMaxUnits);
  if (threadIdx.x == 0 && u1 - u0 > kMaxUnits && device_status) atomicOr(device_status, FASTAV_DEV_SHAPE_MISMATCH);
  // Unit `target` of the global order -> what to work on.  `b` is its sequence, `off` its index inside it.
  auto describe = [&](int b, int off, Unit& un) {
    const Span seq = seq_span(s, cu_seqlens, b), rows = row_span(s, cu_qlens, b);
    if ((seq.bad || rows.bad) && device_status) atomicOr(device_status, FASTAV_DEV_SHAPE_MISMATCH);
    un.tok0 = seq.first;
    un.n = seq.count;
    un.row0 = rows.first;
    const int flat_rows = rows.count * s.group;
    const int row_chunks = (flat_rows + rows_per_chunk - 1) / rows_per_chunk;
    const int key_chunks = (un.n + chunk_keys - 1) / chunk_keys;
    const int grc = off / key_chunks;
    un.g = grc / row_chunks;
    un.rc = grc % row_chunks;
    un.kc = off % key_chunks;
    un.rows_here = min(rows_per_chunk, flat_rows - un.rc * rows_per_chunk);
    un.new_q = 1;
  };
  if (table) {
    __syncthreads();
    if (threadIdx.x < n_mine) {
      const int target = u0 + threadIdx.x;
      int lo = 0, hi = s.batch;  // smallest hi with first_unit[hi] > target; the sequence is hi - 1 (empty ones are skipped)
      while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        const int first_next = mid + 1 < s.batch ? ctl.seq_first_unit[mid + 1] : total_units;
        if (first_next > target) hi = mid; else lo = mid + 1;
      }
      Unit un;
      describe(lo, target - ctl.seq_first_unit[lo], un);
      ctl.units[threadIdx.x] = un;
    }
    __syncthreads();
    if (threadIdx.x > 0 && threadIdx.x < n_mine) {  // same sequence, KV head and row chunk as the unit before: same query tile
      const Unit &a = ctl.units[threadIdx.x - 1], &c = ctl.units[threadIdx.x];
      if (a.tok0 == c.tok0 && a.g == c.g && a.rc == c.rc) ctl.units[threadIdx.x].new_q = 0;
    }
  } else {
    int before = 0;  // units of the sequences before the current batch slice
    for (int b0 = 0; b0 < s.batch; b0 += kThreads) {
      const int b = b0 + threadIdx.x;
      const int mine = b < s.batch ? units_of_sequence(s, cu_seqlens, cu_qlens, b, rows_per_chunk, chunk_keys) : 0;
      int incl = mine;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int t = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= d) incl += t;
      }
      __syncthreads();
      if (lane == 31) ctl.warp_sums[warp] = incl;
      __syncthreads();
      int warp_base = 0, slice_total = 0;
#pragma unroll
      for (int w = 0; w < kThreads / 32; ++w) {
        if (w < warp) warp_base += ctl.warp_sums[w];
        slice_total += ctl.warp_sums[w];
      }
      const int excl = before + warp_base + incl - mine;
      if (mine > 0 && excl <= u0 && u0 < excl + mine) {  // exactly one thread of one slice
        ctl.start_b = b;
        ctl.start_off = u0 - excl;
      }
      before += slice_total;
    }
    __syncthreads();
    if (threadIdx.x == 0) {  // very large batches: one thread walks this block's units
      int b = ctl.start_b, off = ctl.start_off;
      for (int i = 0; i < n_mine; ++i) {
        while (off >= units_of_sequence(s, cu_seqlens, cu_qlens, b, rows_per_chunk, chunk_keys)) {
          ++b;  // sequence exhausted (or empty): on to the next one
          off = 0;
        }
        Unit un;
        describe(b, off, un);
        if (i > 0 && ctl.units[i - 1].tok0 == un.tok0 && ctl.units[i - 1].g == un.g && ctl.units[i - 1].rc == un.rc) un.new_q = 0;
        ctl.units[i] = un;
        ++off;
      }
    }
  }
  if (threadIdx.x == 0) {
    const int count = n_mine;
    ctl.n_units = count;
    for (int i = 0; i < kStages; ++i) {
      ptx::mbar_init(ptx::smem_u32(&ctl.full_k[i]), 1);
      ptx::mbar_init(ptx::smem_u32(&ctl.empty_k[i]), 1);
    }
    ptx::mbar_init(ptx::smem_u32(&ctl.q_ready), 1);
    ptx::mbar_init(ptx::smem_u32(&ctl.q_free), 1);
    for (int i = 0; i < 4; ++i) {
      ptx::mbar_init(ptx::smem_u32(&ctl.tmem_full[i]), 1);
      // sweep 1: accumulator (e, i) is read by the two warpgroups of row tile e; sweep 2: accumulator i by all four
      ptx::mbar_init(ptx::smem_u32(&ctl.tmem_empty[i]), SWEEP == 1 ? 256 : 128 * kGroups);
    }
    for (int i = 0; i < 2; ++i) ptx::mbar_init(ptx::smem_u32(&ctl.sums_ready[i]), 128 * (kGroups - 1));
    ctl.abort = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(&k_map);
    ptx::prefetch_tensormap(&q_map);
  }
  // The query tile starts as zeros: rows no copy ever fills are then harmless operands.
  for (int i = threadIdx.x; i < L::kQBytes / 16; i += kThreads)
    asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(q_smem + i * 16), "r"(0) : "memory");
  ptx::fence_proxy_async_smem();  // ordered before the TMA writes that follow the barrier
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(&ctl.tmem_base), kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem = ctl.tmem_base;
  const int n_units = ctl.n_units;

  if (warp == 0) {
    // ---- TMA producer: one elected lane streams query tiles and K tiles ---------------------------
    if (lane == 0) {
      // q and k may be what the previous kernel in the stream wrote.  Sweep 2 is never the first kernel of a call,
      // so it may fetch them ahead of its wait -- unless the call's first kernel was itself launched
      // programmatically (FASTAV_CHAIN_CALLS): then the previous call's last kernel may still be running.
      if (SWEEP != 2 || (s.flags & FASTAV_CHAIN_CALLS)) pdl_wait();
      int tile_no = 0, q_gen = 0;  // K tiles / query tiles issued so far
      bool ok = true;
      for (int u = 0; u < n_units && ok; ++u) {
        const Unit un = ctl.units[u];
        if (un.new_q) {
          // The previous query tile must have been read by its last MMA before it is overwritten.
          if (q_gen > 0) ok = ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.q_free), (q_gen - 1) & 1, abort);
          if (!ok) break;
          // Boxes of 8 scored rows x G heads x 64 columns land as 8 G consecutive 128-byte rows, which is the
          // flat (scored row, head) order of the tile; 8 G rows are a whole number of 1024-byte swizzle groups.
          const int boxes = (un.rows_here / s.group + 7) / 8;
          const uint32_t box_bytes = 8u * s.group * 128u;
          const uint32_t bar = ptx::smem_u32(&ctl.q_ready);
          ptx::mbar_arrive_expect_tx(bar, boxes * box_bytes * L::kSubTiles);
          for (int sub = 0; sub < L::kSubTiles; ++sub)
            for (int i = 0; i < boxes; ++i)
              ptx::tma_load_3d(q_smem + sub * L::kQSubBytes + i * box_bytes, &q_map, sub * 64, un.g * s.group,
                               un.row0 + un.rc * scored_per_chunk + 8 * i, bar);
          ++q_gen;
        }
        const int key_begin = un.kc * chunk_keys;
        const int tiles = (min(un.n - key_begin, chunk_keys) + kTileKeys - 1) / kTileKeys;
        for (int t = 0; t < tiles; ++t, ++tile_no) {
          const int stage = tile_no % kStages;
          ok = ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.empty_k[stage]), ((tile_no / kStages) & 1) ^ 1u, abort);
          if (!ok) break;
          const uint32_t bar = ptx::smem_u32(&ctl.full_k[stage]);
          ptx::mbar_arrive_expect_tx(bar, L::kKTileBytes);
#pragma unroll
          for (int sub = 0; sub < L::kSubTiles; ++sub)
            ptx::tma_load_3d(k_smem + stage * L::kKTileBytes + sub * L::kKSubBytes, &k_map, sub * 64, un.g,
                             un.tok0 + key_begin + t * kTileKeys, bar);
        }
      }
      if (*abort) {
        // Giving up: copies already issued still write into this block's shared memory, so wait (bounded
        // once more) for each of them before the block may exit.
        int never = 0;
        for (int t = max(0, tile_no - kStages); t < tile_no; ++t)
          ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.full_k[t % kStages]), (t / kStages) & 1, &never);
        if (q_gen > 0) ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.q_ready), (q_gen - 1) & 1, &never);
      }
    }
  } else if (warp == 1) {
    // ---- MMA issuer: one elected lane -------------------------------------------------------------
    if (lane == 0) {
      int tile_no = 0, q_gen = 0;
      int uses0 = 0, uses1 = 0;  // sweep 1: how often the accumulators of 128-row tile e have been used
      bool ok = true;
      for (int u = 0; u < n_units && ok; ++u) {
        const Unit un = ctl.units[u];
        if (un.new_q) {
          ok = ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.q_ready), q_gen & 1, abort);
          if (!ok) break;
          ptx::tc_fence_after_sync();
          ++q_gen;
        }
        const int key_begin = un.kc * chunk_keys;
        const int tiles = (min(un.n - key_begin, chunk_keys) + kTileKeys - 1) / kTileKeys;
        const int mtiles = (un.rows_here + 127) / 128;     // sweep 1: 128-row MMA tiles in use
        const int n_cols = (un.rows_here + 31) / 32 * 32;  // sweep 2: MMA N (query rows as columns)
        for (int t = 0; t < tiles && ok; ++t, ++tile_no) {
          const int stage = tile_no % kStages;
          ok = ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.full_k[stage]), (tile_no / kStages) & 1, abort);
          if (!ok) break;
          const uint32_t k_tile = k_smem + stage * L::kKTileBytes;
          if constexpr (SWEEP == 1) {
            // S = Q K^T: A = 128 query rows, B = 128 keys; accumulator (e, i) at columns i*256 + e*128.
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              if (e >= mtiles || !ok) break;
              const int uses = e == 0 ? uses0 : uses1;
              const int i = uses & 1;
              ok = ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.tmem_empty[i * 2 + e]), ((uses >> 1) & 1) ^ 1u, abort);
              if (!ok) break;
              ptx::tc_fence_after_sync();
#pragma unroll
              for (int ks = 0; ks < DIM / 16; ++ks) {
                const uint32_t sub = ks / 4, off = (ks % 4) * 32;
                ptx::umma_bf16(tmem + i * 256 + e * 128, ptx::umma_desc_sw128(q_smem + sub * L::kQSubBytes + e * 128 * 128, off),
                               ptx::umma_desc_sw128(k_tile + sub * L::kKSubBytes, off), ptx::umma_idesc_bf16(128, kTileKeys),
                               ks > 0);
              }
              ptx::umma_commit(ptx::smem_u32(&ctl.tmem_full[i * 2 + e]));
              if (e == 0) ++uses0; else ++uses1;
            }
            if (!ok) break;
            ptx::umma_commit(ptx::smem_u32(&ctl.empty_k[stage]));
          } else {
            // S^T = K Q^T: A = 128 keys, B = n_cols query rows; accumulator i at columns i*256.
            const int i = tile_no & 1;
            ok = ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.tmem_empty[i]), ((tile_no >> 1) & 1) ^ 1u, abort);
            if (!ok) break;
            ptx::tc_fence_after_sync();
            const uint32_t idesc = ptx::umma_idesc_bf16(kTileKeys, n_cols);
#pragma unroll
            for (int ks = 0; ks < DIM / 16; ++ks) {
              const uint32_t sub = ks / 4, off = (ks % 4) * 32;
              ptx::umma_bf16(tmem + i * 256, ptx::umma_desc_sw128(k_tile + sub * L::kKSubBytes, off),
                             ptx::umma_desc_sw128(q_smem + sub * L::kQSubBytes, off), idesc, ks > 0);
            }
            ptx::umma_commit(ptx::smem_u32(&ctl.empty_k[stage]));
            ptx::umma_commit(ptx::smem_u32(&ctl.tmem_full[i]));
          }
        }
        // Once the MMAs issued so far are done, the query tile may be replaced.
        if (ok && u + 1 < n_units && ctl.units[u + 1].new_q) ptx::umma_commit(ptx::smem_u32(&ctl.q_free));
      }
    }
  } else {
    // ---- softmax warps: four warpgroups, so that every scheduler has four of them to pick from ---------
    const int wg = (warp - 2) >> 2;           // warpgroup 0..3
    const int quarter = warp & 3;             // the 32 TMEM lanes this warp may read
    const int my_lane = quarter * 32 + lane;  // row (sweep 1) or key (sweep 2) inside the tile
    const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
    pdl_wait();  // before the first read of lse (sweep 2) and the first write of stats / partial
    pdl_acquire(lse);

    if constexpr (SWEEP == 1) {
      // Warpgroup (e, h) owns the rows of 128-row tile e and the keys [64 h, 64 h + 64) of every K tile:
      // thread <-> row, its running (max, sum) over that half of the keys -> one stats entry per half.
      const int e = wg & 1, h = wg >> 1;
      int uses = 0;
      bool ok = true;
      for (int u = 0; u < n_units && ok; ++u) {
        const Unit un = ctl.units[u];
        if (e * 128 >= un.rows_here) continue;  // this 128-row tile is not in use for the unit
        const int key_begin = un.kc * chunk_keys;
        const int tiles = (min(un.n - key_begin, chunk_keys) + kTileKeys - 1) / kTileKeys;
        const int f = un.rc * rows_per_chunk + e * 128 + my_lane;
        const bool row_valid = e * 128 + my_lane < un.rows_here;
        const int r = row_valid ? f / s.group : 0;
        const int last_visible = min(un.n - 1, (causal && row_valid) ? q_idx[un.row0 + r] : INT_MAX);
        float zmax = -INFINITY;
        float2 sum2 = make_float2(0.f, 0.f);
        for (int t = 0; t < tiles; ++t, ++uses) {
          const int i = uses & 1;
          ok = ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.tmem_full[i * 2 + e]), (uses >> 1) & 1, abort);
          if (!ok) break;
          ptx::tc_fence_after_sync();
          const int bound = last_visible - (key_begin + t * kTileKeys + h * 64);  // columns 0..bound of this half are visible
          const uint32_t taddr = lane_addr + i * 256 + e * 128 + h * 64;
          uint32_t va[32], vb[32];
          ptx::tmem_ld32(taddr, va);
          tmem_ld_wait_for(va);
          ptx::tmem_ld32(taddr + 32, vb);
          fold_row_piece_any(va, bound, s.scale_log2, zmax, sum2);
          tmem_ld_wait_for(vb);
          ptx::tc_fence_before_sync();
          ptx::mbar_arrive(ptx::smem_u32(&ctl.tmem_empty[i * 2 + e]));  // the accumulator may be overwritten
          fold_row_piece_any(vb, bound - 32, s.scale_log2, zmax, sum2);
        }
        if (ok && row_valid) {
          const long long rh = (long long)(un.row0 + r) * s.hq + un.g * s.group + f % s.group;
          stats[rh * stat_chunks + un.kc * 2 + h] = make_float2(zmax * s.scale_log2, sum2.x + sum2.y);
        }
      }
    } else if constexpr (SWEEP == 0) {
      // Logits only (few scored rows: the matrix-vector case done as a skinny MMA, bound by streaming K).
      // Thread <-> key, warpgroup w owns the query-row columns [32 w, 32 w + 32) and writes their scaled,
      // masked logits to the [Hq, rq, N] workspace; consecutive lanes write consecutive tokens.
      int tile_no = 0;
      bool ok = true;
      int* slot_of = reinterpret_cast<int*>(ctl.neg_lse[warp - 2]);  // per column: head * rq + scored row
      int* limit = ctl.limit[warp - 2];
      for (int u = 0; u < n_units && ok; ++u) {
        const Unit un = ctl.units[u];
        const int key_begin = un.kc * chunk_keys;
        const int tiles = (min(un.n - key_begin, chunk_keys) + kTileKeys - 1) / kTileKeys;
        const int my_cols = max(0, min(32, un.rows_here - wg * 32));
        if (un.new_q) {
          __syncwarp();
          const int f = un.rc * rows_per_chunk + wg * 32 + lane;
          const int r = f / s.group;
          slot_of[lane] = (un.g * s.group + f % s.group) * rq + r;
          limit[lane] = (causal && lane < my_cols) ? q_idx[un.row0 + r] : INT_MAX;
          __syncwarp();
        }
        float* out = logits + un.tok0;
        for (int t = 0; t < tiles; ++t, ++tile_no) {
          const int i = tile_no & 1;
          ok = ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.tmem_full[i]), (tile_no >> 1) & 1, abort);
          if (!ok) break;
          ptx::tc_fence_after_sync();
          const int key = key_begin + t * kTileKeys + my_lane;
          if (my_cols > 0) {
            uint32_t v[32];
            ptx::tmem_ld32(lane_addr + i * 256 + wg * 32, v);
            tmem_ld_wait_for(v);
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(ptx::smem_u32(&ctl.tmem_empty[i]));
            if (key < un.n) {
#pragma unroll
              for (int c = 0; c < 32; ++c)
                if (c < my_cols)
                  out[(long long)slot_of[c] * s.total_tokens + key] = key <= limit[c] ? __uint_as_float(v[c]) * s.scale_log2 : -INFINITY;
            }
          } else {
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(ptx::smem_u32(&ctl.tmem_empty[i]));
          }
        }
      }
    } else {
      // Every K tile is shared by the four warpgroups: thread <-> key, warpgroup w sums the query-row columns
      // [64 w, 64 w + 64); warpgroups 1-3 publish their sums in shared memory and warpgroup 0 adds them in a
      // fixed order and writes the partial.  Each warp keeps its own copy of the per-column -lse and mask
      // limits (no block-level barrier between softmax warps).
      int tile_no = 0, min_limit = INT_MAX;
      bool ok = true;
      float* neg_lse = ctl.neg_lse[warp - 2];
      int* limit = ctl.limit[warp - 2];
      for (int u = 0; u < n_units && ok; ++u) {
        const Unit un = ctl.units[u];
        const int key_begin = un.kc * chunk_keys;
        const int tiles = (min(un.n - key_begin, chunk_keys) + kTileKeys - 1) / kTileKeys;
        const int my_cols = max(0, min(64, un.rows_here - wg * 64));  // columns of this warpgroup that exist
        const int pieces = (my_cols + 31) / 32;
        if (un.new_q) {
          __syncwarp();
          min_limit = INT_MAX;
          for (int c = lane; c < 64; c += 32) {
            const int f = un.rc * rows_per_chunk + wg * 64 + c;
            float nl = -INFINITY;
            int lim = -1;
            if (c < my_cols) {
              const int r = f / s.group;
              nl = -chain_load(lse + (long long)(un.row0 + r) * s.hq + un.g * s.group + f % s.group);
              lim = causal ? q_idx[un.row0 + r] : INT_MAX;
              min_limit = min(min_limit, lim);
            }
            neg_lse[c] = nl;
            limit[c] = lim;
          }
          min_limit = __reduce_min_sync(0xFFFFFFFFu, min_limit);
          __syncwarp();
        }
        float* out = partial + (long long)(un.g * rc_max + un.rc) * s.total_tokens + un.tok0;
        for (int t = 0; t < tiles; ++t, ++tile_no) {
          const int i = tile_no & 1;
          const uint32_t parity = (tile_no >> 1) & 1;
          ok = ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.tmem_full[i]), parity, abort);
          if (!ok) break;
          ptx::tc_fence_after_sync();
          const int key = key_begin + t * kTileKeys + my_lane;
          const bool masked = causal && (key_begin + t * kTileKeys + kTileKeys - 1 > min_limit);
          const uint32_t taddr = lane_addr + i * 256 + wg * 64;
          float sum = 0.f;
          if (pieces > 0)
            sum = masked ? sum_key_columns<true>(taddr, pieces, neg_lse, limit, key, s.scale_log2)
                         : sum_key_columns<false>(taddr, pieces, neg_lse, limit, key, s.scale_log2);
          if (wg > 0) {
            // sums[i] is free again: warpgroup 0 read it before it released accumulator i two tiles ago
            ctl.sums[i][wg - 1][my_lane] = sum;
            ptx::mbar_arrive(ptx::smem_u32(&ctl.sums_ready[i]));
          } else {
            ok = ptx::mbar_wait_bounded(ptx::smem_u32(&ctl.sums_ready[i]), parity, abort);
            if (!ok) break;
#pragma unroll
            for (int w = 0; w < kGroups - 1; ++w) sum += ctl.sums[i][w][my_lane];
            if (key < un.n) out[key] = sum;
          }
          ptx::tc_fence_before_sync();
          ptx::mbar_arrive(ptx::smem_u32(&ctl.tmem_empty[i]));
        }
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
  pdl_trigger();
  // which sequence this warp's row belongs to: from the caller's arrays, so before the wait
  const int w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  const bool active = w < s.total_q * s.hq;
  int chunks = 0;
  if (active) {
    const int row = w / s.hq;
    int lo = 0, hi = s.batch;
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (cu_qlens[mid] <= row) lo = mid; else hi = mid;
    }
    const int n = seq_span(s, cu_seqlens, lo).count;
    chunks = 2 * ((n + chunk_keys - 1) / chunk_keys);  // one entry per 64-key half of every tile run
  }
  pdl_wait();
  pdl_acquire(stats);
  if (!active) return;
  const float2* mine = stats + (long long)w * stat_chunks;
  // the first 32 entries stay in a register (usually all of them); the rest, if any, is read twice
  const float2 first = lane < chunks ? chain_load(mine + lane) : make_float2(-INFINITY, 0.f);
  float m = first.x;
  for (int t = lane + 32; t < chunks; t += 32) m = fmaxf(m, chain_load(mine + t).x);
#pragma unroll
  for (int d = 16; d; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, d));
  float l = 0.f;
  if (m > -INFINITY) {
    if (first.x > -INFINITY) l = first.y * exp2f(first.x - m);
    for (int t = lane + 32; t < chunks; t += 32) {
      const float2 v = chain_load(mine + t);
      if (v.x > -INFINITY) l += v.y * exp2f(v.x - m);
    }
  }
#pragma unroll
  for (int d = 16; d; d >>= 1) l += __shfl_xor_sync(0xFFFFFFFFu, l, d);
  if (lane == 0) lse[w] = (l > 0.f) ? m + log2f(l) : INFINITY;  // a row that sees no key contributes 0
}

constexpr int kFinalizeThreads = 64;

__global__ void __launch_bounds__(kFinalizeThreads) score_wide_finalize_kernel(Shapes s, const int32_t* __restrict__ cu_seqlens,
                                                                               const int32_t* __restrict__ cu_qlens, int rc_max,
                                                                               int rows_per_chunk, const float* __restrict__ partial,
                                                                               float* __restrict__ scores) {
  pdl_trigger();
  const int b = blockIdx.y;
  const Span seq = seq_span(s, cu_seqlens, b);
  const int tok0 = seq.first, n = seq.count;
  const int rows = row_span(s, cu_qlens, b).count;
  const int row_chunks = (rows * s.group + rows_per_chunk - 1) / rows_per_chunk;
  const float inv = rows > 0 ? 1.0f / ((float)s.hq * (float)rows) : 0.f;
  pdl_wait();
  pdl_acquire(partial);
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= n) return;
  // Partial i = (KV head, row chunk) in that order; eight loads in flight, one running sum in fixed order.
  const int terms = s.hkv * row_chunks;
  const float* col = partial + tok0 + j;
  float total = 0.f;
  int g = 0, rc = 0;  // (KV head, row chunk) of the next term, stepped along instead of divided out
  for (int i0 = 0; i0 < terms; i0 += 8) {
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      v[u] = i0 + u < terms ? chain_load(col + (long long)(g * rc_max + rc) * s.total_tokens) : 0.f;
      if (++rc == row_chunks) {
        rc = 0;
        ++g;
      }
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) total += v[u];
  }
  scores[tok0 + j] = total * inv;
}

// ---- host side -----------------------------------------------------------------------------------

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                   const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() { return reinterpret_cast<EncodeTiledFn>(tensor_map_encode_entry()); }

// A [rows, heads, d] bf16 tensor with element strides (st, sh, 1) as a rank-3 tensor (d, heads, rows); a box
// is a 64-element (128-byte) column block of `box_heads` heads of `box_rows` consecutive rows.
bool make_map(const void* ptr, int dim, int heads, long long rows, long long st, long long sh, int box_heads, int box_rows,
              CUtensorMap* map) {
  EncodeTiledFn encode = encode_tiled_fn();
  if (!encode || rows <= 0) return false;
  const cuuint64_t dims[3] = {(cuuint64_t)dim, (cuuint64_t)heads, (cuuint64_t)rows};
  const cuuint64_t strides[2] = {(cuuint64_t)sh * 2, (cuuint64_t)st * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)box_heads, (cuuint32_t)box_rows};
  const cuuint32_t elem[3] = {1, 1, 1};
  return encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, elem,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Persistent grid and key chunk: one block per SM; chunks sized so that a block gets about a dozen units (fine
// enough to balance, and never more than its table holds).
void plan_units(const Shapes& s, int rc_max, int* grid_out, int* chunk_tiles_out) {
  const long long tiles_upper = (long long)s.total_tokens / kTileKeys + s.batch;  // >= sum over sequences of ceil(n / 128)
  const long long tile_units = tiles_upper * s.hkv * rc_max;
  const int grid = (int)(tile_units < kNumSMs ? tile_units : kNumSMs);
  long long chunk_tiles = (tile_units + (long long)grid * kUnitsPerBlock - 1) / ((long long)grid * kUnitsPerBlock);
  if (chunk_tiles < 1) chunk_tiles = 1;
  // units <= hkv * rc_max * (tokens / chunk + batch); keep the per-block share within the table
  while (((long long)s.hkv * rc_max * (s.total_tokens / (chunk_tiles * kTileKeys) + s.batch) + grid - 1) / grid + 1 > kMaxUnits)
    ++chunk_tiles;
  *grid_out = grid;
  *chunk_tiles_out = (int)chunk_tiles;
}

template <int DIM>
cudaError_t run_logits(const Shapes& s, const CUtensorMap& k_map, const CUtensorMap& q_map, const int32_t* q_idx,
                       const int32_t* cu_qlens, const int32_t* cu_seqlens, float* logits, int rq, int32_t* device_status,
                       cudaStream_t stream) {
  int grid, chunk_tiles;
  plan_units(s, 1, &grid, &chunk_tiles);
  const int smem = Layout<DIM>::kTotal;
  cudaError_t e = cudaFuncSetAttribute(score_wide_kernel<DIM, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  return launch_chained(score_wide_kernel<DIM, 0>, dim3(grid), dim3(kThreads), smem, stream, k_map, q_map, s, q_idx, cu_qlens,
                        cu_seqlens, chunk_tiles, 0, 1, wide_rows_per_chunk(s.group), (float2*)nullptr, (const float*)nullptr,
                        (float*)nullptr, logits, rq, device_status);
}

template <int DIM>
cudaError_t run(const Shapes& s, const Workspace& w, const CUtensorMap& k_map, const CUtensorMap& q_map, const int32_t* q_idx,
                const int32_t* cu_qlens, const int32_t* cu_seqlens, const float* lse_in, float* scores_out, unsigned char* ws,
                int32_t* device_status, cudaStream_t stream) {
  float2* stats = reinterpret_cast<float2*>(ws + w.stats_off);
  float* lse = reinterpret_cast<float*>(ws + w.lse_off);
  float* partial = reinterpret_cast<float*>(ws + w.partial_off);
  const int rows_per_chunk = wide_rows_per_chunk(s.group);
  const int rc_max = wide_row_chunks(s.max_qlen, s.group);
  int grid, chunk_tiles;
  plan_units(s, rc_max, &grid, &chunk_tiles);
  const int chunk_keys = chunk_tiles * kTileKeys;
  const int stat_chunks = 2 * ((s.max_seqlen + chunk_keys - 1) / chunk_keys);  // (max, sum) entries per (row, head)
  const int smem = Layout<DIM>::kTotal;
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(score_wide_kernel<DIM, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(score_wide_kernel<DIM, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)) != cudaSuccess) return e;
  if (lse_in) {
    // The caller already has log-sum-exp per (row, head) (the layer's attention kernel returns it): one sweep.
    if ((e = launch_lse_import(s, lse_in, lse, stream)) != cudaSuccess) return e;
  } else {
    if ((e = launch_chained(score_wide_kernel<DIM, 1>, dim3(grid), dim3(kThreads), smem, stream, k_map, q_map, s, q_idx, cu_qlens,
                            cu_seqlens, chunk_tiles, stat_chunks, rc_max, rows_per_chunk, stats, (const float*)nullptr,
                            (float*)nullptr, (float*)nullptr, 0, device_status)) != cudaSuccess)
      return e;
    const int warps = s.total_q * s.hq;
    if ((e = launch_chained(score_wide_merge_kernel, dim3((warps + 7) / 8), dim3(256), 0, stream, s, cu_qlens, cu_seqlens,
                            (const float2*)stats, stat_chunks, chunk_keys, lse)) != cudaSuccess)
      return e;
    count_launches(2);
  }
  if (!scores_out) return cudaGetLastError();  // only the statistics were asked for (fastav_lse)
  if ((e = launch_chained(score_wide_kernel<DIM, 2>, dim3(grid), dim3(kThreads), smem, stream, k_map, q_map, s, q_idx, cu_qlens,
                          cu_seqlens, chunk_tiles, stat_chunks, rc_max, rows_per_chunk, (float2*)nullptr, (const float*)lse,
                          partial, (float*)nullptr, 0, device_status)) != cudaSuccess)
    return e;
  if ((e = launch_chained(score_wide_finalize_kernel, dim3((s.max_seqlen + kFinalizeThreads - 1) / kFinalizeThreads, s.batch),
                          dim3(kFinalizeThreads), 0, stream, s,
                          cu_seqlens, cu_qlens, rc_max, rows_per_chunk, (const float*)partial, scores_out)) != cudaSuccess)
    return e;
  count_launches(2);
  return cudaGetLastError();
}

}  // namespace

void* tensor_map_encode_entry() {
  static void* entry = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult res;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &res) != cudaSuccess ||
        res != cudaDriverEntryPointSuccess)
      p = nullptr;
    return p;
  }();
  return entry;
}

// Query rows per block: whole TMA boxes of 8 scored rows x G heads, as many as fit in 256 rows.
int wide_rows_per_chunk(int group) { return group >= 1 && group <= 32 ? kRowsPerCta / (8 * group) * (8 * group) : 0; }

int wide_row_chunks(int max_qlen, int group) {
  const int per = wide_rows_per_chunk(group);
  if (per == 0) return 1;
  const int c = (max_qlen * group + per - 1) / per;
  return c < 1 ? 1 : c;
}

bool score_wide_applies(const Shapes& s) {
  const auto ok_stride = [](long long v) { return v > 0 && v % 8 == 0 && (v >> 36) == 0; };
  return s.max_qlen >= 1 && s.total_q >= 1 && s.max_seqlen >= 1 && (s.dim == 64 || s.dim == 128) && s.group <= 32 &&
         ok_stride(s.k_st) && ok_stride(s.k_sh) && ok_stride(s.q_st) && ok_stride(s.q_sh);
}

// Logits [Hq, rq, N] of a batch with at most rq <= 4 scored rows per sequence, by the tensor-core kernel.
cudaError_t launch_logits_wide(const Shapes& s, const void* q, const int32_t* q_idx, const int32_t* cu_qlens, const void* k,
                               const int32_t* cu_seqlens, float* logits, int rq, int32_t* device_status, cudaStream_t stream,
                               bool* used) {
  CUtensorMap k_map, q_map;
  *used = rq * s.group <= 128 && make_map(k, s.dim, s.hkv, s.total_tokens, s.k_st, s.k_sh, 1, kTileKeys, &k_map) &&
          make_map(q, s.dim, s.hq, s.total_q, s.q_st, s.q_sh, s.group, 8, &q_map);
  if (!*used) return cudaSuccess;
  count_launches(1);
  if (s.dim == 128) return run_logits<128>(s, k_map, q_map, q_idx, cu_qlens, cu_seqlens, logits, rq, device_status, stream);
  return run_logits<64>(s, k_map, q_map, q_idx, cu_qlens, cu_seqlens, logits, rq, device_status, stream);
}

cudaError_t launch_score_wide(const Shapes& s, const Workspace& w, const void* q, const int32_t* q_idx,
                              const int32_t* cu_qlens, const void* k, const int32_t* cu_seqlens, const float* lse_in,
                              float* scores_out, unsigned char* ws, int32_t* device_status, cudaStream_t stream, bool* used) {
  CUtensorMap k_map, q_map;
  *used = make_map(k, s.dim, s.hkv, s.total_tokens, s.k_st, s.k_sh, 1, kTileKeys, &k_map) &&
          make_map(q, s.dim, s.hq, s.total_q, s.q_st, s.q_sh, s.group, 8, &q_map);
  if (!*used) return cudaSuccess;  // the caller falls back to the CUDA-core path
  if (s.dim == 128) return run<128>(s, w, k_map, q_map, q_idx, cu_qlens, cu_seqlens, lse_in, scores_out, ws, device_status, stream);
  return run<64>(s, w, k_map, q_map, q_idx, cu_qlens, cu_seqlens, lse_in, scores_out, ws, device_status, stream);
}

}  // namespace fastav
