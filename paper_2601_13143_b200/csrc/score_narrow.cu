// Importance score, Eq. 4 (Section 2.2), for FEW scored rows per sequence -- the shape the paper
// itself uses in the fine-pruning stage: Q_last is one row per head, so Q K^T is a matrix-vector
// product and the step is bound by reading K once from HBM.
//
//   logits   : K streams through a ring of shared-memory slots filled by bulk asynchronous copies; every
//              16-byte piece of a key row is read once by one lane and multiplied with up to eight query
//              rows held in registers (the rows and heads of one KV group); a butterfly
//              of shuffles that halves the row set at each step leaves one finished logit per lane.
//              Logits [Hq, R, N] (base-2 units, -inf where the causal mask hides the key) go to the
//              workspace: R * Hq * 4 bytes per token next to the Hkv * d * 2 bytes of K read.
//   stats    : one block per (sequence, head, row): max and sum 2^(z - max) -> log2-sum-exp2.
//   finalize : per token, sum over heads and rows of 2^(z - lse) in a fixed order, times 1/(Hq R).
//
// Every key goes through the same arithmetic in the same order, whatever its position, so equal
// keys get bit-equal scores and runs are bit-reproducible.
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace fastav {
namespace {

constexpr int kComputeThreads = 256;             // 8 warps that multiply
constexpr int kThreads = kComputeThreads + 32;   // + 1 warp that issues the copies
constexpr int kStages = 3;                       // K slots in flight per block
constexpr int kSlotKeys = 16;                    // tokens per slot

__device__ __forceinline__ void unpack8(const uint4& v, float2 (&out)[4]) {
  out[0] = make_float2(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xFFFF0000u));
  out[1] = make_float2(__uint_as_float(v.y << 16), __uint_as_float(v.y & 0xFFFF0000u));
  out[2] = make_float2(__uint_as_float(v.z << 16), __uint_as_float(v.z & 0xFFFF0000u));
  out[3] = make_float2(__uint_as_float(v.w << 16), __uint_as_float(v.w & 0xFFFF0000u));
}

__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_smem),
               "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar)
               : "memory");
}

// DIM: head_dim; ROWS: query rows handled per pass (4 or 8).  One block covers `heads_per_block` KV heads
// of a chunk of keys.  A producer warp streams the K rows of those heads, 16 tokens per slot, into a ring
// of shared-memory slots with bulk asynchronous copies; eight warps multiply.  A "lane group" is the DIM/8
// lanes that together read one key row of one KV head; its query rows stay in registers.
template <int DIM, int ROWS>
__global__ void __launch_bounds__(kThreads, ROWS == 8 ? 1 : 2)
score_narrow_logits_kernel(Shapes s, const uint16_t* __restrict__ q, const int32_t* __restrict__ q_idx,
                           const int32_t* __restrict__ cu_qlens, const uint16_t* __restrict__ k,
                           const int32_t* __restrict__ cu_seqlens, float* __restrict__ logits, int rq, int heads_per_block,
                           int chunk_keys, int32_t* device_status) {
  constexpr int kLanes = DIM / 8;                     // lanes per key row
  constexpr int kGroups = kComputeThreads / kLanes;   // key rows per block per step
  constexpr int kHalvings = ROWS == 8 ? 3 : 2;        // butterfly steps that halve the row set
  constexpr int kPlainBits = (kLanes == 16 ? 4 : 3) - kHalvings;
  extern __shared__ __align__(128) unsigned char ring_smem[];
  __shared__ uint64_t full[kStages], empty[kStages];
  __shared__ int abort_flag;

  pdl_trigger();
  const int warp = threadIdx.x >> 5;
  const int row_bytes = heads_per_block * DIM * 2;  // bytes of one token in a slot
  const int slot_bytes = kSlotKeys * row_bytes;
  if (threadIdx.x == 0) {
    for (int i = 0; i < kStages; ++i) {
      ptx::mbar_init(ptx::smem_u32(&full[i]), 1);
      ptx::mbar_init(ptx::smem_u32(&empty[i]), kComputeThreads / 32);
    }
    abort_flag = 0;
    ptx::fence_barrier_init();
  }
  __syncthreads();
  pdl_wait();  // q and k may be what the previous kernel wrote; the logits may still be read by it
  pdl_acquire(q);
  pdl_acquire(k);
  const int b = blockIdx.z;
  const Span seq = seq_span(s, cu_seqlens, b), qrows = row_span(s, cu_qlens, b);
  if ((seq.bad || qrows.bad) && threadIdx.x == 0 && device_status) atomicOr(device_status, FASTAV_DEV_SHAPE_MISMATCH);
  const int tok0 = seq.first, n = seq.count;
  const int key_begin = blockIdx.x * chunk_keys;
  if (key_begin >= n) return;
  const int key_end = min(n, key_begin + chunk_keys);
  const int row0 = qrows.first, rows = min(qrows.count, rq);
  const int flat_rows = rows * s.group;
  if (flat_rows == 0) return;
  const int passes = (flat_rows + ROWS - 1) / ROWS;
  const int slots = (key_end - key_begin + kSlotKeys - 1) / kSlotKeys;  // per pass
  const int head0 = blockIdx.y * heads_per_block;
  const uint32_t ring = ptx::smem_u32(ring_smem);

  if (warp == kComputeThreads / 32) {
    // ---- producer: slot `it` (over all passes) holds tokens [key, key + 16) x heads [head0, head0 + hb) -------
    const int lane = threadIdx.x & 31;
    const bool packed = s.k_sh == DIM;  // the heads of a token are contiguous
    const int pieces_per_token = packed ? 1 : heads_per_block;
    const uint32_t piece_bytes = packed ? row_bytes : DIM * 2;
    bool ok = true;
    for (int it = 0; it < passes * slots && ok; ++it) {
      const int stage = it % kStages;
      ok = ptx::mbar_wait_bounded(ptx::smem_u32(&empty[stage]), ((it / kStages) & 1) ^ 1u, &abort_flag);
      if (!ok) break;
      const int key = key_begin + (it % slots) * kSlotKeys;
      const int tokens = min(kSlotKeys, key_end - key);
      const uint32_t bar = ptx::smem_u32(&full[stage]);
      if (lane == 0) ptx::mbar_arrive_expect_tx(bar, tokens * row_bytes);
      __syncwarp();
      for (int piece = lane; piece < tokens * pieces_per_token; piece += 32) {
        const int t = piece / pieces_per_token, h = piece % pieces_per_token;
        bulk_load(ring + stage * slot_bytes + t * row_bytes + h * DIM * 2,
                  k + (long long)(tok0 + key + t) * s.k_st + (long long)(head0 + h) * s.k_sh, piece_bytes, bar);
      }
    }
    if (!ok && lane == 0 && device_status) atomicOr(device_status, FASTAV_DEV_WAIT_EXPIRED);
    return;
  }

  // ---- consumers ---------------------------------------------------------------------------------------
  const int group = threadIdx.x / kLanes, lane = threadIdx.x % kLanes;
  const int head_local = group % heads_per_block, head = head0 + head_local;  // KV head of this lane group
  const int keys_per_step = kGroups / heads_per_block;
  const int key_lane = group / heads_per_block;
  const bool causal = (s.flags & FASTAV_CAUSAL) != 0;
  const int my_row = (lane >> kPlainBits) & (ROWS - 1);  // the row whose finished logit lands in this lane
  const bool writer = (lane & ((1 << kPlainBits) - 1)) == 0;
  const uint32_t lane_off = head_local * DIM * 2 + lane * 16;

  int it = 0;
  for (int pass = 0; pass < passes; ++pass) {
    const int pass0 = pass * ROWS;
    // Query rows of this pass: flat index f = r * G + (head within the group).
    float2 qv[ROWS][4];
#pragma unroll
    for (int i = 0; i < ROWS; ++i) {
      const int f = pass0 + i;
      uint4 raw = make_uint4(0, 0, 0, 0);
      if (f < flat_rows)
        raw = chain_load(reinterpret_cast<const uint4*>(q + (long long)(row0 + f / s.group) * s.q_st +
                                                   (long long)(head * s.group + f % s.group) * s.q_sh + lane * 8));
      unpack8(raw, qv[i]);
    }
    const int f_mine = pass0 + my_row;
    const bool row_valid = f_mine < flat_rows;
    const int r_mine = row_valid ? f_mine / s.group : 0;
    const int limit = (causal && row_valid) ? q_idx[row0 + r_mine] : 0x7FFFFFFF;
    float* out = logits + ((long long)(head * s.group + (row_valid ? f_mine % s.group : 0)) * rq + r_mine) * s.total_tokens + tok0;

    for (int sl = 0; sl < slots; ++sl, ++it) {
      const int stage = it % kStages;
      if (!ptx::mbar_wait_bounded(ptx::smem_u32(&full[stage]), (it / kStages) & 1, &abort_flag)) {
        // the producer may have issued everything and left already: report here as well
        if ((threadIdx.x & 31) == 0 && device_status) atomicOr(device_status, FASTAV_DEV_WAIT_EXPIRED);
        return;
      }
      const int key_base = key_begin + sl * kSlotKeys;
      const uint32_t slot = ring + stage * slot_bytes + lane_off;
      // The trip count is the same for every lane (the shuffles below need whole warps).
#pragma unroll 2
      for (int t0 = 0; t0 < kSlotKeys; t0 += keys_per_step) {
        const int t = t0 + key_lane, key = key_base + t;
        uint4 raw = make_uint4(0, 0, 0, 0);
        if (t < kSlotKeys)
          asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                       : "=r"(raw.x), "=r"(raw.y), "=r"(raw.z), "=r"(raw.w)
                       : "r"(slot + t * row_bytes));
        float2 kv[4];
        unpack8(raw, kv);
        float vals[ROWS];
#pragma unroll
        for (int i = 0; i < ROWS; ++i) {
          float2 acc = make_float2(0.f, 0.f);
#pragma unroll
          for (int c = 0; c < 4; ++c) acc = __ffma2_rn(kv[c], qv[i][c], acc);
          vals[i] = acc.x + acc.y;
        }
        // Butterfly: at each halving step a lane gives away the half of the rows its partner keeps.
        int count = ROWS;
#pragma unroll
        for (int off = kLanes / 2; off >= 1; off >>= 1) {
          if (count > 1) {
            const int half = count / 2;
            const bool upper = (lane & off) != 0;
#pragma unroll
            for (int i = 0; i < ROWS / 2; ++i) {
              if (i < half) {
                const float send = upper ? vals[i] : vals[i + half];
                const float keep = upper ? vals[i + half] : vals[i];
                vals[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, off);
              }
            }
            count = half;
          } else {
            vals[0] += __shfl_xor_sync(0xFFFFFFFFu, vals[0], off);
          }
        }
        // Tokens past the end of the chunk hold stale bytes of an earlier slot: computed, never written.
        if (writer && row_valid && t < kSlotKeys && key < key_end) out[key] = key <= limit ? vals[0] * s.scale_log2 : -INFINITY;
      }
      __syncwarp();
      if ((threadIdx.x & 31) == 0) ptx::mbar_arrive(ptx::smem_u32(&empty[stage]));  // this warp is done with the slot
    }
  }
}

// One block per (head, row, sequence): log2-sum-exp2 of a row of logits.
__global__ void __launch_bounds__(256) score_narrow_stats_kernel(Shapes s, const int32_t* __restrict__ cu_qlens,
                                                                 const int32_t* __restrict__ cu_seqlens,
                                                                 const float* __restrict__ logits, int rq,
                                                                 float* __restrict__ lse) {
  __shared__ float red[8];
  pdl_trigger();
  // the caller's arrays first: these loads overlap the predecessor's tail
  const int b = blockIdx.y, head = blockIdx.x / rq, r = blockIdx.x % rq;
  const Span seq = seq_span(s, cu_seqlens, b), qrows = row_span(s, cu_qlens, b);
  const int row0 = qrows.first, rows = min(qrows.count, rq);
  const int tok0 = seq.first, n = seq.count;
  pdl_wait();
  pdl_acquire(logits);
  if (r >= rows) return;
  const float* z = logits + ((long long)head * rq + r) * s.total_tokens + tok0;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // One pass: every thread keeps a running (max, sum 2^(z - max)) over its strided share, sixteen loads at a time.
  float m = -INFINITY, l = 0.f;
  for (int j0 = threadIdx.x; j0 < n; j0 += 256 * 16) {  // sixteen loads in flight per thread: two trips for 8k tokens
    float v[16];
#pragma unroll
    for (int u = 0; u < 16; ++u) v[u] = j0 + u * 256 < n ? chain_load(z + j0 + u * 256) : -INFINITY;
    float m_new = m;
#pragma unroll
    for (int u = 0; u < 16; ++u) m_new = fmaxf(m_new, v[u]);
    if (m_new > -INFINITY) {
      l = l * exp2f(m - m_new);
#pragma unroll
      for (int u = 0; u < 16; ++u) l += exp2f(v[u] - m_new);
      m = m_new;
    }
  }
  // Merge the per-thread pairs: first the maximum, then the rescaled sums, both in a fixed order.
  float bm = m;
#pragma unroll
  for (int d = 16; d; d >>= 1) bm = fmaxf(bm, __shfl_xor_sync(0xFFFFFFFFu, bm, d));
  if (lane == 0) red[warp] = bm;
  __syncthreads();
  bm = red[0];
#pragma unroll
  for (int w = 1; w < 8; ++w) bm = fmaxf(bm, red[w]);
  __syncthreads();
  float part = (m > -INFINITY) ? l * exp2f(m - bm) : 0.f;
#pragma unroll
  for (int d = 16; d; d >>= 1) part += __shfl_xor_sync(0xFFFFFFFFu, part, d);
  if (lane == 0) red[warp] = part;
  __syncthreads();
  if (threadIdx.x == 0) {
    float total = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) total += red[w];
    lse[(long long)(row0 + r) * s.hq + head] = total > 0.f ? bm + log2f(total) : INFINITY;  // a row that sees no key adds 0
  }
}

constexpr int kFinalizeThreads = 64;  // small blocks: a few thousand tokens still spread over all SMs

__global__ void __launch_bounds__(kFinalizeThreads) score_narrow_finalize_kernel(Shapes s, const int32_t* __restrict__ cu_qlens,
                                                                                 const int32_t* __restrict__ cu_seqlens,
                                                                                 const float* __restrict__ logits, int rq,
                                                                                 const float* __restrict__ lse,
                                                                                 float* __restrict__ scores) {
  extern __shared__ float lse_sh[];  // [Hq][rows], then the term offsets
  pdl_trigger();
  // the caller's arrays first: these loads overlap the predecessor's tail
  const int b = blockIdx.y;
  const Span seq = seq_span(s, cu_seqlens, b), qrows = row_span(s, cu_qlens, b);
  const int tok0 = seq.first, n = seq.count;
  const int row0 = qrows.first, all_rows = qrows.count, rows = min(all_rows, rq);
  const int terms = s.hq * rows;
  pdl_wait();
  pdl_acquire(logits);
  pdl_acquire(lse);
  if ((int)(blockIdx.x * blockDim.x) >= n) return;
  // where term i's logits start, in units of N floats: worked out once per block (no integer division per logit below)
  int* term_row = reinterpret_cast<int*>(lse_sh + s.hq * rq);
  for (int i = threadIdx.x; i < terms; i += blockDim.x) {
    const int head = i / rows, r = i % rows;
    lse_sh[i] = chain_load(lse + (long long)(row0 + r) * s.hq + head);
    term_row[i] = head * rq + r;
  }
  __syncthreads();
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= n) return;
  // Term i = (head, row) in head-major order; sixteen loads in flight, one running sum in that fixed order.
  const float* z = logits + tok0 + j;
  float total = 0.f;
  for (int i0 = 0; i0 < terms; i0 += 16) {
    float v[16];
#pragma unroll
    for (int u = 0; u < 16; ++u) {
      const int i = i0 + u;
      v[u] = i < terms ? chain_load(z + (long long)term_row[i] * s.total_tokens) : -INFINITY;
    }
#pragma unroll
    for (int u = 0; u < 16; ++u)
      if (i0 + u < terms) total += exp2f(v[u] - lse_sh[i0 + u]);
  }
  scores[tok0 + j] = all_rows > 0 ? total / ((float)s.hq * (float)all_rows) : 0.f;
}

template <int DIM, int ROWS>
cudaError_t launch_logits(const Shapes& s, const uint16_t* q, const int32_t* q_idx, const int32_t* cu_qlens, const uint16_t* k,
                          const int32_t* cu_seqlens, float* logits, int rq, int32_t* device_status, cudaStream_t stream) {
  constexpr int kGroups = kComputeThreads / (DIM / 8);
  // One block covers `hb` KV heads so that a step of the block reads whole contiguous token rows.
  int hb = 1;
  while (hb * 2 <= s.hkv && s.hkv % (hb * 2) == 0 && hb * 2 <= kGroups) hb *= 2;
  // Key chunk per block: a multiple of the slot size, about two blocks per SM over the whole batch, 64..1024 keys.
  long long chunk = ((long long)s.total_tokens * (s.hkv / hb) + 2 * kNumSMs - 1) / (2 * kNumSMs);
  chunk = (chunk + kSlotKeys - 1) / kSlotKeys * kSlotKeys;
  if (chunk < 4 * kSlotKeys) chunk = 4 * kSlotKeys;
  if (chunk > 64 * kSlotKeys) chunk = 64 * kSlotKeys;
  const size_t smem = (size_t)kStages * kSlotKeys * hb * DIM * 2;
  cudaError_t e = cudaFuncSetAttribute(score_narrow_logits_kernel<DIM, ROWS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const dim3 grid((unsigned)((s.max_seqlen + chunk - 1) / chunk), s.hkv / hb, s.batch);
  return launch_chained(score_narrow_logits_kernel<DIM, ROWS>, grid, dim3(kThreads), smem, stream, s, q, q_idx, cu_qlens, k, cu_seqlens,
                        logits, rq, hb, (int)chunk, device_status);
}

}  // namespace

bool score_narrow_applies(const Shapes& s) { return s.max_qlen >= 1 && s.max_qlen <= kNarrowMaxRows && s.hq <= 256; }

cudaError_t launch_narrow_logits(const Shapes& s, const Workspace& w, const void* q, const int32_t* q_idx,
                                 const int32_t* cu_qlens, const void* k, const int32_t* cu_seqlens, unsigned char* ws,
                                 int32_t* device_status, cudaStream_t stream) {
  const uint16_t* qq = static_cast<const uint16_t*>(q);
  const uint16_t* kk = static_cast<const uint16_t*>(k);
  float* logits = reinterpret_cast<float*>(ws + w.logits_off);
  const int rq = s.max_qlen;
  const bool four = s.max_qlen * s.group <= 4;
  cudaError_t e;
  // The logits come from a skinny tensor-core MMA over TMA-streamed K tiles where that kernel takes the shapes
  // (and the caller did not ask for the CUDA-core kernel); otherwise from the lane-group kernel above.
  bool by_mma = false;
  if ((s.flags & FASTAV_SCORE_PATH_MASK) != FASTAV_SCORE_PATH_NARROW && score_wide_applies(s)) {
    e = launch_logits_wide(s, q, q_idx, cu_qlens, k, cu_seqlens, logits, rq, device_status, stream, &by_mma);
    if (e != cudaSuccess || by_mma) return e;
  }
  if (s.dim == 128) {
    e = four ? launch_logits<128, 4>(s, qq, q_idx, cu_qlens, kk, cu_seqlens, logits, rq, device_status, stream)
             : launch_logits<128, 8>(s, qq, q_idx, cu_qlens, kk, cu_seqlens, logits, rq, device_status, stream);
  } else {
    e = four ? launch_logits<64, 4>(s, qq, q_idx, cu_qlens, kk, cu_seqlens, logits, rq, device_status, stream)
             : launch_logits<64, 8>(s, qq, q_idx, cu_qlens, kk, cu_seqlens, logits, rq, device_status, stream);
  }
  count_launches(1);
  return e;
}

cudaError_t launch_score_narrow(const Shapes& s, const Workspace& w, const void* q, const int32_t* q_idx,
                                const int32_t* cu_qlens, const void* k, const int32_t* cu_seqlens, const float* lse_in,
                                float* scores_out, unsigned char* ws, int32_t* device_status, cudaStream_t stream) {
  float* logits = reinterpret_cast<float*>(ws + w.logits_off);
  float* lse = reinterpret_cast<float*>(ws + w.lse_off);
  const int rq = s.max_qlen;
  cudaError_t e = launch_narrow_logits(s, w, q, q_idx, cu_qlens, k, cu_seqlens, ws, device_status, stream);
  if (e != cudaSuccess) return e;
  if (!lse_in && scores_out && narrow_tail_applies(s))  // short sequences: statistics and scores in one kernel
    return launch_narrow_tail(s, logits, rq, scores_out, false, cu_seqlens, nullptr, nullptr, q_idx, cu_qlens, nullptr, nullptr,
                              device_status, stream);
  if (lse_in) e = launch_lse_import(s, lse_in, lse, stream);
  else e = launch_chained(score_narrow_stats_kernel, dim3(s.hq * rq, s.batch), dim3(256), 0, stream, s, cu_qlens, cu_seqlens,
                          (const float*)logits, rq, lse);
  if (e != cudaSuccess) return e;
  if (!scores_out) {  // only the statistics were asked for (fastav_lse)
    count_launches(lse_in ? 0 : 1);
    return cudaGetLastError();
  }
  if ((e = launch_chained(score_narrow_finalize_kernel, dim3((s.max_seqlen + kFinalizeThreads - 1) / kFinalizeThreads, s.batch),
                          dim3(kFinalizeThreads),
                          s.hq * rq * (sizeof(float) + sizeof(int)), stream, s, cu_qlens, cu_seqlens, (const float*)logits, rq, (const float*)lse,
                          scores_out)) != cudaSuccess)
    return e;
  count_launches((lse_in ? 0 : 1) + 1);  // the lse import counts itself
  return cudaGetLastError();
}

}  // namespace fastav
