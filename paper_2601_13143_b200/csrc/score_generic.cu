// Importance score, Eq. 4 (Section 2.2):  s = mean_h softmax(Q_last K^T), for R scored rows,
// grouped-query heads and packed varlen batches -- the shape-agnostic CUDA-core path.
//
// The L x L attention map is never formed and neither is the [Hq R, n] block of logits: two sweeps
// over the keys recompute 64-key x 32-row logit tiles in shared memory.
//   sweep 1: per (row, head) and key tile, (max, sum 2^(z - max))     -> merged into log2-sum-exp2
//   sweep 2: p = 2^(z - lse) summed over the rows and heads of one KV head -> partial[kv head][token]
//   finalize: scores = (sum over KV heads, ascending) / (Hq R_b)
// Logits are kept in base-2 units (scale * log2 e folded in), all sums are taken in a fixed order,
// so a run is bit-reproducible and equal keys get bit-equal scores.
#include "common.cuh"

namespace fastav {
namespace {

constexpr int kTileKeys = 64;
constexpr int kTileRows = 32;
constexpr int kThreads = 256;

__device__ __forceinline__ float bf16_lo(unsigned v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16_hi(unsigned v) { return __uint_as_float(v & 0xFFFF0000u); }

template <int DIM>
struct TileShared {
  float k[kTileKeys][DIM + 1];
  float q[kTileRows][DIM + 1];
  float z[kTileRows][kTileKeys + 1];
  int q_tok[kTileRows];  // sequence-local token index of each row of the chunk (causal mask)
};

// Rows of `count` bf16 vectors of DIM elements -> fp32 shared tile; rows >= count are zero-filled.
template <int DIM, int ROWS>
__device__ __forceinline__ void load_rows(float (*dst)[DIM + 1], int count, const uint16_t* (*row_ptr)(int, const void*),
                                          const void* ctx) {
  constexpr int kChunks = DIM / 8;
  for (int idx = threadIdx.x; idx < ROWS * kChunks; idx += kThreads) {
    const int row = idx / kChunks, chunk = idx % kChunks;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (row < count) v = *reinterpret_cast<const uint4*>(row_ptr(row, ctx) + chunk * 8);
    float* d = &dst[row][chunk * 8];
    d[0] = bf16_lo(v.x); d[1] = bf16_hi(v.x); d[2] = bf16_lo(v.y); d[3] = bf16_hi(v.y);
    d[4] = bf16_lo(v.z); d[5] = bf16_hi(v.z); d[6] = bf16_lo(v.w); d[7] = bf16_hi(v.w);
  }
}

struct KeyCtx { const uint16_t* base; long long stride; };
struct QueryCtx { const uint16_t* base; long long st, sh; int group, head0, first; };

__device__ const uint16_t* key_row(int row, const void* c) {
  const KeyCtx* k = static_cast<const KeyCtx*>(c);
  return k->base + (long long)row * k->stride;
}
__device__ const uint16_t* query_row(int row, const void* c) {
  const QueryCtx* q = static_cast<const QueryCtx*>(c);
  const int f = q->first + row;  // flat (row, head-in-group) index
  return q->base + (long long)(f / q->group) * q->st + (long long)(q->head0 + f % q->group) * q->sh;
}

// z[row][key] = scale_log2 * <q_row, k_key>, or -inf where the row may not see the key.
template <int DIM>
__device__ __forceinline__ void tile_logits(TileShared<DIM>& sh, float scale_log2, int key0, int keys_valid, bool causal) {
  const int tk = threadIdx.x & 15, tr = threadIdx.x >> 4;
  float acc[2][4] = {};
#pragma unroll 4
  for (int c = 0; c < DIM; ++c) {
    const float q0 = sh.q[tr * 2][c], q1 = sh.q[tr * 2 + 1][c];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float kv = sh.k[tk + 16 * i][c];
      acc[0][i] = fmaf(q0, kv, acc[0][i]);
      acc[1][i] = fmaf(q1, kv, acc[1][i]);
    }
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int limit = causal ? sh.q_tok[tr * 2 + r] : 0x7FFFFFFF;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int key = tk + 16 * i;
      const bool visible = key < keys_valid && (key0 + key) <= limit;
      sh.z[tr * 2 + r][key] = visible ? acc[r][i] * scale_log2 : -INFINITY;
    }
  }
}

// Common prologue of both sweeps: returns false when the block has nothing to do.
template <int DIM>
__device__ __forceinline__ bool load_key_tile(TileShared<DIM>& sh, const Shapes& s, const uint16_t* k,
                                              const int32_t* cu_seqlens, int& tok0, int& n, int& key0, int& keys_valid) {
  const int b = blockIdx.z, g = blockIdx.y;
  const Span seq = seq_span(s, cu_seqlens, b);
  tok0 = seq.first;
  n = seq.count;
  key0 = blockIdx.x * kTileKeys;
  if (key0 >= n) return false;
  keys_valid = min(kTileKeys, n - key0);
  KeyCtx kc{k + (long long)(tok0 + key0) * s.k_st + (long long)g * s.k_sh, s.k_st};
  load_rows<DIM, kTileKeys>(sh.k, keys_valid, key_row, &kc);
  return true;
}

template <int DIM>
__device__ __forceinline__ void load_query_chunk(TileShared<DIM>& sh, const Shapes& s, const uint16_t* q, const int32_t* q_idx,
                                                 int row0, int flat0, int flat_count) {
  QueryCtx qc{q + (long long)row0 * s.q_st, s.q_st, s.q_sh, s.group, (int)blockIdx.y * s.group, flat0};
  const int count = min(kTileRows, flat_count - flat0);
  load_rows<DIM, kTileRows>(sh.q, count, query_row, &qc);
  if (threadIdx.x < kTileRows) {
    const int f = flat0 + threadIdx.x;
    sh.q_tok[threadIdx.x] = f < flat_count ? q_idx[row0 + f / s.group] : -1;
  }
}

template <int DIM>
__global__ void __launch_bounds__(kThreads) score_tile_stats_kernel(Shapes s, const uint16_t* __restrict__ q,
                                                                    const int32_t* __restrict__ q_idx,
                                                                    const int32_t* __restrict__ cu_qlens,
                                                                    const uint16_t* __restrict__ k,
                                                                    const int32_t* __restrict__ cu_seqlens,
                                                                    float2* __restrict__ stats, int stat_tiles) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  TileShared<DIM>& sh = *reinterpret_cast<TileShared<DIM>*>(smem_raw);
  int tok0, n, key0, keys_valid;
  if (!load_key_tile<DIM>(sh, s, k, cu_seqlens, tok0, n, key0, keys_valid)) return;
  const int b = blockIdx.z;
  const Span qrows = row_span(s, cu_qlens, b);
  const int row0 = qrows.first, rows = qrows.count;
  const int flat_count = rows * s.group;
  const bool causal = (s.flags & FASTAV_CAUSAL) != 0;
  for (int flat0 = 0; flat0 < flat_count; flat0 += kTileRows) {
    __syncthreads();
    load_query_chunk<DIM>(sh, s, q, q_idx, row0, flat0, flat_count);
    __syncthreads();
    tile_logits<DIM>(sh, s.scale_log2, key0, keys_valid, causal);
    __syncthreads();
    // 8 threads per row, 8 keys each; combine with shuffles inside the 8-lane group.
    const int row = threadIdx.x >> 3, part = threadIdx.x & 7;
    float m = -INFINITY;
#pragma unroll
    for (int i = 0; i < 8; ++i) m = fmaxf(m, sh.z[row][part + 8 * i]);
#pragma unroll
    for (int d = 1; d < 8; d <<= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, d));
    float l = 0.f;
    if (m > -INFINITY) {
#pragma unroll
      for (int i = 0; i < 8; ++i) l += exp2f(sh.z[row][part + 8 * i] - m);
    }
#pragma unroll
    for (int d = 1; d < 8; d <<= 1) l += __shfl_xor_sync(0xFFFFFFFFu, l, d);
    const int f = flat0 + row;
    if (part == 0 && f < flat_count) {
      const long long rh = (long long)(row0 + f / s.group) * s.hq + (blockIdx.y * s.group + f % s.group);
      stats[rh * stat_tiles + blockIdx.x] = make_float2(m, l);
    }
  }
}

// One warp per (scored row, head): fold the per-tile (max, sum) pairs into log2-sum-exp2.
__global__ void __launch_bounds__(256) score_merge_stats_kernel(Shapes s, const int32_t* __restrict__ cu_qlens,
                                                                const int32_t* __restrict__ cu_seqlens,
                                                                const float2* __restrict__ stats, int stat_tiles,
                                                                float* __restrict__ lse) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= s.total_q * s.hq) return;
  const int row = warp / s.hq;
  int lo = 0, hi = s.batch;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (cu_qlens[mid] <= row) lo = mid; else hi = mid;
  }
  const int n = seq_span(s, cu_seqlens, lo).count;
  const int tiles = (n + kTileKeys - 1) / kTileKeys;
  const float2* mine = stats + (long long)warp * stat_tiles;
  float m = -INFINITY;
  for (int t = lane; t < tiles; t += 32) m = fmaxf(m, mine[t].x);
#pragma unroll
  for (int d = 16; d; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, d));
  float l = 0.f;
  if (m > -INFINITY)
    for (int t = lane; t < tiles; t += 32) {
      const float2 v = mine[t];
      if (v.x > -INFINITY) l += v.y * exp2f(v.x - m);
    }
#pragma unroll
  for (int d = 16; d; d >>= 1) l += __shfl_xor_sync(0xFFFFFFFFu, l, d);
  if (lane == 0) lse[warp] = (l > 0.f) ? m + log2f(l) : INFINITY;  // a row that sees no key contributes 0
}

template <int DIM>
__global__ void __launch_bounds__(kThreads) score_tile_accumulate_kernel(Shapes s, const uint16_t* __restrict__ q,
                                                                         const int32_t* __restrict__ q_idx,
                                                                         const int32_t* __restrict__ cu_qlens,
                                                                         const uint16_t* __restrict__ k,
                                                                         const int32_t* __restrict__ cu_seqlens,
                                                                         const float* __restrict__ lse,
                                                                         float* __restrict__ partial) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  TileShared<DIM>& sh = *reinterpret_cast<TileShared<DIM>*>(smem_raw);
  int tok0, n, key0, keys_valid;
  if (!load_key_tile<DIM>(sh, s, k, cu_seqlens, tok0, n, key0, keys_valid)) return;
  const int b = blockIdx.z;
  const Span qrows = row_span(s, cu_qlens, b);
  const int row0 = qrows.first, rows = qrows.count;
  const int flat_count = rows * s.group;
  const bool causal = (s.flags & FASTAV_CAUSAL) != 0;
  // 4 threads per key, 8 rows of the chunk each.
  const int key = threadIdx.x >> 2, part = threadIdx.x & 3;
  float sum = 0.f;
  for (int flat0 = 0; flat0 < flat_count; flat0 += kTileRows) {
    __syncthreads();
    load_query_chunk<DIM>(sh, s, q, q_idx, row0, flat0, flat_count);
    __syncthreads();
    tile_logits<DIM>(sh, s.scale_log2, key0, keys_valid, causal);
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int row = part * 8 + i, f = flat0 + row;
      if (f < flat_count) {
        const float z = sh.z[row][key];
        const float l = lse[(long long)(row0 + f / s.group) * s.hq + (blockIdx.y * s.group + f % s.group)];
        if (z > -INFINITY) sum += exp2f(z - l);
      }
    }
  }
  sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 1);
  sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 2);
  if (part == 0 && key < keys_valid) partial[(long long)blockIdx.y * s.total_tokens + tok0 + key0 + key] = sum;
}

__global__ void __launch_bounds__(256) score_finalize_kernel(Shapes s, const int32_t* __restrict__ cu_seqlens,
                                                             const int32_t* __restrict__ cu_qlens,
                                                             const float* __restrict__ partial, float* __restrict__ scores) {
  const int b = blockIdx.y;
  const Span seq = seq_span(s, cu_seqlens, b);
  const int tok0 = seq.first, n = seq.count;
  const int rows = row_span(s, cu_qlens, b).count;
  const float inv = rows > 0 ? 1.0f / ((float)s.hq * (float)rows) : 0.f;
  for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < n; j += gridDim.x * blockDim.x) {
    float total = 0.f;
    if (rows > 0)
      for (int g = 0; g < s.hkv; ++g) total += partial[(long long)g * s.total_tokens + tok0 + j];
    scores[tok0 + j] = total * inv;
  }
}

__global__ void __launch_bounds__(256) lse_import_kernel(int count, const float* __restrict__ lse_in, float* __restrict__ lse_ws) {
  pdl_trigger();
  pdl_wait();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= count) return;
  const float v = lse_in[i];
  lse_ws[i] = (v == v && fabsf(v) != INFINITY) ? v * kLog2e : INFINITY;
}

// The way back: log2-sum-exp2 of the workspace -> natural-log log-sum-exp as attention kernels report it
// (-inf for a row that sees no key).
__global__ void __launch_bounds__(256) lse_export_kernel(int count, const float* __restrict__ lse_ws, float* __restrict__ lse_out) {
  pdl_trigger();
  pdl_wait();
  pdl_acquire(lse_ws);
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= count) return;
  const float v = chain_load(lse_ws + i);
  lse_out[i] = v == INFINITY ? -INFINITY : v * kLn2;
}

template <int DIM>
cudaError_t run(const Shapes& s, const Workspace& w, const uint16_t* q, const int32_t* q_idx, const int32_t* cu_qlens,
                const uint16_t* k, const int32_t* cu_seqlens, const float* lse_in, float* scores_out, unsigned char* ws,
                cudaStream_t stream) {
  float2* stats = reinterpret_cast<float2*>(ws + w.stats_off);
  float* lse = reinterpret_cast<float*>(ws + w.lse_off);
  float* partial = reinterpret_cast<float*>(ws + w.partial_off);
  const size_t smem = sizeof(TileShared<DIM>);
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(score_tile_stats_kernel<DIM>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(score_tile_accumulate_kernel<DIM>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
  if (s.total_q > 0 && s.max_seqlen > 0) {
    const dim3 grid(w.stat_tiles, s.hkv, s.batch);
    if (lse_in) {
      if ((e = launch_lse_import(s, lse_in, lse, stream)) != cudaSuccess) return e;
    } else {
      score_tile_stats_kernel<DIM><<<grid, kThreads, smem, stream>>>(s, q, q_idx, cu_qlens, k, cu_seqlens, stats, w.stat_tiles);
      const int warps = s.total_q * s.hq;
      score_merge_stats_kernel<<<(warps + 7) / 8, 256, 0, stream>>>(s, cu_qlens, cu_seqlens, stats, w.stat_tiles, lse);
      count_launches(2);
    }
    if (!scores_out) return cudaGetLastError();  // only the statistics were asked for (fastav_lse)
    score_tile_accumulate_kernel<DIM><<<grid, kThreads, smem, stream>>>(s, q, q_idx, cu_qlens, k, cu_seqlens, lse, partial);
    count_launches(1);
  }
  if (s.max_seqlen > 0 && scores_out) {
    const dim3 grid((s.max_seqlen + 255) / 256, s.batch);
    score_finalize_kernel<<<grid, 256, 0, stream>>>(s, cu_seqlens, cu_qlens, partial, scores_out);
    count_launches(1);
  }
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_lse_import(const Shapes& s, const float* lse_in, float* lse_ws, cudaStream_t stream) {
  const int count = s.total_q * s.hq;
  if (count <= 0) return cudaSuccess;
  count_launches(1);
  return launch_chained(lse_import_kernel, dim3((count + 255) / 256), dim3(256), 0, stream, count, lse_in, lse_ws);
}

cudaError_t launch_lse_export(const Shapes& s, const float* lse_ws, float* lse_out, cudaStream_t stream) {
  const int count = s.total_q * s.hq;
  if (count <= 0) return cudaSuccess;
  count_launches(1);
  return launch_chained(lse_export_kernel, dim3((count + 255) / 256), dim3(256), 0, stream, count, lse_ws, lse_out);
}

cudaError_t launch_score_generic(const Shapes& s, const Workspace& w, const void* q, const int32_t* q_idx,
                                 const int32_t* cu_qlens, const void* k, const int32_t* cu_seqlens, const float* lse_in,
                                 float* scores_out, unsigned char* ws, cudaStream_t stream) {
  const uint16_t* qq = static_cast<const uint16_t*>(q);
  const uint16_t* kk = static_cast<const uint16_t*>(k);
  if (s.dim == 128) return run<128>(s, w, qq, q_idx, cu_qlens, kk, cu_seqlens, lse_in, scores_out, ws, stream);
  return run<64>(s, w, qq, q_idx, cu_qlens, kk, cu_seqlens, lse_in, scores_out, ws, stream);
}

}  // namespace fastav
