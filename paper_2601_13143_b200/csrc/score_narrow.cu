// Importance score, Eq. 4 (Section 2.2), for FEW scored rows per sequence -- the shape the paper
// itself uses in the fine-pruning stage: Q_last is one row per head, so Q K^T is a matrix-vector
// product and the step is bound by reading K once from HBM.
//
//   logits   : every 16-byte piece of a key row is loaded once by one lane and multiplied with up to
//              eight query rows held in registers (the rows and heads of one KV group); a butterfly
//              of shuffles that halves the row set at each step leaves one finished logit per lane.
//              Logits [Hq, R, N] (base-2 units, -inf where the causal mask hides the key) go to the
//              workspace: R * Hq * 4 bytes per token next to the Hkv * d * 2 bytes of K read.
//   stats    : one block per (sequence, head, row): max and sum 2^(z - max) -> log2-sum-exp2.
//   finalize : per token, sum over heads and rows of 2^(z - lse) in a fixed order, times 1/(Hq R).
//
// Every key goes through the same arithmetic in the same order, whatever its position, so equal
// keys get bit-equal scores and runs are bit-reproducible.
#include "common.cuh"

namespace fastav {
namespace {

constexpr int kThreads = 256;
// Key rows in flight per lane group: more when fewer query rows occupy the registers.
template <int ROWS> struct Unroll { static constexpr int value = ROWS == 4 ? 8 : 4; };

__device__ __forceinline__ void unpack8(const uint4& v, float2 (&out)[4]) {
  out[0] = make_float2(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xFFFF0000u));
  out[1] = make_float2(__uint_as_float(v.y << 16), __uint_as_float(v.y & 0xFFFF0000u));
  out[2] = make_float2(__uint_as_float(v.z << 16), __uint_as_float(v.z & 0xFFFF0000u));
  out[3] = make_float2(__uint_as_float(v.w << 16), __uint_as_float(v.w & 0xFFFF0000u));
}

// DIM: head_dim; ROWS: query rows handled per pass (4 or 8); HB: KV heads covered by one block.
// A "lane group" is the DIM/8 lanes that together read one key row of one KV head.
template <int DIM, int ROWS>
__global__ void __launch_bounds__(kThreads, ROWS == 4 ? 3 : 2)
score_narrow_logits_kernel(Shapes s, const uint16_t* __restrict__ q, const int32_t* __restrict__ q_idx,
                           const int32_t* __restrict__ cu_qlens, const uint16_t* __restrict__ k,
                           const int32_t* __restrict__ cu_seqlens, float* __restrict__ logits, int rq, int heads_per_block,
                           int chunk_keys) {
  constexpr int kUnroll = Unroll<ROWS>::value;
  constexpr int kLanes = DIM / 8;               // lanes per key row
  constexpr int kGroups = kThreads / kLanes;    // key rows per block per step
  constexpr int kHalvings = ROWS == 8 ? 3 : 2;  // butterfly steps that halve the row set
  constexpr int kPlainBits = (kLanes == 16 ? 4 : 3) - kHalvings;

  pdl_trigger();
  pdl_wait();  // q and k may be what the previous kernel wrote; the logits may still be read by it
  pdl_acquire(q);
  pdl_acquire(k);
  const int b = blockIdx.z;
  const int tok0 = cu_seqlens[b], n = cu_seqlens[b + 1] - tok0;
  const int key_begin = blockIdx.x * chunk_keys;
  if (key_begin >= n) return;
  const int key_end = min(n, key_begin + chunk_keys);
  const int row0 = cu_qlens[b], rows = min(cu_qlens[b + 1] - row0, rq);
  const int flat_rows = rows * s.group;
  if (flat_rows == 0) return;

  const int group = threadIdx.x / kLanes, lane = threadIdx.x % kLanes;
  const int head = blockIdx.y * heads_per_block + group % heads_per_block;  // KV head of this lane group
  const int keys_per_step = kGroups / heads_per_block;
  const int key_lane = group / heads_per_block;
  const bool causal = (s.flags & FASTAV_CAUSAL) != 0;
  const int my_row = (lane >> kPlainBits) & (ROWS - 1);  // the row whose finished logit lands in this lane
  const bool writer = (lane & ((1 << kPlainBits) - 1)) == 0;
  const uint16_t* kbase = k + (long long)tok0 * s.k_st + (long long)head * s.k_sh + lane * 8;

  for (int pass0 = 0; pass0 < flat_rows; pass0 += ROWS) {
    // Query rows of this pass: flat index f = r * G + (head within the group).
    float2 qv[ROWS][4];
#pragma unroll
    for (int i = 0; i < ROWS; ++i) {
      const int f = pass0 + i;
      uint4 raw = make_uint4(0, 0, 0, 0);
      if (f < flat_rows)
        raw = __ldg(reinterpret_cast<const uint4*>(q + (long long)(row0 + f / s.group) * s.q_st +
                                                   (long long)(head * s.group + f % s.group) * s.q_sh + lane * 8));
      unpack8(raw, qv[i]);
    }
    const int f_mine = pass0 + my_row;
    const bool row_valid = f_mine < flat_rows;
    const int r_mine = row_valid ? f_mine / s.group : 0;
    const int limit = (causal && row_valid) ? q_idx[row0 + r_mine] : 0x7FFFFFFF;
    float* out = logits + ((long long)(head * s.group + (row_valid ? f_mine % s.group : 0)) * rq + r_mine) * s.total_tokens + tok0;

    // The trip count is the same for every lane of the block (the shuffles below need whole warps).
    for (int base = key_begin; base < key_end; base += keys_per_step * kUnroll) {
      const int key0 = base + key_lane;
      uint4 raw[kUnroll];
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int key = key0 + u * keys_per_step;
        raw[u] = make_uint4(0, 0, 0, 0);
        if (key < key_end) raw[u] = __ldg(reinterpret_cast<const uint4*>(kbase + (long long)key * s.k_st));
      }
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int key = key0 + u * keys_per_step;
        float2 kv[4];
        unpack8(raw[u], kv);
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
        if (writer && row_valid && key < key_end) out[key] = key <= limit ? vals[0] * s.scale_log2 : -INFINITY;
      }
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
  pdl_wait();
  pdl_acquire(logits);
  const int b = blockIdx.y, head = blockIdx.x / rq, r = blockIdx.x % rq;
  const int row0 = cu_qlens[b], rows = min(cu_qlens[b + 1] - row0, rq);
  if (r >= rows) return;
  const int tok0 = cu_seqlens[b], n = cu_seqlens[b + 1] - tok0;
  const float* z = logits + ((long long)head * rq + r) * s.total_tokens + tok0;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // One pass: every thread keeps a running (max, sum 2^(z - max)) over its strided share, four loads at a time.
  float m = -INFINITY, l = 0.f;
  for (int j0 = threadIdx.x; j0 < n; j0 += 256 * 4) {
    float v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) v[u] = j0 + u * 256 < n ? z[j0 + u * 256] : -INFINITY;
    const float m_new = fmaxf(fmaxf(m, fmaxf(v[0], v[1])), fmaxf(v[2], v[3]));
    if (m_new > -INFINITY) {
      l = l * exp2f(m - m_new);
#pragma unroll
      for (int u = 0; u < 4; ++u) l += exp2f(v[u] - m_new);
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
  extern __shared__ float lse_sh[];  // [Hq][rows]
  pdl_trigger();
  pdl_wait();
  pdl_acquire(logits);
  pdl_acquire(lse);
  const int b = blockIdx.y;
  const int tok0 = cu_seqlens[b], n = cu_seqlens[b + 1] - tok0;
  if ((int)(blockIdx.x * blockDim.x) >= n) return;
  const int row0 = cu_qlens[b], all_rows = cu_qlens[b + 1] - row0, rows = min(all_rows, rq);
  const int terms = s.hq * rows;
  for (int i = threadIdx.x; i < terms; i += blockDim.x) {
    const int head = i / rows, r = i % rows;
    lse_sh[i] = lse[(long long)(row0 + r) * s.hq + head];
  }
  __syncthreads();
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= n) return;
  // Term i = (head, row) in head-major order; eight loads in flight, one running sum in that fixed order.
  const float* z = logits + tok0 + j;
  float total = 0.f;
  for (int i0 = 0; i0 < terms; i0 += 8) {
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = i0 + u;
      v[u] = i < terms ? z[((long long)(i / rows) * rq + i % rows) * s.total_tokens] : -INFINITY;
    }
#pragma unroll
    for (int u = 0; u < 8; ++u)
      if (i0 + u < terms) total += exp2f(v[u] - lse_sh[i0 + u]);
  }
  scores[tok0 + j] = all_rows > 0 ? total / ((float)s.hq * (float)all_rows) : 0.f;
}

template <int DIM, int ROWS>
cudaError_t launch_logits(const Shapes& s, const uint16_t* q, const int32_t* q_idx, const int32_t* cu_qlens, const uint16_t* k,
                   const int32_t* cu_seqlens, float* logits, int rq, cudaStream_t stream) {
  constexpr int kGroups = kThreads / (DIM / 8);
  // One block covers `hb` KV heads so that a step of the block reads whole contiguous token rows.
  int hb = 1;
  while (hb * 2 <= s.hkv && s.hkv % (hb * 2) == 0 && hb * 2 <= kGroups) hb *= 2;
  const int keys_per_step = kGroups / hb;
  const int quantum = keys_per_step * Unroll<ROWS>::value;
  // Enough blocks to fill the machine a few times over, but never less than one unrolled step each.
  const long long want_blocks = (long long)kNumSMs * 8;
  long long chunk = ((long long)s.total_tokens * (s.hkv / hb) + want_blocks - 1) / want_blocks;
  chunk = (chunk + quantum - 1) / quantum * quantum;
  if (chunk < quantum) chunk = quantum;
  if (chunk > 8 * quantum) chunk = 8 * quantum;
  const dim3 grid((unsigned)((s.max_seqlen + chunk - 1) / chunk), s.hkv / hb, s.batch);
  return launch_chained(score_narrow_logits_kernel<DIM, ROWS>, grid, dim3(kThreads), 0, stream, s, q, q_idx, cu_qlens, k, cu_seqlens,
                        logits, rq, hb, (int)chunk);
}

}  // namespace

bool score_narrow_applies(const Shapes& s) { return s.max_qlen >= 1 && s.max_qlen <= kNarrowMaxRows && s.hq <= 256; }

cudaError_t launch_score_narrow(const Shapes& s, const Workspace& w, const void* q, const int32_t* q_idx,
                                const int32_t* cu_qlens, const void* k, const int32_t* cu_seqlens, float* scores_out,
                                unsigned char* ws, cudaStream_t stream) {
  const uint16_t* qq = static_cast<const uint16_t*>(q);
  const uint16_t* kk = static_cast<const uint16_t*>(k);
  float* logits = reinterpret_cast<float*>(ws + w.logits_off);
  float* lse = reinterpret_cast<float*>(ws + w.lse_off);
  const int rq = s.max_qlen;
  const bool four = s.max_qlen * s.group <= 4;
  cudaError_t e;
  if (s.dim == 128) {
    e = four ? launch_logits<128, 4>(s, qq, q_idx, cu_qlens, kk, cu_seqlens, logits, rq, stream)
             : launch_logits<128, 8>(s, qq, q_idx, cu_qlens, kk, cu_seqlens, logits, rq, stream);
  } else {
    e = four ? launch_logits<64, 4>(s, qq, q_idx, cu_qlens, kk, cu_seqlens, logits, rq, stream)
             : launch_logits<64, 8>(s, qq, q_idx, cu_qlens, kk, cu_seqlens, logits, rq, stream);
  }
  if (e != cudaSuccess) return e;
  if ((e = launch_chained(score_narrow_stats_kernel, dim3(s.hq * rq, s.batch), dim3(256), 0, stream, s, cu_qlens, cu_seqlens,
                          (const float*)logits, rq, lse)) != cudaSuccess)
    return e;
  if ((e = launch_chained(score_narrow_finalize_kernel, dim3((s.max_seqlen + kFinalizeThreads - 1) / kFinalizeThreads, s.batch),
                          dim3(kFinalizeThreads),
                          s.hq * rq * sizeof(float), stream, s, cu_qlens, cu_seqlens, (const float*)logits, rq, (const float*)lse,
                          scores_out)) != cudaSuccess)
    return e;
  count_launches(3);
  return cudaGetLastError();
}

}  // namespace fastav
