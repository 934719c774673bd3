// Top-k keep set per sequence: the bottom-P % rule of Section 2.2 ("Fine pruning"), stated as "keep the k best".
//
// One thread block per sequence.  Scores become order-preserving 32-bit keys (protected tokens get
// the largest key), held in shared memory when the sequence fits.  The k-th largest key T is found
// by an MSB-first radix select over the bits in which the keys of the sequence actually differ
// (the common leading bits come from a min/max reduction; softmax scores share most of their
// exponent, so without this the first histogram would pile into a handful of bins): at most three
// passes of 13-bit digits (11-bit ones for sequences of at most 2,048 tokens), shared-memory histograms, a block-wide suffix scan to pick the bin; as soon
// as the chosen bin holds at most 256 keys (usually after the first pass) they are collected and T is
// the one whose rank among them is the wanted one, which saves the remaining passes.
// A single blocked prefix scan in index order then keeps every key above T plus the first
// (k - #above) keys equal to T: ties go to the lower index and survivors come out ascending, which
// is exactly the order the gather that follows needs.  Integer work throughout: the result is a
// unique function of the fp32 score bits.
#include <mutex>

#include "common.cuh"
#include "select_block.cuh"

namespace fastav {
namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kDigitBits = 13;  // long sequences; short ones (kShortKeys or fewer) take kShortDigitBits, their passes being cheap
constexpr int kShortDigitBits = 11, kShortKeys = 2048;
constexpr int kBins = 1 << kDigitBits;
constexpr int kBinsPerThread = kBins / kThreads;  // bins one thread owns in the suffix scan, at most
struct SelectShared {
  unsigned hist[kBins];
  unsigned warp_a[kWarps], warp_b[kWarps];
  unsigned key_min, key_max;
  unsigned prefix;      // bits of T fixed so far
  int remaining;        // how many more keys (from the top of the current bucket) are still to take
  int base;             // output offset of this sequence
  int protected_count;
  int bucket;           // how many keys the chosen bin of the last pass holds
  int list_n;           // direct finish: the keys of a small bucket, in no particular order
  unsigned list[kDirectMax];
};

// Shared-memory slot of key j: one word of padding per 32 keeps both the strided and the blocked
// access patterns below (nearly) free of bank conflicts.
template <bool kKeysInShared>
__device__ __forceinline__ int slot(int j) { return kKeysInShared ? j + (j >> 5) : j; }

// Few scored rows, short sequences: the scores themselves are made here, from the logits the previous
// kernel left in the workspace (one block per sequence: log2-sum-exp2 per (head, row) by one warp each,
// then per token the fixed-order sum over heads and rows), so that a pruning layer of a small prompt is
// three kernels (logits, this one, the gather) instead of five.
struct FromLogits {
  const float* logits;  // [Hq, rq, N] base-2 logits, -inf where masked
  float* scores_out;    // [N]
  int rq;               // scored rows per sequence the logits are laid out for
  int do_select;        // 0: only the scores are wanted (fastav_score)
};

template <bool kKeysInShared, bool kFromLogits>
__global__ void __launch_bounds__(kThreads) select_topk_kernel(Shapes s, const float* __restrict__ scores,
                                                               const int32_t* __restrict__ cu_seqlens,
                                                               const int32_t* __restrict__ keep_counts,
                                                               const uint8_t* __restrict__ protect,
                                                               const int32_t* __restrict__ q_idx,
                                                               const int32_t* __restrict__ cu_qlens,
                                                               int32_t* __restrict__ keep_idx, int32_t* __restrict__ cu_keep,
                                                               unsigned* __restrict__ keys_global, int32_t* device_status,
                                                               FromLogits fl) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  SelectShared& sh = *reinterpret_cast<SelectShared*>(smem_raw);
  unsigned* keys = kKeysInShared ? reinterpret_cast<unsigned*>(smem_raw + sizeof(SelectShared)) : nullptr;

  pdl_trigger();
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const Span seq = seq_span(s, cu_seqlens, b);  // never beyond what the key storage was sized for
  const int tok0 = seq.first, n = seq.count;
  if (!kKeysInShared) keys = keys_global + tok0;

  const bool selecting = !kFromLogits || fl.do_select != 0;
  // Output offset: prefix sum of the clamped keep counts of the sequences before this one.
  if (tid == 0) { sh.base = 0; sh.protected_count = 0; sh.key_min = 0xFFFFFFFFu; sh.key_max = 0u; }
  __syncthreads();
  if (selecting) {
    int part = 0;
    bool clamped = false, mismatch = false;
    for (int i = tid; i <= b; i += kThreads) {
      const Span si = seq_span(s, cu_seqlens, i);
      const int ni = si.count;
      mismatch |= si.bad;
      int ki = keep_counts[i];
      if (ki < 0 || ki > ni) { clamped = true; ki = ki < 0 ? 0 : ni; }
      if (i < b) part += ki;
    }
    if (part) atomicAdd(&sh.base, part);
    if (clamped && device_status) atomicOr(device_status, FASTAV_DEV_K_CLAMPED);
    if (mismatch && device_status) atomicOr(device_status, FASTAV_DEV_SHAPE_MISMATCH);
  }
  int k = selecting ? keep_counts[b] : 0;
  k = k < 0 ? 0 : (k > n ? n : k);

  pdl_wait();  // the scores (or logits) are the previous kernel's output
  pdl_acquire(scores);

  // Keys.  Under FASTAV_SELECT_LOWEST the ranking is reversed by negating the scores (ties still go to the lower index).
  const bool lowest = (s.flags & FASTAV_SELECT_LOWEST) != 0;
  if constexpr (kFromLogits) {
    pdl_acquire(fl.logits);
    float* lse_sh = reinterpret_cast<float*>(keys + (s.max_seqlen + s.max_seqlen / 32 + 1));
    const int all_rows = row_span(s, cu_qlens, b).count, rows = min(all_rows, fl.rq);
    const int terms = s.hq * rows;  // term i = (head i / rows, row i % rows)
    // where term i's logits start, in units of N floats: worked out once, not per token (no integer division in the loop below)
    int* term_row = reinterpret_cast<int*>(lse_sh + s.hq * fl.rq);
    for (int i = tid; i < terms; i += kThreads) term_row[i] = (i / rows) * fl.rq + i % rows;
    for (int i = warp; i < terms; i += kWarps) {
      // log2-sum-exp2 of one row of logits by one warp: running (max, sum) per lane, merged in a fixed order
      const float* z = fl.logits + ((long long)(i / rows) * fl.rq + i % rows) * s.total_tokens + tok0;
      float m = -INFINITY, l = 0.f;
      for (int j0 = lane; j0 < n; j0 += 512) {  // sixteen loads in flight per lane: at most two trips for 1,024 tokens
        float v[16];
#pragma unroll
        for (int u = 0; u < 16; ++u) v[u] = j0 + 32 * u < n ? chain_load(z + j0 + 32 * u) : -INFINITY;
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
      float bm = m;
#pragma unroll
      for (int d = 16; d; d >>= 1) bm = fmaxf(bm, __shfl_xor_sync(0xFFFFFFFFu, bm, d));
      float part = (m > -INFINITY) ? l * exp2f(m - bm) : 0.f;
#pragma unroll
      for (int d = 16; d; d >>= 1) part += __shfl_xor_sync(0xFFFFFFFFu, part, d);
      if (lane == 0) lse_sh[i] = part > 0.f ? bm + log2f(part) : INFINITY;  // a row that sees no key adds 0
    }
    __syncthreads();
    for (int j = tid; j < n; j += kThreads) {
      const float* z = fl.logits + tok0 + j;
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
      const float score = all_rows > 0 ? total / ((float)s.hq * (float)all_rows) : 0.f;
      fl.scores_out[tok0 + j] = score;
      unsigned key = order_key(lowest ? -score : score);
      if (key == kProtectedKey) key = kProtectedKey - 1;
      if (protect && protect[tok0 + j]) key = kProtectedKey;
      keys[slot<kKeysInShared>(j)] = key;
    }
    if (!selecting) return;  // uniform for the block
  } else
  for (int j0 = tid; j0 < n; j0 += kThreads * 16) {
    float v[16];  // sixteen independent loads in flight per thread: one block serves a whole sequence
#pragma unroll
    for (int u = 0; u < 16; ++u) {
      const int j = j0 + u * kThreads;
      v[u] = j < n ? chain_load(scores + tok0 + j) : 0.f;
    }
#pragma unroll
    for (int u = 0; u < 16; ++u) {
      const int j = j0 + u * kThreads;
      if (j < n) {
        unsigned key = order_key(lowest ? -v[u] : v[u]);
        if (key == kProtectedKey) key = kProtectedKey - 1;  // only a NaN pattern lands here
        if (protect && protect[tok0 + j]) key = kProtectedKey;
        keys[slot<kKeysInShared>(j)] = key;
      }
    }
  }
  __syncthreads();
  if (s.flags & FASTAV_PROTECT_QUERY_ROWS) {
    const Span rows = checked_span(cu_qlens, b, s.total_q, s.total_q);
    for (int r = rows.first + tid; r < rows.first + rows.count; r += kThreads) {
      const int j = q_idx[r];
      if (j >= 0 && j < n) keys[slot<kKeysInShared>(j)] = kProtectedKey;
    }
    __syncthreads();
  }
  // Range of the unprotected keys and number of protected ones.
  {
    unsigned lo = 0xFFFFFFFFu, hi = 0u;
    int prot = 0;
    for (int j = tid; j < n; j += kThreads) {
      const unsigned key = keys[slot<kKeysInShared>(j)];
      if (key == kProtectedKey) ++prot;
      else { lo = min(lo, key); hi = max(hi, key); }
    }
    lo = __reduce_min_sync(0xFFFFFFFFu, lo);
    hi = __reduce_max_sync(0xFFFFFFFFu, hi);
    prot = __reduce_add_sync(0xFFFFFFFFu, prot);
    if (lane == 0) {
      atomicMin(&sh.key_min, lo);
      atomicMax(&sh.key_max, hi);
      if (prot) atomicAdd(&sh.protected_count, prot);
    }
  }
  __syncthreads();
  const int base = sh.base, n_protected = sh.protected_count;
  const unsigned key_min = sh.key_min, key_max = sh.key_max;
  if (tid == 0) {
    cu_keep[b + 1] = base + k;
    if (b == 0) cu_keep[0] = 0;
    if (n_protected > k && device_status) atomicOr(device_status, FASTAV_DEV_PROTECT_OVERFLOW);
  }
  if (k == 0 || n == 0) return;

  unsigned T;
  int need_eq;  // how many keys equal to T are kept (the lowest-index ones)
  if (k <= n_protected) {
    T = kProtectedKey;  // protected tokens alone fill the keep set
    need_eq = k;
  } else if (key_min == key_max) {
    T = key_min;  // every unprotected key is the same
    need_eq = k - n_protected;
  } else {
    // Radix select of the (k - #protected)-th largest unprotected key over the bits below the common prefix.
    int bits_left = 32 - __clz(key_min ^ key_max);  // >= 1
    if (tid == 0) {
      sh.prefix = bits_left == 32 ? 0u : (key_min >> bits_left) << bits_left;
      sh.remaining = k - n_protected;
    }
    while (bits_left > 0) {
      const int digit_bits = n > kShortKeys ? kDigitBits : kShortDigitBits;
      const int per_thread = (1 << digit_bits) / kThreads;  // 8 or 2 (uniform)
      const int width = min(digit_bits, bits_left), shift = bits_left - width;
      for (int i = tid; i < (1 << digit_bits); i += kThreads) sh.hist[i] = 0;
      __syncthreads();
      const unsigned prefix = sh.prefix;
      const unsigned digit_mask = (1u << width) - 1u;
      const int rounds = (n + kThreads - 1) / kThreads;
      for (int rd = 0; rd < rounds; ++rd) {
        const int j = rd * kThreads + tid;
        const unsigned key = j < n ? keys[slot<kKeysInShared>(j)] : kProtectedKey;
        // in the bucket: unprotected and equal to the prefix in the bits above this digit
        const bool in_bucket = key != kProtectedKey && (bits_left == 32 || (key >> bits_left) == (prefix >> bits_left));
        const unsigned digit = in_bucket ? ((key >> shift) & digit_mask) : 0xFFFFu;
        int same;
        __match_all_sync(0xFFFFFFFFu, digit, &same);
        if (same) {  // a run of equal scores (typically zeros): one add for the warp
          if (in_bucket && lane == 0) atomicAdd(&sh.hist[digit], 32u);
        } else if (in_bucket) {
          atomicAdd(&sh.hist[digit], 1u);
        }
      }
      __syncthreads();
      // Suffix sums over the bins, per_thread consecutive bins per thread, to find the bin holding the wanted key.
      unsigned h[kBinsPerThread];
      unsigned own = 0;
#pragma unroll
      for (int i = 0; i < kBinsPerThread; i += 2) {
        uint2 q = make_uint2(0u, 0u);
        if (i < per_thread) q = *reinterpret_cast<const uint2*>(&sh.hist[per_thread * tid + i]);
        h[i] = q.x; h[i + 1] = q.y;
        own += q.x + q.y;
      }
      unsigned incl = own;  // inclusive suffix sum over threads (higher threads = larger digits)
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const unsigned t = __shfl_down_sync(0xFFFFFFFFu, incl, d);
        if (lane + d < 32) incl += t;
      }
      if (lane == 0) sh.warp_a[warp] = incl;
      __syncthreads();
      // keys in the bins of higher warps: suffix sum of the 32 warp totals with shuffles (every warp does the same)
      unsigned suffix = sh.warp_a[lane];
      const unsigned own_total = suffix;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const unsigned t = __shfl_down_sync(0xFFFFFFFFu, suffix, d);
        if (lane + d < 32) suffix += t;
      }
      const unsigned above_warp = __shfl_sync(0xFFFFFFFFu, suffix - own_total, warp);
      const unsigned above_me = above_warp + incl - own;  // keys in bins above this thread's own
      const unsigned rem = (unsigned)sh.remaining;
      __syncthreads();  // everyone has read `remaining` before the one owner rewrites it
      if (above_me < rem && rem <= above_me + own) {
        unsigned above = above_me;  // walk this thread's bins from the top
#pragma unroll
        for (int i = kBinsPerThread - 1; i >= 0; --i) {
          if (i < per_thread && above < rem && rem <= above + h[i]) {
            sh.prefix = prefix | ((unsigned)(per_thread * tid + i) << shift);
            sh.remaining = (int)(rem - above);
            sh.bucket = (int)h[i];
            sh.list_n = 0;
          }
          above += h[i];
        }
      }
      __syncthreads();
      bits_left = shift;
      if (bits_left > 0 && sh.bucket <= kDirectMax) {
        // Few keys left in the bucket (the usual case after the first pass): collect them and let each find its
        // rank among them; the one whose rank range covers `remaining` is the threshold.
        const unsigned want = sh.prefix >> bits_left;
        for (int rd = 0; rd < rounds; ++rd) {
          const int j = rd * kThreads + tid;
          const unsigned key = j < n ? keys[slot<kKeysInShared>(j)] : kProtectedKey;
          if (key != kProtectedKey && (key >> bits_left) == want) sh.list[atomicAdd(&sh.list_n, 1)] = key;
        }
        __syncthreads();
        const int count = sh.list_n, rem_in = sh.remaining;
        __syncthreads();  // everyone has read `remaining` before an owner rewrites it
        if (tid < count) {
          const unsigned mine = sh.list[tid];
          int above = 0, not_below = 0;
          for (int i = 0; i < count; ++i) {
            const unsigned other = sh.list[i];
            above += other > mine;
            not_below += other >= mine;
          }
          if (above < rem_in && rem_in <= not_below) {  // equal keys all write the same two values
            sh.prefix = mine;
            sh.remaining = rem_in - above;
          }
        }
        __syncthreads();
        bits_left = 0;
      }
    }
    T = sh.prefix;
    need_eq = sh.remaining;
  }

  // Stable compaction in index order: thread t owns the `per` consecutive tokens starting at t * per.
  const bool global_idx = (s.flags & FASTAV_KEEP_IDX_GLOBAL) != 0;
  const int per = (n + kThreads - 1) / kThreads;
  const int j0 = tid * per, j1 = min(n, j0 + per);
  unsigned my_gt = 0, my_eq = 0;
  for (int j = j0; j < j1; ++j) {
    const unsigned key = keys[slot<kKeysInShared>(j)];
    my_gt += key > T;
    my_eq += key == T;
  }
  unsigned gt_incl = my_gt, eq_incl = my_eq;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const unsigned a = __shfl_up_sync(0xFFFFFFFFu, gt_incl, d), c = __shfl_up_sync(0xFFFFFFFFu, eq_incl, d);
    if (lane >= d) { gt_incl += a; eq_incl += c; }
  }
  if (lane == 31) { sh.warp_a[warp] = gt_incl; sh.warp_b[warp] = eq_incl; }
  __syncthreads();
  unsigned gt_before = gt_incl - my_gt, eq_before = eq_incl - my_eq;
  {  // plus the totals of the warps before this one: prefix sums of the 32 warp totals with shuffles
    unsigned pa = sh.warp_a[lane], pb = sh.warp_b[lane];
    const unsigned ta = pa, tb = pb;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const unsigned a = __shfl_up_sync(0xFFFFFFFFu, pa, d), c = __shfl_up_sync(0xFFFFFFFFu, pb, d);
      if (lane >= d) { pa += a; pb += c; }
    }
    gt_before += __shfl_sync(0xFFFFFFFFu, pa - ta, warp);
    eq_before += __shfl_sync(0xFFFFFFFFu, pb - tb, warp);
  }
  for (int j = j0; j < j1; ++j) {
    const unsigned key = keys[slot<kKeysInShared>(j)];
    const bool gt = key > T, eq = key == T;
    if (gt || (eq && (int)eq_before < need_eq)) {
      const int out = (int)gt_before + min((int)eq_before, need_eq);
      keep_idx[base + out] = global_idx ? tok0 + j : j;
    }
    gt_before += gt;
    eq_before += eq;
  }
}

// Sequences of kBlockedMinKeys < n <= kBlockedMaxKeys tokens: one block per sequence with the BLOCKED layout (see
// select_block.cuh) -- thread t owns PER consecutive tokens, the scores staged in shared memory and turned into
// keys in place, the stable scan one prefix sum over the threads.
constexpr int kBlockedMinKeys = kShortKeys;
constexpr int kBlockedMaxKeys = kThreads * 32;
using BlockedShared = SelectBlockedShared<kThreads, kDigitBits>;

template <int PER>
__global__ void __launch_bounds__(kThreads) select_topk_blocked_kernel(Shapes s, const float* __restrict__ scores,
                                                                       const int32_t* __restrict__ cu_seqlens,
                                                                       const int32_t* __restrict__ keep_counts,
                                                                       const uint8_t* __restrict__ protect,
                                                                       const int32_t* __restrict__ q_idx,
                                                                       const int32_t* __restrict__ cu_qlens,
                                                                       int32_t* __restrict__ keep_idx, int32_t* __restrict__ cu_keep,
                                                                       int32_t* device_status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  BlockedShared& shared = *reinterpret_cast<BlockedShared*>(smem_raw);
  float* stage = reinterpret_cast<float*>(smem_raw + sizeof(BlockedShared));
  pdl_trigger();
  select_sequence_blocked<kThreads, PER, kDigitBits>(
      shared, stage, s, blockIdx.x, threadIdx.x, scores, cu_seqlens, keep_counts, protect, q_idx, cu_qlens, keep_idx, cu_keep,
      device_status, [] { __syncthreads(); }, [] { pdl_wait(); /* the scores are the previous kernel's output */ });
}

template <int PER>
cudaError_t launch_blocked(const Shapes& s, const float* scores, const int32_t* cu_seqlens, const int32_t* keep_counts,
                           const uint8_t* protect, const int32_t* q_idx, const int32_t* cu_qlens, int32_t* keep_idx, int32_t* cu_keep,
                           int32_t* device_status, cudaStream_t stream) {
  const size_t smem = sizeof(BlockedShared) + ((size_t)s.max_seqlen + s.max_seqlen / 32 + 1) * sizeof(float);
  cudaError_t e = cudaFuncSetAttribute(select_topk_blocked_kernel<PER>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 1024);
  if (e != cudaSuccess) return e;
  return launch_chained(select_topk_blocked_kernel<PER>, dim3(s.batch), dim3(kThreads), smem, stream, s, scores, cu_seqlens,
                        keep_counts, protect, q_idx, cu_qlens, keep_idx, cu_keep, device_status);
}

}  // namespace

cudaError_t launch_select(const Shapes& s, const Workspace& w, const float* scores, const int32_t* cu_seqlens,
                          const int32_t* keep_counts, const uint8_t* protect, const int32_t* q_idx,
                          const int32_t* cu_qlens, int32_t* keep_idx, int32_t* cu_keep, unsigned char* ws,
                          int32_t* device_status, cudaStream_t stream) {
  const size_t fixed = sizeof(SelectShared);
  const size_t want = fixed + ((size_t)s.max_seqlen + s.max_seqlen / 32 + 1) * sizeof(unsigned);
  constexpr size_t kMaxDynamic = 227 * 1024 - 1024;
  cudaError_t e;
  if (s.max_seqlen > kBlockedMinKeys && s.max_seqlen <= kBlockedMaxKeys) {
    // the fewest tokens per thread that cover the longest sequence: all 1024 threads share the work
    if (s.max_seqlen <= kThreads * 4) e = launch_blocked<4>(s, scores, cu_seqlens, keep_counts, protect, q_idx, cu_qlens, keep_idx, cu_keep, device_status, stream);
    else if (s.max_seqlen <= kThreads * 8) e = launch_blocked<8>(s, scores, cu_seqlens, keep_counts, protect, q_idx, cu_qlens, keep_idx, cu_keep, device_status, stream);
    else if (s.max_seqlen <= kThreads * 16) e = launch_blocked<16>(s, scores, cu_seqlens, keep_counts, protect, q_idx, cu_qlens, keep_idx, cu_keep, device_status, stream);
    else e = launch_blocked<32>(s, scores, cu_seqlens, keep_counts, protect, q_idx, cu_qlens, keep_idx, cu_keep, device_status, stream);
  } else if (want <= kMaxDynamic) {
    e = cudaFuncSetAttribute(select_topk_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxDynamic);
    if (e != cudaSuccess) return e;
    e = launch_chained(select_topk_kernel<true, false>, dim3(s.batch), dim3(kThreads), want, stream, s, scores, cu_seqlens,
                       keep_counts, protect, q_idx, cu_qlens, keep_idx, cu_keep, (unsigned*)nullptr, device_status, FromLogits{});
  } else {
    e = launch_chained(select_topk_kernel<false, false>, dim3(s.batch), dim3(kThreads), fixed, stream, s, scores, cu_seqlens,
                       keep_counts, protect, q_idx, cu_qlens, keep_idx, cu_keep, reinterpret_cast<unsigned*>(ws + w.keys_off),
                       device_status, FromLogits{});
  }
  count_launches(1);
  return e != cudaSuccess ? e : cudaGetLastError();
}

// Scores (and, with `do_select`, the keep list) of a batch of short sequences with few scored rows, straight
// from the logits in the workspace.
bool narrow_tail_applies(const Shapes& s) {
  const size_t smem = sizeof(SelectShared) + ((size_t)s.max_seqlen + s.max_seqlen / 32 + 1) * sizeof(unsigned) +
                      (size_t)s.hq * s.max_qlen * (sizeof(float) + sizeof(int));
  // one block per sequence does all of it: worth it only while a sequence is short (measured: up to about 1k tokens)
  return s.max_qlen >= 1 && s.max_qlen <= kNarrowMaxRows && s.max_seqlen >= 1 && s.max_seqlen <= 1024 && smem <= 200 * 1024;
}

cudaError_t launch_narrow_tail(const Shapes& s, const float* logits, int rq, float* scores_out, bool do_select,
                               const int32_t* cu_seqlens, const int32_t* keep_counts, const uint8_t* protect,
                               const int32_t* q_idx, const int32_t* cu_qlens, int32_t* keep_idx, int32_t* cu_keep,
                               int32_t* device_status, cudaStream_t stream) {
  const size_t smem = sizeof(SelectShared) + ((size_t)s.max_seqlen + s.max_seqlen / 32 + 1) * sizeof(unsigned) +
                      (size_t)s.hq * rq * (sizeof(float) + sizeof(int));  // keys, log-sum-exp per term, term offsets
  cudaError_t e = cudaFuncSetAttribute(select_topk_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  if (e != cudaSuccess) return e;
  e = launch_chained(select_topk_kernel<true, true>, dim3(s.batch), dim3(kThreads), smem, stream, s, (const float*)nullptr,
                     cu_seqlens, keep_counts, protect, q_idx, cu_qlens, keep_idx, cu_keep, (unsigned*)nullptr, device_status,
                     FromLogits{logits, scores_out, rq, do_select ? 1 : 0});
  count_launches(1);
  return e != cudaSuccess ? e : cudaGetLastError();
}

// ---- keep set given as a mask (the paper's positional global rule) ---------------------------------
namespace {

// counts[b] = number of kept tokens of sequence b.
__global__ void __launch_bounds__(256) mask_count_kernel(Shapes s, const uint8_t* __restrict__ keep_mask,
                                                         const int32_t* __restrict__ cu_seqlens, int32_t* __restrict__ counts) {
  __shared__ int warp_sums[8];
  pdl_trigger();
  pdl_wait();
  pdl_acquire(keep_mask);
  const int b = blockIdx.x;
  const Span seq = checked_span(cu_seqlens, b, s.total_tokens, s.total_tokens);
  const int tok0 = seq.first, n = seq.count;
  int c = 0;
  for (int j = threadIdx.x; j < n; j += 256) c += keep_mask[tok0 + j] != 0;
  c = __reduce_add_sync(0xFFFFFFFFu, c);
  if ((threadIdx.x & 31) == 0) warp_sums[threadIdx.x >> 5] = c;
  __syncthreads();
  if (threadIdx.x == 0) {
    int total = 0;
    for (int w = 0; w < 8; ++w) total += warp_sums[w];
    counts[b] = total;
  }
}

// Survivors of sequence b in ascending order, after those of the sequences before it.
__global__ void __launch_bounds__(kThreads) mask_emit_kernel(Shapes s, const uint8_t* __restrict__ keep_mask,
                                                             const int32_t* __restrict__ cu_seqlens,
                                                             const int32_t* __restrict__ counts, int32_t* __restrict__ keep_idx,
                                                             int32_t* __restrict__ cu_keep, int32_t* device_status) {
  __shared__ unsigned warp_a[kWarps];
  __shared__ int base_sh;
  pdl_trigger();
  pdl_wait();
  pdl_acquire(counts);
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const Span seq = checked_span(cu_seqlens, b, s.total_tokens, s.total_tokens);
  const int tok0 = seq.first, n = seq.count;
  if (tid == 0 && seq.bad && device_status) atomicOr(device_status, FASTAV_DEV_SHAPE_MISMATCH);
  if (tid == 0) base_sh = 0;
  __syncthreads();
  int part = 0;
  for (int i = tid; i < b; i += kThreads) part += chain_load(counts + i);
  if (part) atomicAdd(&base_sh, part);
  __syncthreads();
  const int base = base_sh;
  if (tid == 0) {
    const int mine = chain_load(counts + b);
    cu_keep[b + 1] = min(base + mine, s.total_keep);
    if (b == 0) cu_keep[0] = 0;
    if (base + mine > s.total_keep && device_status) atomicOr(device_status, FASTAV_DEV_K_CLAMPED);
  }
  const bool global_idx = (s.flags & FASTAV_KEEP_IDX_GLOBAL) != 0;
  const int per = (n + kThreads - 1) / kThreads;
  const int j0 = min(n, tid * per), j1 = min(n, j0 + per);
  unsigned mine = 0;
  for (int j = j0; j < j1; ++j) mine += keep_mask[tok0 + j] != 0;
  unsigned incl = mine;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const unsigned t = __shfl_up_sync(0xFFFFFFFFu, incl, d);
    if (lane >= d) incl += t;
  }
  if (lane == 31) warp_a[warp] = incl;
  __syncthreads();
  unsigned before = incl - mine;
  for (int w = 0; w < warp; ++w) before += warp_a[w];
  for (int j = j0; j < j1; ++j)
    if (keep_mask[tok0 + j]) {
      const int out = base + (int)before++;
      if (out < s.total_keep) keep_idx[out] = global_idx ? tok0 + j : j;  // never past the caller's buffer
    }
}

}  // namespace
}  // namespace fastav

extern "C" int32_t fastav_select_mask(const fastav_params* p, const uint8_t* keep_mask, const int32_t* cu_seqlens,
                                      int32_t* keep_idx_out, int32_t* cu_keep_out, void* workspace, size_t workspace_bytes,
                                      int32_t* device_status, void* stream) {
  fastav::chain_begin(p ? p->flags : 0u);
  using namespace fastav;
  if (!p || p->batch < 1 || p->total_tokens < 0 || p->total_keep < 0 || p->total_keep > p->total_tokens) return FASTAV_ERR_INVALID_ARG;
  if (!cu_seqlens || !cu_keep_out || (p->total_tokens > 0 && !keep_mask) || (p->total_keep > 0 && !keep_idx_out))
    return FASTAV_ERR_INVALID_ARG;
  const size_t need = align_up((size_t)p->batch * sizeof(int32_t), 256);
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < need) return FASTAV_ERR_WORKSPACE;
  Shapes s{};
  s.batch = p->batch; s.total_tokens = p->total_tokens; s.max_seqlen = p->max_seqlen; s.total_keep = p->total_keep;
  s.flags = p->flags;
  int32_t* counts = static_cast<int32_t*>(workspace);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e = launch_chained(mask_count_kernel, dim3(s.batch), dim3(256), 0, st, s, keep_mask, cu_seqlens, counts);
  if (e == cudaSuccess)
    e = launch_chained(mask_emit_kernel, dim3(s.batch), dim3(kThreads), 0, st, s, keep_mask, cu_seqlens, (const int32_t*)counts,
                       keep_idx_out, cu_keep_out, device_status);
  count_launches(2);
  return e == cudaSuccess && cudaGetLastError() == cudaSuccess ? FASTAV_OK : FASTAV_ERR_CUDA;
}

namespace fastav {

// ---- fastav_select_noalloc: the same selection with its scratch inside the library ----------
//
// The radix select keeps one 32-bit key per token.  fastav_select puts them in shared memory or in
// the caller's workspace; this variant always puts them in the array below, so a caller that owns
// no device scratch (and may not obtain any) can still run the step.  The array lives in every
// CUDA context that loads the library, from load to exit.
namespace {

static __device__ __align__(256) unsigned g_noalloc_keys[FASTAV_NOALLOC_MAX_TOKENS];

constexpr int kMaxDevices = 64;
std::mutex g_noalloc_mutex;
unsigned* g_noalloc_ptr[kMaxDevices] = {};  // device address of g_noalloc_keys, per device ordinal

// Device address of the scratch array on the current device.  In host code `g_noalloc_keys` is only
// a handle for the symbol, not an address a kernel may use: the runtime translates it, once per
// device, with that device current.
cudaError_t noalloc_scratch(unsigned** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  if (!g_noalloc_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_keys);
    if (e != cudaSuccess) return e;
    g_noalloc_ptr[dev] = static_cast<unsigned*>(p);
  }
  *out = g_noalloc_ptr[dev];
  return cudaSuccess;
}

}  // namespace
}  // namespace fastav

extern "C" int32_t fastav_select_noalloc(const fastav_params* p, const float* scores, const int32_t* cu_seqlens,
                                         const int32_t* keep_counts, const uint8_t* protect_opt, const int32_t* q_idx,
                                         const int32_t* cu_qlens, int32_t* keep_idx_out, int32_t* cu_keep_out,
                                         int32_t* device_status, void* stream) {
  fastav::chain_begin(p ? p->flags : 0u);
  using namespace fastav;
  if (!p || p->batch < 1 || p->total_tokens < 0 || p->max_seqlen < 0 || p->max_seqlen > p->total_tokens ||
      p->total_keep < 0 || p->total_keep > p->total_tokens || p->total_q < 0)
    return FASTAV_ERR_INVALID_ARG;
  if (p->total_tokens > FASTAV_NOALLOC_MAX_TOKENS) return FASTAV_ERR_UNSUPPORTED;  // beyond the built-in scratch
  if (!cu_seqlens || !keep_counts || !cu_keep_out) return FASTAV_ERR_INVALID_ARG;
  if (p->total_tokens > 0 && !scores) return FASTAV_ERR_INVALID_ARG;
  if (p->total_keep > 0 && !keep_idx_out) return FASTAV_ERR_INVALID_ARG;
  if ((p->flags & FASTAV_PROTECT_QUERY_ROWS) && (!cu_qlens || (p->total_q > 0 && !q_idx))) return FASTAV_ERR_INVALID_ARG;
  unsigned* keys = nullptr;
  if (noalloc_scratch(&keys) != cudaSuccess || !keys) return FASTAV_ERR_CUDA;
  Shapes s{};
  s.batch = p->batch; s.total_tokens = p->total_tokens; s.max_seqlen = p->max_seqlen;
  s.total_q = p->total_q; s.max_qlen = p->max_qlen; s.total_keep = p->total_keep; s.max_keep = p->max_keep;
  s.flags = p->flags;
  // Every key a block reads was written by that block earlier in the same launch, so what an
  // earlier call left in the array never matters and nothing has to be cleared.
  select_topk_kernel<false, false><<<s.batch, kThreads, sizeof(SelectShared), static_cast<cudaStream_t>(stream)>>>(
      s, scores, cu_seqlens, keep_counts, protect_opt, q_idx, cu_qlens, keep_idx_out, cu_keep_out, keys, device_status, FromLogits{});
  count_launches(1);
  return cudaGetLastError() == cudaSuccess ? FASTAV_OK : FASTAV_ERR_CUDA;
}
