// Top-k keep set of ONE sequence by one thread block (the bottom-P % rule of Section 2.2, "Fine pruning", stated as
// "keep the k best"; ties to the lower index).  Scores become order-preserving 32-bit keys (protected tokens get
// the largest key); min/max of the unprotected keys gives their common leading bits; one MSB-first histogram pass
// of DIGIT_BITS-bit digits over the bits below, then the direct finish on the chosen bin (its keys are collected and
// each finds its rank among them by counting; further passes only if the bin holds more than kDirectMax keys);
// then ONE stable scan in index order.  Integer work throughout: the result is a unique function of the fp32
// score bits.
#pragma once

#include "common.cuh"

namespace fastav {

constexpr unsigned kProtectedKey = 0xFFFFFFFFu;
constexpr int kDirectMax = 256;  // a bucket of at most this many keys is finished by counting ranks, not by more passes

// fp32 -> uint32 with the same ordering as the float comparison (-0 and +0 compare equal).
__device__ __forceinline__ unsigned order_key(float x) {
  if (x == 0.0f) x = 0.0f;
  const unsigned u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// BLOCKED layout: thread t owns the PER consecutive tokens PER t .. PER t + PER - 1.
//
// The scores are staged in shared memory with coalesced loads (one word of padding per 32 keeps the blocked reads free
// of bank conflicts) and turned into keys in place; every later step is a short loop of a thread over its own
// keys in token order.  That makes the stable scan trivial -- per-thread counts, one prefix scan over the
// threads, then each thread writes its survivors as one run -- where a strided layout (thread t holding tokens
// t, t + THREADS, ...) needs a vote per key and a scan over (round, warp) cells; protection (mask and scored rows alike) is a few bits of one 32-bit word per
// thread; and runs of equal keys inside a thread (typically zeros) cost one histogram update.  The loops are
// deliberately NOT unrolled over a thread's keys: the selection runs once per sequence, so straight-line code would be fetched
// from memory once and never reused, and instruction fetch, not arithmetic, would set its speed.
template <int THREADS, int DIGIT_BITS>
struct alignas(16) SelectBlockedShared {
  static constexpr int kBins = 1 << DIGIT_BITS;
  unsigned hist[kBins];
  unsigned warp_a[32], warp_b[32];
  unsigned key_min, key_max;
  unsigned prefix;
  int remaining, base, protected_count, bucket, list_n;
  unsigned list[kDirectMax];
  unsigned prot_bits[THREADS];  // bit j of the array: token j is protected (at most 32 THREADS tokens)
};

// `stage` holds at least n + n / 32 + 1 floats of shared memory.  n <= PER * THREADS; PER divides 32.
// `scores_ready()` is called once, after the caller-provided index arrays have been read and before the first
// score is loaded (a kernel launched programmatically waits for its predecessor there).
template <int THREADS, int PER, int DIGIT_BITS, typename Sync, typename Ready>
__device__ __forceinline__ void select_sequence_blocked(SelectBlockedShared<THREADS, DIGIT_BITS>& sh, float* stage, const Shapes& s, int b,
                                                        int tid, const float* scores, const int32_t* cu_seqlens,
                                                        const int32_t* keep_counts, const uint8_t* protect, const int32_t* q_idx,
                                                        const int32_t* cu_qlens, int32_t* keep_idx, int32_t* cu_keep,
                                                        int32_t* device_status, Sync sync, Ready scores_ready) {
  using Sh = SelectBlockedShared<THREADS, DIGIT_BITS>;
  constexpr int kBins = Sh::kBins, kWarps = THREADS / 32, kPer = PER;
  static_assert(32 % PER == 0, "a thread's tokens lie inside one 32-token word");
  constexpr int kBinsPerThread = kBins / THREADS;
  static_assert(kBins % THREADS == 0 && kBinsPerThread % 4 == 0, "every thread owns whole 16-byte groups of bins");
  const int lane = tid & 31, warp = tid >> 5;
  const Span seq = seq_span(s, cu_seqlens, b);
  const int tok0 = seq.first, n = min(seq.count, THREADS * kPer);
  const bool by_rows = (s.flags & FASTAV_PROTECT_QUERY_ROWS) != 0;

  if (tid == 0) { sh.base = 0; sh.protected_count = 0; sh.key_min = 0xFFFFFFFFu; sh.key_max = 0u; }
  for (int i = tid; i < kBins; i += THREADS) sh.hist[i] = 0u;
  sh.prot_bits[tid] = 0u;
  sync();
  {
    int part = 0;
    bool clamped = false, mismatch = false;
    for (int i = tid; i <= b; i += THREADS) {
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
  if (by_rows) {
    const Span rows = checked_span(cu_qlens, b, s.total_q, s.total_q);
    for (int r = rows.first + tid; r < rows.first + rows.count; r += THREADS) {
      const int j = q_idx[r];
      if (j >= 0 && j < n) atomicOr(&sh.prot_bits[j >> 5], 1u << (j & 31));
    }
  }
  int k = keep_counts[b];
  k = k < 0 ? 0 : (k > n ? n : k);
  scores_ready();
  pdl_acquire(scores);
  // Stage the scores (and fold the protect mask into the protection bits): coalesced, several loads in flight.
  for (int j0 = tid; j0 < n; j0 += THREADS * 8) {
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int j = j0 + u * THREADS;
      v[u] = j < n ? chain_load(scores + tok0 + j) : 0.f;
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int j = j0 + u * THREADS;
      if (j < n) stage[j + (j >> 5)] = v[u];  // (turned into a key in place below)
    }
  }
  if (protect) {
    for (int j0 = warp * 32; j0 < n; j0 += THREADS) {  // a warp covers tokens j0 .. j0 + 31: one word
      const int j = j0 + lane;
      const unsigned word = __ballot_sync(0xFFFFFFFFu, j < n && protect[tok0 + j] != 0);
      if (lane == 0 && word) atomicOr(&sh.prot_bits[j0 >> 5], word);
    }
  }
  sync();

  const int j_first = tid * kPer;
  const int mine = max(0, min(kPer, n - j_first));  // tokens of this thread that exist
  const unsigned prot = sh.prot_bits[j_first >> 5] >> (j_first & 31);  // bit u: token j_first + u is protected
  const bool lowest = (s.flags & FASTAV_SELECT_LOWEST) != 0;
  unsigned* const key = reinterpret_cast<unsigned*>(stage) + j_first + (j_first >> 5);  // key[u]: the padded slot of token j_first + u
  {
    unsigned lo = 0xFFFFFFFFu, hi = 0u;
    int n_prot = 0;
#pragma unroll 4
    for (int u = 0; u < mine; ++u) {
      const float v = __uint_as_float(key[u]);
      unsigned x = order_key(lowest ? -v : v);
      if (x == kProtectedKey) x = kProtectedKey - 1;  // only a NaN pattern lands here
      if ((prot >> u) & 1u) x = kProtectedKey;
      if (x == kProtectedKey) ++n_prot;
      else { lo = min(lo, x); hi = max(hi, x); }
      key[u] = x;
    }
    lo = __reduce_min_sync(0xFFFFFFFFu, lo);
    hi = __reduce_max_sync(0xFFFFFFFFu, hi);
    n_prot = __reduce_add_sync(0xFFFFFFFFu, n_prot);
    if (lane == 0) {
      atomicMin(&sh.key_min, lo);
      atomicMax(&sh.key_max, hi);
      if (n_prot) atomicAdd(&sh.protected_count, n_prot);
    }
  }
  sync();
  const int base = sh.base, n_protected = sh.protected_count;
  const unsigned key_min = sh.key_min, key_max = sh.key_max;
  if (tid == 0) {
    cu_keep[b + 1] = base + k;
    if (b == 0) cu_keep[0] = 0;
    if (n_protected > k && device_status) atomicOr(device_status, FASTAV_DEV_PROTECT_OVERFLOW);
  }
  if (k == 0 || n == 0) return;  // uniform for the group

  unsigned T;
  int need_eq;
  if (k <= n_protected) {
    T = kProtectedKey;
    need_eq = k;
  } else if (key_min == key_max) {
    T = key_min;
    need_eq = k - n_protected;
  } else {
    int bits_left = 32 - __clz(key_min ^ key_max);  // >= 1
    if (tid == 0) {
      sh.prefix = bits_left == 32 ? 0u : (key_min >> bits_left) << bits_left;
      sh.remaining = k - n_protected;
    }
    sync();
    for (int pass = 0; bits_left > 0; ++pass) {
      const int width = min(DIGIT_BITS, bits_left), shift = bits_left - width;
      if (pass > 0) {
        for (int i = tid; i < kBins; i += THREADS) sh.hist[i] = 0u;
        sync();
      }
      const unsigned prefix = sh.prefix;
      const unsigned digit_mask = (1u << width) - 1u;
      const unsigned above_want = __funnelshift_rc(prefix, 0u, bits_left);
      {
        unsigned run_digit = 0xFFFFFFFFu, run_len = 0u;  // equal digits of consecutive tokens: one update
#pragma unroll 4
        for (int u = 0; u < mine; ++u) {
          const unsigned x = key[u];
          const bool in_bucket = x != kProtectedKey && __funnelshift_rc(x, 0u, bits_left) == above_want;
          const unsigned digit = in_bucket ? ((x >> shift) & digit_mask) : 0xFFFFFFFFu;
          if (digit != run_digit) {
            if (run_len) atomicAdd(&sh.hist[run_digit], run_len);
            run_digit = digit;
            run_len = 0u;
          }
          if (in_bucket) ++run_len;
        }
        if (run_len) atomicAdd(&sh.hist[run_digit], run_len);
      }
      sync();
      unsigned h[kBinsPerThread];
      unsigned own = 0;
#pragma unroll
      for (int i = 0; i < kBinsPerThread; i += 4) {
        const uint4 q = *reinterpret_cast<const uint4*>(&sh.hist[kBinsPerThread * tid + i]);
        h[i] = q.x; h[i + 1] = q.y; h[i + 2] = q.z; h[i + 3] = q.w;
        own += q.x + q.y + q.z + q.w;
      }
      unsigned incl = own;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const unsigned t = __shfl_down_sync(0xFFFFFFFFu, incl, d);
        if (lane + d < 32) incl += t;
      }
      if (lane == 0) sh.warp_a[warp] = incl;
      sync();
      unsigned suffix = lane < kWarps ? sh.warp_a[lane] : 0u;
      const unsigned own_total = suffix;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const unsigned t = __shfl_down_sync(0xFFFFFFFFu, suffix, d);
        if (lane + d < 32) suffix += t;
      }
      const unsigned above_warp = __shfl_sync(0xFFFFFFFFu, suffix - own_total, warp);
      const unsigned above_me = above_warp + incl - own;
      const unsigned rem = (unsigned)sh.remaining;
      sync();  // everyone has read `remaining` (and warp_a) before the one owner rewrites it
      if (above_me < rem && rem <= above_me + own) {
        unsigned above = above_me;
#pragma unroll
        for (int i = kBinsPerThread - 1; i >= 0; --i) {
          if (above < rem && rem <= above + h[i]) {
            sh.prefix = prefix | ((unsigned)(kBinsPerThread * tid + i) << shift);
            sh.remaining = (int)(rem - above);
            sh.bucket = (int)h[i];
            sh.list_n = 0;
          }
          above += h[i];
        }
      }
      sync();
      bits_left = shift;
      if (bits_left > 0 && sh.bucket <= kDirectMax) {
        const unsigned want = sh.prefix >> bits_left;
#pragma unroll 4
        for (int u = 0; u < mine; ++u) {
          const unsigned x = key[u];
          if (x != kProtectedKey && (x >> bits_left) == want) sh.list[atomicAdd(&sh.list_n, 1)] = x;
        }
        sync();
        const int count = sh.list_n, rem_in = sh.remaining;
        sync();  // everyone has read `remaining` before an owner rewrites it
        if (tid < count) {
          const unsigned me = sh.list[tid];
          int above = 0, not_below = 0;
          for (int i = 0; i < count; ++i) {
            const unsigned other = sh.list[i];
            above += other > me;
            not_below += other >= me;
          }
          if (above < rem_in && rem_in <= not_below) {  // equal keys all write the same two values
            sh.prefix = me;
            sh.remaining = rem_in - above;
          }
        }
        sync();
        bits_left = 0;
      }
    }
    T = sh.prefix;
    need_eq = sh.remaining;
  }

  // Stable compaction: per-thread counts, one exclusive scan over the threads, each thread writes its run.
  // (A token that does not exist carries the protected key: it is left out by its index.)
  unsigned my_gt = 0, my_eq = 0;
#pragma unroll 4
  for (int u = 0; u < mine; ++u) {
    const unsigned x = key[u];
    my_gt += x > T ? 1u : 0u;
    my_eq += x == T ? 1u : 0u;
  }
  unsigned gt_incl = my_gt, eq_incl = my_eq;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const unsigned ga = __shfl_up_sync(0xFFFFFFFFu, gt_incl, d), ea = __shfl_up_sync(0xFFFFFFFFu, eq_incl, d);
    if (lane >= d) { gt_incl += ga; eq_incl += ea; }
  }
  if (lane == 31) { sh.warp_a[warp] = gt_incl; sh.warp_b[warp] = eq_incl; }
  sync();
  unsigned gt_before = gt_incl - my_gt, eq_before = eq_incl - my_eq;
  {
    unsigned pa = lane < kWarps ? sh.warp_a[lane] : 0u, pb = lane < kWarps ? sh.warp_b[lane] : 0u;
    const unsigned ta = pa, tb = pb;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const unsigned ga = __shfl_up_sync(0xFFFFFFFFu, pa, d), ea = __shfl_up_sync(0xFFFFFFFFu, pb, d);
      if (lane >= d) { pa += ga; pb += ea; }
    }
    gt_before += __shfl_sync(0xFFFFFFFFu, pa - ta, warp);
    eq_before += __shfl_sync(0xFFFFFFFFu, pb - tb, warp);
  }
  const bool global_idx = (s.flags & FASTAV_KEEP_IDX_GLOBAL) != 0;
#pragma unroll 4
  for (int u = 0; u < mine; ++u) {
    const unsigned x = key[u];
    const bool gt = x > T, eq = x == T;
    if (gt || (eq && (int)eq_before < need_eq))
      keep_idx[base + (int)gt_before + min((int)eq_before, need_eq)] = global_idx ? tok0 + j_first + u : j_first + u;
    gt_before += gt;
    eq_before += eq;
  }
}

}  // namespace fastav
