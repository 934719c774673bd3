// Top-k keep set per sequence: "tokens with the lowest P% scores are removed" (Section 2.2).
//
// One thread block per sequence.  Scores become order-preserving 32-bit keys (protected tokens get
// the largest key), held in shared memory when the sequence fits.  The k-th largest key T is found
// by an MSB-first radix select (4 passes of 8 bits, shared-memory histograms fed by warp-aggregated
// atomics).  A block-wide prefix scan in index order then keeps every key above T plus the first
// (k - #above) keys equal to T: ties go to the lower index and survivors come out ascending, which
// is exactly the order the gather that follows needs.  Integer work throughout: the result is a
// unique function of the fp32 score bits.
#include <mutex>

#include "common.cuh"

namespace fastav {
namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr unsigned kProtectedKey = 0xFFFFFFFFu;

// fp32 -> uint32 with the same ordering as the float comparison (-0 and +0 compare equal).
__device__ __forceinline__ unsigned order_key(float x) {
  if (x == 0.0f) x = 0.0f;
  const unsigned u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct SelectShared {
  unsigned hist[256];
  unsigned warp_totals[2][kWarps];
  unsigned prefix;      // bits of T fixed so far
  int remaining;        // how many more keys (from the top of the current bucket) are still to take
  int base;             // output offset of this sequence
  int protected_count;
};

template <bool kKeysInShared>
__global__ void __launch_bounds__(kThreads) select_topk_kernel(Shapes s, const float* __restrict__ scores,
                                                               const int32_t* __restrict__ cu_seqlens,
                                                               const int32_t* __restrict__ keep_counts,
                                                               const uint8_t* __restrict__ protect,
                                                               const int32_t* __restrict__ q_idx,
                                                               const int32_t* __restrict__ cu_qlens,
                                                               int32_t* __restrict__ keep_idx, int32_t* __restrict__ cu_keep,
                                                               unsigned* __restrict__ keys_global, int32_t* device_status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  SelectShared& sh = *reinterpret_cast<SelectShared*>(smem_raw);
  unsigned* keys = kKeysInShared ? reinterpret_cast<unsigned*>(smem_raw + sizeof(SelectShared)) : nullptr;

  pdl_trigger();
  pdl_wait();  // the scores are the previous kernel's output
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int tok0 = cu_seqlens[b], n = cu_seqlens[b + 1] - tok0;
  if (!kKeysInShared) keys = keys_global + tok0;

  // Output offset: prefix sum of the clamped keep counts of the sequences before this one.
  if (tid == 0) { sh.base = 0; sh.protected_count = 0; }
  __syncthreads();
  {
    int part = 0;
    bool clamped = false;
    for (int i = tid; i <= b; i += kThreads) {
      const int ni = cu_seqlens[i + 1] - cu_seqlens[i];
      int ki = keep_counts[i];
      if (ki < 0 || ki > ni) { clamped = true; ki = ki < 0 ? 0 : ni; }
      if (i < b) part += ki;
    }
    if (part) atomicAdd(&sh.base, part);
    if (clamped && device_status) atomicOr(device_status, FASTAV_DEV_K_CLAMPED);
  }
  int k = keep_counts[b];
  k = k < 0 ? 0 : (k > n ? n : k);

  // Keys.
  for (int j = tid; j < n; j += kThreads) {
    unsigned key = order_key(scores[tok0 + j]);
    if (key == kProtectedKey) key = kProtectedKey - 1;  // only a NaN pattern lands here
    if (protect && protect[tok0 + j]) key = kProtectedKey;
    keys[j] = key;
  }
  __syncthreads();
  if (s.flags & FASTAV_PROTECT_QUERY_ROWS) {
    for (int r = cu_qlens[b] + tid; r < cu_qlens[b + 1]; r += kThreads) {
      const int j = q_idx[r];
      if (j >= 0 && j < n) keys[j] = kProtectedKey;
    }
    __syncthreads();
  }
  const int base = sh.base;
  if (tid == 0) {
    cu_keep[b + 1] = base + k;
    if (b == 0) cu_keep[0] = 0;
    sh.prefix = 0;
    sh.remaining = k;
  }
  if (k == 0 || n == 0) return;

  // Radix select: after pass p the top 8(p+1) bits of T are known.
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    for (int i = tid; i < 256; i += kThreads) sh.hist[i] = 0;
    __syncthreads();
    const unsigned prefix = sh.prefix;
    const unsigned high_mask = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
    const int rounds = (n + kThreads - 1) / kThreads;
    for (int rd = 0; rd < rounds; ++rd) {
      const int j = rd * kThreads + tid;
      const bool in_bucket = j < n && ((keys[j] & high_mask) == prefix);
      const unsigned digit = in_bucket ? ((keys[j] >> shift) & 0xFFu) : 0x100u;
      const unsigned peers = __match_any_sync(0xFFFFFFFFu, digit);
      if (in_bucket && lane == (__ffs(peers) - 1)) atomicAdd(&sh.hist[digit], (unsigned)__popc(peers));
    }
    __syncthreads();
    if (warp == 0) {
      // Walk the 256 bins from the top; lane l owns bins [8l, 8l+8).
      unsigned local[8], sum = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) { local[i] = sh.hist[lane * 8 + i]; sum += local[i]; }
      unsigned above = sum;  // inclusive suffix sum over lanes (higher lanes = larger digits)
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const unsigned t = __shfl_down_sync(0xFFFFFFFFu, above, d);
        if (lane + d < 32) above += t;
      }
      const unsigned rem = (unsigned)sh.remaining;
      const unsigned strictly_above = above - sum;  // keys in bins of higher lanes
      if (strictly_above < rem && rem <= above) {   // the k-th key falls in one of this lane's bins
        unsigned acc = strictly_above;
        for (int i = 7; i >= 0; --i) {
          if (acc + local[i] >= rem) {
            sh.prefix = prefix | ((unsigned)(lane * 8 + i) << shift);
            sh.remaining = (int)(rem - acc);
            break;
          }
          acc += local[i];
        }
      }
    }
    __syncthreads();
  }
  const unsigned T = sh.prefix;
  const int need_eq = sh.remaining;  // how many keys equal to T are kept (the lowest-index ones)

  // Stable compaction in index order.
  int run_gt = 0, run_eq = 0;
  const bool global_idx = (s.flags & FASTAV_KEEP_IDX_GLOBAL) != 0;
  const int rounds = (n + kThreads - 1) / kThreads;
  for (int rd = 0; rd < rounds; ++rd) {
    const int j = rd * kThreads + tid;
    const unsigned key = j < n ? keys[j] : 0u;
    const bool gt = j < n && key > T, eq = j < n && key == T;
    const unsigned m_gt = __ballot_sync(0xFFFFFFFFu, gt), m_eq = __ballot_sync(0xFFFFFFFFu, eq);
    const unsigned lt_mask = (1u << lane) - 1u;
    unsigned* totals = sh.warp_totals[rd & 1];
    if (lane == 0) totals[warp] = (unsigned)__popc(m_gt) | ((unsigned)__popc(m_eq) << 16);
    __syncthreads();
    unsigned incl = totals[lane];  // packed (gt, eq) counts never exceed 1024 per round: no carry between halves
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const unsigned t = __shfl_up_sync(0xFFFFFFFFu, incl, d);
      if (lane >= d) incl += t;
    }
    const unsigned round_total = __shfl_sync(0xFFFFFFFFu, incl, 31);
    const unsigned before_warp = warp == 0 ? 0u : __shfl_sync(0xFFFFFFFFu, incl, warp - 1);
    const int gt_before = run_gt + (int)(before_warp & 0xFFFFu) + __popc(m_gt & lt_mask);
    const int eq_before = run_eq + (int)(before_warp >> 16) + __popc(m_eq & lt_mask);
    if (gt || (eq && eq_before < need_eq)) {
      const int out = gt_before + (eq_before < need_eq ? eq_before : need_eq);
      keep_idx[base + out] = global_idx ? tok0 + j : j;
    }
    if (key == kProtectedKey && j < n) atomicAdd(&sh.protected_count, 1);
    run_gt += (int)(round_total & 0xFFFFu);
    run_eq += (int)(round_total >> 16);
  }
  __syncthreads();
  if (tid == 0 && sh.protected_count > k && device_status) atomicOr(device_status, FASTAV_DEV_PROTECT_OVERFLOW);
}

}  // namespace

cudaError_t launch_select(const Shapes& s, const Workspace& w, const float* scores, const int32_t* cu_seqlens,
                          const int32_t* keep_counts, const uint8_t* protect, const int32_t* q_idx,
                          const int32_t* cu_qlens, int32_t* keep_idx, int32_t* cu_keep, unsigned char* ws,
                          int32_t* device_status, cudaStream_t stream) {
  const size_t fixed = sizeof(SelectShared);
  const size_t want = fixed + (size_t)s.max_seqlen * sizeof(unsigned);
  constexpr size_t kMaxDynamic = 227 * 1024 - 1024;
  cudaError_t e;
  if (want <= kMaxDynamic) {
    e = cudaFuncSetAttribute(select_topk_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kMaxDynamic);
    if (e != cudaSuccess) return e;
    e = launch_chained(select_topk_kernel<true>, dim3(s.batch), dim3(kThreads), want, stream, s, scores, cu_seqlens, keep_counts,
                       protect, q_idx, cu_qlens, keep_idx, cu_keep, (unsigned*)nullptr, device_status);
  } else {
    e = launch_chained(select_topk_kernel<false>, dim3(s.batch), dim3(kThreads), fixed, stream, s, scores, cu_seqlens, keep_counts,
                       protect, q_idx, cu_qlens, keep_idx, cu_keep, reinterpret_cast<unsigned*>(ws + w.keys_off), device_status);
  }
  count_launches(1);
  return e != cudaSuccess ? e : cudaGetLastError();
}

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
  select_topk_kernel<false><<<s.batch, kThreads, sizeof(SelectShared), static_cast<cudaStream_t>(stream)>>>(
      s, scores, cu_seqlens, keep_counts, protect_opt, q_idx, cu_qlens, keep_idx_out, cu_keep_out, keys, device_status);
  count_launches(1);
  return cudaGetLastError() == cudaSuccess ? FASTAV_OK : FASTAV_ERR_CUDA;
}
