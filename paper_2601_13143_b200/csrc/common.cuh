// Internal declarations shared by the kernels and the C-ABI layer.  Nothing here is exported.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "fastav.h"

namespace fastav {

constexpr int kNumSMs = 148;          // B200: 2 dies x 74 SMs; grids are sized in multiples of this
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// Device-side view of one call's shapes (a trimmed fastav_params, passed by value).
struct Shapes {
  int batch, total_tokens, max_seqlen, total_q, max_qlen, total_keep, max_keep;
  int hq, hkv, group, dim, hidden;
  long long q_st, q_sh, k_st, k_sh, v_st, v_sh, ko_st, ko_sh, vo_st, vo_sh;
  float scale_log2;  // softmax scale * log2(e): logits are kept in base-2 units
  unsigned flags;
};

// Carved from the caller's workspace by plan_workspace(); all offsets 256-byte aligned.
struct Workspace {
  size_t total = 0;
  // generic / narrow score
  size_t stats_off = 0;     // float2 [total_q * Hq][stat_tiles]   per-tile (max, sum-exp2)
  size_t lse_off = 0;       // float  [total_q * Hq]               log2-sum-exp2 per (row, head)
  size_t partial_off = 0;   // float  [Hkv * row chunks][N]        score partials per KV head and chunk of query rows
  size_t logits_off = 0;    // float  [Hq][max_qlen][N] (matrix-vector path only; 0 bytes otherwise)
  // select
  size_t keys_off = 0;      // uint32 [N] (only when a sequence does not fit in shared memory)
  int stat_tiles = 0;
};

Workspace plan_workspace(const fastav_params& p);

// ---- launchers (each returns cudaGetLastError() after its launches) -------------------------
cudaError_t launch_score(const Shapes& s, const Workspace& w, const void* q, const int32_t* q_idx,
                         const int32_t* cu_qlens, const void* k, const int32_t* cu_seqlens, const float* lse_in,
                         float* scores_out, unsigned char* ws, int32_t* device_status, cudaStream_t stream);

// `lse_in` (optional, everywhere below): the caller's natural-log log-sum-exp per (scored row, head); when
// given, the softmax statistics are not recomputed.
cudaError_t launch_score_generic(const Shapes& s, const Workspace& w, const void* q, const int32_t* q_idx,
                                 const int32_t* cu_qlens, const void* k, const int32_t* cu_seqlens, const float* lse_in,
                                 float* scores_out, unsigned char* ws, cudaStream_t stream);

// lse_ws[i] = log2(e) * lse_in[i] (the kernels work in base-2 units); a non-finite entry (a row that saw no
// key) becomes +inf, i.e. the row contributes nothing.
cudaError_t launch_lse_import(const Shapes& s, const float* lse_in, float* lse_ws, cudaStream_t stream);
// ... and back: the workspace's statistics as natural-log log-sum-exp [total_q, Hq] (-inf where a row sees no key).
cudaError_t launch_lse_export(const Shapes& s, const float* lse_ws, float* lse_out, cudaStream_t stream);

// Few scored rows per sequence (the paper's fine stage scores the last token only): matrix-vector path.
constexpr int kNarrowMaxRows = 4;
bool score_narrow_applies(const Shapes& s);
cudaError_t launch_score_narrow(const Shapes& s, const Workspace& w, const void* q, const int32_t* q_idx,
                                const int32_t* cu_qlens, const void* k, const int32_t* cu_seqlens, const float* lse_in,
                                float* scores_out, unsigned char* ws, int32_t* device_status, cudaStream_t stream);

// Many scored rows per sequence: tensor-core path (tcgen05 + TMA).  `*used` is false when the TMA
// descriptor for K could not be built; nothing was launched then and the caller takes another path.
int wide_rows_per_chunk(int group);
int wide_row_chunks(int max_qlen, int group);
bool score_wide_applies(const Shapes& s);
cudaError_t launch_score_wide(const Shapes& s, const Workspace& w, const void* q, const int32_t* q_idx,
                              const int32_t* cu_qlens, const void* k, const int32_t* cu_seqlens, const float* lse_in,
                              float* scores_out, unsigned char* ws, int32_t* device_status, cudaStream_t stream, bool* used);

cudaError_t launch_logits_wide(const Shapes& s, const void* q, const int32_t* q_idx, const int32_t* cu_qlens, const void* k,
                               const int32_t* cu_seqlens, float* logits, int rq, int32_t* device_status, cudaStream_t stream,
                               bool* used);

// Short sequences with few scored rows: one kernel turns the logits into scores and (optionally) the keep list.
bool narrow_tail_applies(const Shapes& s);
cudaError_t launch_narrow_tail(const Shapes& s, const float* logits, int rq, float* scores_out, bool do_select,
                               const int32_t* cu_seqlens, const int32_t* keep_counts, const uint8_t* protect,
                               const int32_t* q_idx, const int32_t* cu_qlens, int32_t* keep_idx, int32_t* cu_keep,
                               int32_t* device_status, cudaStream_t stream);
// Only the logits [Hq, max_qlen, N] of the few-rows path, into the workspace.
cudaError_t launch_narrow_logits(const Shapes& s, const Workspace& w, const void* q, const int32_t* q_idx,
                                 const int32_t* cu_qlens, const void* k, const int32_t* cu_seqlens, unsigned char* ws,
                                 int32_t* device_status, cudaStream_t stream);

cudaError_t launch_select(const Shapes& s, const Workspace& w, const float* scores, const int32_t* cu_seqlens,
                          const int32_t* keep_counts, const uint8_t* protect, const int32_t* q_idx,
                          const int32_t* cu_qlens, int32_t* keep_idx, int32_t* cu_keep, unsigned char* ws,
                          int32_t* device_status, cudaStream_t stream);

cudaError_t launch_compact(const Shapes& s, const int32_t* keep_idx, const int32_t* cu_keep,
                           const int32_t* cu_seqlens, const void* hidden_in, void* hidden_out, const int32_t* pos_in,
                           int32_t* pos_out, const void* k_in, void* k_out, const void* v_in, void* v_out,
                           int32_t* device_status, cudaStream_t stream);

int32_t validate_prune(const fastav_params* params, const void* q, const int32_t* q_idx, const int32_t* cu_qlens, const void* k,
                       const void* v, const int32_t* cu_seqlens, const int32_t* keep_counts, const void* hidden_in,
                       const int32_t* pos_in, const float* scores_out, const int32_t* keep_idx_out, const int32_t* cu_keep_out,
                       const void* hidden_out, const int32_t* pos_out, const void* k_out, const void* v_out, const void* workspace,
                       size_t workspace_bytes);

// Diagnostic launch counter (fastav_kernel_launches).
void count_launches(int n);

// The driver's tensor-map encoder (cuTensorMapEncodeTiled), looked up once through the runtime; nullptr if absent.
void* tensor_map_encode_entry();

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---- programmatic dependent launch ----------------------------------------------------------------
// The kernels of one prune call form a chain in which each reads what its predecessor wrote.  They
// are launched with programmatic stream serialization: a kernel lets its successor start early
// (pdl_trigger, first thing) so that the successor's set-up overlaps this kernel's tail, and every
// block of the successor calls pdl_wait -- which returns once the predecessor has completed and its
// writes are visible -- before it touches global memory another kernel may have written, or writes
// global memory another kernel may still read.  Every block waits before it exits, so completion of a
// kernel implies completion of all its predecessors.
#ifdef __CUDACC__
// Sequence b of a packed batch as the device sees it in a prefix-sum array, cut down to what the host scalars
// promise: buffers and grids are sized from total_tokens / max_seqlen (total_q / max_qlen), loop bounds come from
// the device array, and a caller whose two views disagree must get a status bit, not an out-of-bounds access.
struct Span {
  int first, count;
  bool bad;  // the array and the host scalars disagree: the span was clamped (FASTAV_DEV_SHAPE_MISMATCH)
};
__device__ __forceinline__ Span checked_span(const int32_t* cu, int b, int total, int max_count) {
  const int a = cu[b], e = cu[b + 1];
  Span sp{a, e - a, false};
  if (a < 0 || a > total) {
    sp = Span{0, 0, true};
  } else {
    const int room = min(max_count, total - a);
    if (sp.count < 0) { sp.count = 0; sp.bad = true; }
    else if (sp.count > room) { sp.count = room; sp.bad = true; }
  }
  return sp;
}
__device__ __forceinline__ Span seq_span(const Shapes& s, const int32_t* cu_seqlens, int b) {
  return checked_span(cu_seqlens, b, s.total_tokens, s.max_seqlen);
}
__device__ __forceinline__ Span row_span(const Shapes& s, const int32_t* cu_qlens, int b) {
  return checked_span(cu_qlens, b, s.total_q, s.max_qlen);
}

__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// A pointer to data the predecessor writes must be passed through this after pdl_wait: the compiler
// may otherwise hoist loads through a `const __restrict__` pointer above the wait (it is entitled to
// assume nobody writes such data while the kernel runs).
#define pdl_acquire(ptr) asm volatile("" : "+l"(ptr) : : "memory")
// ... and must never be read through the non-coherent path (ld.global.nc, which __ldg forces): such a load can
// be served from a line this SM cached during an earlier launch, before the predecessor rewrote it (seen with a
// kernel that started early under programmatic launch and re-read a buffer of the previous call).  chain_load
// reads through L2.
template <typename T>
__device__ __forceinline__ T chain_load(const T* p) { return __ldcg(p); }
// The same for values read many times (a table that is searched): an ordinary coherent load that may stay in L1,
// spelled out so that it can never turn into the non-coherent form.
template <typename T>
__device__ __forceinline__ T chain_load_cached(const T* p) { return __ldca(p); }

// The FIRST kernel an entry point launches takes an ordinary stream dependency: it starts only when all earlier
// work on the stream has completed, so that the arrays the kernels read before their wait (cu_seqlens, cu_qlens,
// q_idx, keep_counts, protect: possibly the output of the call before, e.g. its cu_keep) are final.  Every later
// kernel of the call is launched programmatically.  Under FASTAV_CHAIN_CALLS the caller vouches for those arrays
// and the first kernel is launched programmatically as well.  chain_begin() marks the start of a call (per host
// thread).
inline thread_local bool g_chain_head = true;
inline void chain_begin(uint32_t flags) { g_chain_head = (flags & FASTAV_CHAIN_CALLS) == 0; }

template <typename... KArgs, typename... Args>
cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = g_chain_head ? 0 : 1;
  g_chain_head = false;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

}  // namespace fastav
