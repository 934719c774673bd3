// C-ABI layer: argument validation, workspace carving and kernel dispatch.  See fastav.h for the
// contract of every entry point; nothing here computes anything.
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>

#include "common.cuh"

namespace fastav {
namespace {

thread_local char g_cuda_error[256] = "";
std::atomic<long long> g_launches{0};

int32_t cuda_failed(cudaError_t e) {
  std::snprintf(g_cuda_error, sizeof g_cuda_error, "%s: %s", cudaGetErrorName(e), cudaGetErrorString(e));
  return FASTAV_ERR_CUDA;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Shape checks shared by all entry points.
int32_t check_params(const fastav_params* p) {
  if (!p) return FASTAV_ERR_INVALID_ARG;
  if (p->batch < 1 || p->total_tokens < 0 || p->max_seqlen < 0 || p->max_seqlen > p->total_tokens) return FASTAV_ERR_INVALID_ARG;
  if (p->total_q < 0 || p->max_qlen < 0 || p->max_qlen > p->total_q) return FASTAV_ERR_INVALID_ARG;
  if (p->total_keep < 0 || p->max_keep < 0 || p->total_keep > p->total_tokens || p->max_keep > p->total_keep) return FASTAV_ERR_INVALID_ARG;
  if (p->num_q_heads < 1 || p->num_kv_heads < 1 || p->num_q_heads % p->num_kv_heads != 0) return FASTAV_ERR_INVALID_ARG;
  if (p->head_dim != 64 && p->head_dim != 128) return FASTAV_ERR_UNSUPPORTED;
  if (p->hidden < 0 || p->hidden % 8 != 0) return FASTAV_ERR_UNSUPPORTED;
  return FASTAV_OK;
}

// A [tokens, heads, dim] view: the head stride must hold a row, the token stride must hold all heads,
// and both must keep rows 16-byte aligned.
// Two layouts pass: heads inside a token (st >= heads * sh, e.g. a view into a packed projection output) and
// tokens inside a head (sh > st, a head-major cache; its extent is the caller's business).  What is rejected is
// the one case that is certainly wrong: heads inside a token whose rows overlap the next token's.
int32_t check_strides(int64_t st, int64_t sh, int heads, int dim) {
  if (sh < dim || st < dim) return FASTAV_ERR_INVALID_ARG;
  if (st % 8 != 0 || sh % 8 != 0) return FASTAV_ERR_UNSUPPORTED;
  if (heads > 1 && st >= sh && st < (int64_t)(heads - 1) * sh + dim) return FASTAV_ERR_INVALID_ARG;
  return FASTAV_OK;
}

bool overlaps(const void* a, size_t a_bytes, const void* b, size_t b_bytes) {
  if (!a || !b || !a_bytes || !b_bytes) return false;
  const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
  return a0 < b0 + b_bytes && b0 < a0 + a_bytes;
}

size_t view_bytes(int64_t rows, int64_t st, int64_t sh, int heads, int dim) {
  if (rows <= 0) return 0;
  return (size_t)(((rows - 1) * st + (int64_t)(heads - 1) * sh + dim) * 2);
}

Shapes make_shapes(const fastav_params& p) {
  Shapes s{};
  s.batch = p.batch; s.total_tokens = p.total_tokens; s.max_seqlen = p.max_seqlen;
  s.total_q = p.total_q; s.max_qlen = p.max_qlen; s.total_keep = p.total_keep; s.max_keep = p.max_keep;
  s.hq = p.num_q_heads; s.hkv = p.num_kv_heads; s.group = p.num_q_heads / p.num_kv_heads;
  s.dim = p.head_dim; s.hidden = p.hidden;
  s.q_st = p.q_stride_tok; s.q_sh = p.q_stride_head;
  s.k_st = p.k_stride_tok; s.k_sh = p.k_stride_head; s.v_st = p.v_stride_tok; s.v_sh = p.v_stride_head;
  s.ko_st = p.ko_stride_tok; s.ko_sh = p.ko_stride_head; s.vo_st = p.vo_stride_tok; s.vo_sh = p.vo_stride_head;
  const float scale = p.softmax_scale > 0.f ? p.softmax_scale : 1.0f / std::sqrt((float)p.head_dim);
  s.scale_log2 = scale * kLog2e;
  s.flags = p.flags;
  return s;
}

int32_t check_workspace(const Workspace& w, const void* ws, size_t bytes) {
  if (w.total == 0) return FASTAV_OK;
  if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u) || bytes < w.total) return FASTAV_ERR_WORKSPACE;
  return FASTAV_OK;
}

int32_t check_score_args(const fastav_params* p, const void* q, const int32_t* q_idx, const int32_t* cu_qlens,
                         const void* k, const int32_t* cu_seqlens, const float* scores_out) {
  if (!cu_seqlens || !cu_qlens) return FASTAV_ERR_INVALID_ARG;
  if (p->total_tokens > 0 && (!k || !scores_out)) return FASTAV_ERR_INVALID_ARG;
  if (p->total_q > 0 && (!q || !q_idx)) return FASTAV_ERR_INVALID_ARG;
  int32_t rc;
  if ((rc = check_strides(p->q_stride_tok, p->q_stride_head, p->num_q_heads, p->head_dim)) != FASTAV_OK) return rc;
  if ((rc = check_strides(p->k_stride_tok, p->k_stride_head, p->num_kv_heads, p->head_dim)) != FASTAV_OK) return rc;
  if (!aligned16(q) || !aligned16(k)) return FASTAV_ERR_UNSUPPORTED;
  return FASTAV_OK;
}

int32_t check_select_args(const fastav_params* p, const float* scores, const int32_t* cu_seqlens, const int32_t* keep_counts,
                          const int32_t* q_idx, const int32_t* cu_qlens, const int32_t* keep_idx_out, const int32_t* cu_keep_out) {
  if (!cu_seqlens || !keep_counts || !cu_keep_out) return FASTAV_ERR_INVALID_ARG;
  if (p->total_tokens > 0 && !scores) return FASTAV_ERR_INVALID_ARG;
  if (p->total_keep > 0 && !keep_idx_out) return FASTAV_ERR_INVALID_ARG;
  if ((p->flags & FASTAV_PROTECT_QUERY_ROWS) && (!cu_qlens || (p->total_q > 0 && !q_idx))) return FASTAV_ERR_INVALID_ARG;
  return FASTAV_OK;
}

int32_t check_compact_args(const fastav_params* p, const int32_t* keep_idx, const int32_t* cu_keep, const int32_t* cu_seqlens,
                           const void* hidden_in, const void* hidden_out, const int32_t* pos_in, const int32_t* pos_out,
                           const void* k_in, const void* k_out, const void* v_in, const void* v_out) {
  if (!cu_keep || !cu_seqlens) return FASTAV_ERR_INVALID_ARG;
  if (p->total_keep > 0 && !keep_idx) return FASTAV_ERR_INVALID_ARG;
  if ((hidden_in == nullptr) != (hidden_out == nullptr) || (pos_in == nullptr) != (pos_out == nullptr) ||
      (k_in == nullptr) != (k_out == nullptr) || (v_in == nullptr) != (v_out == nullptr))
    return FASTAV_ERR_INVALID_ARG;
  int32_t rc;
  if (k_in) {
    if ((rc = check_strides(p->k_stride_tok, p->k_stride_head, p->num_kv_heads, p->head_dim)) != FASTAV_OK) return rc;
    if ((rc = check_strides(p->ko_stride_tok, p->ko_stride_head, p->num_kv_heads, p->head_dim)) != FASTAV_OK) return rc;
  }
  if (v_in) {
    if ((rc = check_strides(p->v_stride_tok, p->v_stride_head, p->num_kv_heads, p->head_dim)) != FASTAV_OK) return rc;
    if ((rc = check_strides(p->vo_stride_tok, p->vo_stride_head, p->num_kv_heads, p->head_dim)) != FASTAV_OK) return rc;
  }
  if (!aligned16(hidden_in) || !aligned16(hidden_out) || !aligned16(k_in) || !aligned16(k_out) || !aligned16(v_in) ||
      !aligned16(v_out))
    return FASTAV_ERR_UNSUPPORTED;
  const int N = p->total_tokens, K = p->total_keep, H = p->num_kv_heads, d = p->head_dim;
  if (overlaps(hidden_in, (size_t)N * p->hidden * 2, hidden_out, (size_t)K * p->hidden * 2)) return FASTAV_ERR_INVALID_ARG;
  if (overlaps(pos_in, (size_t)N * 4, pos_out, (size_t)K * 4)) return FASTAV_ERR_INVALID_ARG;
  if (overlaps(k_in, view_bytes(N, p->k_stride_tok, p->k_stride_head, H, d), k_out, view_bytes(K, p->ko_stride_tok, p->ko_stride_head, H, d)))
    return FASTAV_ERR_INVALID_ARG;
  if (overlaps(v_in, view_bytes(N, p->v_stride_tok, p->v_stride_head, H, d), v_out, view_bytes(K, p->vo_stride_tok, p->vo_stride_head, H, d)))
    return FASTAV_ERR_INVALID_ARG;
  return FASTAV_OK;
}

}  // namespace

void count_launches(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

Workspace plan_workspace(const fastav_params& p) {
  Workspace w;
  size_t off = 0;
  auto carve = [&](size_t bytes) { const size_t at = off; off = align_up(off + bytes, 256); return at; };
  const size_t rows_heads = (size_t)p.total_q * p.num_q_heads;
  w.stat_tiles = (p.max_seqlen + 63) / 64;
  // per (row, head): one (max, sum) per 64-key tile on the CUDA-core path, at most two per 128-key tile on the tensor-core path
  const size_t stat_entries = (size_t)2 * ((p.max_seqlen + 127) / 128);
  w.stats_off = carve(rows_heads * (stat_entries > (size_t)w.stat_tiles ? stat_entries : (size_t)w.stat_tiles) * sizeof(float2));
  w.lse_off = carve(rows_heads * sizeof(float));
  w.partial_off = carve((size_t)p.num_kv_heads * wide_row_chunks(p.max_qlen, p.num_q_heads / p.num_kv_heads) *
                        p.total_tokens * sizeof(float));
  const bool narrow = p.max_qlen >= 1 && p.max_qlen <= kNarrowMaxRows;
  w.logits_off = carve(narrow ? (size_t)p.num_q_heads * p.max_qlen * p.total_tokens * sizeof(float) : 0);
  w.keys_off = carve((size_t)p.total_tokens * sizeof(uint32_t));
  w.total = off;
  return w;
}

__global__ void status_or_kernel(int32_t* device_status, int32_t bits) {
  pdl_trigger();
  pdl_wait();
  atomicOr(device_status, bits);
}

// A forced score path (FASTAV_SCORE_PATH_*) must support the shapes; the shape-based choice always does.
bool score_path_ok(const Shapes& s) {
  const unsigned forced = s.flags & FASTAV_SCORE_PATH_MASK;
  if (forced == FASTAV_SCORE_PATH_NARROW) return score_narrow_applies(s);
  if (forced == FASTAV_SCORE_PATH_WIDE) return score_wide_applies(s);
  return true;
}

// Shape-based choice: few scored rows -> matrix-vector path; otherwise the tensor-core path; the
// CUDA-core tiles take whatever is left (and whatever the TMA descriptor cannot express).
cudaError_t launch_score(const Shapes& s, const Workspace& w, const void* q, const int32_t* q_idx,
                         const int32_t* cu_qlens, const void* k, const int32_t* cu_seqlens, const float* lse_in,
                         float* scores_out, unsigned char* ws, int32_t* device_status, cudaStream_t stream) {
  const unsigned forced = s.flags & FASTAV_SCORE_PATH_MASK;
  if (forced == FASTAV_SCORE_PATH_GENERIC) return launch_score_generic(s, w, q, q_idx, cu_qlens, k, cu_seqlens, lse_in, scores_out, ws, stream);
  if (score_narrow_applies(s) && (forced == 0 || forced == FASTAV_SCORE_PATH_NARROW))
    return launch_score_narrow(s, w, q, q_idx, cu_qlens, k, cu_seqlens, lse_in, scores_out, ws, device_status, stream);
  if (score_wide_applies(s)) {
    bool used = false;
    const cudaError_t e = launch_score_wide(s, w, q, q_idx, cu_qlens, k, cu_seqlens, lse_in, scores_out, ws, device_status, stream, &used);
    if (used || e != cudaSuccess) return e;
    if (forced == FASTAV_SCORE_PATH_WIDE) return cudaErrorNotSupported;
    // The tensor map could not be encoded: the CUDA-core tiles below are correct but far slower, so say so.
    if (device_status) {
      const cudaError_t es = launch_chained(status_or_kernel, dim3(1), dim3(1), 0, stream, device_status, (int32_t)FASTAV_DEV_SLOW_PATH);
      if (es != cudaSuccess) return es;
      count_launches(1);
    }
  }
  return launch_score_generic(s, w, q, q_idx, cu_qlens, k, cu_seqlens, lse_in, scores_out, ws, stream);
}

// Everything fastav_prune checks before it enqueues anything (also used by the host-buffer entry point, which must
// not start its uploads for a call that will be refused).
int32_t validate_prune(const fastav_params* params, const void* q, const int32_t* q_idx, const int32_t* cu_qlens, const void* k,
                       const void* v, const int32_t* cu_seqlens, const int32_t* keep_counts, const void* hidden_in,
                       const int32_t* pos_in, const float* scores_out, const int32_t* keep_idx_out, const int32_t* cu_keep_out,
                       const void* hidden_out, const int32_t* pos_out, const void* k_out, const void* v_out, const void* workspace,
                       size_t workspace_bytes) {
  int32_t rc = check_params(params);
  if (rc != FASTAV_OK) return rc;
  if ((rc = check_score_args(params, q, q_idx, cu_qlens, k, cu_seqlens, scores_out)) != FASTAV_OK) return rc;
  if ((rc = check_select_args(params, scores_out, cu_seqlens, keep_counts, q_idx, cu_qlens, keep_idx_out, cu_keep_out)) != FASTAV_OK) return rc;
  if ((rc = check_compact_args(params, keep_idx_out, cu_keep_out, cu_seqlens, hidden_in, hidden_out, pos_in, pos_out, k, k_out,
                               v, v_out)) != FASTAV_OK)
    return rc;
  if ((rc = check_workspace(plan_workspace(*params), workspace, workspace_bytes)) != FASTAV_OK) return rc;
  if (!score_path_ok(make_shapes(*params))) return FASTAV_ERR_UNSUPPORTED;
  return FASTAV_OK;
}

}  // namespace fastav

using namespace fastav;

extern "C" {

int32_t fastav_version(void) { return FASTAV_VERSION; }

const char* fastav_status_string(int32_t status) {
  switch (status) {
    case FASTAV_OK: return "ok";
    case FASTAV_ERR_INVALID_ARG: return "invalid argument";
    case FASTAV_ERR_UNSUPPORTED: return "unsupported shape, stride or alignment";
    case FASTAV_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case FASTAV_ERR_CUDA: return "CUDA launch failed (see fastav_last_cuda_error)";
    case FASTAV_ERR_TIMEOUT: return "bounded device wait expired";
    default: return "unknown status";
  }
}

const char* fastav_last_cuda_error(void) { return g_cuda_error; }

int64_t fastav_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }

int32_t fastav_workspace_bytes(const fastav_params* params, size_t* out_bytes) {
  int32_t rc = check_params(params);
  if (rc != FASTAV_OK) return rc;
  if (!out_bytes) return FASTAV_ERR_INVALID_ARG;
  *out_bytes = plan_workspace(*params).total;
  return FASTAV_OK;
}

int32_t fastav_score(const fastav_params* params, const void* q, const int32_t* q_idx, const int32_t* cu_qlens,
                     const void* k, const int32_t* cu_seqlens, const float* lse_opt, float* scores_out,
                     void* workspace, size_t workspace_bytes, int32_t* device_status, void* stream) {
  int32_t rc = check_params(params);
  if (rc != FASTAV_OK) return rc;
  chain_begin(params->flags);
  if ((rc = check_score_args(params, q, q_idx, cu_qlens, k, cu_seqlens, scores_out)) != FASTAV_OK) return rc;
  const Workspace w = plan_workspace(*params);
  if ((rc = check_workspace(w, workspace, workspace_bytes)) != FASTAV_OK) return rc;
  if (!score_path_ok(make_shapes(*params))) return FASTAV_ERR_UNSUPPORTED;
  if (params->total_tokens == 0) return FASTAV_OK;
  const cudaError_t e = launch_score(make_shapes(*params), w, q, q_idx, cu_qlens, k, cu_seqlens, lse_opt, scores_out,
                                     static_cast<unsigned char*>(workspace), device_status, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? FASTAV_OK : cuda_failed(e);
}

int32_t fastav_lse(const fastav_params* params, const void* q, const int32_t* q_idx, const int32_t* cu_qlens, const void* k,
                   const int32_t* cu_seqlens, float* lse_out, void* workspace, size_t workspace_bytes, int32_t* device_status,
                   void* stream) {
  int32_t rc = check_params(params);
  if (rc != FASTAV_OK) return rc;
  chain_begin(params->flags);
  if (!lse_out && params->total_q > 0) return FASTAV_ERR_INVALID_ARG;
  // the scores pointer only has to be non-null for the shared argument check; nothing is written through it
  if ((rc = check_score_args(params, q, q_idx, cu_qlens, k, cu_seqlens, lse_out)) != FASTAV_OK) return rc;
  const Workspace w = plan_workspace(*params);
  if ((rc = check_workspace(w, workspace, workspace_bytes)) != FASTAV_OK) return rc;
  const Shapes s = make_shapes(*params);
  if (!score_path_ok(s)) return FASTAV_ERR_UNSUPPORTED;
  if (params->total_tokens == 0 || params->total_q == 0) return FASTAV_OK;
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e = launch_score(s, w, q, q_idx, cu_qlens, k, cu_seqlens, nullptr, nullptr, ws, device_status, st);
  if (e == cudaSuccess) e = launch_lse_export(s, reinterpret_cast<const float*>(ws + w.lse_off), lse_out, st);
  return e == cudaSuccess ? FASTAV_OK : cuda_failed(e);
}

int32_t fastav_select(const fastav_params* params, const float* scores, const int32_t* cu_seqlens,
                      const int32_t* keep_counts, const uint8_t* protect_opt, const int32_t* q_idx,
                      const int32_t* cu_qlens, int32_t* keep_idx_out, int32_t* cu_keep_out, void* workspace,
                      size_t workspace_bytes, int32_t* device_status, void* stream) {
  int32_t rc = check_params(params);
  if (rc != FASTAV_OK) return rc;
  chain_begin(params->flags);
  if ((rc = check_select_args(params, scores, cu_seqlens, keep_counts, q_idx, cu_qlens, keep_idx_out, cu_keep_out)) != FASTAV_OK) return rc;
  const Workspace w = plan_workspace(*params);
  if ((rc = check_workspace(w, workspace, workspace_bytes)) != FASTAV_OK) return rc;
  const cudaError_t e = launch_select(make_shapes(*params), w, scores, cu_seqlens, keep_counts, protect_opt, q_idx, cu_qlens,
                                      keep_idx_out, cu_keep_out, static_cast<unsigned char*>(workspace), device_status,
                                      static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? FASTAV_OK : cuda_failed(e);
}

int32_t fastav_compact(const fastav_params* params, const int32_t* keep_idx, const int32_t* cu_keep,
                       const int32_t* cu_seqlens, const void* hidden_in, void* hidden_out, const int32_t* pos_in,
                       int32_t* pos_out, const void* k_in, void* k_out, const void* v_in, void* v_out,
                       int32_t* device_status, void* stream) {
  int32_t rc = check_params(params);
  if (rc != FASTAV_OK) return rc;
  chain_begin(params->flags);
  if ((rc = check_compact_args(params, keep_idx, cu_keep, cu_seqlens, hidden_in, hidden_out, pos_in, pos_out, k_in, k_out,
                               v_in, v_out)) != FASTAV_OK)
    return rc;
  const cudaError_t e = launch_compact(make_shapes(*params), keep_idx, cu_keep, cu_seqlens, hidden_in, hidden_out, pos_in,
                                       pos_out, k_in, k_out, v_in, v_out, device_status, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? FASTAV_OK : cuda_failed(e);
}

int32_t fastav_prune(const fastav_params* params, const void* q, const int32_t* q_idx, const int32_t* cu_qlens,
                     const void* k, const void* v, const int32_t* cu_seqlens, const float* lse_opt, const int32_t* keep_counts,
                     const uint8_t* protect_opt, const void* hidden_in, const int32_t* pos_in, float* scores_out,
                     int32_t* keep_idx_out, int32_t* cu_keep_out, void* hidden_out, int32_t* pos_out, void* k_out,
                     void* v_out, void* workspace, size_t workspace_bytes, int32_t* device_status, void* stream) {
  // Validate everything first so that an error leaves nothing enqueued.
  int32_t rc = validate_prune(params, q, q_idx, cu_qlens, k, v, cu_seqlens, keep_counts, hidden_in, pos_in, scores_out, keep_idx_out,
                              cu_keep_out, hidden_out, pos_out, k_out, v_out, workspace, workspace_bytes);
  if (rc != FASTAV_OK) return rc;
  chain_begin(params->flags);
  const Workspace w = plan_workspace(*params);
  const Shapes s = make_shapes(*params);
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaSuccess;
  const unsigned forced = s.flags & FASTAV_SCORE_PATH_MASK;
  if (params->total_tokens > 0 && !lse_opt && score_narrow_applies(s) && narrow_tail_applies(s) &&
      (forced == 0 || forced == FASTAV_SCORE_PATH_NARROW)) {
    // Short sequences, few scored rows: logits, then ONE kernel for the softmax statistics, the scores and the keep list.
    e = launch_narrow_logits(s, w, q, q_idx, cu_qlens, k, cu_seqlens, ws, device_status, st);
    if (e == cudaSuccess)
      e = launch_narrow_tail(s, reinterpret_cast<const float*>(ws + w.logits_off), s.max_qlen, scores_out, true, cu_seqlens,
                             keep_counts, protect_opt, q_idx, cu_qlens, keep_idx_out, cu_keep_out, device_status, st);
  } else {
    if (params->total_tokens > 0) e = launch_score(s, w, q, q_idx, cu_qlens, k, cu_seqlens, lse_opt, scores_out, ws, device_status, st);
    if (e == cudaSuccess)
      e = launch_select(s, w, scores_out, cu_seqlens, keep_counts, protect_opt, q_idx, cu_qlens, keep_idx_out, cu_keep_out, ws,
                        device_status, st);
  }
  if (e == cudaSuccess)
    e = launch_compact(s, keep_idx_out, cu_keep_out, cu_seqlens, hidden_in, hidden_out, pos_in, pos_out, k, k_out, v, v_out,
                       device_status, st);
  return e == cudaSuccess ? FASTAV_OK : cuda_failed(e);
}

}  // extern "C"
