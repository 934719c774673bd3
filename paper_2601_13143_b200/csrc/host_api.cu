// Host-buffer entry point: the same prune step for callers whose tensors live in host memory
// (offloaded activations / KV cache).  Copies in, runs fastav_prune, copies out -- all enqueued on
// the caller's stream, staged through a device arena the caller provides.
#include <atomic>

#include "common.cuh"

namespace fastav {
namespace {

struct Arena {
  size_t q, q_idx, cu_qlens, k, v, cu_seqlens, lse, keep_counts, protect, hidden, pos;
  size_t scores, keep_idx, cu_keep, hidden_out, pos_out, k_out, v_out, status, workspace, workspace_bytes, total;
};

bool packed(const fastav_params& p) {
  const int64_t d = p.head_dim;
  return p.q_stride_head == d && p.q_stride_tok == d * p.num_q_heads && p.k_stride_head == d &&
         p.k_stride_tok == d * p.num_kv_heads && p.v_stride_head == d && p.v_stride_tok == d * p.num_kv_heads &&
         p.ko_stride_head == d && p.ko_stride_tok == d * p.num_kv_heads && p.vo_stride_head == d &&
         p.vo_stride_tok == d * p.num_kv_heads;
}

Arena plan_arena(const fastav_params& p) {
  Arena a{};
  size_t off = 0;
  auto carve = [&](size_t bytes) { const size_t at = off; off = align_up(off + bytes, 256); return at; };
  const size_t N = p.total_tokens, K = p.total_keep, B = p.batch, R = p.total_q;
  const size_t kv_row = (size_t)p.num_kv_heads * p.head_dim * 2;
  a.q = carve(R * p.num_q_heads * p.head_dim * 2);
  a.q_idx = carve(R * 4);
  a.cu_qlens = carve((B + 1) * 4);
  a.k = carve(N * kv_row);
  a.v = carve(N * kv_row);
  a.cu_seqlens = carve((B + 1) * 4);
  a.lse = carve(R * p.num_q_heads * 4);
  a.keep_counts = carve(B * 4);
  a.protect = carve(N);
  a.hidden = carve(N * (size_t)p.hidden * 2);
  a.pos = carve(N * 4);
  a.scores = carve(N * 4);
  a.keep_idx = carve(K * 4);
  a.cu_keep = carve((B + 1) * 4);
  a.hidden_out = carve(K * (size_t)p.hidden * 2);
  a.pos_out = carve(K * 4);
  a.k_out = carve(K * kv_row);
  a.v_out = carve(K * kv_row);
  a.status = carve(4);
  a.workspace_bytes = plan_workspace(p).total;
  a.workspace = carve(a.workspace_bytes);
  a.total = off;
  return a;
}

}  // namespace
}  // namespace fastav

using namespace fastav;

extern "C" {

int32_t fastav_host_arena_bytes(const fastav_params* params, size_t* out_bytes) {
  size_t ws = 0;
  const int32_t rc = fastav_workspace_bytes(params, &ws);  // validates the shapes
  if (rc != FASTAV_OK) return rc;
  if (!out_bytes) return FASTAV_ERR_INVALID_ARG;
  if (!packed(*params)) return FASTAV_ERR_UNSUPPORTED;
  *out_bytes = plan_arena(*params).total;
  return FASTAV_OK;
}

int32_t fastav_prune_host(const fastav_params* params, const void* q, const int32_t* q_idx, const int32_t* cu_qlens,
                          const void* k, const void* v, const int32_t* cu_seqlens, const float* lse_opt,
                          const int32_t* keep_counts, const uint8_t* protect_opt, const void* hidden_in, const int32_t* pos_in,
                          float* scores_out, int32_t* keep_idx_out, int32_t* cu_keep_out, void* hidden_out, int32_t* pos_out,
                          void* k_out, void* v_out, int32_t* status_out, void* device_arena, size_t arena_bytes, void* stream) {
  size_t need = 0;
  int32_t rc = fastav_host_arena_bytes(params, &need);
  if (rc != FASTAV_OK) return rc;
  if (!device_arena || (reinterpret_cast<uintptr_t>(device_arena) & 255u) || arena_bytes < need) return FASTAV_ERR_WORKSPACE;
  if (!q_idx || !cu_qlens || !cu_seqlens || !keep_counts || !scores_out || !keep_idx_out || !cu_keep_out || !k || !q)
    return FASTAV_ERR_INVALID_ARG;
  if ((v == nullptr) != (v_out == nullptr) || (hidden_in == nullptr) != (hidden_out == nullptr) ||
      (pos_in == nullptr) != (pos_out == nullptr) || !k_out)
    return FASTAV_ERR_INVALID_ARG;
  // The index arrays are uploaded by this very call, so its first kernel must not start before earlier work on
  // the stream has completed: the chaining flag is not forwarded.
  fastav_params p = *params;
  p.flags &= ~FASTAV_CHAIN_CALLS;
  const Arena a = plan_arena(p);
  unsigned char* base = static_cast<unsigned char*>(device_arena);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t N = p.total_tokens, K = p.total_keep, B = p.batch, R = p.total_q;
  const size_t kv_row = (size_t)p.num_kv_heads * p.head_dim * 2;
  auto dev = [&](size_t off, const void* host) -> void* { return host ? base + off : nullptr; };
  // Everything the fused call would refuse is refused here, before the first copy is enqueued.
  rc = validate_prune(&p, base + a.q, (const int32_t*)(base + a.q_idx), (const int32_t*)(base + a.cu_qlens), base + a.k, dev(a.v, v),
                      (const int32_t*)(base + a.cu_seqlens), (const int32_t*)(base + a.keep_counts), dev(a.hidden, hidden_in),
                      (const int32_t*)dev(a.pos, pos_in), (const float*)(base + a.scores), (const int32_t*)(base + a.keep_idx),
                      (const int32_t*)(base + a.cu_keep), dev(a.hidden_out, hidden_out), (const int32_t*)dev(a.pos_out, pos_out),
                      base + a.k_out, dev(a.v_out, v_out), base + a.workspace, a.workspace_bytes);
  if (rc != FASTAV_OK) return rc;
  cudaError_t e = cudaSuccess;
  auto h2d = [&](size_t off, const void* src, size_t bytes) {
    if (e == cudaSuccess && src && bytes) e = cudaMemcpyAsync(base + off, src, bytes, cudaMemcpyHostToDevice, st);
  };
  auto d2h = [&](void* dst, size_t off, size_t bytes) {
    if (e == cudaSuccess && dst && bytes) e = cudaMemcpyAsync(dst, base + off, bytes, cudaMemcpyDeviceToHost, st);
  };
  h2d(a.q, q, R * p.num_q_heads * p.head_dim * 2);
  h2d(a.q_idx, q_idx, R * 4);
  h2d(a.cu_qlens, cu_qlens, (B + 1) * 4);
  h2d(a.k, k, N * kv_row);
  h2d(a.v, v, N * kv_row);
  h2d(a.cu_seqlens, cu_seqlens, (B + 1) * 4);
  h2d(a.lse, lse_opt, R * p.num_q_heads * 4);
  h2d(a.keep_counts, keep_counts, B * 4);
  h2d(a.protect, protect_opt, N);
  h2d(a.hidden, hidden_in, N * (size_t)p.hidden * 2);
  h2d(a.pos, pos_in, N * 4);
  if (e == cudaSuccess) e = cudaMemsetAsync(base + a.status, 0, 4, st);
  if (e != cudaSuccess) return FASTAV_ERR_CUDA;
  rc = fastav_prune(&p, base + a.q, (const int32_t*)(base + a.q_idx), (const int32_t*)(base + a.cu_qlens), base + a.k,
                    dev(a.v, v), (const int32_t*)(base + a.cu_seqlens), (const float*)dev(a.lse, lse_opt),
                    (const int32_t*)(base + a.keep_counts),
                    (const uint8_t*)dev(a.protect, protect_opt), dev(a.hidden, hidden_in), (const int32_t*)dev(a.pos, pos_in),
                    (float*)(base + a.scores), (int32_t*)(base + a.keep_idx), (int32_t*)(base + a.cu_keep),
                    dev(a.hidden_out, hidden_out), (int32_t*)dev(a.pos_out, pos_out), base + a.k_out, dev(a.v_out, v_out),
                    base + a.workspace, a.workspace_bytes, (int32_t*)(base + a.status), stream);
  if (rc != FASTAV_OK) return rc;
  d2h(scores_out, a.scores, N * 4);
  d2h(keep_idx_out, a.keep_idx, K * 4);
  d2h(cu_keep_out, a.cu_keep, (B + 1) * 4);
  d2h(hidden_out, a.hidden_out, K * (size_t)p.hidden * 2);
  d2h(pos_out, a.pos_out, K * 4);
  d2h(k_out, a.k_out, K * kv_row);
  d2h(v_out, a.v_out, K * kv_row);
  d2h(status_out, a.status, 4);
  return e == cudaSuccess ? FASTAV_OK : FASTAV_ERR_CUDA;
}

}  // extern "C"
