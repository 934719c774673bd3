// Survivor gather: out[i] = in[source(i)] for hidden states, K, V and position ids.
//
// The step the paper implies by "iteratively refining the token set" (Section 2.2): the following
// layers only ever see the survivors, so their rows are packed into a dense layout.  It moves
// about 85-90 % of all bytes of a prune call and is bound by HBM bandwidth: each row (7-8 KB of
// hidden state, 1-2 KB each of K and V) is read once and written once with 16-byte accesses, the
// whole thread block walking one row so that every warp instruction covers 512 contiguous bytes.
#include "common.cuh"

namespace fastav {
namespace {

constexpr int kThreads = 256;
constexpr int kUnroll = 4;  // 16-byte loads in flight per thread

__device__ __forceinline__ uint4 load_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

__device__ __forceinline__ void store_row(uint4* p, const uint4& v) {
  asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

struct RowStreams {
  const uint16_t* hidden_in;
  uint16_t* hidden_out;
  const uint16_t* k_in;
  uint16_t* k_out;
  const uint16_t* v_in;
  uint16_t* v_out;
  const int32_t* pos_in;
  int32_t* pos_out;
};

__global__ void __launch_bounds__(kThreads) compact_rows_kernel(Shapes s, RowStreams t, const int32_t* __restrict__ keep_idx,
                                                                const int32_t* __restrict__ cu_keep,
                                                                const int32_t* __restrict__ cu_seqlens,
                                                                int32_t* device_status) {
  pdl_trigger();
  pdl_wait();  // keep_idx and cu_keep are the previous kernel's output
  // 16-byte chunks per output row: [hidden | K heads | V heads]
  const int per_head = s.dim >> 3;
  const int n_hidden = t.hidden_in ? (s.hidden >> 3) : 0;
  const int n_k = t.k_in ? s.hkv * per_head : 0;
  const int n_v = t.v_in ? s.hkv * per_head : 0;
  const int n_chunks = n_hidden + n_k + n_v;
  const int head_shift = (s.dim == 128) ? 4 : 3;
  const bool global_idx = (s.flags & FASTAV_KEEP_IDX_GLOBAL) != 0;
  int rows = cu_keep[s.batch];
  if (rows > s.total_keep) rows = s.total_keep;  // never write past the caller's buffers

  for (int row = blockIdx.x; row < rows; row += gridDim.x) {
    int lo = 0, hi = s.batch;  // largest b with cu_keep[b] <= row
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (cu_keep[mid] <= row) lo = mid; else hi = mid;
    }
    const long long src = global_idx ? (long long)keep_idx[row] : (long long)cu_seqlens[lo] + keep_idx[row];
    const long long dst = row;
    if (src < cu_seqlens[lo] || src >= cu_seqlens[lo + 1]) {  // an index outside its sequence: skip the row, report
      if (threadIdx.x == 0 && device_status) atomicOr(device_status, FASTAV_DEV_BAD_INDEX);
      continue;
    }
    if (threadIdx.x == 0 && t.pos_in) t.pos_out[dst] = t.pos_in[src];

    for (int base = 0; base < n_chunks; base += kThreads * kUnroll) {
      uint4 regs[kUnroll];
      uint4* out_ptr[kUnroll];
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int c = base + u * kThreads + threadIdx.x;
        out_ptr[u] = nullptr;
        if (c < n_chunks) {
          const uint16_t* in;
          uint16_t* out;
          if (c < n_hidden) {
            in = t.hidden_in + src * s.hidden + (c << 3);
            out = t.hidden_out + dst * s.hidden + (c << 3);
          } else if (c < n_hidden + n_k) {
            const int cc = c - n_hidden, head = cc >> head_shift, off = (cc & (per_head - 1)) << 3;
            in = t.k_in + src * s.k_st + head * s.k_sh + off;
            out = t.k_out + dst * s.ko_st + head * s.ko_sh + off;
          } else {
            const int cc = c - n_hidden - n_k, head = cc >> head_shift, off = (cc & (per_head - 1)) << 3;
            in = t.v_in + src * s.v_st + head * s.v_sh + off;
            out = t.v_out + dst * s.vo_st + head * s.vo_sh + off;
          }
          regs[u] = load_stream(reinterpret_cast<const uint4*>(in));
          out_ptr[u] = reinterpret_cast<uint4*>(out);
        }
      }
#pragma unroll
      for (int u = 0; u < kUnroll; ++u)
        if (out_ptr[u]) store_row(out_ptr[u], regs[u]);
    }
  }
}

}  // namespace

cudaError_t launch_compact(const Shapes& s, const int32_t* keep_idx, const int32_t* cu_keep,
                           const int32_t* cu_seqlens, const void* hidden_in, void* hidden_out, const int32_t* pos_in,
                           int32_t* pos_out, const void* k_in, void* k_out, const void* v_in, void* v_out,
                           int32_t* device_status, cudaStream_t stream) {
  if (s.total_keep <= 0) return cudaSuccess;
  RowStreams t{static_cast<const uint16_t*>(hidden_in), static_cast<uint16_t*>(hidden_out),
               static_cast<const uint16_t*>(k_in),      static_cast<uint16_t*>(k_out),
               static_cast<const uint16_t*>(v_in),      static_cast<uint16_t*>(v_out),
               pos_in,                                  pos_out};
  int blocks = kNumSMs * 8;
  if (blocks > s.total_keep) blocks = s.total_keep;
  const cudaError_t e = launch_chained(compact_rows_kernel, dim3(blocks), dim3(kThreads), 0, stream, s, t, keep_idx, cu_keep,
                                       cu_seqlens, device_status);
  count_launches(1);
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace fastav
