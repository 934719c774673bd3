// Survivor gather: out[i] = in[source(i)] for hidden states, K, V and position ids.
//
// The step Section 2.2 ("Fine pruning") implies when it shrinks the token set layer after layer: the following
// layers only ever see the survivors, so their rows are packed into a dense layout.  It moves
// about 85-90 % of all bytes of a prune call and is bound by HBM bandwidth: each row (7-8 KB of
// hidden state, 1-2 KB each of K and V) is read once and written once with 16-byte accesses, the
// whole thread block walking one row so that every warp instruction covers 512 contiguous bytes.
//
// Main path: bulk asynchronous copies.  A row is a handful of contiguous segments (the hidden state,
// K and V of the token); each warp runs its own ring of row-sized shared-memory slots, one lane per
// segment issuing cp.async.bulk global -> shared (completion on an mbarrier) and then shared ->
// global, several rows in flight per warp and no register staging.  Rows whose segments are not
// 16-byte friendly, or too long for the ring, take the load/store kernel below.
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace fastav {
namespace {

constexpr int kThreads = 256;
constexpr int kUnroll = 4;  // 16-byte loads in flight per thread

__device__ __forceinline__ uint4 load_stream(const uint4* p) {
  uint4 v;
  // a plain (coherent) load: under programmatic launch the rows may be what the previous kernel wrote
  asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
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
  pdl_acquire(keep_idx);
  pdl_acquire(cu_keep);
  // 16-byte chunks per output row: [hidden | K heads | V heads]
  const int per_head = s.dim >> 3;
  const int n_hidden = t.hidden_in ? (s.hidden >> 3) : 0;
  const int n_k = t.k_in ? s.hkv * per_head : 0;
  const int n_v = t.v_in ? s.hkv * per_head : 0;
  const int n_chunks = n_hidden + n_k + n_v;
  const int head_shift = (s.dim == 128) ? 4 : 3;
  const bool global_idx = (s.flags & FASTAV_KEEP_IDX_GLOBAL) != 0;
  int rows = chain_load_cached(cu_keep + s.batch);
  if (rows > s.total_keep) rows = s.total_keep;  // never write past the caller's buffers

  for (int row = blockIdx.x; row < rows; row += gridDim.x) {
    int lo = 0, hi = s.batch;  // largest b with cu_keep[b] <= row
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (chain_load_cached(cu_keep + mid) <= row) lo = mid; else hi = mid;
    }
    const long long src = (global_idx ? 0ll : (long long)cu_seqlens[lo]) + chain_load(keep_idx + row);
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

// ---- bulk-copy path ---------------------------------------------------------------------------------
constexpr int kBulkStages = 4;          // row slots per warp
constexpr int kBulkMaxWarps = 8;
constexpr int kBulkSmemBudget = 200 * 1024;

struct Segment {  // one contiguous piece of a row
  const unsigned char* in;
  unsigned char* out;
  long long in_stride, out_stride;  // bytes between consecutive tokens
  unsigned bytes, slot_off;         // size, offset inside the row slot
};

__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_smem),
               "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void bulk_store(void* dst, uint32_t src_smem, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(reinterpret_cast<uint64_t>(dst)),
               "r"(src_smem), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// Segment `idx` of a row: [hidden] [K: one piece if packed, else one per head] [V: likewise].
__device__ __forceinline__ bool make_segment(const Shapes& s, const RowStreams& t, int idx, bool packed_k, bool packed_v, Segment& seg) {
  unsigned off = 0;
  int at = 0;
  if (t.hidden_in) {
    if (idx == at) {
      seg = {reinterpret_cast<const unsigned char*>(t.hidden_in), reinterpret_cast<unsigned char*>(t.hidden_out),
             (long long)s.hidden * 2, (long long)s.hidden * 2, (unsigned)s.hidden * 2, off};
      return true;
    }
    ++at;
    off += s.hidden * 2;
  }
  if (t.k_in) {
    const int pieces = packed_k ? 1 : s.hkv;
    if (idx < at + pieces) {
      const int h = idx - at;
      seg = {reinterpret_cast<const unsigned char*>(t.k_in + (long long)h * s.k_sh), reinterpret_cast<unsigned char*>(t.k_out + (long long)h * s.ko_sh),
             s.k_st * 2, s.ko_st * 2, (unsigned)((packed_k ? s.hkv : 1) * s.dim * 2), off + (unsigned)h * s.dim * 2};
      return true;
    }
    at += pieces;
    off += s.hkv * s.dim * 2;
  }
  if (t.v_in) {
    const int pieces = packed_v ? 1 : s.hkv;
    if (idx < at + pieces) {
      const int h = idx - at;
      seg = {reinterpret_cast<const unsigned char*>(t.v_in + (long long)h * s.v_sh), reinterpret_cast<unsigned char*>(t.v_out + (long long)h * s.vo_sh),
             s.v_st * 2, s.vo_st * 2, (unsigned)((packed_v ? s.hkv : 1) * s.dim * 2), off + (unsigned)h * s.dim * 2};
      return true;
    }
  }
  return false;
}

__global__ void __launch_bounds__(kBulkMaxWarps * 32, 1)
compact_rows_bulk_kernel(Shapes s, RowStreams t, const int32_t* __restrict__ keep_idx, const int32_t* __restrict__ cu_keep,
                         const int32_t* __restrict__ cu_seqlens, int n_segments, int packed_k, int packed_v, int row_bytes,
                         int32_t* device_status) {
  extern __shared__ __align__(128) unsigned char bulk_smem[];
  __shared__ uint64_t full[kBulkMaxWarps][kBulkStages];
  pdl_trigger();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, warps = blockDim.x >> 5;
  const uint32_t ring = ptx::smem_u32(bulk_smem) + (uint32_t)warp * kBulkStages * row_bytes;
  Segment seg{};
  const bool active = lane < n_segments && make_segment(s, t, lane, packed_k != 0, packed_v != 0, seg);
  if (lane == 0) {
    for (int i = 0; i < kBulkStages; ++i) ptx::mbar_init(ptx::smem_u32(&full[warp][i]), n_segments);
    ptx::fence_barrier_init();
  }
  __syncwarp();
  const bool global_idx = (s.flags & FASTAV_KEEP_IDX_GLOBAL) != 0;
  pdl_wait();  // keep_idx and cu_keep are the previous kernel's output
  pdl_acquire(keep_idx);
  pdl_acquire(cu_keep);
  int rows = chain_load_cached(cu_keep + s.batch);
  if (rows > s.total_keep) rows = s.total_keep;  // never write past the caller's buffers
  const int first = blockIdx.x * warps + warp, step = gridDim.x * warps;
  const int my_rows = first < rows ? (rows - first + step - 1) / step : 0;

  // Source token of this warp's i-th row, or -1 for an index outside its sequence (row skipped, reported).
  auto source_of = [&](int i) -> long long {
    const int row = first + i * step;
    int lo = 0, hi = s.batch;  // largest b with cu_keep[b] <= row
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (chain_load_cached(cu_keep + mid) <= row) lo = mid; else hi = mid;
    }
    const long long src = (global_idx ? 0ll : (long long)cu_seqlens[lo]) + chain_load(keep_idx + row);
    if (src < cu_seqlens[lo] || src >= cu_seqlens[lo + 1]) {
      if (lane == 0 && device_status) atomicOr(device_status, FASTAV_DEV_BAD_INDEX);
      return -1;
    }
    return src;
  };
  // Issue the loads of row i into slot i % stages (all lanes call; one lane per segment copies).
  auto issue_load = [&](int i) -> bool {
    const long long src = source_of(i);
    if (src < 0) {  // skipped row: the slot's barrier still completes its phase, so later rows keep their parity
      if (active) ptx::mbar_arrive(ptx::smem_u32(&full[warp][i % kBulkStages]));
      return false;
    }
    if (active) {
      const uint32_t bar = ptx::smem_u32(&full[warp][i % kBulkStages]);
      ptx::mbar_arrive_expect_tx(bar, seg.bytes);
      bulk_load(ring + (i % kBulkStages) * row_bytes + seg.slot_off, seg.in + src * seg.in_stride, seg.bytes, bar);
    }
    if (lane == 0 && t.pos_in) t.pos_out[first + i * step] = t.pos_in[src];
    return true;
  };

  int abort_flag = 0;
  unsigned loaded = 0;  // bit i % 32: row i has loads in flight or done (not skipped)
  constexpr int kAhead = kBulkStages - 2;  // rows loaded ahead of the one being stored
  for (int i = 0; i < min(kAhead, my_rows); ++i)
    if (issue_load(i)) loaded |= 1u << (i & 31);
  for (int i = 0; i < my_rows; ++i) {
    // The slot of row i + kAhead last held row i - 2: its store must have finished reading shared memory.
    if (i + kAhead < my_rows) {
      bulk_wait_read<1>();
      if (issue_load(i + kAhead)) loaded |= 1u << ((i + kAhead) & 31);
      else loaded &= ~(1u << ((i + kAhead) & 31));
    }
    if (loaded & (1u << (i & 31))) {
      const uint32_t bar = ptx::smem_u32(&full[warp][i % kBulkStages]);
      if (!ptx::mbar_wait_bounded(bar, (i / kBulkStages) & 1, &abort_flag)) {
        if (lane == 0 && device_status) atomicOr(device_status, FASTAV_DEV_WAIT_EXPIRED);
        break;
      }
      if (active) bulk_store(seg.out + (long long)(first + i * step) * seg.out_stride, ring + (i % kBulkStages) * row_bytes + seg.slot_off, seg.bytes);
    }
    bulk_commit();  // one group per row, empty or not, so that the wait above always counts rows
  }
  bulk_wait_all();  // the slots and the outputs are this kernel's until every store has landed
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
  // Bulk-copy path: every segment must be 16-byte friendly (it is: rows and strides are multiples of 8 elements),
  // a row must fit a slot, and there may be at most one segment per lane.
  const bool packed_k = k_in && s.k_sh == s.dim && s.ko_sh == s.dim, packed_v = v_in && s.v_sh == s.dim && s.vo_sh == s.dim;
  const int n_segments = (hidden_in ? 1 : 0) + (k_in ? (packed_k ? 1 : s.hkv) : 0) + (v_in ? (packed_v ? 1 : s.hkv) : 0);
  const int row_bytes = (hidden_in ? s.hidden * 2 : 0) + ((k_in ? 1 : 0) + (v_in ? 1 : 0)) * s.hkv * s.dim * 2;
  const int forced = (s.flags & FASTAV_COMPACT_PATH_MASK);
  if (forced != FASTAV_COMPACT_PATH_LOADSTORE && n_segments >= 1 && n_segments <= 32 && row_bytes > 0 &&
      kBulkStages * row_bytes <= kBulkSmemBudget) {
    int warps = kBulkSmemBudget / (kBulkStages * row_bytes);
    if (warps > kBulkMaxWarps) warps = kBulkMaxWarps;
    const size_t smem = (size_t)warps * kBulkStages * row_bytes;
    cudaError_t e = cudaFuncSetAttribute(compact_rows_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int blocks = (s.total_keep + warps - 1) / warps;
    if (blocks > kNumSMs) blocks = kNumSMs;
    e = launch_chained(compact_rows_bulk_kernel, dim3(blocks), dim3(warps * 32), smem, stream, s, t, keep_idx, cu_keep, cu_seqlens,
                       n_segments, (int)packed_k, (int)packed_v, row_bytes, device_status);
    count_launches(1);
    return e != cudaSuccess ? e : cudaGetLastError();
  }
  int blocks = kNumSMs * 8;
  if (blocks > s.total_keep) blocks = s.total_keep;
  const cudaError_t e = launch_chained(compact_rows_kernel, dim3(blocks), dim3(kThreads), 0, stream, s, t, keep_idx, cu_keep,
                                       cu_seqlens, device_status);
  count_launches(1);
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace fastav
