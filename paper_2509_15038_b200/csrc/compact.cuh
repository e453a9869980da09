// Gather of the selected rows into the compacted cache (Alg. 1 (gather step)):
// byte copies with 16-byte vectors, a half-warp per row (K in lanes 0-15, V in
// lanes 16-31), eight rows in flight per warp.
#pragma once
#include "common.cuh"

namespace curdkv {

struct CompactArgs {
  KvView K, V;
  const int32_t* seqlens;
  int heads, n_max, d;
  const int32_t* idx;
  int64_t idx_stride;
  const int32_t* counts;
  const int32_t* offsets;
  __nv_bfloat16* K_out;
  __nv_bfloat16* V_out;
  int64_t out_stride_h;     // > 0: fixed layout, 0: packed
  uint32_t* status;
  // Set when the launch may start before the kernel that selects has finished (programmatic
  // dependent launch behind the fused score + select kernel): ready[p] becomes non-zero once
  // head p's indices and count are written and fenced; a CTA waits for its head's entry.
  const int32_t* ready = nullptr;
  unsigned long long wait_ns = 2000000000ull;
};

constexpr int kCompactWarps = 8;
constexpr int kCompactRowsPerWarp = 8;
constexpr int kCompactRowsPerCta = kCompactWarps * kCompactRowsPerWarp;

// grid = batch*heads*ctas_per_head; the CTAs of a head stride over its rows.
// BEHIND: the launch is a programmatic dependent of the kernel that selects (a.ready is set).
template <bool BEHIND>
__global__ void __launch_bounds__(kCompactWarps * 32) compact_kernel(const CompactArgs a,
                                                                     const int ctas_per_head) {
  const int p = blockIdx.x / ctas_per_head, part = blockIdx.x % ctas_per_head;
  const int b = p / a.heads, h = p % a.heads;
  const int n = seq_len_of(a.seqlens, b, a.n_max);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, half = lane >> 4, l16 = lane & 15;
  const bool fixed = a.out_stride_h > 0;
  if constexpr (BEHIND) {
    __shared__ int head_missing;
    if (threadIdx.x == 0) {
      head_missing = 0;
      unsigned long long t0 = 0;
      for (uint32_t spin = 1; *(volatile const int32_t*)(a.ready + p) == 0; ++spin) {
        __nanosleep(500);
        if ((spin & 0x3fu) == 0) {
          const unsigned long long now = global_ns();
          if (t0 == 0) t0 = now;
          // the selecting kernel flags its own failures; here the head simply never arrived
          if ((*(volatile uint32_t*)a.status & CURDKV_DEV_TIMEOUT) != 0 || now - t0 > a.wait_ns) {
            flag_status(a.status, CURDKV_DEV_TIMEOUT);
            head_missing = 1;
            break;
          }
        }
      }
      __threadfence();                                     // the head's indices were written by another CTA
    }
    __syncthreads();
    if (head_missing) return;
  }
  // a count the layout cannot hold (a stale or unwritten counts buffer) is cut to what it can
  // hold and flagged, so that neither the index row nor the output rows of a neighbour are touched
  // (behind a kernel that may still be running, what it wrote is read from L2, not through the
  // read-only path)
  int count = BEHIND ? __ldcg(a.counts + p) : a.counts[p];
  const int64_t room = fixed ? (a.idx_stride < a.out_stride_h ? a.idx_stride : a.out_stride_h)
                             : (int64_t)a.offsets[p + 1] - a.offsets[p];
  if (count < 0 || count > room) {
    if (threadIdx.x == 0 && part == 0) flag_status(a.status, CURDKV_DEV_BAD_INDEX);
    count = count < 0 ? 0 : (int)(room > 0 ? room : 0);
  }
  const int32_t* ix = fixed ? a.idx + (size_t)p * a.idx_stride : a.idx + a.offsets[p];
  const size_t out_row0 = fixed ? (size_t)p * a.out_stride_h : (size_t)a.offsets[p];
  const KvView& T = half ? a.V : a.K;
  const __nv_bfloat16* src = T.base + b * T.stride_b + h * T.stride_h;
  __nv_bfloat16* dst = (half ? a.V_out : a.K_out) + out_row0 * a.d;
  const int chunks = a.d >> 3;

  for (int t0 = (part * kCompactWarps + warp) * kCompactRowsPerWarp; t0 < count;
       t0 += ctas_per_head * kCompactRowsPerCta) {
    // the warp's eight indices in one request (lane i holds the i-th), then handed round
    int mine = -1;
    if (lane < kCompactRowsPerWarp && t0 + lane < count) {
      mine = BEHIND ? __ldcg(ix + t0 + lane) : __ldg(ix + t0 + lane);
      if (mine < 0 || mine >= n) {
        flag_status(a.status, CURDKV_DEV_BAD_INDEX);
        mine = -1;
      }
    }
    int j[kCompactRowsPerWarp];
#pragma unroll
    for (int i = 0; i < kCompactRowsPerWarp; ++i) j[i] = __shfl_sync(0xffffffffu, mine, i);
    for (int c = l16; c < chunks; c += 16) {
      uint4 v[kCompactRowsPerWarp];
#pragma unroll
      for (int i = 0; i < kCompactRowsPerWarp; ++i)
        if (j[i] >= 0) v[i] = __ldg(reinterpret_cast<const uint4*>(src + j[i] * T.stride_n) + c);
#pragma unroll
      for (int i = 0; i < kCompactRowsPerWarp; ++i)
        if (j[i] >= 0) __stcs(reinterpret_cast<uint4*>(dst + (size_t)(t0 + i) * a.d) + c, v[i]);
    }
  }
}

// GQA group map (Sec. 3.2): query head q reads KV head q / (q_heads / kv_heads).
__global__ void gqa_map_kernel(int32_t* kv_head_of_q, int q_heads, int kv_heads) {
  const int q = blockIdx.x * blockDim.x + threadIdx.x;
  if (q < q_heads) kv_head_of_q[q] = q / (q_heads / kv_heads);
}

// Per-query-head copy of a fixed-layout selection: query head q of sequence b gets the indices
// and the count of its KV head (for attention code that wants one index list per query head).
// grid = batch*q_heads, block = 256.
__global__ void __launch_bounds__(256) gqa_expand_kernel(const int32_t* idx, const int32_t* counts,
                                                         int q_heads, int kv_heads, int budget,
                                                         int32_t* idx_q, int32_t* counts_q) {
  const int b = blockIdx.x / q_heads, q = blockIdx.x % q_heads;
  const int h = q / (q_heads / kv_heads);
  const int32_t* src = idx + ((size_t)b * kv_heads + h) * budget;
  int32_t* dst = idx_q + (size_t)blockIdx.x * budget;
  for (int t = threadIdx.x; t < budget; t += blockDim.x) dst[t] = src[t];
  if (threadIdx.x == 0) counts_q[blockIdx.x] = counts[b * kv_heads + h];
}

}  // namespace curdkv
