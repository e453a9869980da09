// Shared device/host helpers of the CurDKV kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "curdkv.h"

namespace curdkv {

// Rows of one (batch, head) problem are processed in tiles of this many tokens;
// every tile leaves one fp32 partial sum of its scores in the workspace.
constexpr int kTileRows = 128;

// Workspace layout: [0, 256) status words, then tile partial sums.
constexpr size_t kStatusBytes = 256;

// Adds one to the library's launch counter (defined beside the C ABI).
void count_launch();

// curdkv_score without its last step: `scores` receive l^K l^V (Alg. 1 (product step)) as the score
// kernels leave them, entries at or beyond a sequence's length are unspecified, head sums are not
// formed.  For callers that read the valid entries only (defined beside the C ABI).
curdkv_status score_unnormalised(const void* K, const void* V, const float* G, int32_t g_per_head,
                                 const curdkv_desc* desc, float* scores, void* workspace,
                                 size_t workspace_bytes, void* cuda_stream);

struct KvView {          // one bf16 tensor [batch][heads][n_max][d], strides in elements
  const __nv_bfloat16* base;
  int64_t stride_b, stride_h, stride_n;
};

__device__ __forceinline__ int seq_len_of(const int32_t* seqlens, int b, int n_max) {
  if (seqlens == nullptr) return n_max;
  int n = seqlens[b];
  return n < 0 ? 0 : (n > n_max ? n_max : n);
}

__device__ __forceinline__ void flag_status(uint32_t* status, uint32_t bits) {
  if (status != nullptr) atomicOr(status, bits);
}

// Nanoseconds of the device-wide timer (the clock every bounded wait is measured on).
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Eight bf16 values packed in a 16-byte vector -> fp32.
__device__ __forceinline__ void unpack_bf16x8(const uint4& v, float (&f)[8]) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(w[i] << 16);
    f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}

__device__ __forceinline__ float combine_scores(float lk, float lv, int score_mode) {
  return score_mode == 1 ? lk : (score_mode == 2 ? lv : lk * lv);
}

}  // namespace curdkv
