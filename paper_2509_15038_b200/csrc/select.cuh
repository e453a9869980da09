// Token selection (Alg. 1 lines 7-9): forced sinks + window, then an exact
// top-k of the remaining scores by radix select on the fp32 bit patterns
// (scores are >= 0, so the patterns order like the values), ties to the lower
// token index, output in ascending token order.
#pragma once
#include "common.cuh"

namespace curdkv {

constexpr int kSelThreads = 1024;
constexpr int kSelItems = 4;                               // consecutive tokens per thread
constexpr int kSelChunk = kSelThreads * kSelItems;

// NaN and non-positive scores rank as 0.
__device__ __forceinline__ uint32_t score_key(float s) { return s > 0.f ? __float_as_uint(s) : 0u; }

// The forced-keep set of a sequence of n rows under a budget of k_eff rows:
// sinks [0, sinks) and window [hi, n); candidates are [sinks, hi).
struct ForcedSet {
  int sinks, hi, free_slots;
};

__device__ __forceinline__ ForcedSet forced_set(int n, int k_eff, int num_sink, int window) {
  ForcedSet f;
  const int w_eff = min(window, k_eff);                    // k_eff <= n
  const int s_cand = min(num_sink, n - w_eff);
  f.sinks = min(s_cand, k_eff - w_eff);
  f.hi = n - w_eff;
  f.free_slots = k_eff - w_eff - f.sinks;
  return f;
}

// One radix-select step over an 8-bit digit histogram held in shared memory.
// Finds the digit holding the `remaining`-th largest key, returns it and
// updates `remaining` to the rank inside that digit's bucket.  Called by one
// full warp; every lane returns the same values.
__device__ __forceinline__ uint32_t pick_digit(const uint32_t* hist, uint32_t& remaining) {
  const int lane = threadIdx.x & 31;
  uint32_t c[8], mine = 0;
#pragma unroll
  for (int u = 0; u < 8; ++u) { c[u] = hist[lane * 8 + u]; mine += c[u]; }
  uint32_t above = mine;                                   // inclusive suffix sum over lanes
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t v = __shfl_down_sync(0xffffffffu, above, o);
    if (lane + o < 32) above += v;
  }
  above -= mine;                                           // keys in higher lanes' bins
  uint32_t found = 0xffffffffu, rank = 0;
#pragma unroll
  for (int u = 7; u >= 0; --u) {
    if (above < remaining && above + c[u] >= remaining) { found = lane * 8 + u; rank = remaining - above; }
    above += c[u];
  }
  const uint32_t who = __ballot_sync(0xffffffffu, found != 0xffffffffu);
  const int src = who ? __ffs(who) - 1 : 0;
  remaining = __shfl_sync(0xffffffffu, rank, src);
  return __shfl_sync(0xffffffffu, found, src);
}

// Adds the keys of candidates [lo, hi) whose bits under `mask` equal `prefix`
// to the 256-bin histogram of digit (key >> shift).  Runs of equal digits are
// merged per thread before touching shared memory: normalised scores share
// their exponent bits, so the leading digits are nearly constant.
__device__ __forceinline__ void digit_histogram(const float* row, int lo, int hi, uint32_t mask,
                                                uint32_t prefix, int shift, uint32_t* hist) {
  uint32_t run_digit = 0, run = 0;
  for (int j = lo + threadIdx.x; j < hi; j += blockDim.x) {
    const uint32_t key = score_key(__ldg(row + j));
    if ((key & mask) != prefix) continue;
    const uint32_t dgt = (key >> shift) & 0xffu;
    if (dgt == run_digit) { ++run; continue; }
    if (run) atomicAdd(&hist[run_digit], run);
    run_digit = dgt;
    run = 1;
  }
  if (run) atomicAdd(&hist[run_digit], run);
}

// Exclusive block scan of a packed (lo16 | hi16 << 16) counter; returns the
// exclusive prefix of this thread and the block total.  blockDim = 1024.
__device__ __forceinline__ uint32_t block_scan_packed(uint32_t v, uint32_t* warp_tot,
                                                      uint32_t& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  if (lane == 31) warp_tot[warp] = inc;
  __syncthreads();
  uint32_t w = warp_tot[lane];
  uint32_t winc = w;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t t = __shfl_up_sync(0xffffffffu, winc, o);
    if (lane >= o) winc += t;
  }
  total = __shfl_sync(0xffffffffu, winc, 31);
  const uint32_t wexc = __shfl_sync(0xffffffffu, winc - w, warp);
  __syncthreads();                                         // warp_tot may be reused
  return wexc + inc - v;
}

// ---------------------------------------------------------------------------
// Fixed per-head budget.  grid = batch*heads, block = 1024.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(kSelThreads) select_fixed_kernel(
    const float* __restrict__ scores, const int32_t* __restrict__ seqlens, int heads, int n_max,
    int budget, const int32_t* __restrict__ head_budgets, int num_sink, int window,
    int32_t* __restrict__ idx, int32_t* __restrict__ counts, int32_t* __restrict__ offsets) {
  __shared__ uint32_t hist[256];
  __shared__ uint32_t warp_tot[32];
  __shared__ uint32_t s_digit, s_remaining;

  const int p = blockIdx.x, b = p / heads, tid = threadIdx.x;
  const int n = seq_len_of(seqlens, b, n_max);
  int k = budget;
  if (head_budgets != nullptr) k = max(0, min(head_budgets[p], budget));
  const int k_eff = min(k, n);
  const ForcedSet F = forced_set(n, k_eff, num_sink, window);
  const float* row = scores + (size_t)p * n_max;
  int32_t* out = idx + (size_t)p * budget;

  // threshold key T and how many candidates equal to T are taken
  uint32_t T = 0, eq_take = 0;
  bool any = F.free_slots > 0;
  if (F.free_slots >= F.hi - F.sinks) {                    // every candidate is kept
    T = 0;
    eq_take = (uint32_t)max(F.hi - F.sinks, 0);
  } else if (any) {
    uint32_t prefix = 0, mask = 0, remaining = (uint32_t)F.free_slots;
    for (int shift = 24; shift >= 0; shift -= 8) {
      if (tid < 256) hist[tid] = 0;
      __syncthreads();
      digit_histogram(row, F.sinks, F.hi, mask, prefix, shift, hist);
      __syncthreads();
      if (tid < 32) {
        uint32_t rem = remaining;
        const uint32_t dgt = pick_digit(hist, rem);
        if (tid == 0) { s_digit = dgt; s_remaining = rem; }
      }
      __syncthreads();
      prefix |= s_digit << shift;
      mask |= 0xffu << shift;
      remaining = s_remaining;
      __syncthreads();
    }
    T = prefix;
    eq_take = remaining;
  }

  // ordered compaction: forced tokens, keys above T, and the first eq_take keys equal to T
  uint32_t def_base = 0, eq_base = 0;
  for (int j0 = 0; j0 < n; j0 += kSelChunk) {
    const int j = j0 + tid * kSelItems;
    uint32_t def_f = 0, eq_f = 0;                          // bit i: item i
#pragma unroll
    for (int i = 0; i < kSelItems; ++i) {
      const int jj = j + i;
      if (jj < n) {
        const bool forced = jj < F.sinks || jj >= F.hi;
        if (forced) {
          def_f |= 1u << i;
        } else if (any) {
          const uint32_t key = score_key(__ldg(row + jj));
          if (key > T) def_f |= 1u << i;
          else if (key == T) eq_f |= 1u << i;
        }
      }
    }
    uint32_t total;
    const uint32_t exc =
        block_scan_packed((uint32_t)__popc(def_f) | ((uint32_t)__popc(eq_f) << 16), warp_tot, total);
    uint32_t def_before = def_base + (exc & 0xffffu);
    uint32_t eq_before = eq_base + (exc >> 16);
#pragma unroll
    for (int i = 0; i < kSelItems; ++i) {
      if (def_f & (1u << i)) {
        out[def_before + min(eq_before, eq_take)] = j + i;
        ++def_before;
      } else if (eq_f & (1u << i)) {
        if (eq_before < eq_take) out[def_before + eq_before] = j + i;
        ++eq_before;
      }
    }
    def_base += total & 0xffffu;
    eq_base += total >> 16;
  }
  for (int t = k_eff + tid; t < budget; t += kSelThreads) out[t] = -1;
  if (tid == 0) {
    counts[p] = k_eff;
    if (offsets != nullptr) {
      // fixed layout: heads sit at multiples of `budget` rows
      offsets[p] = p * budget;
      if (p == gridDim.x - 1) offsets[p + 1] = (p + 1) * budget;
    }
  }
}

}  // namespace curdkv
