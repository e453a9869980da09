// Token selection (Alg. 1 lines 7-9 and AdaCurDKV, Sec. 3.2): forced sinks +
// window, then an exact top-k of the remaining scores by radix select on the
// fp32 bit patterns (scores are >= 0, so the patterns order like the values),
// ties to the lower token index, output in ascending token order.
#pragma once
#include <cooperative_groups.h>

#include "common.cuh"

namespace curdkv {

namespace cg = cooperative_groups;

constexpr int kSelThreads = 1024;
constexpr int kSelItems = 4;                               // consecutive tokens per thread
constexpr int kSelChunk = kSelThreads * kSelItems;
constexpr int kMaxAdaptiveHeads = 16;                      // one CTA per head in a cluster

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

// What the ordered compaction keeps besides the forced tokens: every candidate
// key above T and the first eq_take candidates (by token index) equal to T.
struct Cut {
  uint32_t T, eq_take;
  bool any;                                                // false: forced tokens only
};

// One radix-select step over a 256-bin digit histogram in shared memory.
// Finds the digit holding the `remaining`-th largest key, returns it, sets
// `remaining` to the rank inside that digit's bucket and `above` to the number
// of keys in higher bins.  Called by one full warp; all lanes get the results.
__device__ __forceinline__ uint32_t pick_digit(const uint32_t* hist, uint32_t& remaining,
                                               uint32_t& above_out) {
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
  uint32_t found = 0xffffffffu, rank = 0, found_above = 0;
#pragma unroll
  for (int u = 7; u >= 0; --u) {
    if (above < remaining && above + c[u] >= remaining) {
      found = lane * 8 + u;
      rank = remaining - above;
      found_above = above;
    }
    above += c[u];
  }
  const uint32_t who = __ballot_sync(0xffffffffu, found != 0xffffffffu);
  const int src = who ? __ffs(who) - 1 : 0;
  remaining = __shfl_sync(0xffffffffu, rank, src);
  above_out = __shfl_sync(0xffffffffu, found_above, src);
  return __shfl_sync(0xffffffffu, found, src);
}

// Number of keys in bins above `digit` (one full warp; all lanes get the sum).
__device__ __forceinline__ uint32_t count_above(const uint32_t* hist, uint32_t digit) {
  const int lane = threadIdx.x & 31;
  uint32_t s = 0;
#pragma unroll
  for (int u = 0; u < 8; ++u) {
    const uint32_t bin = lane * 8 + u;
    if (bin > digit) s += hist[bin];
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  return s;
}

// Adds the candidates [lo, hi) with key <= ceiling whose bits under `mask`
// equal `prefix` to the 256-bin histogram of digit (key >> shift).  Runs of
// equal digits are merged per thread before touching shared memory:
// normalised scores share their exponent bits, so the leading digits are
// nearly constant.
__device__ __forceinline__ void digit_histogram(const float* row, int lo, int hi, uint32_t ceiling,
                                                uint32_t mask, uint32_t prefix, int shift,
                                                uint32_t* hist) {
  uint32_t run_digit = 0, run = 0;
  for (int j = lo + threadIdx.x; j < hi; j += blockDim.x) {
    const uint32_t key = score_key(__ldg(row + j));
    if (key > ceiling || (key & mask) != prefix) continue;
    const uint32_t dgt = (key >> shift) & 0xffu;
    if (dgt == run_digit) { ++run; continue; }
    if (run) atomicAdd(&hist[run_digit], run);
    run_digit = dgt;
    run = 1;
  }
  if (run) atomicAdd(&hist[run_digit], run);
}

struct SelectSmem {
  uint32_t hist[256];
  uint32_t warp_tot[32];
  uint32_t digit, remaining, above;
};

// Top-kk cut of the candidates [lo, hi) of one row (0 < kk < hi - lo).  Whole CTA.
__device__ __forceinline__ Cut local_cut(const float* row, int lo, int hi, int kk, SelectSmem& sm) {
  const int tid = threadIdx.x;
  uint32_t prefix = 0, mask = 0, remaining = (uint32_t)kk;
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (tid < 256) sm.hist[tid] = 0;
    __syncthreads();
    digit_histogram(row, lo, hi, 0xffffffffu, mask, prefix, shift, sm.hist);
    __syncthreads();
    if (tid < 32) {
      uint32_t rem = remaining, above;
      const uint32_t dgt = pick_digit(sm.hist, rem, above);
      if (tid == 0) { sm.digit = dgt; sm.remaining = rem; }
    }
    __syncthreads();
    prefix |= sm.digit << shift;
    mask |= 0xffu << shift;
    remaining = sm.remaining;
    __syncthreads();
  }
  return Cut{prefix, remaining, true};
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

// Ordered compaction of one row: forced tokens, keys above cut.T and the first
// cut.eq_take keys equal to cut.T, written to `out` in ascending token order.
__device__ __forceinline__ void ordered_compact(const float* row, int n, const ForcedSet& F,
                                                const Cut& cut, int32_t* out, SelectSmem& sm) {
  const int tid = threadIdx.x;
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
        } else if (cut.any) {
          const uint32_t key = score_key(__ldg(row + jj));
          if (key > cut.T) def_f |= 1u << i;
          else if (key == cut.T) eq_f |= 1u << i;
        }
      }
    }
    uint32_t total;
    const uint32_t exc = block_scan_packed(
        (uint32_t)__popc(def_f) | ((uint32_t)__popc(eq_f) << 16), sm.warp_tot, total);
    uint32_t def_before = def_base + (exc & 0xffffu);
    uint32_t eq_before = eq_base + (exc >> 16);
#pragma unroll
    for (int i = 0; i < kSelItems; ++i) {
      if (def_f & (1u << i)) {
        out[def_before + min(eq_before, cut.eq_take)] = j + i;
        ++def_before;
      } else if (eq_f & (1u << i)) {
        if (eq_before < cut.eq_take) out[def_before + eq_before] = j + i;
        ++eq_before;
      }
    }
    def_base += total & 0xffffu;
    eq_base += total >> 16;
  }
}

// ---------------------------------------------------------------------------
// Fixed per-head budget.  grid = batch*heads, block = 1024.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(kSelThreads) select_fixed_kernel(
    const float* __restrict__ scores, const int32_t* __restrict__ seqlens, int heads, int n_max,
    int budget, const int32_t* __restrict__ head_budgets, int num_sink, int window,
    int32_t* __restrict__ idx, int32_t* __restrict__ counts, int32_t* __restrict__ offsets) {
  __shared__ SelectSmem sm;
  const int p = blockIdx.x, b = p / heads, tid = threadIdx.x;
  const int n = seq_len_of(seqlens, b, n_max);
  int k = budget;
  if (head_budgets != nullptr) k = max(0, min(head_budgets[p], budget));
  const int k_eff = min(k, n);
  const ForcedSet F = forced_set(n, k_eff, num_sink, window);
  const float* row = scores + (size_t)p * n_max;
  int32_t* out = idx + (size_t)p * budget;
  const int cand = F.hi - F.sinks;

  Cut cut{0u, 0u, F.free_slots > 0};
  if (F.free_slots >= cand) cut.eq_take = (uint32_t)max(cand, 0);   // every candidate is kept
  else if (cut.any) cut = local_cut(row, F.sinks, F.hi, F.free_slots, sm);

  ordered_compact(row, n, F, cut, out, sm);
  for (int t = k_eff + tid; t < budget; t += kSelThreads) out[t] = -1;
  if (tid == 0) {
    counts[p] = k_eff;
    if (offsets != nullptr) {                              // heads sit at multiples of `budget` rows
      offsets[p] = p * budget;
      if (p == (int)gridDim.x - 1) offsets[p + 1] = (p + 1) * budget;
    }
  }
}

// ---------------------------------------------------------------------------
// AdaCurDKV.  One thread-block cluster per (layer, sequence), one CTA per KV
// head.  Every head first protects its forced tokens and its best tokens up to
// p = min(max(floor(alpha k), forced), k_eff); the remaining heads*(k_eff - p)
// slots go to the best unprotected keys of all heads (ties: lower head, then
// lower token), found by a radix select whose digit histograms are summed
// across the cluster through distributed shared memory.
// grid = batch*heads, cluster = heads, block = 1024.
// ---------------------------------------------------------------------------
struct AdaptiveSmem {
  SelectSmem s;
  uint32_t hist_local[256];                                // read by the other CTAs of the cluster
  uint32_t pub_eq;                                         // unprotected keys equal to the global cut
  uint32_t pub_count;                                      // rows this head keeps
};

__global__ void __launch_bounds__(kSelThreads) select_adaptive_kernel(
    const float* __restrict__ scores, const int32_t* __restrict__ seqlens, int heads, int n_max,
    int budget, int num_sink, int window, int min_protected, int32_t* __restrict__ idx,
    int32_t* __restrict__ counts, int32_t* __restrict__ offsets) {
  __shared__ AdaptiveSmem sm;
  cg::cluster_group cluster = cg::this_cluster();
  const int tid = threadIdx.x;
  const int h = (int)cluster.block_rank();
  const int b = blockIdx.x / heads, p = b * heads + h;
  const int n = seq_len_of(seqlens, b, n_max);
  const int k_eff = min(budget, n);
  const ForcedSet F = forced_set(n, k_eff, num_sink, window);
  const float* row = scores + (size_t)p * n_max;
  const int cand = F.hi - F.sinks;
  const int forced = k_eff - F.free_slots;
  const int prot = min(max(min_protected, forced), k_eff);  // protected rows per head, forced included
  const int pp = prot - forced;                             // protected candidates

  // ---- this head's safeguard share
  const bool prot_all = pp >= cand;                         // every candidate is protected
  const bool prot_none = pp == 0 && !prot_all;
  Cut own{0u, 0u, false};
  if (!prot_all && !prot_none) own = local_cut(row, F.sinks, F.hi, pp, sm.s);
  // unprotected keys: candidates with key <= ceiling, minus the first own.eq_take equal to it
  const uint32_t ceiling = prot_none ? 0xffffffffu : own.T;

  // ---- layer-wide cut over the unprotected keys of all heads
  const uint32_t pool = (uint32_t)heads * (uint32_t)(k_eff - prot);
  uint32_t Tg = 0, eq_g = 0, local_gt = 0, local_eq = 0;
  if (pool > 0) {
    uint32_t prefix = 0, mask = 0, remaining = pool;
    for (int shift = 24; shift >= 0; shift -= 8) {
      if (tid < 256) sm.hist_local[tid] = 0;
      __syncthreads();
      if (!prot_all) digit_histogram(row, F.sinks, F.hi, ceiling, mask, prefix, shift, sm.hist_local);
      __syncthreads();
      if (tid == 0 && !prot_all && !prot_none && (own.T & mask) == prefix)
        sm.hist_local[(own.T >> shift) & 0xffu] -= own.eq_take;   // those are protected
      cluster.sync();
      if (tid < 256) {
        uint32_t s = 0;
        for (int r = 0; r < heads; ++r) s += cluster.map_shared_rank(sm.hist_local, r)[tid];
        sm.s.hist[tid] = s;
      }
      __syncthreads();
      if (tid < 32) {
        uint32_t rem = remaining, above;
        const uint32_t dgt = pick_digit(sm.s.hist, rem, above);
        const uint32_t mine_above = count_above(sm.hist_local, dgt);
        if (tid == 0) { sm.s.digit = dgt; sm.s.remaining = rem; sm.s.above = mine_above; }
      }
      __syncthreads();
      prefix |= sm.s.digit << shift;
      mask |= 0xffu << shift;
      remaining = sm.s.remaining;
      local_gt += sm.s.above;
      if (shift == 0) local_eq = sm.hist_local[sm.s.digit];
      cluster.sync();                                      // peers are done reading hist_local
    }
    Tg = prefix;
    eq_g = remaining;
  }
  // share of the keys equal to the global cut: lower heads first
  if (tid == 0) sm.pub_eq = local_eq;
  cluster.sync();
  uint32_t eq_before_me = 0;
  for (int r = 0; r < h; ++r) eq_before_me += *cluster.map_shared_rank(&sm.pub_eq, r);
  const uint32_t e_h = eq_g > eq_before_me ? min(eq_g - eq_before_me, local_eq) : 0u;

  // ---- this head's final cut and row count
  Cut cut;
  uint32_t kept;
  if (prot_all) {
    cut = Cut{0u, (uint32_t)max(cand, 0), cand > 0};
    kept = (uint32_t)(forced + max(cand, 0));
  } else {
    kept = (uint32_t)prot + local_gt + e_h;
    if (pool == 0) cut = Cut{own.T, own.eq_take, !prot_none};
    else if (prot_none || Tg < own.T) cut = Cut{Tg, e_h, true};
    else if (Tg == own.T) cut = Cut{own.T, own.eq_take + e_h, true};
    else cut = Cut{own.T, own.eq_take, true};
  }
  if (tid == 0) sm.pub_count = kept;
  cluster.sync();

  // ---- packed output position: rows of earlier sequences, then earlier heads
  uint32_t part = 0;
  for (int bb = tid; bb < b; bb += kSelThreads)
    part += (uint32_t)heads * (uint32_t)min(budget, seq_len_of(seqlens, bb, n_max));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
  if ((tid & 31) == 0) sm.s.warp_tot[tid >> 5] = part;
  __syncthreads();
  uint32_t off = 0;
  for (int w = 0; w < kSelThreads / 32; ++w) off += sm.s.warp_tot[w];
  for (int r = 0; r < h; ++r) off += *cluster.map_shared_rank(&sm.pub_count, r);
  __syncthreads();

  ordered_compact(row, n, F, cut, idx + off, sm.s);
  if (tid == 0) {
    counts[p] = (int32_t)kept;
    offsets[p] = (int32_t)off;
    if (p == (int)gridDim.x - 1) offsets[p + 1] = (int32_t)(off + kept);
  }
  cluster.sync();                                          // keep shared memory alive for peers
}

}  // namespace curdkv
