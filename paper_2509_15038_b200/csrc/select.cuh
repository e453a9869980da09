// Token selection (Alg. 1 (sinks, top-k, union) and AdaCurDKV, Sec. 3.2): forced sinks +
// window, then an exact top-k of the remaining scores by radix select on the
// fp32 bit patterns (scores are >= 0, so the patterns order like the values),
// ties to the lower token index, output in ascending token order.
//
// Every token of a row gets a 32-bit rank key:
//   0             position at or beyond the sequence length (never kept)
//   bits(s) + 1   candidate with score s (NaN and s <= 0 rank as score 0)
//   0xffffffff    forced token (sink or window; always kept)
// so "keep the forced tokens and the best k - |forced| candidates" becomes
// "keep the k largest keys", and no pass needs the token index again.
#pragma once
#include <cooperative_groups.h>

#include "common.cuh"

namespace curdkv {

namespace cg = cooperative_groups;

constexpr int kSelThreads = 1024;
constexpr int kSelStageBytes = 144 * 1024;                 // largest row copy kept in shared memory
// After the leading digit of a cut is known, the keys that share it (a few per cent of a row)
// are copied with their token index into a list in shared memory; the remaining digits, the
// tie count and the per-warp totals of the compaction then come from the list instead of from
// further sweeps over the row.  A list that overflows falls back to sweeping.
constexpr int kSelListCap = 6144;                          // (key, index) pairs per list
constexpr int kSelListBytes = kSelListCap * 8;
constexpr int kMaxAdaptiveHeads = 16;                      // one CTA per head in a cluster
constexpr uint32_t kForcedKey = 0xffffffffu;

__device__ __forceinline__ uint32_t score_key(float s) { return s > 0.f ? __float_as_uint(s) + 1u : 1u; }

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

// What the ordered compaction keeps: every key above T and the first eq_take
// keys (by token index) equal to T.
struct Cut {
  uint32_t T, eq_take;
};
__device__ __forceinline__ Cut keep_nothing() { return Cut{0xffffffffu, 0u}; }
__device__ __forceinline__ Cut keep_forced_only() { return Cut{0xfffffffeu, 0u}; }
__device__ __forceinline__ Cut keep_every_token() { return Cut{0u, 0u}; }

// The keys are consumed most significant digit first in three radix passes of
// 12, 12 and 8 bits.  A wide leading digit matters: normalised scores of one
// head span only a few binades, so an 8-bit leading digit would send nearly
// every key to the same two or three histogram bins and serialise the
// shared-memory atomics.
constexpr int kSelPasses = 3;
constexpr int kSelBins = 4096;
__device__ __forceinline__ int pass_shift(int pass) { return pass == 0 ? 20 : (pass == 1 ? 8 : 0); }
__device__ __forceinline__ uint32_t pass_digit_mask(int pass) { return pass == 2 ? 0xffu : 0xfffu; }

struct SelectSmem {
  alignas(16) uint32_t hist[kSelBins];                     // read and cleared as 16-byte vectors
  uint32_t warp_def[32], warp_eq[32];
  uint32_t seg_def[32], seg_eq[32];                        // per-segment totals of the compaction
  uint32_t digit, remaining, above;
  uint32_t list_count[2];
};

struct KeyList {
  uint2* items;            // (rank key, token index)
  uint32_t* count;         // entries offered; more than cap means the list is incomplete
  uint32_t cap;
  __device__ __forceinline__ bool complete() const { return *count <= cap; }
  __device__ __forceinline__ int size() const { return (int)min(*count, cap); }
};

// The helpers below are written for a group G of threads that works on one row together: a whole
// CTA, or a run of warps inside a larger, warp-specialised CTA (the fused score + select kernel).
// G supplies the thread's rank in the group, the group's size and its barrier.  Sizes: 1024 threads
// (four histogram bins per thread), 512 (eight; short rows run as two such CTAs per SM, which hides
// more of the latency of their many short phases) or 256 (sixteen).
struct WholeCta {
  static constexpr int kUnroll = 4;                        // quads in flight per thread
  static __device__ __forceinline__ int tid() { return (int)threadIdx.x; }
  static __device__ __forceinline__ int size() { return (int)blockDim.x; }
  static __device__ __forceinline__ void sync() { __syncthreads(); }
};
// Threads [FIRST, FIRST + N) of the CTA, synchronised by the named hardware barrier BAR.
template <int FIRST, int N, int BAR>
struct WarpRange {
  static_assert(N % 32 == 0 && FIRST % 32 == 0 && BAR >= 1 && BAR <= 15, "whole warps, a free barrier");
  static constexpr int kUnroll = 4;                        // (eight spill under this kernel's register cap)
  static __device__ __forceinline__ int tid() { return (int)threadIdx.x - FIRST; }
  static __device__ __forceinline__ int size() { return N; }
  static __device__ __forceinline__ void sync() { asm volatile("bar.sync %0, %1;" ::"n"(BAR), "n"(N) : "memory"); }
};

template <class G>
__device__ __forceinline__ void clear_hist(uint32_t* hist) {
  for (int i = G::tid(); i < kSelBins / 4; i += G::size())
    reinterpret_cast<uint4*>(hist)[i] = make_uint4(0u, 0u, 0u, 0u);
}

// One radix-select step over the kSelBins-bin histogram `hist`: finds the digit
// holding the `remaining`-th largest key and leaves it in sm.digit, the rank
// inside that digit's bucket in sm.remaining and the number of keys in higher
// bins in sm.above.  Whole CTA (B consecutive bins per thread); the results are
// readable after the call.
template <class G, int B>
__device__ __forceinline__ void pick_digit_impl(const uint32_t* hist, uint32_t remaining, SelectSmem& sm) {
  constexpr int kWarps = kSelBins / (32 * B);
  const int tid = G::tid(), lane = tid & 31, warp = tid >> 5;
  uint32_t c[B];
#pragma unroll
  for (int q = 0; q < B / 4; ++q) {
    const uint4 c4 = reinterpret_cast<const uint4*>(hist)[tid * (B / 4) + q];
    c[4 * q] = c4.x; c[4 * q + 1] = c4.y; c[4 * q + 2] = c4.z; c[4 * q + 3] = c4.w;
  }
  uint32_t mine = 0;
#pragma unroll
  for (int u = 0; u < B; ++u) mine += c[u];
  uint32_t suffix = mine;                                  // inclusive suffix sum over the warp
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t v = __shfl_down_sync(0xffffffffu, suffix, o);
    if (lane + o < 32) suffix += v;
  }
  if (lane == 0) sm.warp_def[warp] = suffix;
  if (tid == 0) { sm.digit = 0; sm.remaining = 0; sm.above = 0; }
  G::sync();
  uint32_t w = lane < kWarps ? sm.warp_def[lane] : 0u, wsuf = w;   // inclusive suffix sum over the warps
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t v = __shfl_down_sync(0xffffffffu, wsuf, o);
    if (lane + o < 32) wsuf += v;
  }
  uint32_t above = __shfl_sync(0xffffffffu, wsuf - w, warp) + (suffix - mine);
#pragma unroll
  for (int u = B - 1; u >= 0; --u) {
    if (above < remaining && above + c[u] >= remaining) {
      sm.digit = (uint32_t)(tid * B + u);
      sm.remaining = remaining - above;
      sm.above = above;
    }
    above += c[u];
  }
  G::sync();
}
template <class G>
__device__ __forceinline__ void pick_digit(const uint32_t* hist, uint32_t remaining, SelectSmem& sm) {
  if (G::size() == 1024) pick_digit_impl<G, 4>(hist, remaining, sm);
  else if (G::size() == 512) pick_digit_impl<G, 8>(hist, remaining, sm);
  else pick_digit_impl<G, 16>(hist, remaining, sm);
}

// Number of keys of `hist` in bins above `digit`.  Whole CTA; every thread gets the sum.
template <class G, int B>
__device__ __forceinline__ uint32_t count_above_impl(const uint32_t* hist, uint32_t digit, SelectSmem& sm) {
  constexpr int kWarps = kSelBins / (32 * B);
  const int tid = G::tid(), lane = tid & 31, warp = tid >> 5;
  uint32_t v = 0;
#pragma unroll
  for (int u = 0; u < B; ++u)
    if ((uint32_t)(tid * B + u) > digit) v += hist[tid * B + u];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if (lane == 0) sm.warp_eq[warp] = v;
  G::sync();
  uint32_t t = lane < kWarps ? sm.warp_eq[lane] : 0u;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
  G::sync();
  return t;
}
template <class G>
__device__ __forceinline__ uint32_t count_above(const uint32_t* hist, uint32_t digit, SelectSmem& sm) {
  if (G::size() == 1024) return count_above_impl<G, 4>(hist, digit, sm);
  if (G::size() == 512) return count_above_impl<G, 8>(hist, digit, sm);
  return count_above_impl<G, 16>(hist, digit, sm);
}

// Rank keys of one row, four tokens at a time ("quad" q holds tokens
// 4q .. 4q+3).  They come from the copy staged in shared memory when the row
// fits there, otherwise they are rebuilt from the fp32 scores in global memory
// (16-byte loads when the row is aligned).
struct RowKeys {
  const float* row;
  const uint4* staged;                                     // nullptr: read global memory
  int n, sinks, hi;                                        // candidates are [sinks, hi)
  bool vec;                                                // row is 16-byte aligned
  bool written_here = false;                               // the row was written by this kernel: read it
                                                           // from L2, never through the read-only path

  __device__ __forceinline__ int quads() const { return (n + 3) >> 2; }

  __device__ __forceinline__ uint32_t key_of(float s, int j) const {
    if (j >= n) return 0u;
    if (j < sinks || j >= hi) return kForcedKey;
    return score_key(s);
  }

  __device__ __forceinline__ uint4 load4(int q) const {
    if (staged != nullptr) return staged[q];
    const int j = 4 * q;
    if (vec && j >= sinks && j + 3 < hi) {                 // interior quad: four candidates
      const float4* at = reinterpret_cast<const float4*>(row) + q;
      const float4 f = written_here ? __ldcg(at) : __ldg(at);
      return make_uint4(score_key(f.x), score_key(f.y), score_key(f.z), score_key(f.w));
    }
    float f[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) f[i] = j + i < n ? (written_here ? __ldcg(row + j + i) : __ldg(row + j + i)) : 0.f;
    return make_uint4(key_of(f[0], j), key_of(f[1], j + 1), key_of(f[2], j + 2), key_of(f[3], j + 3));
  }
};

__device__ __forceinline__ RowKeys global_keys(const float* row, int n, const ForcedSet& F) {
  return RowKeys{row, nullptr, n, F.sinks, F.hi, (reinterpret_cast<uintptr_t>(row) & 15u) == 0, false};
}

// Running (digit, count) pair of one thread: equal neighbouring digits are
// merged before they reach the shared-memory histogram, which keeps runs of
// equal scores (padding, constant rows) from hammering one bin.
struct DigitRun {
  uint32_t digit = 0, count = 0;
  __device__ __forceinline__ void add(uint32_t d, uint32_t* hist) {
    if (d == digit) { ++count; return; }
    if (count) atomicAdd(&hist[digit], count);
    digit = d;
    count = 1;
  }
  __device__ __forceinline__ void flush(uint32_t* hist) {
    if (count) atomicAdd(&hist[digit], count);
    count = 0;
  }
};

constexpr int kSelRankDirect = 192;                        // lists up to this size are ranked without histograms

// Adds the keys <= ceiling whose bits under `mask` equal `prefix` to the
// histogram of this pass's digit.  Whole CTA.
template <class G>
__device__ __forceinline__ void digit_histogram(const RowKeys& keys, uint32_t ceiling, uint32_t mask,
                                                uint32_t prefix, int pass, uint32_t* hist) {
  const int quads = keys.quads(), step = (int)G::size();
  const int shift = pass_shift(pass);
  const uint32_t dmask = pass_digit_mask(pass);
  DigitRun run;
  for (int q0 = (int)G::tid(); q0 < quads; q0 += G::kUnroll * step) {
    uint4 v[G::kUnroll];
#pragma unroll
    for (int u = 0; u < G::kUnroll; ++u)
      if (q0 + u * step < quads) v[u] = keys.load4(q0 + u * step);
#pragma unroll
    for (int u = 0; u < G::kUnroll; ++u) {
      if (q0 + u * step < quads) {
        const uint32_t k4[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint32_t key = k4[i];
          if (pass == 0) {                                 // every key takes part: merge runs
            if (key <= ceiling) run.add(key >> shift, hist);
          } else if ((key & mask) == prefix && key <= ceiling) {
            atomicAdd(&hist[(key >> shift) & dmask], 1u);  // few keys share the prefix
          }
        }
      }
    }
  }
  run.flush(hist);
}

// Copies the rank keys of a row into shared memory and, on the way, builds the
// histogram of their leading digit.  Whole CTA; hist must be zero on entry.
template <class G>
__device__ __forceinline__ void stage_keys(const RowKeys& src, uint4* staged, uint32_t* hist) {
  const int quads = src.quads(), step = (int)G::size();
  DigitRun run;
  for (int q0 = (int)G::tid(); q0 < quads; q0 += G::kUnroll * step) {
    uint4 v[G::kUnroll];
#pragma unroll
    for (int u = 0; u < G::kUnroll; ++u)
      if (q0 + u * step < quads) v[u] = src.load4(q0 + u * step);
#pragma unroll
    for (int u = 0; u < G::kUnroll; ++u) {
      if (q0 + u * step < quads) {
        staged[q0 + u * step] = v[u];
        run.add(v[u].x >> 20, hist);
        run.add(v[u].y >> 20, hist);
        run.add(v[u].z >> 20, hist);
        run.add(v[u].w >> 20, hist);
      }
    }
  }
  run.flush(hist);
}

// Quads of a row are dealt to the CTA's warps in contiguous runs ("segments"), so that the kept
// tokens of warp w precede those of warp w + 1 in token order.
struct Segments {
  int per_warp, quads;
  __device__ __forceinline__ Segments(int quads_, int warps) : quads(quads_) {
    per_warp = ((quads_ + warps - 1) / warps + 31) & ~31;  // whole-warp sweeps
  }
  __device__ __forceinline__ int begin(int warp) const { return min(warp * per_warp, quads); }
  __device__ __forceinline__ int end(int warp) const { return min(begin(warp) + per_warp, quads); }
  __device__ __forceinline__ int of_token(uint32_t j) const { return (int)(j >> 2) / per_warp; }
};

// flags of the four tokens of a quad: bits 0-3 key above T, bits 4-7 key equal to T
__device__ __forceinline__ uint32_t classify(const uint4& v, uint32_t T) {
  return (v.x > T ? 1u : 0u) | (v.y > T ? 2u : 0u) | (v.z > T ? 4u : 0u) | (v.w > T ? 8u : 0u) |
         (v.x == T ? 16u : 0u) | (v.y == T ? 32u : 0u) | (v.z == T ? 64u : 0u) | (v.w == T ? 128u : 0u);
}

// Per-segment numbers of keys above / equal to the cut, by sweeping the row.  Whole CTA;
// the totals land in sm.seg_def / sm.seg_eq (visible after the caller's next barrier).
template <class G>
__device__ __forceinline__ void count_sweep(const RowKeys& keys, const Cut& cut, SelectSmem& sm) {
  const int lane = G::tid() & 31, warp = G::tid() >> 5;
  const Segments seg(keys.quads(), G::size() >> 5);
  const int q_end = seg.end(warp);
  uint32_t def_cnt = 0, eq_cnt = 0;
  for (int q0 = seg.begin(warp) + lane; q0 < q_end; q0 += G::kUnroll * 32) {
    uint4 v[G::kUnroll];
#pragma unroll
    for (int u = 0; u < G::kUnroll; ++u)
      if (q0 + u * 32 < q_end) v[u] = keys.load4(q0 + u * 32);
#pragma unroll
    for (int u = 0; u < G::kUnroll; ++u) {
      if (q0 + u * 32 < q_end) {
        const uint32_t f = classify(v[u], cut.T);
        def_cnt += __popc(f & 15u);
        eq_cnt += __popc(f >> 4);
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    def_cnt += __shfl_xor_sync(0xffffffffu, def_cnt, o);
    eq_cnt += __shfl_xor_sync(0xffffffffu, eq_cnt, o);
  }
  if (lane == 0) { sm.seg_def[warp] = def_cnt; sm.seg_eq[warp] = eq_cnt; }
}

// One sweep over the row once the leading digits are known: counts, per segment, the keys whose
// leading digit is above `d_cut` (they are kept whatever the rest of the cut turns out to be) and
// copies the keys with leading digit d_a (and d_b, if use_b) into the lists.  Whole CTA; totals in
// sm.seg_def (sm.seg_eq is cleared); list counters must be zero on entry.
template <class G>
__device__ __forceinline__ void collect_sweep(const RowKeys& keys, uint32_t d_cut, uint32_t d_a,
                                              const KeyList& list_a, bool use_b, uint32_t d_b,
                                              const KeyList& list_b, SelectSmem& sm) {
  const int lane = G::tid() & 31, warp = G::tid() >> 5;
  const Segments seg(keys.quads(), G::size() >> 5);
  const int q_end = seg.end(warp);
  uint32_t def_cnt = 0;
  for (int q0 = seg.begin(warp) + lane; q0 < q_end; q0 += G::kUnroll * 32) {
    uint4 v[G::kUnroll];
#pragma unroll
    for (int u = 0; u < G::kUnroll; ++u)
      if (q0 + u * 32 < q_end) v[u] = keys.load4(q0 + u * 32);
#pragma unroll
    for (int u = 0; u < G::kUnroll; ++u) {
      if (q0 + u * 32 < q_end) {
        const uint32_t k4[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint32_t dgt = k4[i] >> 20;
          def_cnt += dgt > d_cut ? 1u : 0u;
          if (dgt == d_a) {
            const uint32_t at = atomicAdd(list_a.count, 1u);
            if (at < list_a.cap) list_a.items[at] = make_uint2(k4[i], 4u * (q0 + u * 32) + i);
          }
          if (use_b && dgt == d_b) {
            const uint32_t at = atomicAdd(list_b.count, 1u);
            if (at < list_b.cap) list_b.items[at] = make_uint2(k4[i], 4u * (q0 + u * 32) + i);
          }
        }
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) def_cnt += __shfl_xor_sync(0xffffffffu, def_cnt, o);
  if (lane == 0) { sm.seg_def[warp] = def_cnt; sm.seg_eq[warp] = 0; }
}

// digit_histogram over a (complete) list instead of the row.
template <class G>
__device__ __forceinline__ void list_histogram(const KeyList& list, uint32_t ceiling, uint32_t mask,
                                               uint32_t prefix, int pass, uint32_t* hist) {
  const int shift = pass_shift(pass), n = list.size();
  const uint32_t dmask = pass_digit_mask(pass);
  for (int e = G::tid(); e < n; e += G::size()) {
    const uint32_t key = list.items[e].x;
    if ((key & mask) == prefix && key <= ceiling) atomicAdd(&hist[(key >> shift) & dmask], 1u);
  }
}

// Adds the list's keys above / equal to the cut to the per-segment totals (the list holds every
// key whose leading digit equals the cut's; keys with a higher digit were counted by collect_sweep).
template <class G>
__device__ __forceinline__ void count_from_list(const KeyList& list, const Cut& cut, const Segments& seg,
                                                SelectSmem& sm) {
  const int n = list.size();
  for (int e = G::tid(); e < n; e += G::size()) {
    const uint2 it = list.items[e];
    if (it.x > cut.T) atomicAdd(&sm.seg_def[seg.of_token(it.y)], 1u);
    else if (it.x == cut.T) atomicAdd(&sm.seg_eq[seg.of_token(it.y)], 1u);
  }
}

// Remaining digits of a cut whose leading digit `d0` is known: the `rank`-th largest key (1-based)
// among the keys of leading digit d0.  Uses the list if it is complete, else sweeps the row.  Whole CTA.
template <class G>
__device__ __forceinline__ Cut finish_cut(const RowKeys& keys, const KeyList& list, uint32_t d0,
                                          uint32_t rank, SelectSmem& sm) {
  uint32_t prefix = d0 << 20, mask = 0xfffu << 20, remaining = rank;
  const bool from_list = list.complete();
  if (from_list && list.size() <= kSelRankDirect) {
    // a short list is ranked directly: thread t counts the keys above and equal to key t (equal
    // keys find the same cut, so it does not matter which of their threads writes it)
    const int L = list.size();
    if ((int)G::tid() < L) {
      const uint32_t key = list.items[G::tid()].x;
      uint32_t gt = 0, eq = 0;
      for (int e = 0; e < L; ++e) {
        const uint32_t other = list.items[e].x;
        gt += other > key ? 1u : 0u;
        eq += other == key ? 1u : 0u;
      }
      if (gt < rank && rank <= gt + eq) {
        sm.digit = key;
        sm.remaining = rank - gt;
      }
    }
    G::sync();
    const Cut cut{sm.digit, sm.remaining};
    G::sync();                                       // sm.digit may be rewritten
    return cut;
  }
  for (int pass = 1; pass < kSelPasses; ++pass) {
    clear_hist<G>(sm.hist);
    G::sync();
    if (from_list) list_histogram<G>(list, 0xffffffffu, mask, prefix, pass, sm.hist);
    else digit_histogram<G>(keys, 0xffffffffu, mask, prefix, pass, sm.hist);
    G::sync();
    pick_digit<G>(sm.hist, remaining, sm);
    prefix |= sm.digit << pass_shift(pass);
    mask |= pass_digit_mask(pass) << pass_shift(pass);
    remaining = sm.remaining;
    G::sync();
  }
  return Cut{prefix, remaining};
}

// Ordered write of one row: the tokens whose key is above cut.T and the first cut.eq_take tokens
// whose key equals cut.T go to `out` in ascending token order.  The per-segment totals must be in
// sm.seg_def / sm.seg_eq (from count_sweep, or collect_sweep + count_from_list).  Whole CTA.
template <class G>
__device__ __forceinline__ void write_sweep(const RowKeys& keys, const Cut& cut, int32_t* out,
                                            SelectSmem& sm) {
  const int lane = G::tid() & 31, warp = G::tid() >> 5;
  const Segments seg(keys.quads(), G::size() >> 5);
  const int q_begin = seg.begin(warp), q_end = seg.end(warp);
  G::sync();
  uint32_t def_before = 0, eq_before = 0;                  // kept / equal tokens of earlier warps
  {
    const bool live = lane < ((int)G::size() >> 5);       // one segment per warp of the CTA
    const uint32_t d = live ? sm.seg_def[lane] : 0u, e = live ? sm.seg_eq[lane] : 0u;
    uint32_t di = d, ei = e;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t td = __shfl_up_sync(0xffffffffu, di, o), te = __shfl_up_sync(0xffffffffu, ei, o);
      if (lane >= o) { di += td; ei += te; }
    }
    def_before = __shfl_sync(0xffffffffu, di - d, warp);
    eq_before = __shfl_sync(0xffffffffu, ei - e, warp);
  }
  const uint32_t lt = (1u << lane) - 1u;                   // lanes before this one
  for (int q0 = q_begin; q0 < q_end; q0 += 32) {           // uniform trip count across the warp
    const int q = q0 + lane;
    uint32_t f = 0;
    if (q < q_end) f = classify(keys.load4(q), cut.T);
    // tokens run lane-major, then by position in the quad: ranks from one ballot per flag bit
    uint32_t d = def_before, dtot = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t bal = __ballot_sync(0xffffffffu, f & (1u << i));
      d += __popc(bal & lt);
      dtot += __popc(bal);
    }
    uint32_t e = eq_before, etot = 0;
    if (__any_sync(0xffffffffu, f >> 4)) {                 // ties at the cut are rare
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t bal = __ballot_sync(0xffffffffu, f & (16u << i));
        e += __popc(bal & lt);
        etot += __popc(bal);
      }
    }
    if (f) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (f & (1u << i)) {
          out[d + min(e, cut.eq_take)] = 4 * q + i;
          ++d;
        } else if (f & (16u << i)) {
          if (e < cut.eq_take) out[d + e] = 4 * q + i;
          ++e;
        }
      }
    }
    def_before += dtot;
    eq_before += etot;
  }
  G::sync();                                         // sm.warp_* may be reused
}

// The head normaliser S = sum_j lK_j lV_j from the per-tile partial sums, in the one order every
// kernel of this library uses (256 threads: thread t adds partials t, t + 256, ...; a shuffle tree
// per warp; the eight warp sums in warp order), so that S is the same bit pattern wherever it is
// formed.  Group G of at least 256 threads; the partials may have been written by this launch.
template <class G>
__device__ __forceinline__ float head_sum_fixed_order(const float* partials, int count, SelectSmem& sm) {
  const int tid = G::tid(), lane = tid & 31, warp = tid >> 5;
  float part = 0.f;
  if (tid < 256)
    for (int i = tid; i < count; i += 256) part += __ldcg(partials + i);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
  if (lane == 0 && warp < 8) sm.warp_def[warp] = __float_as_uint(part);
  G::sync();
  float S = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) S += __uint_as_float(sm.warp_def[w]);
  return S;
}

// Alg. 1 (normalisation step) for one row, on the way to the selection: row[j] <- row[j] / S for j < n (0 when the
// sum is not positive; left as it is with `raw`), row[j] <- 0 for first_unwritten <= j < n_max, and
// the leading-digit histogram of the resulting rank keys in `hist` (zero on entry).  With `staged`
// (16-byte aligned rows only) the rank keys are also left there, a quad per four tokens.  The row
// may have been written by other CTAs of this launch: it is read from L2.  Group G.
template <class G>
__device__ __forceinline__ void scale_row_and_histogram(float* row, const RowKeys& keys, int n_max,
                                                        int first_unwritten, float S, bool raw,
                                                        uint32_t* hist, uint4* staged) {
  const int n = keys.n, step = G::size();
  const bool live = S > 0.f;
  auto scaled = [&](float x) { return raw ? x : (live ? __fdiv_rn(x, S) : 0.f); };
  DigitRun run;
  if (keys.vec) {
    const int quads = n >> 2;                              // whole quads of valid tokens
    for (int q0 = G::tid(); q0 < quads; q0 += G::kUnroll * step) {
      float4 f[G::kUnroll];
#pragma unroll
      for (int u = 0; u < G::kUnroll; ++u)
        if (q0 + u * step < quads) f[u] = __ldcg(reinterpret_cast<const float4*>(row) + q0 + u * step);
#pragma unroll
      for (int u = 0; u < G::kUnroll; ++u) {
        const int q = q0 + u * step;
        if (q < quads) {
          const float4 o = make_float4(scaled(f[u].x), scaled(f[u].y), scaled(f[u].z), scaled(f[u].w));
          if (!raw) reinterpret_cast<float4*>(row)[q] = o;
          const uint4 k4 = make_uint4(keys.key_of(o.x, 4 * q), keys.key_of(o.y, 4 * q + 1),
                                      keys.key_of(o.z, 4 * q + 2), keys.key_of(o.w, 4 * q + 3));
          if (staged != nullptr) staged[q] = k4;
          run.add(k4.x >> 20, hist);
          run.add(k4.y >> 20, hist);
          run.add(k4.z >> 20, hist);
          run.add(k4.w >> 20, hist);
        }
      }
    }
    if (G::tid() == 0 && (n & 3) != 0) {                   // the last, partial quad
      uint32_t k4[4] = {0u, 0u, 0u, 0u};
      for (int j = quads << 2; j < n; ++j) {
        const float o = scaled(__ldcg(row + j));
        if (!raw) row[j] = o;
        k4[j & 3] = keys.key_of(o, j);
        run.add(k4[j & 3] >> 20, hist);
      }
      if (staged != nullptr) staged[quads] = make_uint4(k4[0], k4[1], k4[2], k4[3]);
    }
  } else {
    for (int j = G::tid(); j < n; j += step) {
      const float o = scaled(__ldcg(row + j));
      if (!raw) row[j] = o;
      run.add(keys.key_of(o, j) >> 20, hist);
    }
  }
  run.flush(hist);
  for (int j = first_unwritten + G::tid(); j < n_max; j += step) row[j] = 0.f;
}

// What a selection kernel needs to finish Alg. 1 (normalisation step) itself (the scores then arrive as the
// score kernels leave them: unnormalised, with per-tile partial sums).  tile_sums = nullptr: the
// scores are final already.
struct Normaliser {
  const float* tile_sums;  // [heads][tiles_per_head][parts_per_tile]
  float* head_sums;        // [heads]
  int tiles_per_head, parts_per_tile, raw;
};

// ---------------------------------------------------------------------------
// Fixed per-head budget, one row, by the group G: Alg. 1 (sinks, top-k, union) on the scores `keys` describes.
// k_eff = min(k, n) rows are kept; their ascending indices go to out[0, k_eff), -1 to
// out[k_eff, budget).  `staged` (stage_quads quads, or nothing) may hold a copy of the keys;
// `hist_ready` says that sm.hist already holds the leading-digit histogram of the row's keys (the
// caller built it while it had the scores in hand).
// ---------------------------------------------------------------------------
template <class G>
__device__ __forceinline__ void select_fixed_row(RowKeys keys, const ForcedSet& F, int k_eff, int budget,
                                                 uint4* staged, int stage_quads, const KeyList& list,
                                                 bool hist_ready, int32_t* out, SelectSmem& sm) {
  const int tid = G::tid(), n = keys.n;
  Cut cut;
  bool counted = false;                                    // per-segment totals already in sm.seg_*
  if (k_eff == 0) {
    cut = keep_nothing();
  } else if (k_eff == n) {
    cut = keep_every_token();
  } else if (F.free_slots == 0) {
    cut = keep_forced_only();
  } else {
    // sweep 1: leading-digit histogram (staging the keys on the way if the row fits)
    if (!hist_ready) {
      clear_hist<G>(sm.hist);
      if (tid == 0) *list.count = 0;
      G::sync();
      if (keys.quads() <= stage_quads) {
        stage_keys<G>(keys, staged, sm.hist);
        keys.staged = staged;
      } else {
        digit_histogram<G>(keys, 0xffffffffu, 0u, 0u, 0, sm.hist);
      }
    } else if (tid == 0) {
      *list.count = 0;
    }
    G::sync();
    pick_digit<G>(sm.hist, (uint32_t)k_eff, sm);
    const uint32_t d0 = sm.digit, rank = sm.remaining;
    G::sync();
    // sweep 2: keys above the digit are counted per segment, keys of the digit go to the list
    collect_sweep<G>(keys, d0, d0, list, false, 0u, list, sm);
    G::sync();
    cut = finish_cut<G>(keys, list, d0, rank, sm);
    if (list.complete()) {
      count_from_list<G>(list, cut, Segments(keys.quads(), G::size() >> 5), sm);
      counted = true;
    }
  }
  if (!counted) count_sweep<G>(keys, cut, sm);
  write_sweep<G>(keys, cut, out, sm);
  for (int t = k_eff + tid; t < budget; t += G::size()) out[t] = -1;
}

}  // namespace curdkv
