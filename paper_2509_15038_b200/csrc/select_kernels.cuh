// The two selection kernels (Alg. 1 (sinks, top-k, union) with a fixed budget per head, and AdaCurDKV of
// Sec. 3.2), built from the per-row routines of select.cuh.
#pragma once
#include "select.cuh"

namespace curdkv {

// grid = batch*heads, block = 1024, 512 or 256, dynamic shared memory = 16 * stage_quads bytes
// (0: rows are read from global memory) followed by one candidate list of list_cap entries.
// With norm.tile_sums the kernel first finishes Alg. 1 (normalisation step) for its row (head sum, division on the
// way into the staged keys) and `scores` is written.
__global__ void __launch_bounds__(kSelThreads) select_fixed_kernel(
    float* __restrict__ scores, const int32_t* __restrict__ seqlens, int heads, int n_max,
    int budget, const int32_t* __restrict__ head_budgets, int num_sink, int window, int stage_quads,
    int list_cap, int32_t* __restrict__ idx, int32_t* __restrict__ counts, int32_t* __restrict__ offsets,
    const Normaliser norm) {
  __shared__ SelectSmem sm;
  extern __shared__ uint4 staged_keys[];                   // stage_quads quads, or nothing
  using G = WholeCta;
  const int p = blockIdx.x, b = p / heads;
  const int n = seq_len_of(seqlens, b, n_max);
  int k = budget;
  if (head_budgets != nullptr) k = max(0, min(head_budgets[p], budget));
  const int k_eff = min(k, n);
  const ForcedSet F = forced_set(n, k_eff, num_sink, window);
  float* row = scores + (size_t)p * n_max;
  RowKeys keys = global_keys(row, n, F);
  const KeyList list{reinterpret_cast<uint2*>(staged_keys + stage_quads), &sm.list_count[0], (uint32_t)list_cap};
  bool hist_ready = false;
  if (norm.tile_sums != nullptr) {
    const int tiles = (n + kTileRows - 1) / kTileRows;
    const float S = head_sum_fixed_order<G>(
        norm.tile_sums + (size_t)p * norm.tiles_per_head * norm.parts_per_tile, tiles * norm.parts_per_tile, sm);
    if (threadIdx.x == 0) norm.head_sums[p] = S;
    clear_hist<G>(sm.hist);
    G::sync();
    const bool stage = keys.vec && keys.quads() <= stage_quads;
    scale_row_and_histogram<G>(row, keys, n_max, tiles * kTileRows, S, norm.raw != 0, sm.hist,
                               stage ? staged_keys : nullptr);
    keys.written_here = true;
    if (stage) keys.staged = staged_keys;
    hist_ready = true;
    G::sync();
  }
  select_fixed_row<G>(keys, F, k_eff, budget, staged_keys, stage_quads, list, hist_ready,
                      idx + (size_t)p * budget, sm);
  if (threadIdx.x == 0) {
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
// grid = batch*heads, cluster = heads, block = THREADS (1024, or 512 with lists
// of half the size so that two CTAs share an SM: more clusters are resident at
// once, which pays when there are more clusters than fit in one round).
// ---------------------------------------------------------------------------
struct AdaptiveSmem {
  SelectSmem s;
  alignas(16) uint32_t hist_local[kSelBins];               // read by the other CTAs of the cluster
  uint32_t pub_eq;                                         // unprotected keys equal to the global cut
  uint32_t pub_count;                                      // rows this head keeps
};
// dynamic shared memory: leading-digit histogram + two lists
__host__ __device__ constexpr int adaptive_list_cap(int threads) { return threads == 1024 ? kSelListCap : kSelListCap / 2; }
__host__ __device__ constexpr int adaptive_dynamic_bytes(int threads) { return kSelBins * 4 + 2 * adaptive_list_cap(threads) * 8; }

template <int THREADS>
__global__ void __launch_bounds__(THREADS, 1024 / THREADS) select_adaptive_kernel(
    float* __restrict__ scores, const int32_t* __restrict__ seqlens, int heads, int n_max,
    int budget, int num_sink, int window, int min_protected, int32_t* __restrict__ idx,
    int32_t* __restrict__ counts, int32_t* __restrict__ offsets, const Normaliser norm) {
  __shared__ AdaptiveSmem sm;
  using G = WholeCta;
  extern __shared__ uint4 adaptive_dyn[];
  uint32_t* hist_all = reinterpret_cast<uint32_t*>(adaptive_dyn);          // leading digits of all keys
  constexpr int B = kSelBins / THREADS, Q = B / 4;         // histogram bins (quads of bins) per thread
  constexpr int kCap = adaptive_list_cap(THREADS);
  const KeyList list_a{reinterpret_cast<uint2*>(hist_all + kSelBins), &sm.s.list_count[0], (uint32_t)kCap};
  const KeyList list_b{list_a.items + kCap, &sm.s.list_count[1], (uint32_t)kCap};
  cg::cluster_group cluster = cg::this_cluster();
  const int tid = threadIdx.x;
  const int h = (int)cluster.block_rank();
  const int b = blockIdx.x / heads, p = b * heads + h;
  const int n = seq_len_of(seqlens, b, n_max);
  const int k_eff = min(budget, n);
  const ForcedSet F = forced_set(n, k_eff, num_sink, window);
  RowKeys keys = global_keys(scores + (size_t)p * n_max, n, F);
  const int forced = k_eff - F.free_slots;
  const int prot = min(max(min_protected, forced), k_eff);  // protected rows per head, forced included
  const bool none = prot == 0, all = prot >= n;             // nothing / everything is protected
  const uint32_t pool = (uint32_t)heads * (uint32_t)(k_eff - prot);   // same for every head of b

  // ---- sweep 1: leading-digit histogram of the row; leading digit of this head's safeguard cut
  // (its `prot` largest keys) and how many keys of that digit the cut takes
  clear_hist<G>(hist_all);
  if (tid == 0) sm.s.list_count[0] = sm.s.list_count[1] = 0;
  if (norm.tile_sums != nullptr) {
    // Alg. 1 (normalisation step) first: the scores arrive unnormalised, with per-tile partial sums
    const int tiles = (n + kTileRows - 1) / kTileRows;
    const float S = head_sum_fixed_order<G>(
        norm.tile_sums + (size_t)p * norm.tiles_per_head * norm.parts_per_tile, tiles * norm.parts_per_tile, sm.s);
    if (tid == 0) norm.head_sums[p] = S;
    scale_row_and_histogram<G>(scores + (size_t)p * n_max, keys, n_max, tiles * kTileRows, S, norm.raw != 0,
                               hist_all, nullptr);
    keys.written_here = true;
  } else {
    __syncthreads();
    if (!all) digit_histogram<G>(keys, 0xffffffffu, 0u, 0u, 0, hist_all);
  }
  __syncthreads();
  uint32_t d0 = 0xffffffffu, rank_own = 0;
  if (!none && !all) {
    pick_digit_impl<G, B>(hist_all, (uint32_t)prot, sm.s);
    d0 = sm.s.digit;
    rank_own = sm.s.remaining;
    __syncthreads();
  }

  // ---- leading digit of the layer-wide cut over the unprotected keys of all heads.  Their
  // leading-digit histogram follows from the row's: bins below d0 whole, bin d0 minus the
  // protected keys in it, nothing above.
  uint32_t dg = 0, remaining = pool, local_gt = 0, local_eq = 0;
  if (pool > 0) {
#pragma unroll
    for (int q = 0; q < Q; ++q) {
      const uint4 v = reinterpret_cast<const uint4*>(hist_all)[tid * Q + q];
      uint32_t c[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const uint32_t bin = (uint32_t)(B * tid + 4 * q + u);
        if (all) c[u] = 0;
        else if (!none && bin > d0) c[u] = 0;
        else if (!none && bin == d0) c[u] -= rank_own;
      }
      reinterpret_cast<uint4*>(sm.hist_local)[tid * Q + q] = make_uint4(c[0], c[1], c[2], c[3]);
    }
    cluster.sync();
#pragma unroll
    for (int q = 0; q < Q; ++q) {
      uint4 acc = make_uint4(0u, 0u, 0u, 0u);              // four of this thread's bins over all heads
      for (int r = 0; r < heads; ++r) {
        const uint4 v = reinterpret_cast<const uint4*>(cluster.map_shared_rank(sm.hist_local, r))[tid * Q + q];
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
      }
      reinterpret_cast<uint4*>(sm.s.hist)[tid * Q + q] = acc;
    }
    __syncthreads();
    pick_digit_impl<G, B>(sm.s.hist, remaining, sm.s);
    dg = sm.s.digit;
    remaining = sm.s.remaining;
    local_gt = count_above_impl<G, B>(sm.hist_local, dg, sm.s);
    cluster.sync();                                        // peers are done reading hist_local
  }

  // ---- sweep 2: keys with a leading digit above the final cut's are kept for sure (counted per
  // segment); keys with the digits d0 and dg go to the lists
  // (the layer-wide cut can lie above this head's own cut when other heads score higher: then
  // this head keeps its protected keys only and its final cut is its own)
  const bool global_lower = pool > 0 && (none || dg < d0); // the final cut has leading digit dg
  const uint32_t d_cut = global_lower ? dg : d0;
  const bool share = !none && dg == d0;                    // one list serves both cuts
  const bool swept = !all && (pool > 0 || !none);
  if (swept) collect_sweep<G>(keys, d_cut, d0, list_a, pool > 0 && !share, dg, list_b, sm.s);
  __syncthreads();

  // ---- this head's safeguard cut
  Cut own = keep_nothing();
  if (all) own = keep_every_token();
  else if (!none) own = finish_cut<G>(keys, list_a, d0, rank_own, sm.s);
  // unprotected keys: those <= own.T, minus the first own.eq_take equal to it
  const uint32_t ceiling = own.T;

  // ---- remaining digits of the layer-wide cut
  const KeyList& list_g = share ? list_a : list_b;
  uint32_t Tg = 0, eq_g = 0;
  if (pool > 0) {
    uint32_t prefix = dg << 20, mask = 0xfffu << 20;
    for (int pass = 1; pass < kSelPasses; ++pass) {
      const int shift = pass_shift(pass);
      clear_hist<G>(sm.hist_local);
      __syncthreads();
      if (!all) {
        if (list_g.complete()) list_histogram<G>(list_g, ceiling, mask, prefix, pass, sm.hist_local);
        else digit_histogram<G>(keys, ceiling, mask, prefix, pass, sm.hist_local);
      }
      __syncthreads();
      if (tid == 0 && own.eq_take > 0 && (own.T & mask) == prefix)
        sm.hist_local[(own.T >> shift) & pass_digit_mask(pass)] -= own.eq_take;   // those are protected
      cluster.sync();
#pragma unroll
      for (int q = 0; q < Q; ++q) {
        uint4 acc = make_uint4(0u, 0u, 0u, 0u);
        for (int r = 0; r < heads; ++r) {
          const uint4 v =
              reinterpret_cast<const uint4*>(cluster.map_shared_rank(sm.hist_local, r))[tid * Q + q];
          acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        reinterpret_cast<uint4*>(sm.s.hist)[tid * Q + q] = acc;
      }
      __syncthreads();
      pick_digit_impl<G, B>(sm.s.hist, remaining, sm.s);
      const uint32_t dgt = sm.s.digit;
      remaining = sm.s.remaining;
      prefix |= dgt << shift;
      mask |= pass_digit_mask(pass) << shift;
      local_gt += count_above_impl<G, B>(sm.hist_local, dgt, sm.s);
      if (pass == kSelPasses - 1) local_eq = sm.hist_local[dgt];
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
  const uint32_t kept = (uint32_t)prot + local_gt + e_h;
  Cut cut = own;
  if (pool > 0) {
    if (Tg < own.T) cut = Cut{Tg, e_h};
    else if (Tg == own.T) cut = Cut{own.T, own.eq_take + e_h};
  }
  if (tid == 0) sm.pub_count = kept;
  cluster.sync();

  // ---- packed output position: rows of earlier sequences, then earlier heads
  uint32_t part = 0;
  for (int bb = tid; bb < b; bb += THREADS)
    part += (uint32_t)heads * (uint32_t)min(budget, seq_len_of(seqlens, bb, n_max));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
  if ((tid & 31) == 0) sm.s.warp_def[tid >> 5] = part;
  __syncthreads();
  uint32_t off = 0;
  for (int w = 0; w < THREADS / 32; ++w) off += sm.s.warp_def[w];
  for (int r = 0; r < h; ++r) off += *cluster.map_shared_rank(&sm.pub_count, r);
  __syncthreads();

  // ---- per-segment totals, then the ordered write (sweep 3)
  const KeyList& list_c = global_lower ? list_b : list_a;  // holds the keys of the cut's leading digit
  if (swept && list_c.complete()) count_from_list<G>(list_c, cut, Segments(keys.quads(), THREADS >> 5), sm.s);
  else count_sweep<G>(keys, cut, sm.s);
  write_sweep<G>(keys, cut, idx + off, sm.s);
  if (tid == 0) {
    counts[p] = (int32_t)kept;
    offsets[p] = (int32_t)off;
    if (p == (int)gridDim.x - 1) offsets[p + 1] = (int32_t)(off + kept);
  }
  cluster.sync();                                          // keep shared memory alive for peers
}

}  // namespace curdkv
