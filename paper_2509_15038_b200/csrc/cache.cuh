// Bookkeeping kernels of the generation-phase cache (Sec. 3.2: the method also
// applies while tokens are generated): rows are appended with their
// unnormalised scores l^KV (Alg. 1 (sketch, row norms, product)) and original positions, and a
// compression step carries scores and positions along with the gathered rows.
#pragma once
#include "common.cuh"
#include "select.cuh"

namespace curdkv {

struct CacheView {
  __nv_bfloat16* K;
  __nv_bfloat16* V;        // [batch][heads][capacity][d]
  float* raw;              // [batch][heads][capacity]
  int32_t* pos;            // [batch][heads][capacity]
  int32_t* count;          // [batch]
  int32_t* total;          // [batch]
  int capacity;
};

struct AppendArgs {
  CacheView cache;
  KvView K_new, V_new;     // [batch][heads][t][d]
  const float* raw_new;    // [batch][heads][t]
  const int32_t* t_new;    // [batch] or nullptr (every sequence brings t rows)
  int heads, t, d;
  uint32_t* status;
};

constexpr int kAppendWarps = 8;
constexpr int kAppendRowsPerCta = 32;

// grid = batch*heads*ceil(t / 32), block = 256: a half-warp per row (K in lanes
// 0-15, V in lanes 16-31).  Rows that do not fit under `capacity` are dropped
// and flagged.  Reads count/total, never writes them (cache_advance_kernel does).
__global__ void __launch_bounds__(kAppendWarps * 32) cache_append_kernel(const AppendArgs a) {
  const int chunks_per_head = (a.t + kAppendRowsPerCta - 1) / kAppendRowsPerCta;
  const int p = blockIdx.x / chunks_per_head, chunk = blockIdx.x % chunks_per_head;
  const int b = p / a.heads, h = p % a.heads;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, half = lane >> 4, l16 = lane & 15;
  int tb = a.t_new != nullptr ? a.t_new[b] : a.t;
  tb = tb < 0 ? 0 : (tb > a.t ? a.t : tb);
  int held = a.cache.count[b];
  if (held < 0 || held > a.cache.capacity) {               // counters the caller never set up
    if (threadIdx.x == 0 && chunk == 0) flag_status(a.status, CURDKV_DEV_BAD_INDEX);
    held = held < 0 ? 0 : a.cache.capacity;
  }
  const int room = a.cache.capacity - held;
  if (tb > room) {
    if (threadIdx.x == 0 && chunk == 0) flag_status(a.status, CURDKV_DEV_CACHE_FULL);
    tb = room > 0 ? room : 0;
  }
  const int first_pos = a.cache.total[b];
  const KvView& T = half ? a.V_new : a.K_new;
  const __nv_bfloat16* src = T.base + b * T.stride_b + h * T.stride_h;
  __nv_bfloat16* dst = (half ? a.cache.V : a.cache.K) + ((size_t)p * a.cache.capacity + held) * a.d;
  const int chunks = a.d >> 3;
  // four rows per warp in flight (rows warp, warp + 8, warp + 16, warp + 24 of the chunk)
  const int row0 = chunk * kAppendRowsPerCta + warp;
  for (int c = l16; c < chunks; c += 16) {
    uint4 v[kAppendRowsPerCta / kAppendWarps];
#pragma unroll
    for (int j = 0; j < kAppendRowsPerCta / kAppendWarps; ++j) {
      const int i = row0 + j * kAppendWarps;
      if (i < tb) v[j] = __ldg(reinterpret_cast<const uint4*>(src + i * T.stride_n) + c);
    }
#pragma unroll
    for (int j = 0; j < kAppendRowsPerCta / kAppendWarps; ++j) {
      const int i = row0 + j * kAppendWarps;
      if (i < tb) reinterpret_cast<uint4*>(dst + (size_t)i * a.d)[c] = v[j];
    }
  }
  if (lane == 0) {
#pragma unroll
    for (int j = 0; j < kAppendRowsPerCta / kAppendWarps; ++j) {
      const int i = row0 + j * kAppendWarps;
      if (i < tb) {
        a.cache.raw[(size_t)p * a.cache.capacity + held + i] = a.raw_new[(size_t)p * a.t + i];
        a.cache.pos[(size_t)p * a.cache.capacity + held + i] = first_pos + i;
      }
    }
  }
}

// count[b] += rows that fitted, total[b] += rows offered.  grid = ceil(batch / 256).
__global__ void cache_advance_kernel(CacheView cache, const int32_t* t_new, int t, int batch) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= batch) return;
  int tb = t_new != nullptr ? t_new[b] : t;
  tb = tb < 0 ? 0 : (tb > t ? t : tb);
  const int held = min(max(cache.count[b], 0), cache.capacity);   // as cache_append_kernel read it
  const int room = cache.capacity - held;
  cache.count[b] = held + (tb < room ? tb : room);
  cache.total[b] += tb;
}

// Scores, positions and counters of the rows a compression keeps.
// grid = batch*heads, block = 256.  idx: [batch][heads][budget]; counts: [batch][heads].
__global__ void __launch_bounds__(256) cache_gather_meta_kernel(const CacheView in, const CacheView out,
                                                                const int32_t* idx, int budget,
                                                                const int32_t* counts, int heads) {
  const int p = blockIdx.x, b = p / heads, h = p % heads;
  const int kept = min(counts[p], out.capacity);
  const int held = in.count[b];
  for (int t = threadIdx.x; t < kept; t += blockDim.x) {
    const int j = idx[(size_t)p * budget + t];
    if (j >= 0 && j < held) {
      out.raw[(size_t)p * out.capacity + t] = in.raw[(size_t)p * in.capacity + j];
      out.pos[(size_t)p * out.capacity + t] = in.pos[(size_t)p * in.capacity + j];
    }
  }
  if (h == 0 && threadIdx.x == 0) {
    out.count[b] = kept;
    out.total[b] = in.total[b];
  }
}

// ---- in-place compression: the cache keeps no particular row order ----------

// Selection keys of the held rows: +inf for forced rows (positions < num_sink or among the most
// recent `window`), otherwise the row's l^KV, lifted to the smallest positive float if it is 0 so
// that a real row always outranks an unused slot.  grid = batch*heads, block = 256.
__global__ void __launch_bounds__(256) cache_keyed_scores_kernel(const CacheView c, int heads, int num_sink,
                                                                 int window, float* keyed) {
  const int p = blockIdx.x, b = p / heads;
  const int held = min(max(c.count[b], 0), c.capacity);
  const int recent = c.total[b] - window;
  const int32_t* pos_row = c.pos + (size_t)p * c.capacity;
  const float* raw_row = c.raw + (size_t)p * c.capacity;
  float* key_row = keyed + (size_t)p * c.capacity;
  auto key_of = [&](int pos, float raw) {
    return (pos < num_sink || pos >= recent) ? __int_as_float(0x7f800000) : fmaxf(raw, 1.17549435e-38f);
  };
  int done = 0;
  if ((c.capacity & 3) == 0 && ((reinterpret_cast<uintptr_t>(c.pos) | reinterpret_cast<uintptr_t>(c.raw) |
                                 reinterpret_cast<uintptr_t>(keyed)) & 15u) == 0) {
    const int quads = held >> 2;                           // four slots per thread and step
    for (int q = threadIdx.x; q < quads; q += blockDim.x) {
      const int4 ps = reinterpret_cast<const int4*>(pos_row)[q];
      const float4 rw = reinterpret_cast<const float4*>(raw_row)[q];
      reinterpret_cast<float4*>(key_row)[q] =
          make_float4(key_of(ps.x, rw.x), key_of(ps.y, rw.y), key_of(ps.z, rw.z), key_of(ps.w, rw.w));
    }
    done = quads << 2;
  }
  for (int s = done + threadIdx.x; s < held; s += blockDim.x) key_row[s] = key_of(pos_row[s], raw_row[s]);
}

// After the selection: rows kept at slots >= kept ("movers", the tail of the ascending idx list)
// are copied into the slots < kept that were not kept ("holes"), so that the survivors occupy
// slots [0, kept) again.  At most min(kept, held - kept) rows move.  grid = batch*heads,
// block = 256, dynamic shared memory = capacity bytes (slot flags); holes: int32 [problems][capacity].
// With set_counters the CTA of a sequence's first head also leaves count[b] = rows kept and adds
// `appended` rows (t_new[b], or t) to total[b]: no kernel of this launch reads either.
__global__ void __launch_bounds__(256) cache_fill_holes_kernel(const CacheView c, const int32_t* idx,
                                                               int budget, const int32_t* counts, int heads,
                                                               int d, int32_t* holes, uint32_t* status,
                                                               int set_counters, const int32_t* t_new, int t) {
  extern __shared__ unsigned char slot_kept[];
  __shared__ int s_first_mover, s_base, s_warp_tot[8];
  const int p = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int kept = min(counts[p], c.capacity);
  if (set_counters && tid == 0 && p % heads == 0) {
    const int b = p / heads;
    int tb = t_new != nullptr ? t_new[b] : t;
    tb = tb < 0 ? 0 : (tb > t ? t : tb);
    c.count[b] = kept;
    c.total[b] += tb;
  }
  const int32_t* ix = idx + (size_t)p * budget;
  int32_t* my_holes = holes + (size_t)p * c.capacity;
  for (int s = tid; s < kept; s += 256) slot_kept[s] = 0;
  if (tid == 0) {                                          // idx is ascending: first entry >= kept
    int lo = 0, hi = kept;
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (ix[mid] < kept) lo = mid + 1; else hi = mid;
    }
    s_first_mover = lo;
    s_base = 0;
  }
  __syncthreads();
  const int first_mover = s_first_mover, movers = kept - first_mover;
  for (int t = tid; t < first_mover; t += 256) slot_kept[ix[t]] = 1;
  __syncthreads();
  // holes in ascending slot order, 256 slots per sweep
  for (int s0 = 0; s0 < kept; s0 += 256) {
    const int s = s0 + tid;
    const bool hole = s < kept && slot_kept[s] == 0;
    const uint32_t bal = __ballot_sync(0xffffffffu, hole);
    if (lane == 0) s_warp_tot[warp] = __popc(bal);
    __syncthreads();
    int before = s_base;
    for (int w = 0; w < warp; ++w) before += s_warp_tot[w];
    if (hole) my_holes[before + __popc(bal & ((1u << lane) - 1u))] = s;
    __syncthreads();
    if (tid == 0) {
      int tot = 0;
      for (int w = 0; w < 8; ++w) tot += s_warp_tot[w];
      s_base += tot;
    }
    __syncthreads();
  }
  if (tid == 0 && s_base != movers) flag_status(status, CURDKV_DEV_BAD_INDEX);   // idx was not a valid selection
  const int moves = min(s_base, movers);
  // copy mover i into hole i: a half-warp per tensor row (K in lanes 0-15, V in lanes 16-31)
  const int half = lane >> 4, l16 = lane & 15, chunks = d >> 3;
  __nv_bfloat16* rows = (half ? c.V : c.K) + (size_t)p * c.capacity * d;
  float* raw = c.raw + (size_t)p * c.capacity;
  int32_t* pos = c.pos + (size_t)p * c.capacity;
  if (chunks == 16) {
    // d = 128: one 16-byte piece per lane and row; four rows per warp in flight (sources and
    // destinations are disjoint slot ranges, so the order of the copies is free)
    for (int i0 = warp; i0 < moves; i0 += 32) {
      int src[4], dst[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int i = min(i0 + 8 * q, moves - 1);
        src[q] = ix[first_mover + i];
        dst[q] = my_holes[i];
      }
      uint4 v[4];
      float rv = 0.f;
      int pv = 0;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        v[q] = *reinterpret_cast<const uint4*>(rows + (size_t)src[q] * d + l16 * 8);
        if (lane == q) { rv = raw[src[q]]; pv = pos[src[q]]; }
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        if (i0 + 8 * q < moves) {
          reinterpret_cast<uint4*>(rows + (size_t)dst[q] * d)[l16] = v[q];
          if (lane == q) { raw[dst[q]] = rv; pos[dst[q]] = pv; }
        }
      }
    }
    return;
  }
  for (int i = warp; i < moves; i += 8) {
    const int src = ix[first_mover + i], dst = my_holes[i];
    for (int ch = l16; ch < chunks; ch += 16)
      reinterpret_cast<uint4*>(rows + (size_t)dst * d)[ch] =
          *reinterpret_cast<const uint4*>(rows + (size_t)src * d + ch * 8);
    if (lane == 0) {
      raw[dst] = raw[src];
      pos[dst] = pos[src];
    }
  }
}

// ---- one generation step: append the new rows AND compress in place, in one launch ----------
// One CTA per head.  The selection only needs scores and positions, so it runs first, over the
// held rows' scores and positions and the new rows' fresh scores (keys staged in shared memory;
// forced rows, found by position, carry the top key).  Only then are rows moved, and each at most
// once: a surviving new row goes straight from the caller's block into its final slot (its own,
// or a hole an evicted row leaves), a surviving old row beyond the new row count into a hole;
// evicted new rows are never copied at all.  With s = slot of a row after a plain append (held
// rows 0 .. held-1, new row i at held + i) the result is the cache curdkv_cache_append +
// curdkv_cache_compress_inplace leave.  The last CTA of a sequence sets its counters (every CTA of
// the sequence has read them by then: tickets, zero on entry).
struct StepArgs {
  AppendArgs append;
  int budget, num_sink, window;
  int stage_quads, list_cap;       // shared-memory copy of a head's keys, candidate list
  int32_t* idx;                    // [batch*heads][budget]
  int32_t* counts;                 // [batch*heads]
  int32_t* tickets;                // [batch], zero on entry
};

__global__ void __launch_bounds__(256) cache_step_kernel(const StepArgs s) {
  __shared__ SelectSmem sm;
  __shared__ int s_first_mover, s_first_new, s_base, s_warp_tot[8];
  extern __shared__ uint4 step_keys[];                     // stage_quads quads, then the list
  const AppendArgs& a = s.append;
  const int p = blockIdx.x, b = p / a.heads, h = p % a.heads;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int cap = a.cache.capacity;
  int tb = a.t_new != nullptr ? a.t_new[b] : a.t;
  tb = tb < 0 ? 0 : (tb > a.t ? a.t : tb);
  int held = a.cache.count[b];
  if (held < 0 || held > cap) {                            // counters the caller never set up
    if (tid == 0) flag_status(a.status, CURDKV_DEV_BAD_INDEX);
    held = held < 0 ? 0 : cap;
  }
  const int first_pos = a.cache.total[b], offered = tb;
  if (tb > cap - held) {
    if (tid == 0) flag_status(a.status, CURDKV_DEV_CACHE_FULL);
    tb = cap - held;
  }
  // -------------------------------------------------------------- select (Alg. 1 (sinks, top-k, union))
  using G = WholeCta;
  const int n = held + tb;                                 // rows the head holds after the append
  const int k_eff = min(s.budget, n);
  const int recent = first_pos + offered - s.window;       // positions from here on are the window
  float* raw_row = a.cache.raw + (size_t)p * cap;
  int32_t* pos_row = a.cache.pos + (size_t)p * cap;
  const float* raw_new = a.raw_new + (size_t)p * a.t;
  clear_hist<G>(sm.hist);
  if (tid == 0) sm.list_count[0] = 0;
  __syncthreads();
  {
    DigitRun run;
    uint32_t* keys32 = reinterpret_cast<uint32_t*>(step_keys);
    const int padded = ((n + 3) >> 2) << 2;
    for (int j = tid; j < padded; j += 256) {
      uint32_t key = 0u;                                   // beyond the rows held: never kept
      if (j < n) {
        float raw;
        int pos;
        if (j < held) {
          raw = raw_row[j];
          pos = pos_row[j];
        } else {                                           // a new row: file its score and position
          raw = raw_new[j - held];
          pos = first_pos + (j - held);
          raw_row[j] = raw;
          pos_row[j] = pos;
        }
        key = (pos < s.num_sink || pos >= recent) ? kForcedKey : score_key(raw);
        run.add(key >> 20, sm.hist);
      }
      keys32[j] = key;
    }
    run.flush(sm.hist);
  }
  __syncthreads();
  const ForcedSet F = forced_set(n, k_eff, 0, 0);          // forced rows carry the top key already
  RowKeys keys{nullptr, step_keys, n, 0, n, true, false};
  const KeyList list{reinterpret_cast<uint2*>(step_keys + s.stage_quads), &sm.list_count[0], (uint32_t)s.list_cap};
  int32_t* ix = s.idx + (size_t)p * s.budget;
  select_fixed_row<G>(keys, F, k_eff, s.budget, step_keys, s.stage_quads, list, true, ix, sm);
  if (tid == 0) s.counts[p] = k_eff;

  // -------------------------------------------------------------- place the survivors (Alg. 1 (gather step))
  // ix is ascending: [0, first_new) old rows that stay, [first_new, first_mover) new rows whose
  // own slot lies below k_eff, [first_mover, k_eff) movers (slot >= k_eff) that go into the holes.
  // The staged keys are done with: their space takes the slot flags and the list of holes.
  unsigned char* slot_kept = reinterpret_cast<unsigned char*>(step_keys);
  int32_t* holes = reinterpret_cast<int32_t*>(slot_kept + ((cap + 15) & ~15));
  __syncthreads();                                         // ix (global) and the end of the key sweeps
  if (tid == 0) {
    int lo = 0, hi = k_eff;
    while (lo < hi) { const int mid = (lo + hi) >> 1; if (ix[mid] < k_eff) lo = mid + 1; else hi = mid; }
    s_first_mover = lo;
    lo = 0, hi = k_eff;
    while (lo < hi) { const int mid = (lo + hi) >> 1; if (ix[mid] < held) lo = mid + 1; else hi = mid; }
    s_first_new = lo;
    s_base = 0;
  }
  for (int t = tid; t < k_eff; t += 256) slot_kept[t] = 0;
  __syncthreads();
  const int first_mover = s_first_mover, first_new = min(s_first_new, first_mover);
  const int movers = k_eff - first_mover;
  for (int t = tid; t < first_mover; t += 256) slot_kept[ix[t]] = 1;
  __syncthreads();
  for (int s0 = 0; s0 < k_eff; s0 += 256) {                // holes in ascending slot order
    const int sl = s0 + tid;
    const bool hole = sl < k_eff && slot_kept[sl] == 0;
    const uint32_t bal = __ballot_sync(0xffffffffu, hole);
    if (lane == 0) s_warp_tot[warp] = __popc(bal);
    __syncthreads();
    int before = s_base;
    for (int w = 0; w < warp; ++w) before += s_warp_tot[w];
    if (hole) holes[before + __popc(bal & ((1u << lane) - 1u))] = sl;
    __syncthreads();
    if (tid == 0) {
      int tot = 0;
      for (int w = 0; w < 8; ++w) tot += s_warp_tot[w];
      s_base += tot;
    }
    __syncthreads();
  }
  if (tid == 0 && s_base != movers) flag_status(a.status, CURDKV_DEV_BAD_INDEX);
  const int moves = min(s_base, movers);
  // jobs: natural-slot new rows first, then mover i -> hole i.  A half-warp per tensor row (K in
  // lanes 0-15, V in lanes 16-31), four rows per warp in flight; sources and destinations are
  // disjoint (sources: slots >= k_eff or the caller's block), so the order is free.
  const int half = lane >> 4, l16 = lane & 15, chunks = a.d >> 3;
  const int jobs = (first_mover - first_new) + moves;
  __nv_bfloat16* cache_rows = (half ? a.cache.V : a.cache.K) + (size_t)p * cap * a.d;
  const KvView& T = half ? a.V_new : a.K_new;
  const __nv_bfloat16* new_rows = T.base + b * T.stride_b + h * T.stride_h;
  for (int j0 = warp; j0 < jobs; j0 += 32) {
    const __nv_bfloat16* src[4];
    int dst[4], from[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int j = min(j0 + 8 * q, jobs - 1);
      if (j < first_mover - first_new) {                   // new row, own slot
        from[q] = dst[q] = ix[first_new + j];
      } else {
        from[q] = ix[first_mover + (j - (first_mover - first_new))];
        dst[q] = holes[j - (first_mover - first_new)];
      }
      src[q] = from[q] < held ? cache_rows + (size_t)from[q] * a.d
                              : new_rows + (int64_t)(from[q] - held) * T.stride_n;
    }
    for (int c = l16; c < chunks; c += 16) {
      uint4 v[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) v[q] = *reinterpret_cast<const uint4*>(src[q] + c * 8);
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (j0 + 8 * q < jobs) reinterpret_cast<uint4*>(cache_rows + (size_t)dst[q] * a.d)[c] = v[q];
    }
    if (lane < 4 && j0 + 8 * lane < jobs && from[lane] != dst[lane]) {   // a mover's score and position
      int f = from[0], t2 = dst[0];
#pragma unroll
      for (int q = 1; q < 4; ++q)
        if (lane == q) { f = from[q]; t2 = dst[q]; }
      raw_row[t2] = raw_row[f];
      pos_row[t2] = pos_row[f];
    }
  }
  // -------------------------------------------------------------- counters, by the sequence's last CTA
  __threadfence();
  __syncthreads();
  if (tid == 0 && atomicAdd(s.tickets + b, 1) == a.heads - 1) {
    a.cache.count[b] = k_eff;
    a.cache.total[b] = first_pos + offered;
    s.tickets[b] = 0;
  }
}

}  // namespace curdkv
