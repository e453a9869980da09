// Generation-phase cache (Sec. 3.2): append newly generated rows with their
// l^KV, compress the held rows with Alg. 1 (normalisation, selection, gather).  Built on the public
// entry points of curdkv.h plus the bookkeeping kernels of cache.cuh.
#include <cstdint>

#include "cache.cuh"
#include "common.cuh"

namespace {

using namespace curdkv;

inline size_t round256(size_t x) { return (x + 255) & ~size_t(255); }

struct CacheWorkspace {     // byte offsets from the workspace base
  size_t score_ws, raw_new, sums, idx, counts, keyed, holes, tickets, total;
};

bool layout(int32_t batch, int32_t heads, int32_t t_max, int32_t capacity, int32_t budget,
            CacheWorkspace* L) {
  if (batch < 0 || heads < 1 || t_max < 0 || capacity < 1 || budget < 0) return false;
  curdkv_desc d = {};
  d.batch = batch;
  d.kv_heads = d.q_heads = heads;
  d.n_max = t_max;
  d.d = 128;
  d.r = 1;
  d.use_projection = 1;
  const size_t score_ws = curdkv_workspace_bytes(&d, 0, 0);
  if (score_ws == 0) return false;
  const size_t P = (size_t)batch * heads;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o += round256(bytes ? bytes : 1); return at; };
  L->score_ws = take(score_ws);                 // first: its status word is the cache's too
  L->raw_new = take(P * (size_t)t_max * 4);
  L->sums = take(P * 4);
  L->idx = take(P * (size_t)budget * 4);
  L->counts = take(P * 4);
  L->keyed = take(P * (size_t)capacity * 4);    // in-place compression only
  L->holes = take(P * (size_t)capacity * 4);
  L->tickets = take((size_t)batch * 4);         // curdkv_cache_step only
  L->total = o;
  return true;
}

bool cache_ok(const curdkv_cache* c) {
  return c != nullptr && c->K != nullptr && c->V != nullptr && c->raw != nullptr && c->pos != nullptr &&
         c->count != nullptr && c->total != nullptr && c->capacity >= 1;
}

CacheView view_of(const curdkv_cache* c) {
  return CacheView{static_cast<__nv_bfloat16*>(c->K), static_cast<__nv_bfloat16*>(c->V), c->raw, c->pos,
                   c->count, c->total, c->capacity};
}

}  // namespace

extern "C" {

size_t curdkv_cache_workspace_bytes(int32_t batch, int32_t kv_heads, int32_t t_max, int32_t capacity,
                                    int32_t budget) {
  CacheWorkspace L;
  return layout(batch, kv_heads, t_max, capacity, budget, &L) ? L.total : 0;
}

curdkv_status curdkv_cache_append(const curdkv_cache* cache, const void* K_new, const void* V_new,
                                  const float* G, int32_t g_per_head, const curdkv_desc* desc_new,
                                  void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!cache_ok(cache) || desc_new == nullptr || workspace == nullptr) return CURDKV_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return CURDKV_ERR_INVALID_ARG;
  CacheWorkspace L;
  if (!layout(desc_new->batch, desc_new->kv_heads, desc_new->n_max, cache->capacity, 0, &L))
    return CURDKV_ERR_INVALID_ARG;
  if (workspace_bytes < L.total) return CURDKV_ERR_WORKSPACE;
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  float* raw_new = reinterpret_cast<float*>(ws + L.raw_new);

  curdkv_desc d = *desc_new;
  d.raw_scores = 1;
  d.score_mode = 0;
  d.whiten = 0;                       // a row's score must not depend on the rows it arrives with
  // only the real rows' scores are read below: no normalisation pass, no head sums
  curdkv_status st = score_unnormalised(K_new, V_new, G, g_per_head, &d, raw_new, ws + L.score_ws,
                                        L.raw_new - L.score_ws, cuda_stream);
  if (st != CURDKV_OK) return st;
  const int64_t P = (int64_t)d.batch * d.kv_heads;
  if (P == 0 || d.n_max == 0) return CURDKV_OK;

  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  AppendArgs a;
  a.cache = view_of(cache);
  a.K_new = KvView{static_cast<const __nv_bfloat16*>(K_new), d.k_stride_b, d.k_stride_h, d.k_stride_n};
  a.V_new = KvView{static_cast<const __nv_bfloat16*>(V_new), d.v_stride_b, d.v_stride_h, d.v_stride_n};
  a.raw_new = raw_new;
  a.t_new = d.seqlens;
  a.heads = d.kv_heads;
  a.t = d.n_max;
  a.d = d.d;
  a.status = reinterpret_cast<uint32_t*>(ws + L.score_ws);
  const int64_t chunks = (d.n_max + kAppendRowsPerCta - 1) / kAppendRowsPerCta;
  if (P * chunks > 0x7fffffffLL) return CURDKV_ERR_UNSUPPORTED;
  cache_append_kernel<<<(unsigned)(P * chunks), kAppendWarps * 32, 0, stream>>>(a);
  count_launch();
  if (cudaGetLastError() != cudaSuccess) return CURDKV_ERR_CUDA;
  cache_advance_kernel<<<(unsigned)((d.batch + 255) / 256), 256, 0, stream>>>(a.cache, d.seqlens, d.n_max,
                                                                             d.batch);
  count_launch();
  if (cudaGetLastError() != cudaSuccess) return CURDKV_ERR_CUDA;
  return CURDKV_OK;
}

curdkv_status curdkv_cache_compress(const curdkv_cache* in, const curdkv_cache* out,
                                    const curdkv_desc* desc, int32_t budget, int32_t num_sink,
                                    int32_t window, void* workspace, size_t workspace_bytes,
                                    void* cuda_stream) {
  if (!cache_ok(in) || !cache_ok(out) || desc == nullptr || workspace == nullptr)
    return CURDKV_ERR_INVALID_ARG;
  if (budget < 0 || num_sink < 0 || window < 0) return CURDKV_ERR_INVALID_ARG;
  if ((int64_t)num_sink + window > budget) return CURDKV_ERR_INVALID_ARG;   // forced rows must fit
  if (in->K == out->K || in->V == out->V || in->raw == out->raw || in->pos == out->pos)
    return CURDKV_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return CURDKV_ERR_INVALID_ARG;
  const int32_t most = budget < in->capacity ? budget : in->capacity;
  if (out->capacity < most) return CURDKV_ERR_INVALID_ARG;
  CacheWorkspace L;
  if (!layout(desc->batch, desc->kv_heads, 0, in->capacity, budget, &L)) return CURDKV_ERR_INVALID_ARG;
  if (workspace_bytes < L.total) return CURDKV_ERR_WORKSPACE;
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  int32_t* idx = reinterpret_cast<int32_t*>(ws + L.idx);
  int32_t* counts = reinterpret_cast<int32_t*>(ws + L.counts);
  const int64_t P = (int64_t)desc->batch * desc->kv_heads;
  if (P == 0) return CURDKV_OK;

  // the held rows of every (sequence, head) seen as one [batch][heads][capacity] problem set
  curdkv_desc d = *desc;
  d.q_heads = d.kv_heads;
  d.n_max = in->capacity;
  d.k_stride_n = d.v_stride_n = d.d;
  d.k_stride_h = d.v_stride_h = (int64_t)in->capacity * d.d;
  d.k_stride_b = d.v_stride_b = d.k_stride_h * d.kv_heads;
  d.seqlens = in->count;
  d.score_mode = 0;
  d.use_projection = 1;
  d.raw_scores = 0;
  // Forced rows are found by POSITION (sinks: positions below num_sink; window: the most recent
  // positions), whatever slots they sit in: a cache that curdkv_cache_compress_inplace has left
  // unordered is handled like an ordered one.  They enter the selection with an infinite key.
  float* keyed = reinterpret_cast<float*>(ws + L.keyed);
  cache_keyed_scores_kernel<<<(unsigned)P, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      view_of(in), desc->kv_heads, num_sink, window, keyed);
  count_launch();
  if (cudaGetLastError() != cudaSuccess) return CURDKV_ERR_CUDA;
  curdkv_status st = curdkv_select(keyed, &d, budget, nullptr, 0, 0, 0, 0.0, idx, counts, nullptr,
                                   ws + L.score_ws, L.raw_new - L.score_ws, cuda_stream);
  if (st != CURDKV_OK) return st;
  if (budget > 0) {
    st = curdkv_compact(in->K, in->V, &d, idx, budget, counts, nullptr, out->K, out->V, out->capacity,
                        ws + L.score_ws, cuda_stream);
    if (st != CURDKV_OK) return st;
  }
  cache_gather_meta_kernel<<<(unsigned)P, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      view_of(in), view_of(out), idx, budget, counts, d.kv_heads);
  count_launch();
  if (cudaGetLastError() != cudaSuccess) return CURDKV_ERR_CUDA;
  return CURDKV_OK;
}

curdkv_status curdkv_cache_compress_inplace(const curdkv_cache* cache, const curdkv_desc* desc,
                                            int32_t budget, int32_t num_sink, int32_t window,
                                            void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!cache_ok(cache) || desc == nullptr || workspace == nullptr) return CURDKV_ERR_INVALID_ARG;
  if (budget < 0 || num_sink < 0 || window < 0) return CURDKV_ERR_INVALID_ARG;
  if ((int64_t)num_sink + window > budget) return CURDKV_ERR_INVALID_ARG;   // forced rows must fit
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return CURDKV_ERR_INVALID_ARG;
  if (cache->capacity > 200 * 1024) return CURDKV_ERR_UNSUPPORTED;          // slot flags live in shared memory
  CacheWorkspace L;
  if (!layout(desc->batch, desc->kv_heads, 0, cache->capacity, budget, &L)) return CURDKV_ERR_INVALID_ARG;
  if (workspace_bytes < L.total) return CURDKV_ERR_WORKSPACE;
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  int32_t* idx = reinterpret_cast<int32_t*>(ws + L.idx);
  int32_t* counts = reinterpret_cast<int32_t*>(ws + L.counts);
  float* keyed = reinterpret_cast<float*>(ws + L.keyed);
  const int64_t P = (int64_t)desc->batch * desc->kv_heads;
  if (P == 0 || budget == 0) return budget == 0 && P > 0 ? CURDKV_ERR_INVALID_ARG : CURDKV_OK;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const CacheView view = view_of(cache);

  cache_keyed_scores_kernel<<<(unsigned)P, 256, 0, stream>>>(view, desc->kv_heads, num_sink, window, keyed);
  count_launch();
  if (cudaGetLastError() != cudaSuccess) return CURDKV_ERR_CUDA;

  curdkv_desc d = *desc;
  d.q_heads = d.kv_heads;
  d.n_max = cache->capacity;
  d.seqlens = cache->count;
  d.score_mode = 0;
  d.use_projection = 1;
  d.raw_scores = 0;
  d.whiten = 0;
  // forced rows carry +inf keys, so the selection itself needs no sinks or window
  curdkv_status st = curdkv_select(keyed, &d, budget, nullptr, 0, 0, 0, 0.0, idx, counts, nullptr,
                                   ws + L.score_ws, L.raw_new - L.score_ws, cuda_stream);
  if (st != CURDKV_OK) return st;
  if (cudaFuncSetAttribute(cache_fill_holes_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           200 * 1024) != cudaSuccess)
    return CURDKV_ERR_CUDA;
  cache_fill_holes_kernel<<<(unsigned)P, 256, (size_t)cache->capacity, stream>>>(
      view, idx, budget, counts, d.kv_heads, d.d, reinterpret_cast<int32_t*>(ws + L.holes),
      reinterpret_cast<uint32_t*>(ws + L.score_ws), 1, nullptr, 0);      // sets count[b]; total[b] += 0
  count_launch();
  if (cudaGetLastError() != cudaSuccess) return CURDKV_ERR_CUDA;
  return CURDKV_OK;
}

curdkv_status curdkv_cache_step(const curdkv_cache* cache, const void* K_new, const void* V_new,
                                const float* G, int32_t g_per_head, const curdkv_desc* desc_new,
                                int32_t budget, int32_t num_sink, int32_t window, void* workspace,
                                size_t workspace_bytes, void* cuda_stream) {
  if (!cache_ok(cache) || desc_new == nullptr || workspace == nullptr) return CURDKV_ERR_INVALID_ARG;
  if (budget < 1 || num_sink < 0 || window < 0 || (int64_t)num_sink + window > budget)
    return CURDKV_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return CURDKV_ERR_INVALID_ARG;
  CacheWorkspace L;
  if (!layout(desc_new->batch, desc_new->kv_heads, desc_new->n_max, cache->capacity, budget, &L))
    return CURDKV_ERR_INVALID_ARG;
  if (workspace_bytes < L.total) return CURDKV_ERR_WORKSPACE;
  const int64_t P = (int64_t)desc_new->batch * desc_new->kv_heads;
  // the selection CTAs keep a head's keys and its candidate list in shared memory
  const int list_cap = cache->capacity <= 4096 ? kSelListCap / 4 : (cache->capacity <= 16384 ? kSelListCap / 2 : kSelListCap);
  const size_t stage_bytes = (((size_t)cache->capacity + 3) / 4) * sizeof(uint4);
  if (stage_bytes > (size_t)kSelStageBytes || desc_new->n_max < 1 || P < 1 || P > 0x7fffffffLL ||
      desc_new->d % 8 != 0) {
    // shapes the one-launch form does not cover: the two calls it stands for
    curdkv_status st = curdkv_cache_append(cache, K_new, V_new, G, g_per_head, desc_new, workspace,
                                           workspace_bytes, cuda_stream);
    if (st != CURDKV_OK) return st;
    curdkv_desc d = *desc_new;
    return curdkv_cache_compress_inplace(cache, &d, budget, num_sink, window, workspace, workspace_bytes,
                                         cuda_stream);
  }
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  float* raw_new = reinterpret_cast<float*>(ws + L.raw_new);
  curdkv_desc d = *desc_new;
  d.raw_scores = 1;
  d.score_mode = 0;
  d.whiten = 0;
  curdkv_status st = score_unnormalised(K_new, V_new, G, g_per_head, &d, raw_new, ws + L.score_ws,
                                        L.raw_new - L.score_ws, cuda_stream);
  if (st != CURDKV_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  StepArgs sa;
  sa.append.cache = view_of(cache);
  sa.append.K_new = KvView{static_cast<const __nv_bfloat16*>(K_new), d.k_stride_b, d.k_stride_h, d.k_stride_n};
  sa.append.V_new = KvView{static_cast<const __nv_bfloat16*>(V_new), d.v_stride_b, d.v_stride_h, d.v_stride_n};
  sa.append.raw_new = raw_new;
  sa.append.t_new = d.seqlens;
  sa.append.heads = d.kv_heads;
  sa.append.t = d.n_max;
  sa.append.d = d.d;
  sa.append.status = reinterpret_cast<uint32_t*>(ws + L.score_ws);
  sa.budget = budget;
  sa.num_sink = num_sink;
  sa.window = window;
  sa.stage_quads = (int)(stage_bytes / sizeof(uint4));
  sa.list_cap = list_cap;
  sa.idx = reinterpret_cast<int32_t*>(ws + L.idx);
  sa.counts = reinterpret_cast<int32_t*>(ws + L.counts);
  sa.tickets = reinterpret_cast<int32_t*>(ws + L.tickets);
  if (cudaMemsetAsync(sa.tickets, 0, (size_t)d.batch * sizeof(int32_t), stream) != cudaSuccess)
    return CURDKV_ERR_CUDA;
  // after the selection the staged keys' space takes a flag per slot and the list of holes
  const size_t place_bytes = (((size_t)cache->capacity + 15) & ~size_t(15)) + ((size_t)cache->capacity / 2 + 1) * 4;
  const size_t smem = (stage_bytes > place_bytes ? stage_bytes : place_bytes) + (size_t)list_cap * 8;
  if (cudaFuncSetAttribute(cache_step_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           kSelStageBytes + kSelListBytes) != cudaSuccess)
    return CURDKV_ERR_CUDA;
  cache_step_kernel<<<(unsigned)P, 256, smem, stream>>>(sa);
  count_launch();
  if (cudaGetLastError() != cudaSuccess) return CURDKV_ERR_CUDA;
  return CURDKV_OK;
}

}  // extern "C"
