// curdkv_compress_host: the whole path for a cache that lives in HOST memory.
// Chunks of batch elements are copied to the device, scored, selected and
// gathered, and the results copied back, on two internal streams so that the
// copies of one chunk overlap the kernels and the copies of the next.  Built
// only on the public device entry point curdkv_compress.
#include <cuda_runtime.h>

#include <cstdint>
#include <cstring>

#include "curdkv.h"

namespace {

inline size_t round256(size_t x) { return (x + 255) & ~size_t(255); }

struct SlotLayout {          // byte offsets inside one pipeline slot
  size_t K, V, scores, sums, idx, counts, offsets, K_out, V_out, seqlens, workspace, total;
};

inline int64_t cap_rows(const curdkv_desc* d, int32_t budget) {
  return budget < d->n_max ? budget : d->n_max;
}

bool slot_layout(const curdkv_desc* d, int32_t budget, int32_t adaptive, int32_t cb, SlotLayout* L) {
  curdkv_desc c = *d;
  c.batch = cb;
  const size_t ws = curdkv_workspace_bytes(&c, budget > 0 ? budget : 1, adaptive);
  if (ws == 0) return false;
  const size_t P = (size_t)cb * d->kv_heads;
  const size_t kv = P * (size_t)d->n_max * d->d * 2;
  const size_t rows = P * (size_t)(adaptive ? cap_rows(d, budget) : budget);
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o += round256(bytes ? bytes : 1); return at; };
  L->K = take(kv);
  L->V = take(kv);
  L->scores = take(P * (size_t)d->n_max * 4);
  L->sums = take(P * 4);
  L->idx = take(rows * 4);
  L->counts = take(P * 4);
  L->offsets = take((P + 1) * 4);
  L->K_out = take(rows * (size_t)d->d * 2);
  L->V_out = take(rows * (size_t)d->d * 2);
  L->seqlens = take((size_t)cb * 4);
  L->workspace = take(ws);
  L->total = o;
  return true;
}

bool host_dense(const curdkv_desc* d) {
  const int64_t sn = d->d, sh = (int64_t)d->n_max * sn, sb = (int64_t)d->kv_heads * sh;
  return d->k_stride_n == sn && d->k_stride_h == sh && d->k_stride_b == sb && d->v_stride_n == sn &&
         d->v_stride_h == sh && d->v_stride_b == sb;
}

}  // namespace

extern "C" {

size_t curdkv_host_arena_bytes(const curdkv_desc* desc, int32_t budget, int32_t adaptive,
                               int32_t chunk_batch) {
  if (desc == nullptr || budget < 0 || chunk_batch < 1) return 0;
  SlotLayout L;
  if (!slot_layout(desc, budget, adaptive, chunk_batch, &L)) return 0;
  const size_t g = round256((size_t)desc->kv_heads * desc->d * (desc->r > 0 ? desc->r : 1) * 4);
  const size_t chunks = ((size_t)desc->batch + chunk_batch - 1) / chunk_batch;
  return g + round256(4 * (chunks ? chunks : 1)) + 2 * L.total;
}

curdkv_status curdkv_compress_host(const void* K_host, const void* V_host, const float* G_host,
                                   int32_t g_per_head, const curdkv_desc* desc, int32_t budget,
                                   int32_t num_sink, int32_t window, int32_t adaptive, double alpha,
                                   void* K_out_host, void* V_out_host, int32_t* idx_host,
                                   int32_t* counts_host, int32_t* offsets_host, void* arena,
                                   size_t arena_bytes, int32_t chunk_batch, uint32_t* status_flags_host) {
  if (desc == nullptr || K_host == nullptr || V_host == nullptr || K_out_host == nullptr ||
      V_out_host == nullptr || idx_host == nullptr || counts_host == nullptr || arena == nullptr)
    return CURDKV_ERR_INVALID_ARG;
  if (budget < 0 || chunk_batch < 1 || (adaptive && offsets_host == nullptr))
    return CURDKV_ERR_INVALID_ARG;
  if (desc->use_projection && G_host == nullptr) return CURDKV_ERR_INVALID_ARG;
  if (!host_dense(desc)) return CURDKV_ERR_UNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(arena) & 255u) != 0) return CURDKV_ERR_INVALID_ARG;
  const size_t need = curdkv_host_arena_bytes(desc, budget, adaptive, chunk_batch);
  if (need == 0) return CURDKV_ERR_INVALID_ARG;
  if (arena_bytes < need) return CURDKV_ERR_WORKSPACE;
  if (status_flags_host != nullptr) *status_flags_host = 0;
  if (desc->batch == 0) return CURDKV_OK;

  SlotLayout L;
  slot_layout(desc, budget, adaptive, chunk_batch, &L);
  const int H = desc->kv_heads;
  const size_t g_bytes = (size_t)(g_per_head ? H : 1) * desc->d * (desc->r > 0 ? desc->r : 1) * 4;
  unsigned char* base = static_cast<unsigned char*>(arena);
  float* G_dev = reinterpret_cast<float*>(base);
  // one status word per chunk, so that a flag raised by any chunk survives the next chunk's reset
  const size_t num_chunks = ((size_t)desc->batch + chunk_batch - 1) / chunk_batch;
  uint32_t* flag_log = reinterpret_cast<uint32_t*>(
      base + round256((size_t)H * desc->d * (desc->r > 0 ? desc->r : 1) * 4));
  unsigned char* slot_base[2] = {reinterpret_cast<unsigned char*>(flag_log) + round256(4 * num_chunks),
                                 nullptr};
  slot_base[1] = slot_base[0] + L.total;

  cudaStream_t st[2] = {nullptr, nullptr};
  curdkv_status result = CURDKV_OK;
  auto fail = [&](curdkv_status s) { if (result == CURDKV_OK) result = s; };
  for (int i = 0; i < 2; ++i)
    if (cudaStreamCreateWithFlags(&st[i], cudaStreamNonBlocking) != cudaSuccess) fail(CURDKV_ERR_CUDA);
  uint32_t flags = 0;

  if (result == CURDKV_OK && desc->use_projection) {
    if (cudaMemcpyAsync(G_dev, G_host, g_bytes, cudaMemcpyHostToDevice, st[0]) != cudaSuccess ||
        cudaStreamSynchronize(st[0]) != cudaSuccess)
      fail(CURDKV_ERR_CUDA);
  }

  const size_t row_bytes = (size_t)desc->d * 2;
  const size_t elem_bytes = (size_t)H * desc->n_max * row_bytes;      // one batch element of K or V
  int64_t packed_base = 0;                                            // adaptive: rows before this chunk
  int chunk = 0;
  for (int b0 = 0; result == CURDKV_OK && b0 < desc->batch; b0 += chunk_batch, ++chunk) {
    const int cb = desc->batch - b0 < chunk_batch ? desc->batch - b0 : chunk_batch;
    const int s = chunk & 1;
    cudaStream_t stream = st[s];
    unsigned char* sb = slot_base[s];
    const size_t P = (size_t)cb * H;

    curdkv_desc c = *desc;
    c.batch = cb;
    c.seqlens = nullptr;
    int64_t chunk_rows = 0;                                           // rows this chunk keeps (adaptive)
    for (int b = 0; b < cb; ++b) {
      int n = desc->n_max;
      if (desc->seqlens != nullptr) {
        n = desc->seqlens[b0 + b];
        n = n < 0 ? 0 : (n > desc->n_max ? desc->n_max : n);
      }
      chunk_rows += (int64_t)H * (budget < n ? budget : n);
    }
    bool ok = true;
    auto copy = [&](void* dst, const void* src, size_t bytes, cudaMemcpyKind kind) {
      if (ok && bytes && cudaMemcpyAsync(dst, src, bytes, kind, stream) != cudaSuccess) ok = false;
    };
    copy(sb + L.K, static_cast<const unsigned char*>(K_host) + (size_t)b0 * elem_bytes,
         (size_t)cb * elem_bytes, cudaMemcpyHostToDevice);
    copy(sb + L.V, static_cast<const unsigned char*>(V_host) + (size_t)b0 * elem_bytes,
         (size_t)cb * elem_bytes, cudaMemcpyHostToDevice);
    if (desc->seqlens != nullptr) {
      copy(sb + L.seqlens, desc->seqlens + b0, (size_t)cb * 4, cudaMemcpyHostToDevice);
      c.seqlens = reinterpret_cast<const int32_t*>(sb + L.seqlens);
    }
    if (!ok) { fail(CURDKV_ERR_CUDA); break; }

    float* scores = reinterpret_cast<float*>(sb + L.scores);
    int32_t* idx = reinterpret_cast<int32_t*>(sb + L.idx);
    int32_t* counts = reinterpret_cast<int32_t*>(sb + L.counts);
    int32_t* offsets = reinterpret_cast<int32_t*>(sb + L.offsets);
    const curdkv_status stt =
        curdkv_compress(sb + L.K, sb + L.V, G_dev, g_per_head, &c, budget, nullptr, num_sink, window, adaptive,
                        alpha, scores, reinterpret_cast<float*>(sb + L.sums), idx, counts, offsets,
                        sb + L.K_out, sb + L.V_out, sb + L.workspace, L.total - L.workspace, stream);
    if (stt != CURDKV_OK) { fail(stt); break; }

    copy(counts_host + (size_t)b0 * H, counts, P * 4, cudaMemcpyDeviceToHost);
    if (adaptive) {
      copy(idx_host + packed_base, idx, (size_t)chunk_rows * 4, cudaMemcpyDeviceToHost);
      copy(offsets_host + (size_t)b0 * H, offsets, P * 4, cudaMemcpyDeviceToHost);
      copy(static_cast<unsigned char*>(K_out_host) + (size_t)packed_base * row_bytes, sb + L.K_out,
           (size_t)chunk_rows * row_bytes, cudaMemcpyDeviceToHost);
      copy(static_cast<unsigned char*>(V_out_host) + (size_t)packed_base * row_bytes, sb + L.V_out,
           (size_t)chunk_rows * row_bytes, cudaMemcpyDeviceToHost);
    } else {
      const size_t first = (size_t)b0 * H * budget;
      copy(idx_host + first, idx, P * budget * 4, cudaMemcpyDeviceToHost);
      copy(static_cast<unsigned char*>(K_out_host) + first * row_bytes, sb + L.K_out,
           P * budget * row_bytes, cudaMemcpyDeviceToHost);
      copy(static_cast<unsigned char*>(V_out_host) + first * row_bytes, sb + L.V_out,
           P * budget * row_bytes, cudaMemcpyDeviceToHost);
      if (offsets_host != nullptr)
        for (size_t p = 0; p < P; ++p)
          offsets_host[(size_t)b0 * H + p] = (int32_t)(((size_t)b0 * H + p) * budget);
    }
    copy(flag_log + chunk, sb + L.workspace, 4, cudaMemcpyDeviceToDevice);
    if (!ok) { fail(CURDKV_ERR_CUDA); break; }
    packed_base += chunk_rows;
    // the slot is reused two chunks later on the same stream, which orders the reuse
  }
  for (int i = 0; i < 2; ++i)
    if (st[i] != nullptr && cudaStreamSynchronize(st[i]) != cudaSuccess) fail(CURDKV_ERR_CUDA);

  if (result == CURDKV_OK && adaptive) {        // make the chunk-relative offsets global
    int64_t base_rows = 0;
    for (int b0 = 0; b0 < desc->batch; b0 += chunk_batch) {
      const int cb = desc->batch - b0 < chunk_batch ? desc->batch - b0 : chunk_batch;
      int64_t rows = 0;
      for (size_t p = 0; p < (size_t)cb * H; ++p) {
        offsets_host[(size_t)b0 * H + p] += (int32_t)base_rows;
        rows += counts_host[(size_t)b0 * H + p];
      }
      base_rows += rows;
    }
    offsets_host[(size_t)desc->batch * H] = (int32_t)base_rows;
  } else if (result == CURDKV_OK && offsets_host != nullptr) {
    offsets_host[(size_t)desc->batch * H] = (int32_t)((size_t)desc->batch * H * budget);
  }
  for (int i = 0; i < 2; ++i)
    if (st[i] != nullptr) cudaStreamDestroy(st[i]);
  for (size_t c0 = 0; result == CURDKV_OK && c0 < (size_t)chunk; c0 += 64) {
    uint32_t tmp[64];
    const size_t m = (size_t)chunk - c0 < 64 ? (size_t)chunk - c0 : 64;
    if (cudaMemcpy(tmp, flag_log + c0, m * 4, cudaMemcpyDeviceToHost) != cudaSuccess) fail(CURDKV_ERR_CUDA);
    else for (size_t i = 0; i < m; ++i) flags |= tmp[i];
  }
  if (status_flags_host != nullptr) *status_flags_host = flags;
  if (result == CURDKV_OK && (flags & CURDKV_DEV_TIMEOUT)) result = CURDKV_ERR_TIMEOUT;
  return result;
}

}  // extern "C"
