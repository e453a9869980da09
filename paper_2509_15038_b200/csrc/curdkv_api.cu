// C ABI of the CurDKV library: argument checks and kernel launches.
#include <atomic>
#include <cmath>
#include <cstdint>
#include <mutex>

#include "common.cuh"
#include "compact.cuh"
#include "score_simt.cuh"
#include "score_umma.cuh"
#include "select_kernels.cuh"
#include "whiten_factor.cuh"
#include "whiten_umma.cuh"
#include "attn_umma.cuh"

namespace {

using namespace curdkv;

std::atomic<uint64_t> g_launches{0};

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline bool launch_ok() {
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return cudaGetLastError() == cudaSuccess;
}

curdkv_status check_desc(const curdkv_desc* d) {
  if (d == nullptr) return CURDKV_ERR_INVALID_ARG;
  if (d->batch < 0 || d->kv_heads < 1 || d->n_max < 0 || d->d < 1) return CURDKV_ERR_INVALID_ARG;
  if (d->q_heads < d->kv_heads || d->q_heads % d->kv_heads != 0) return CURDKV_ERR_INVALID_ARG;
  if (d->score_mode < 0 || d->score_mode > 2) return CURDKV_ERR_INVALID_ARG;
  if (d->use_projection != 0 && d->use_projection != 1) return CURDKV_ERR_INVALID_ARG;
  if (d->raw_scores != 0 && d->raw_scores != 1) return CURDKV_ERR_INVALID_ARG;
  if (d->whiten != 0 && d->whiten != 1) return CURDKV_ERR_INVALID_ARG;
  if (d->whiten && !(d->ridge >= 0.0)) return CURDKV_ERR_INVALID_ARG;
  if ((int64_t)d->batch * d->kv_heads > (int64_t)1 << 24) return CURDKV_ERR_UNSUPPORTED;
  return CURDKV_OK;
}

curdkv_status check_kv(const void* K, const void* V, const curdkv_desc* d) {
  if (K == nullptr || V == nullptr) return CURDKV_ERR_INVALID_ARG;
  if (d->d % 8 != 0 || d->d > 1024) return CURDKV_ERR_UNSUPPORTED;
  if (!aligned16(K) || !aligned16(V)) return CURDKV_ERR_INVALID_ARG;
  const int64_t s[6] = {d->k_stride_b, d->k_stride_h, d->k_stride_n,
                        d->v_stride_b, d->v_stride_h, d->v_stride_n};
  for (int64_t x : s)
    if (x < 0 || x % 8 != 0) return CURDKV_ERR_INVALID_ARG;
  if (d->k_stride_n < d->d || d->v_stride_n < d->d) return CURDKV_ERR_INVALID_ARG;
  return CURDKV_OK;
}

inline int tiles_per_head(const curdkv_desc* d) { return (d->n_max + kTileRows - 1) / kTileRows; }

inline size_t round256(size_t x) { return (x + 255) & ~size_t(255); }

// K/V tile loads of the score kernels: evict-first below 4 GB of K + V, the default policy above
// (measured: cfg2, 1 GB, 0.7 % faster with evict-first; cfg3 and cfg5, 17-19 GB, 0.5 % slower).
inline int stream_evict_first(const curdkv_desc* d) {
  return (double)d->batch * d->kv_heads * d->n_max * d->d * 4.0 < 4e9 ? 1 : 0;
}

// What curdkv_compress keeps next to the status words: per head a tile counter and an entry of
// the list of finished heads and a selected flag, and two queue counters.
inline size_t head_counter_bytes(const curdkv_desc* d) {
  return round256((size_t)d->batch * d->kv_heads * 3 * sizeof(int32_t)) + 256;
}

// ---- TMA descriptors for the tensor-core sketch kernel ---------------------
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                   const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                   const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// bf16 tensor [batch][heads][n_max][128] -> 4-D map (channel, row, head, batch) with a
// box of 64 channels x 128 rows and the 128-byte swizzle the MMA descriptors expect.
bool make_tile_map(CUtensorMap* map, const void* base, const curdkv_desc* d, int64_t sb, int64_t sh,
                   int64_t sn) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr) return false;
  const cuuint64_t dims[4] = {(cuuint64_t)d->d, (cuuint64_t)d->n_max, (cuuint64_t)d->kv_heads,
                              (cuuint64_t)d->batch};
  // a size-1 axis never moves: give it any legal stride
  const cuuint64_t row = (cuuint64_t)sn * 2;
  const cuuint64_t strides[3] = {row, d->kv_heads > 1 ? (cuuint64_t)sh * 2 : row,
                                 d->batch > 1 ? (cuuint64_t)sb * 2 : row};
  const cuuint32_t box[4] = {64, (cuuint32_t)kTileRows, 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box,
            estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int sm_count() {
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  return n;
}

// SMs the host-side heuristics plan for: the current device's, or a B200's where no device can be
// asked (workspace sizes are also queried on machines without a GPU).
int planning_sm_count() {
  const int n = sm_count();
  return n > 0 ? n : 148;
}

// Events a caller asked to have recorded around the next sketch kernel of this
// host thread (curdkv_profile_next_score).
thread_local cudaEvent_t g_profile_start = nullptr, g_profile_stop = nullptr;

template <int R, bool FUSED = false>
cudaError_t launch_umma(const CUtensorMap& mk, const CUtensorMap& mv, const umma::Args& a,
                        cudaStream_t stream) {
  using L = umma::Smem<R, FUSED>;
  const int smem = L::dynamic_bytes(a.seqlens != nullptr ? a.batch : 0);
  cudaError_t e = cudaFuncSetAttribute(umma::sketch_umma_kernel<R, FUSED>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       L::dynamic_bytes(FUSED ? 0 : umma::kMaxRaggedBatch));
  if (e != cudaSuccess) return e;
  const int sms = sm_count();
  if (sms <= 0) return cudaErrorUnknown;
  const int64_t tiles = (int64_t)a.batch * a.heads * a.tiles_per_head;   // upper bound if ragged
  const unsigned grid = (unsigned)(tiles < sms ? tiles : sms);
  if (g_profile_start != nullptr) cudaEventRecord(g_profile_start, stream);
  if (FUSED) {
    // the selection groups wait for heads that other CTAs stream: all CTAs must be resident at once
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(umma::kFusedThreads);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, umma::sketch_umma_kernel<R, FUSED>, mk, mv, a);
  } else {
    umma::sketch_umma_kernel<R, FUSED><<<grid, umma::kThreads, smem, stream>>>(mk, mv, a);
  }
  if (g_profile_stop != nullptr) cudaEventRecord(g_profile_stop, stream);
  return e;
}

// ---- built-in scratch of curdkv_score_static --------------------------------
// Status words plus up to kStaticParts fp32 tile partial sums.  The array lives
// in every GPU context that loads this library, for the life of the process.
constexpr size_t kStaticParts = size_t(1) << 20;
constexpr size_t kStaticBytes = kStatusBytes + kStaticParts * sizeof(float);
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void* g_static_ptr[kMaxDevices] = {};

// Device address of the scratch array on the current device.  In host code the
// array's name is only a handle, so the address is looked up once per device.
void* static_scratch_ptr() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (g_static_ptr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess) return nullptr;
    g_static_ptr[dev] = p;
  }
  return g_static_ptr[dev];
}

// Whitened scoring cuts every head into this many runs of tiles (the work items of the two
// streaming kernels).  An item costs its tiles plus a fixed part (staging W, draining and storing
// a partial Gram matrix: about ten tiles' worth, measured), and every CTA walks ceil(P s / SMs)
// items, so the count that minimises rounds x (tiles per item + fixed part) is taken: many
// segments balance the SMs, few keep the fixed part small.
int whiten_segments(const curdkv_desc* d) {
  const int64_t P = (int64_t)d->batch * d->kv_heads;
  if (P <= 0) return 1;
  const int tiles = tiles_per_head(d);
  constexpr int64_t kItemOverheadTiles = 10;
  const int64_t sms = planning_sm_count();
  int best = 1;
  int64_t best_cost = -1;
  for (int s = 1; s <= tiles && s <= 1024; ++s) {
    const int64_t rounds = (P * s + sms - 1) / sms;
    const int64_t cost = rounds * ((tiles + s - 1) / s + kItemOverheadTiles);
    if (best_cost < 0 || cost < best_cost) {
      best_cost = cost;
      best = s;
    }
  }
  return best;
}

struct WhitenLayout {      // byte offsets from the workspace base, after the tile sums
  size_t partials, W, total;
};

WhitenLayout whiten_layout(const curdkv_desc* d, size_t after_tile_sums) {
  WhitenLayout L;
  const size_t P = (size_t)d->batch * d->kv_heads;
  L.partials = after_tile_sums;
  L.W = L.partials + round256(P * whiten_segments(d) * 2 * 128 * 128 * sizeof(float));
  L.total = L.W + round256(P * 2 * 128 * (size_t)(d->r > 0 ? d->r : 1) * sizeof(float));
  return L;
}

// valid key rows of every (sequence, head) when the caller gave none: the sequence lengths
__global__ void rows_from_seqlens_kernel(const int32_t* seqlens, int heads, int n_max, int problems,
                                         int32_t* rows) {
  const int p = blockIdx.x * blockDim.x + threadIdx.x;
  if (p < problems) rows[p] = seq_len_of(seqlens, p / heads, n_max);
}

KvView view_of(const void* base, int64_t sb, int64_t sh, int64_t sn) {
  return KvView{static_cast<const __nv_bfloat16*>(base), sb, sh, sn};
}

}  // namespace

namespace {
curdkv_status score_impl(const void* K, const void* V, const float* G, int32_t g_per_head,
                         const curdkv_desc* desc, float* scores, float* head_sums, void* workspace,
                         size_t workspace_bytes, void* cuda_stream, bool normalise, int* parts_per_tile);
curdkv_status compact_impl(const void* K, const void* V, const curdkv_desc* desc, const int32_t* idx,
                           int64_t idx_stride, const int32_t* head_counts, const int32_t* head_offsets,
                           void* K_out, void* V_out, int64_t out_stride_h, void* workspace,
                           void* cuda_stream, const int32_t* ready);
}  // namespace

namespace curdkv {
void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

curdkv_status score_unnormalised(const void* K, const void* V, const float* G, int32_t g_per_head,
                                 const curdkv_desc* desc, float* scores, void* workspace,
                                 size_t workspace_bytes, void* cuda_stream) {
  float unused_sums = 0.f;                                 // only checked for NULL
  return score_impl(K, V, G, g_per_head, desc, scores, &unused_sums, workspace, workspace_bytes, cuda_stream,
                    false, nullptr);
}
}  // namespace curdkv

extern "C" {

size_t curdkv_workspace_bytes(const curdkv_desc* desc, int32_t max_budget, int32_t adaptive) {
  (void)adaptive;
  if (check_desc(desc) != CURDKV_OK) return 0;
  const size_t tiles = (size_t)desc->batch * desc->kv_heads * tiles_per_head(desc);
  const size_t plain = kStatusBytes + round256(tiles * umma::kPartsPerTile * sizeof(float));
  const size_t score = desc->whiten ? whiten_layout(desc, plain).total : plain;
  // curdkv_compress also keeps one tile counter per head
  return score + (max_budget > 0 ? head_counter_bytes(desc) : 0);
}

}  // extern "C"

namespace {

// curdkv_score; with normalise = false the scores stay as the score kernels leave them
// (unnormalised, one or four partial sums per tile in the workspace: *parts_per_tile) for a
// selection kernel that finishes Alg. 1 (normalisation step) itself.
curdkv_status score_impl(const void* K, const void* V, const float* G, int32_t g_per_head,
                         const curdkv_desc* desc, float* scores, float* head_sums, void* workspace,
                         size_t workspace_bytes, void* cuda_stream, bool normalise, int* parts_per_tile) {
  curdkv_status st = check_desc(desc);
  if (st != CURDKV_OK) return st;
  if ((st = check_kv(K, V, desc)) != CURDKV_OK) return st;
  if (scores == nullptr || head_sums == nullptr || workspace == nullptr) return CURDKV_ERR_INVALID_ARG;
  if (g_per_head != 0 && g_per_head != 1) return CURDKV_ERR_INVALID_ARG;
  if (desc->use_projection) {
    if (G == nullptr || desc->r < 1) return CURDKV_ERR_INVALID_ARG;
    if (desc->d != 128 || desc->r > 64) return CURDKV_ERR_UNSUPPORTED;
  }
  if (desc->whiten && (!desc->use_projection || g_per_head || desc->n_max < kTileRows))
    return CURDKV_ERR_UNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return CURDKV_ERR_INVALID_ARG;
  if (workspace_bytes < curdkv_workspace_bytes(desc, 0, 0)) return CURDKV_ERR_WORKSPACE;

  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(workspace, 0, kStatusBytes, stream) != cudaSuccess) return CURDKV_ERR_CUDA;
  const int64_t P = (int64_t)desc->batch * desc->kv_heads;
  const int tiles = tiles_per_head(desc);
  if (P == 0 || tiles == 0) return CURDKV_OK;
  if (P * tiles > 0x7fffffffLL) return CURDKV_ERR_UNSUPPORTED;

  ScoreArgs a;
  a.K = view_of(K, desc->k_stride_b, desc->k_stride_h, desc->k_stride_n);
  a.V = view_of(V, desc->v_stride_b, desc->v_stride_h, desc->v_stride_n);
  a.G = G;
  a.g_per_head = g_per_head;
  a.seqlens = desc->seqlens;
  a.heads = desc->kv_heads;
  a.n_max = desc->n_max;
  a.d = desc->d;
  a.r = desc->r;
  a.tiles_per_head = tiles;
  a.score_mode = desc->score_mode;
  a.scores = scores;
  a.tile_sums = reinterpret_cast<float*>(static_cast<unsigned char*>(workspace) + kStatusBytes);

  const unsigned grid = (unsigned)(P * tiles);
  int parts = 1;                                  // partial sums per 128-row tile
  bool launched = false;
  if (desc->whiten) {
    // two passes over K and V: Gram matrices, their factors, then the sketch with W = L^-T G
    CUtensorMap mk, mv;
    if (!make_tile_map(&mk, K, desc, desc->k_stride_b, desc->k_stride_h, desc->k_stride_n) ||
        !make_tile_map(&mv, V, desc, desc->v_stride_b, desc->v_stride_h, desc->v_stride_n))
      return CURDKV_ERR_CUDA;
    const size_t plain = kStatusBytes + round256((size_t)P * tiles * umma::kPartsPerTile * sizeof(float));
    const WhitenLayout L = whiten_layout(desc, plain);
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    umma::ItemArgs u;
    u.seqlens = desc->seqlens;
    u.batch = desc->batch;
    u.heads = desc->kv_heads;
    u.n_max = desc->n_max;
    u.segments = whiten_segments(desc);
    u.status = static_cast<uint32_t*>(workspace);
    u.partials = reinterpret_cast<float*>(ws + L.partials);
    u.W = reinterpret_cast<const float*>(ws + L.W);
    u.w_per_problem = u.w_per_tensor = 1;
    u.r = desc->r;
    u.tiles_per_head = tiles;
    u.score_mode = desc->score_mode;
    u.scores = scores;
    u.tile_sums = a.tile_sums;
    const int sms = sm_count();
    if (sms <= 0) return CURDKV_ERR_CUDA;
    const int64_t items = P * u.segments;
    const unsigned grid_items = (unsigned)(items < sms ? items : sms);
    if (cudaFuncSetAttribute(umma::gram_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             umma::kGramDynamic) != cudaSuccess)
      return CURDKV_ERR_CUDA;
    umma::gram_umma_kernel<<<grid_items, umma::kThreads, umma::kGramDynamic, stream>>>(mk, mv, u);
    if (!launch_ok()) return CURDKV_ERR_CUDA;
    FactorArgs f;
    f.partials = u.partials;
    f.G = G;
    f.W = reinterpret_cast<float*>(ws + L.W);
    f.segments = u.segments;
    f.r = desc->r;
    f.ridge = desc->ridge;
    f.status = u.status;
    const size_t fsm = kFactorSmemBytes;
    if (cudaFuncSetAttribute(whiten_factor_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)fsm) != cudaSuccess)
      return CURDKV_ERR_CUDA;
    whiten_factor_kernel<<<(unsigned)(2 * P), kFactorThreads, fsm, stream>>>(f);
    if (!launch_ok()) return CURDKV_ERR_CUDA;
    if (g_profile_start != nullptr) cudaEventRecord(g_profile_start, stream);
    if (desc->r <= 32) {
      using S = umma::ItemSmem<32>;
      if (cudaFuncSetAttribute(umma::sketch_items_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               S::kDynamic) != cudaSuccess)
        return CURDKV_ERR_CUDA;
      umma::sketch_items_kernel<32><<<grid_items, umma::kThreads, S::kDynamic, stream>>>(mk, mv, u);
    } else {
      using S = umma::ItemSmem<64>;
      if (cudaFuncSetAttribute(umma::sketch_items_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               S::kDynamic) != cudaSuccess)
        return CURDKV_ERR_CUDA;
      umma::sketch_items_kernel<64><<<grid_items, umma::kThreads, S::kDynamic, stream>>>(mk, mv, u);
    }
    if (g_profile_stop != nullptr) cudaEventRecord(g_profile_stop, stream);
    if (!launch_ok()) return CURDKV_ERR_CUDA;
    parts = umma::kPartsPerTile;
    launched = true;
  } else if (desc->use_projection && g_per_head && desc->n_max >= kTileRows) {
    // one G per KV head: the item-walking sketch kernel with the head's G staged per item
    CUtensorMap mk, mv;
    if (make_tile_map(&mk, K, desc, desc->k_stride_b, desc->k_stride_h, desc->k_stride_n) &&
        make_tile_map(&mv, V, desc, desc->v_stride_b, desc->v_stride_h, desc->v_stride_n)) {
      umma::ItemArgs u;
      u.seqlens = desc->seqlens;
      u.batch = desc->batch;
      u.heads = desc->kv_heads;
      u.n_max = desc->n_max;
      u.segments = whiten_segments(desc);
      u.status = static_cast<uint32_t*>(workspace);
      u.partials = nullptr;
      u.W = G;
      u.w_per_problem = u.w_per_tensor = 0;
      u.r = desc->r;
      u.tiles_per_head = tiles;
      u.score_mode = desc->score_mode;
      u.scores = scores;
      u.tile_sums = a.tile_sums;
      const int sms = sm_count();
      if (sms <= 0) return CURDKV_ERR_CUDA;
      const int64_t items = P * u.segments;
      const unsigned grid_items = (unsigned)(items < sms ? items : sms);
      if (g_profile_start != nullptr) cudaEventRecord(g_profile_start, stream);
      if (desc->r <= 32) {
        using S = umma::ItemSmem<32>;
        if (cudaFuncSetAttribute(umma::sketch_items_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 S::kDynamic) != cudaSuccess)
          return CURDKV_ERR_CUDA;
        umma::sketch_items_kernel<32><<<grid_items, umma::kThreads, S::kDynamic, stream>>>(mk, mv, u);
      } else {
        using S = umma::ItemSmem<64>;
        if (cudaFuncSetAttribute(umma::sketch_items_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 S::kDynamic) != cudaSuccess)
          return CURDKV_ERR_CUDA;
        umma::sketch_items_kernel<64><<<grid_items, umma::kThreads, S::kDynamic, stream>>>(mk, mv, u);
      }
      if (g_profile_stop != nullptr) cudaEventRecord(g_profile_stop, stream);
      if (!launch_ok()) return CURDKV_ERR_CUDA;
      parts = umma::kPartsPerTile;
      launched = true;
    }
    g_profile_start = g_profile_stop = nullptr;
  } else if (desc->use_projection && !g_per_head && desc->n_max >= kTileRows) {
    // tensor-core path: one G for all heads, TMA tiles of 128 rows.  A ragged batch goes in
    // slices of at most kMaxRaggedBatch sequences (the kernel keeps their tile prefix sums
    // in shared memory).
    const int slice = desc->seqlens != nullptr ? umma::kMaxRaggedBatch : desc->batch;
    bool maps_ok = true;
    for (int b0 = 0; b0 < desc->batch && maps_ok; b0 += slice) {
      curdkv_desc part = *desc;
      part.batch = desc->batch - b0 < slice ? desc->batch - b0 : slice;
      const __nv_bfloat16* Kb = static_cast<const __nv_bfloat16*>(K) + (int64_t)b0 * desc->k_stride_b;
      const __nv_bfloat16* Vb = static_cast<const __nv_bfloat16*>(V) + (int64_t)b0 * desc->v_stride_b;
      CUtensorMap mk, mv;
      maps_ok = make_tile_map(&mk, Kb, &part, desc->k_stride_b, desc->k_stride_h, desc->k_stride_n) &&
                make_tile_map(&mv, Vb, &part, desc->v_stride_b, desc->v_stride_h, desc->v_stride_n);
      if (!maps_ok) break;
      const size_t p0 = (size_t)b0 * desc->kv_heads;
      umma::Args u;
      u.G = G;
      u.seqlens = desc->seqlens != nullptr ? desc->seqlens + b0 : nullptr;
      u.batch = part.batch;
      u.heads = desc->kv_heads;
      u.n_max = desc->n_max;
      u.r = desc->r;
      u.tiles_per_head = tiles;
      u.score_mode = desc->score_mode;
      u.scores = scores + p0 * desc->n_max;
      u.tile_sums = a.tile_sums + p0 * tiles * umma::kPartsPerTile;
      u.status = static_cast<uint32_t*>(workspace);
      u.evict_first = stream_evict_first(desc);
      const cudaError_t e = desc->r <= 32 ? launch_umma<32>(mk, mv, u, stream)
                                          : launch_umma<64>(mk, mv, u, stream);
      if (e != cudaSuccess) return CURDKV_ERR_CUDA;
      if (!launch_ok()) return CURDKV_ERR_CUDA;
      parts = umma::kPartsPerTile;
      launched = true;
    }
    if (launched && !maps_ok) return CURDKV_ERR_CUDA;      // a later slice could not be described
  }
  g_profile_start = g_profile_stop = nullptr;
  if (!launched) {
    if (desc->use_projection) {
      const int r_pad = (desc->r + 31) / 32 * 32;
      const size_t smem = 2 * (size_t)kTileRows * kFmaD * 2 + (size_t)kFmaD * r_pad * sizeof(float);
      if (cudaFuncSetAttribute(sketch_fma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               (int)smem) != cudaSuccess)
        return CURDKV_ERR_CUDA;
      sketch_fma_kernel<<<grid, 256, smem, stream>>>(a, r_pad);
    } else {
      row_norm_kernel<<<grid, 256, 0, stream>>>(a);
    }
    if (!launch_ok()) return CURDKV_ERR_CUDA;
  }

  if (parts_per_tile != nullptr) *parts_per_tile = parts;
  if (!normalise) return CURDKV_OK;
  const int chunks = (desc->n_max + kNormChunk - 1) / kNormChunk;
  normalise_kernel<<<(unsigned)(P * chunks), 256, 0, stream>>>(scores, a.tile_sums, head_sums,
                                                              desc->seqlens, desc->kv_heads,
                                                              desc->n_max, tiles, parts, chunks,
                                                              desc->raw_scores);
  if (!launch_ok()) return CURDKV_ERR_CUDA;
  return CURDKV_OK;
}

// curdkv_select; with norm.tile_sums the selection kernel normalises `scores` first
curdkv_status select_impl(float* scores, const curdkv_desc* desc, int32_t budget,
                          const int32_t* head_budgets, int32_t num_sink, int32_t window,
                          int32_t adaptive, double alpha, int32_t* idx, int32_t* head_counts,
                          int32_t* head_offsets, void* cuda_stream, const Normaliser& norm) {
  curdkv_status st = check_desc(desc);
  if (st != CURDKV_OK) return st;
  if (scores == nullptr || idx == nullptr || head_counts == nullptr) return CURDKV_ERR_INVALID_ARG;
  if (budget < 0 || num_sink < 0 || window < 0) return CURDKV_ERR_INVALID_ARG;
  if (adaptive != 0 && adaptive != 1) return CURDKV_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const int64_t P = (int64_t)desc->batch * desc->kv_heads;
  if (P == 0) return CURDKV_OK;
  if (adaptive) {
    if (!(alpha >= 0.0 && alpha <= 1.0) || head_offsets == nullptr || head_budgets != nullptr)
      return CURDKV_ERR_INVALID_ARG;
    if (desc->kv_heads > kMaxAdaptiveHeads) return CURDKV_ERR_UNSUPPORTED;
    if (P * (int64_t)(budget < desc->n_max ? budget : desc->n_max) > 0x7fffffffLL)
      return CURDKV_ERR_UNSUPPORTED;
    const int min_protected = (int)floor(alpha * (double)budget);
    // With one CTA of 1024 threads per SM, floor(SMs / heads) clusters run at a time.  When the
    // batch needs more than one such round, CTAs of 512 threads (two per SM) keep all clusters
    // resident instead.
    const int64_t one_round = planning_sm_count() / (desc->kv_heads > 0 ? desc->kv_heads : 1);
    const bool small_ctas = desc->batch > one_round;
    auto launch = [&](auto kernel, int threads) -> cudaError_t {
      if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               adaptive_dynamic_bytes(threads)) != cudaSuccess)
        return cudaErrorUnknown;
      if (desc->kv_heads > 8 &&
          cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess)
        return cudaErrorUnknown;
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3((unsigned)P);
      cfg.blockDim = dim3((unsigned)threads);
      cfg.dynamicSmemBytes = (size_t)adaptive_dynamic_bytes(threads);
      cfg.stream = stream;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = (unsigned)desc->kv_heads;
      attr[0].val.clusterDim.y = 1;
      attr[0].val.clusterDim.z = 1;
      cfg.attrs = attr;
      cfg.numAttrs = 1;
      return cudaLaunchKernelEx(&cfg, kernel, scores, desc->seqlens, (int)desc->kv_heads, (int)desc->n_max,
                                (int)budget, (int)num_sink, (int)window, min_protected, idx, head_counts,
                                head_offsets, norm);
    };
    const cudaError_t e = small_ctas ? launch(select_adaptive_kernel<512>, 512)
                                     : launch(select_adaptive_kernel<1024>, 1024);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (e != cudaSuccess || cudaGetLastError() != cudaSuccess) return CURDKV_ERR_CUDA;
    return CURDKV_OK;
  }
  // rows that fit are staged in shared memory once and re-read from there by every pass
  const size_t row_bytes = (((size_t)desc->n_max + 3) / 4) * sizeof(uint4);
  const size_t stage_bytes = row_bytes <= (size_t)kSelStageBytes ? row_bytes : 0;
  if (cudaFuncSetAttribute(select_fixed_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           kSelStageBytes + kSelListBytes) != cudaSuccess)
    return CURDKV_ERR_CUDA;
  // shorter rows run as smaller CTAs with a smaller list, several per SM: the many short phases
  // of a row then overlap with those of its neighbours
  int sel_threads = kSelThreads, list_cap = kSelListCap;
  if (desc->n_max <= 4096) { sel_threads = 256; list_cap = kSelListCap / 4; }
  else if (desc->n_max <= 16384) { sel_threads = 512; list_cap = kSelListCap / 2; }
  select_fixed_kernel<<<(unsigned)P, sel_threads, stage_bytes + (size_t)list_cap * 8, stream>>>(
      scores, desc->seqlens, desc->kv_heads, desc->n_max, budget, head_budgets, num_sink, window,
      (int)(stage_bytes / sizeof(uint4)), list_cap, idx, head_counts, head_offsets, norm);
  if (!launch_ok()) return CURDKV_ERR_CUDA;
  return CURDKV_OK;
}

}  // namespace

extern "C" {

curdkv_status curdkv_score(const void* K, const void* V, const float* G, int32_t g_per_head,
                           const curdkv_desc* desc, float* scores, float* head_sums,
                           void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return score_impl(K, V, G, g_per_head, desc, scores, head_sums, workspace, workspace_bytes, cuda_stream,
                    true, nullptr);
}

curdkv_status curdkv_select(const float* scores, const curdkv_desc* desc, int32_t budget,
                            const int32_t* head_budgets, int32_t num_sink, int32_t window,
                            int32_t adaptive, double alpha, int32_t* idx, int32_t* head_counts,
                            int32_t* head_offsets, void* workspace, size_t workspace_bytes,
                            void* cuda_stream) {
  (void)workspace;
  (void)workspace_bytes;
  // the kernels only write the scores when they are asked to normalise them
  return select_impl(const_cast<float*>(scores), desc, budget, head_budgets, num_sink, window, adaptive,
                     alpha, idx, head_counts, head_offsets, cuda_stream, Normaliser{nullptr, nullptr, 0, 0, 0});
}

curdkv_status curdkv_compact(const void* K, const void* V, const curdkv_desc* desc,
                             const int32_t* idx, int64_t idx_stride, const int32_t* head_counts,
                             const int32_t* head_offsets, void* K_out, void* V_out,
                             int64_t out_stride_h, void* workspace, void* cuda_stream) {
  return compact_impl(K, V, desc, idx, idx_stride, head_counts, head_offsets, K_out, V_out, out_stride_h,
                      workspace, cuda_stream, nullptr);
}

}  // extern "C"

namespace {

// curdkv_compact; with `ready` the launch is a programmatic dependent of the kernel before it
// in the stream (the fused score + select kernel), whose selection groups set ready[p] per head.
curdkv_status compact_impl(const void* K, const void* V, const curdkv_desc* desc, const int32_t* idx,
                           int64_t idx_stride, const int32_t* head_counts, const int32_t* head_offsets,
                           void* K_out, void* V_out, int64_t out_stride_h, void* workspace,
                           void* cuda_stream, const int32_t* ready) {
  curdkv_status st = check_desc(desc);
  if (st != CURDKV_OK) return st;
  if ((st = check_kv(K, V, desc)) != CURDKV_OK) return st;
  if (idx == nullptr || head_counts == nullptr || K_out == nullptr || V_out == nullptr)
    return CURDKV_ERR_INVALID_ARG;
  if (!aligned16(K_out) || !aligned16(V_out)) return CURDKV_ERR_INVALID_ARG;
  if (out_stride_h < 0 || idx_stride < 0) return CURDKV_ERR_INVALID_ARG;
  if (out_stride_h == 0 && head_offsets == nullptr) return CURDKV_ERR_INVALID_ARG;
  if (out_stride_h > 0 && idx_stride == 0) return CURDKV_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const int64_t P = (int64_t)desc->batch * desc->kv_heads;
  if (P == 0) return CURDKV_OK;

  CompactArgs a;
  a.K = view_of(K, desc->k_stride_b, desc->k_stride_h, desc->k_stride_n);
  a.V = view_of(V, desc->v_stride_b, desc->v_stride_h, desc->v_stride_n);
  a.seqlens = desc->seqlens;
  a.heads = desc->kv_heads;
  a.n_max = desc->n_max;
  a.d = desc->d;
  a.idx = idx;
  a.idx_stride = idx_stride;
  a.counts = head_counts;
  a.offsets = head_offsets;
  a.K_out = static_cast<__nv_bfloat16*>(K_out);
  a.V_out = static_cast<__nv_bfloat16*>(V_out);
  a.out_stride_h = out_stride_h;
  a.status = static_cast<uint32_t*>(workspace);
  a.ready = ready;

  // enough CTAs per head to cover a typical head in one sweep; larger heads loop
  const int64_t rows_hint = out_stride_h > 0 ? out_stride_h : (idx_stride > 0 ? idx_stride : 1024);
  int64_t ctas = (rows_hint + kCompactRowsPerCta - 1) / kCompactRowsPerCta;
  // (a CTA that first has to wait for its head's flag pays a round trip to L2 for it: eight
  // sweeps per CTA then)
  if (ready != nullptr) ctas = (ctas + 7) / 8;
  if (ctas < 1) ctas = 1;
  if (ctas > 256) ctas = 256;
  while (P * ctas > 0x7fffffffLL) ctas >>= 1;
  if (ready == nullptr) {
    compact_kernel<false><<<(unsigned)(P * ctas), kCompactWarps * 32, 0, stream>>>(a, (int)ctas);
  } else {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(P * ctas));
    cfg.blockDim = dim3(kCompactWarps * 32);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, compact_kernel<true>, a, (int)ctas) != cudaSuccess) return CURDKV_ERR_CUDA;
  }
  if (!launch_ok()) return CURDKV_ERR_CUDA;
  return CURDKV_OK;
}

}  // namespace

extern "C" {

curdkv_status curdkv_compress(const void* K, const void* V, const float* G, int32_t g_per_head,
                              const curdkv_desc* desc, int32_t budget, const int32_t* head_budgets,
                              int32_t num_sink, int32_t window, int32_t adaptive, double alpha,
                              float* scores, float* head_sums, int32_t* idx, int32_t* head_counts,
                              int32_t* head_offsets, void* K_out, void* V_out, void* workspace,
                              size_t workspace_bytes, void* cuda_stream) {
  curdkv_status st = check_desc(desc);
  if (st != CURDKV_OK) return st;
  if ((st = check_kv(K, V, desc)) != CURDKV_OK) return st;
  if (scores == nullptr || head_sums == nullptr || idx == nullptr || head_counts == nullptr ||
      K_out == nullptr || V_out == nullptr || workspace == nullptr)
    return CURDKV_ERR_INVALID_ARG;
  if (budget < 0 || num_sink < 0 || window < 0) return CURDKV_ERR_INVALID_ARG;
  if (adaptive != 0 && adaptive != 1) return CURDKV_ERR_INVALID_ARG;
  if (adaptive && head_offsets == nullptr) return CURDKV_ERR_INVALID_ARG;
  if (!aligned16(K_out) || !aligned16(V_out)) return CURDKV_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return CURDKV_ERR_INVALID_ARG;
  const size_t score_bytes = curdkv_workspace_bytes(desc, 0, 0);
  if (workspace_bytes < score_bytes + head_counter_bytes(desc)) return CURDKV_ERR_WORKSPACE;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const int64_t P = (int64_t)desc->batch * desc->kv_heads;
  const int tiles = tiles_per_head(desc);

  // One launch scores and selects when the tensor-core sketch applies and every head has its own
  // budget; the selection then hides behind the K/V stream.  Otherwise the three steps follow
  // one another.
  // (With fewer heads than SMs the selection of the last heads, which only starts when the stream
  // ends and runs on a quarter of a selection CTA's threads, costs more than the gather that
  // starts beside it wins back: 64 heads of 8192 rows 0.100 against 0.092 ms, 128 heads 0.149
  // against 0.153 ms, 256 heads 0.259 against 0.266 ms.)
  // Ragged batches keep the three-step route as well: their many short heads make the
  // selection warps busy enough to slow the stream by more than the hidden selection saves.
  const bool fused = !adaptive && budget > 0 && desc->use_projection && !g_per_head && !desc->whiten &&
                     P >= (int64_t)sm_count() && desc->seqlens == nullptr &&
                     desc->d == 128 && desc->r >= 1 && desc->r <= 32 && desc->n_max >= kTileRows &&
                     G != nullptr && P > 0 && P * tiles <= 0x7fffffffLL &&
                     P * (int64_t)budget <= 0x7fffffffLL;
  if (!fused) {
    // the selection kernel forms the head sums and divides on its first sweep over the scores:
    // no separate normalisation pass
    int parts = 1;
    st = score_impl(K, V, G, g_per_head, desc, scores, head_sums, workspace, score_bytes, cuda_stream, false,
                    &parts);
    if (st == CURDKV_OK && P > 0) {
      const Normaliser norm{reinterpret_cast<const float*>(static_cast<unsigned char*>(workspace) + kStatusBytes),
                            head_sums, tiles, parts, desc->raw_scores};
      st = select_impl(scores, desc, budget, head_budgets, num_sink, window, adaptive, alpha, idx, head_counts,
                       head_offsets, cuda_stream, tiles > 0 ? norm : Normaliser{nullptr, nullptr, 0, 0, 0});
    }
  } else {
    // workspace: status words, one tile counter per head (zero on entry), tile partial sums
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    const size_t counters = head_counter_bytes(desc);
    if (cudaMemsetAsync(ws, 0, kStatusBytes + counters, stream) != cudaSuccess) return CURDKV_ERR_CUDA;
    int32_t* head_done = reinterpret_cast<int32_t*>(ws + kStatusBytes);
    int32_t* done_list = head_done + P;
    int32_t* head_ready = done_list + P;
    int32_t* queue_ctr = reinterpret_cast<int32_t*>(ws + kStatusBytes + round256((size_t)P * 3 * sizeof(int32_t)));
    float* tile_sums = reinterpret_cast<float*>(ws + kStatusBytes + counters);
    CUtensorMap mk, mv;
    if (!make_tile_map(&mk, K, desc, desc->k_stride_b, desc->k_stride_h, desc->k_stride_n) ||
        !make_tile_map(&mv, V, desc, desc->v_stride_b, desc->v_stride_h, desc->v_stride_n))
      return CURDKV_ERR_CUDA;
    umma::Args u;
    u.G = G;
    u.seqlens = nullptr;
    u.batch = desc->batch;
    u.heads = desc->kv_heads;
    u.n_max = desc->n_max;
    u.r = desc->r;
    u.tiles_per_head = tiles;
    u.score_mode = desc->score_mode;
    u.scores = scores;
    u.tile_sums = tile_sums;
    u.status = static_cast<uint32_t*>(workspace);
    u.head_sums = head_sums;
    u.head_done = head_done;
    u.done_list = done_list;
    u.queue_ctr = queue_ctr;
    u.head_ready = head_ready;
    u.head_budgets = head_budgets;
    u.idx = idx;
    u.counts = head_counts;
    u.offsets = head_offsets;
    u.budget = budget;
    u.num_sink = num_sink;
    u.window = window;
    u.raw = desc->raw_scores;
    u.first_head = 0;
    u.all_heads = (int)P;
    // chunks of consecutive tiles per CTA visit: long enough to make the per-chunk bookkeeping
    // rare, short enough that the last, uneven round of chunks stays near 1 % of the launch
    const int sms = sm_count();
    const int64_t per_cta = P * tiles / (sms > 0 ? sms : 1);
    u.chunk_tiles = (int)(per_cta / 64 < 1 ? 1 : (per_cta / 64 > 16 ? 16 : per_cta / 64));
    u.evict_first = stream_evict_first(desc);
    if (launch_umma<32, true>(mk, mv, u, stream) != cudaSuccess) return CURDKV_ERR_CUDA;
    if (!launch_ok()) return CURDKV_ERR_CUDA;
    g_profile_start = g_profile_stop = nullptr;
  }
  if (st != CURDKV_OK) return st;
  if (!adaptive && budget == 0) return CURDKV_OK;          // nothing is kept, nothing to gather
  // Behind the fused kernel the gather is launched as its programmatic dependent: its CTAs move in
  // as that kernel's CTAs finish and copy the heads already selected while the last heads'
  // selection, which only starts when the stream ends, is still running.
  const int32_t* ready = nullptr;
  if (fused)
    ready = reinterpret_cast<const int32_t*>(static_cast<unsigned char*>(workspace) + kStatusBytes) + 2 * P;
  return compact_impl(K, V, desc, idx, adaptive ? 0 : budget, head_counts, head_offsets, K_out, V_out,
                      adaptive ? 0 : budget, workspace, cuda_stream, ready);
}

curdkv_status curdkv_gqa_map(const curdkv_desc* desc, int32_t* kv_head_of_q, void* cuda_stream) {
  curdkv_status st = check_desc(desc);
  if (st != CURDKV_OK) return st;
  if (kv_head_of_q == nullptr) return CURDKV_ERR_INVALID_ARG;
  gqa_map_kernel<<<(desc->q_heads + 127) / 128, 128, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      kv_head_of_q, desc->q_heads, desc->kv_heads);
  if (!launch_ok()) return CURDKV_ERR_CUDA;
  return CURDKV_OK;
}

curdkv_status curdkv_gqa_expand(const curdkv_desc* desc, const int32_t* idx, const int32_t* head_counts,
                                int32_t budget, int32_t* idx_q, int32_t* counts_q, void* cuda_stream) {
  curdkv_status st = check_desc(desc);
  if (st != CURDKV_OK) return st;
  if (idx == nullptr || head_counts == nullptr || idx_q == nullptr || counts_q == nullptr || budget < 0)
    return CURDKV_ERR_INVALID_ARG;
  const int64_t blocks = (int64_t)desc->batch * desc->q_heads;
  if (blocks == 0) return CURDKV_OK;
  if (blocks > 0x7fffffffLL) return CURDKV_ERR_UNSUPPORTED;
  gqa_expand_kernel<<<(unsigned)blocks, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      idx, head_counts, desc->q_heads, desc->kv_heads, budget, idx_q, counts_q);
  if (!launch_ok()) return CURDKV_ERR_CUDA;
  return CURDKV_OK;
}

curdkv_status curdkv_device_status(const void* workspace, uint32_t* host_flags, void* cuda_stream) {
  if (workspace == nullptr || host_flags == nullptr) return CURDKV_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemcpyAsync(host_flags, workspace, sizeof(uint32_t), cudaMemcpyDeviceToHost, stream) !=
      cudaSuccess)
    return CURDKV_ERR_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return CURDKV_ERR_CUDA;
  return (*host_flags & CURDKV_DEV_TIMEOUT) ? CURDKV_ERR_TIMEOUT : CURDKV_OK;
}

curdkv_status curdkv_score_static(const void* K, const void* V, const float* G, int32_t g_per_head,
                                  const curdkv_desc* desc, float* scores, float* head_sums,
                                  uint32_t* status_flags, void* cuda_stream) {
  const size_t need = curdkv_workspace_bytes(desc, 0, 0);
  if (need == 0) return CURDKV_ERR_INVALID_ARG;
  // the whitened mode parks Gram matrices and their factors in the workspace: far beyond what
  // the built-in array is sized for
  if (desc->whiten) return CURDKV_ERR_UNSUPPORTED;
  if (need > kStaticBytes) return CURDKV_ERR_STATIC_LIMIT;
  void* scratch = static_scratch_ptr();
  if (scratch == nullptr) return CURDKV_ERR_CUDA;
  // curdkv_score clears the status words itself; the partial sums are all rewritten
  const curdkv_status st = curdkv_score(K, V, G, g_per_head, desc, scores, head_sums, scratch,
                                        kStaticBytes, cuda_stream);
  if (st != CURDKV_OK) return st;
  if (status_flags != nullptr &&
      cudaMemcpyAsync(status_flags, scratch, sizeof(uint32_t), cudaMemcpyDeviceToDevice,
                      static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
    return CURDKV_ERR_CUDA;
  return CURDKV_OK;
}

size_t curdkv_attention_workspace_bytes(const curdkv_desc* desc) {
  if (check_desc(desc) != CURDKV_OK) return 0;
  return kStatusBytes + round256((size_t)desc->batch * desc->kv_heads * sizeof(int32_t));
}

curdkv_status curdkv_attention_out(const void* Q, int32_t q_rows, int64_t q_stride_b, int64_t q_stride_h,
                                   int64_t q_stride_n, const void* K, const void* V,
                                   const curdkv_desc* desc, const int32_t* head_rows,
                                   const int32_t* head_offsets, int64_t packed_rows,
                                   const int32_t* extra_zero_keys, float scale, int32_t weight_split,
                                   float* O, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  curdkv_status st = check_desc(desc);
  if (st == CURDKV_OK && weight_split != 0 && weight_split != 1) st = CURDKV_ERR_INVALID_ARG;
  if (st != CURDKV_OK) return st;
  if (Q == nullptr || K == nullptr || V == nullptr || O == nullptr || workspace == nullptr)
    return CURDKV_ERR_INVALID_ARG;
  if (desc->d != 128) return CURDKV_ERR_UNSUPPORTED;
  if (q_rows < 1 || !(scale == scale)) return CURDKV_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O)) return CURDKV_ERR_INVALID_ARG;
  if (q_stride_b < 0 || q_stride_h < 0 || q_stride_n < 128 || q_stride_b % 8 || q_stride_h % 8 || q_stride_n % 8)
    return CURDKV_ERR_INVALID_ARG;
  const bool packed = head_offsets != nullptr;
  if (packed && (head_rows == nullptr || packed_rows < 1)) return CURDKV_ERR_INVALID_ARG;
  if (!packed && (st = check_kv(K, V, desc)) != CURDKV_OK) return st;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return CURDKV_ERR_INVALID_ARG;
  if (workspace_bytes < curdkv_attention_workspace_bytes(desc)) return CURDKV_ERR_WORKSPACE;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(workspace, 0, kStatusBytes, stream) != cudaSuccess) return CURDKV_ERR_CUDA;
  const int64_t P = (int64_t)desc->batch * desc->kv_heads;
  if (P == 0) return CURDKV_OK;
  const int64_t q_blocks = ((int64_t)q_rows + kTileRows - 1) / kTileRows;
  if (P * q_blocks > 0x7fffffffLL) return CURDKV_ERR_UNSUPPORTED;

  const int32_t* rows = head_rows;
  if (rows == nullptr) {
    int32_t* mine = reinterpret_cast<int32_t*>(static_cast<unsigned char*>(workspace) + kStatusBytes);
    rows_from_seqlens_kernel<<<(unsigned)((P + 255) / 256), 256, 0, stream>>>(
        desc->seqlens, desc->kv_heads, desc->n_max, (int)P, mine);
    if (!launch_ok()) return CURDKV_ERR_CUDA;
    rows = mine;
  }
  curdkv_desc qd = *desc;
  qd.n_max = q_rows;
  CUtensorMap mq, mk, mv;
  if (!make_tile_map(&mq, Q, &qd, q_stride_b, q_stride_h, q_stride_n)) return CURDKV_ERR_CUDA;
  if (packed) {
    curdkv_desc pd = *desc;                                // one [packed_rows, 128] array
    pd.batch = pd.kv_heads = 1;
    if (packed_rows > 0x7fffffffLL) return CURDKV_ERR_UNSUPPORTED;
    pd.n_max = (int32_t)packed_rows;
    if (!make_tile_map(&mk, K, &pd, 0, 0, 128) || !make_tile_map(&mv, V, &pd, 0, 0, 128))
      return CURDKV_ERR_CUDA;
  } else if (!make_tile_map(&mk, K, desc, desc->k_stride_b, desc->k_stride_h, desc->k_stride_n) ||
             !make_tile_map(&mv, V, desc, desc->v_stride_b, desc->v_stride_h, desc->v_stride_n)) {
    return CURDKV_ERR_CUDA;
  }
  umma::AttnArgs a;
  a.rows = rows;
  a.row_start = packed ? head_offsets : nullptr;
  a.extra_zero = extra_zero_keys;
  a.heads = desc->kv_heads;
  a.m = q_rows;
  a.packed = packed ? 1 : 0;
  a.scale = scale;
  a.split = weight_split;
  a.O = O;
  a.status = static_cast<uint32_t*>(workspace);
  auto launch = [&](auto kernel) {
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, umma::kAttnDynamic) !=
        cudaSuccess)
      return false;
    kernel<<<(unsigned)(P * q_blocks), umma::kAttnThreads, umma::kAttnDynamic, stream>>>(mq, mk, mv, a);
    return true;
  };
  if (!(weight_split ? launch(umma::attention_umma_kernel<true>) : launch(umma::attention_umma_kernel<false>)))
    return CURDKV_ERR_CUDA;
  if (!launch_ok()) return CURDKV_ERR_CUDA;
  return CURDKV_OK;
}

curdkv_status curdkv_eviction_loss(const float* O_full, const float* O_compressed, int32_t problems,
                                   int64_t elems_per_problem, float* loss, float* ref_norm,
                                   void* cuda_stream) {
  if (O_full == nullptr || O_compressed == nullptr || loss == nullptr) return CURDKV_ERR_INVALID_ARG;
  if (problems < 0 || elems_per_problem < 0 || elems_per_problem > 0x7fffffffLL)
    return CURDKV_ERR_INVALID_ARG;
  if (problems == 0) return CURDKV_OK;
  umma::frob_diff_kernel<<<(unsigned)problems, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      O_full, O_compressed, (int)elems_per_problem, loss, ref_norm);
  if (!launch_ok()) return CURDKV_ERR_CUDA;
  return CURDKV_OK;
}

curdkv_status curdkv_selftest_bounded_wait(uint64_t limit_ns, void* workspace, void* cuda_stream) {
  if (workspace == nullptr || limit_ns == 0 || limit_ns > 1000000000ull) return CURDKV_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return CURDKV_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(workspace, 0, kStatusBytes, stream) != cudaSuccess) return CURDKV_ERR_CUDA;
  umma::wait_selftest_kernel<<<1, 128, 0, stream>>>(static_cast<uint32_t*>(workspace), limit_ns);
  if (!launch_ok()) return CURDKV_ERR_CUDA;
  return CURDKV_OK;
}

curdkv_status curdkv_selftest_gather_wait(uint64_t limit_ns, void* workspace, void* cuda_stream) {
  if (workspace == nullptr || limit_ns == 0 || limit_ns > 1000000000ull) return CURDKV_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return CURDKV_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(workspace, 0, 2 * kStatusBytes, stream) != cudaSuccess) return CURDKV_ERR_CUDA;
  CompactArgs a = {};                                      // one head; the kernel leaves before it reads any of the rest
  a.heads = 1;
  a.d = 128;
  a.status = static_cast<uint32_t*>(workspace);
  a.ready = reinterpret_cast<const int32_t*>(static_cast<unsigned char*>(workspace) + kStatusBytes);
  a.wait_ns = limit_ns;
  compact_kernel<true><<<1, kCompactWarps * 32, 0, stream>>>(a, 1);
  if (!launch_ok()) return CURDKV_ERR_CUDA;
  return CURDKV_OK;
}

curdkv_status curdkv_profile_next_score(void* start_event, void* stop_event) {
  g_profile_start = static_cast<cudaEvent_t>(start_event);
  g_profile_stop = static_cast<cudaEvent_t>(stop_event);
  return CURDKV_OK;
}

uint64_t curdkv_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* curdkv_status_string(curdkv_status status) {
  switch (status) {
    case CURDKV_OK: return "ok";
    case CURDKV_ERR_INVALID_ARG: return "invalid argument";
    case CURDKV_ERR_UNSUPPORTED: return "unsupported shape";
    case CURDKV_ERR_WORKSPACE: return "workspace too small";
    case CURDKV_ERR_CUDA: return "CUDA call failed";
    case CURDKV_ERR_TIMEOUT: return "device-side wait timed out";
    case CURDKV_ERR_STATIC_LIMIT:
      return "shape exceeds the built-in scratch of curdkv_score_static (2^20 tile partial sums)";
  }
  return "unknown status";
}

}  // extern "C"
