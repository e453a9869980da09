// Score kernels that run on the plain fp32 pipes.
//
//   row_norm_kernel    Alg. 1 without its sampling and projection steps (the "no projection" ablation of
//                      App. C.3): l_j = ||a_j||^2.  Pure streaming, HBM bound.
//   sketch_fma_kernel  Alg. 1 (sketch, row norms, product) with fp32 FMAs: y = a_j G, l_j = ||y||^2.
//                      Kept for sketch shapes the tensor-core kernel does not
//                      cover; fp32 G is used as it is (no splitting).
//
// Both write UNNORMALISED scores and one partial sum per 128-row tile; the
// normalise kernel finishes Alg. 1 (normalisation step).
#pragma once
#include "common.cuh"

namespace curdkv {

struct ScoreArgs {
  KvView K, V;
  const float* G;          // [d][r] or [heads][d][r]
  int g_per_head;
  const int32_t* seqlens;
  int heads, n_max, d, r;
  int tiles_per_head;      // ceil(n_max / kTileRows)
  int score_mode;
  float* scores;           // [batch*heads][n_max]
  float* tile_sums;        // [batch*heads][tiles_per_head]
};

// ---------------------------------------------------------------------------
// l_j = ||K_j||^2 (* ||V_j||^2): a half-warp per tensor row, 16-byte loads.
// grid = batch*heads*tiles_per_head (tile fastest), block = 256 (8 warps x 16 rows).
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256) row_norm_kernel(const ScoreArgs a) {
  __shared__ float warp_sum[8];
  const int p = blockIdx.x / a.tiles_per_head, tile = blockIdx.x % a.tiles_per_head;
  const int b = p / a.heads, h = p % a.heads;
  const int n = seq_len_of(a.seqlens, b, a.n_max);
  const int row0 = tile * kTileRows;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int half = lane >> 4, l16 = lane & 15;
  const KvView& T = half ? a.V : a.K;
  const __nv_bfloat16* base = T.base + b * T.stride_b + h * T.stride_h;
  const int chunks = a.d >> 3;
  float wsum = 0.f;
  for (int i = 0; i < 16; ++i) {
    const int j = row0 + warp * 16 + i;
    if (j >= a.n_max) break;
    float acc = 0.f;
    if (j < n) {
      const uint4* row = reinterpret_cast<const uint4*>(base + j * T.stride_n);
      for (int c = l16; c < chunks; c += 16) {
        float f[8];
        unpack_bf16x8(__ldg(row + c), f);
#pragma unroll
        for (int t = 0; t < 8; ++t) acc = fmaf(f[t], f[t], acc);
      }
    }
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    const float lv = __shfl_sync(0xffffffffu, acc, 16);
    if (lane == 0) {
      const float s = j < n ? combine_scores(acc, lv, a.score_mode) : 0.f;
      a.scores[(size_t)p * a.n_max + j] = s;
      wsum += s;
    }
  }
  if (lane == 0) warp_sum[warp] = wsum;
  __syncthreads();
  if (threadIdx.x == 0) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) s += warp_sum[w];
    a.tile_sums[(size_t)p * a.tiles_per_head + tile] = s;
  }
}

// ---------------------------------------------------------------------------
// fp32 FMA sketch.  A CTA stages one 128-row tile of K and V (d = 128) and G in
// shared memory; lane c of a warp owns sketch column c (+32 per pass) and walks
// 8 rows x 2 tensors at a time, reading row values as shared-memory broadcasts.
// grid = batch*heads*tiles_per_head (tile fastest), block = 256.
// dynamic smem = 2 * 128 * 256 B + 128 * r_pad * 4 B.
// ---------------------------------------------------------------------------
constexpr int kFmaD = 128;

__global__ void __launch_bounds__(256) sketch_fma_kernel(const ScoreArgs a, const int r_pad) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint4* sK = reinterpret_cast<uint4*>(smem_raw);                 // [128 rows][16 chunks]
  uint4* sV = sK + kTileRows * (kFmaD / 8);
  float* sG = reinterpret_cast<float*>(sV + kTileRows * (kFmaD / 8));  // [128][r_pad]
  __shared__ float warp_sum[8];

  const int p = blockIdx.x / a.tiles_per_head, tile = blockIdx.x % a.tiles_per_head;
  const int b = p / a.heads, h = p % a.heads;
  const int n = seq_len_of(a.seqlens, b, a.n_max);
  const int row0 = tile * kTileRows;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (row0 >= n) {      // tile holds no valid row
    for (int i = tid; i < kTileRows && row0 + i < a.n_max; i += 256)
      a.scores[(size_t)p * a.n_max + row0 + i] = 0.f;
    if (tid == 0) a.tile_sums[(size_t)p * a.tiles_per_head + tile] = 0.f;
    return;
  }

  const float* G = a.G + (a.g_per_head ? (size_t)h * a.d * a.r : 0);
  for (int i = tid; i < kFmaD * r_pad; i += 256) {
    const int t = i / r_pad, c = i % r_pad;
    sG[i] = c < a.r ? __ldg(G + (size_t)t * a.r + c) : 0.f;
  }
  const __nv_bfloat16* kb = a.K.base + b * a.K.stride_b + h * a.K.stride_h;
  const __nv_bfloat16* vb = a.V.base + b * a.V.stride_b + h * a.V.stride_h;
  for (int i = tid; i < kTileRows * 16; i += 256) {
    const int rr = i >> 4, c = i & 15, j = row0 + rr;
    uint4 zk = make_uint4(0, 0, 0, 0), zv = zk;
    if (j < n) {
      zk = __ldg(reinterpret_cast<const uint4*>(kb + j * a.K.stride_n) + c);
      zv = __ldg(reinterpret_cast<const uint4*>(vb + j * a.V.stride_n) + c);
    }
    sK[i] = zk;
    sV[i] = zv;
  }
  __syncthreads();

  float wsum = 0.f;
  for (int grp = 0; grp < 2; ++grp) {
    const int rbase = warp * 16 + grp * 8;
    float sqK[8], sqV[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) sqK[i] = sqV[i] = 0.f;
    for (int pass = 0; pass * 32 < r_pad; ++pass) {
      const int c = pass * 32 + lane;
      float yK[8], yV[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) yK[i] = yV[i] = 0.f;
      for (int t8 = 0; t8 < kFmaD / 8; ++t8) {
        float g[8];
#pragma unroll
        for (int tt = 0; tt < 8; ++tt) g[tt] = sG[(t8 * 8 + tt) * r_pad + c];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          float fk[8], fv[8];
          unpack_bf16x8(sK[(rbase + i) * 16 + t8], fk);
          unpack_bf16x8(sV[(rbase + i) * 16 + t8], fv);
#pragma unroll
          for (int tt = 0; tt < 8; ++tt) {
            yK[i] = fmaf(fk[tt], g[tt], yK[i]);
            yV[i] = fmaf(fv[tt], g[tt], yV[i]);
          }
        }
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        sqK[i] = fmaf(yK[i], yK[i], sqK[i]);
        sqV[i] = fmaf(yV[i], yV[i], sqV[i]);
      }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        sqK[i] += __shfl_xor_sync(0xffffffffu, sqK[i], o);
        sqV[i] += __shfl_xor_sync(0xffffffffu, sqV[i], o);
      }
    }
    if (lane == 0) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int j = row0 + rbase + i;
        if (j < a.n_max) {
          const float s = j < n ? combine_scores(sqK[i], sqV[i], a.score_mode) : 0.f;
          a.scores[(size_t)p * a.n_max + j] = s;
          wsum += s;
        }
      }
    }
  }
  if (lane == 0) warp_sum[warp] = wsum;
  __syncthreads();
  if (tid == 0) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) s += warp_sum[w];
    a.tile_sums[(size_t)p * a.tiles_per_head + tile] = s;
  }
}

// ---------------------------------------------------------------------------
// Alg. 1 (normalisation step): S = sum of the partial sums of the head's valid tiles in a
// fixed order, scores /= S; scores at or beyond the sequence length become 0.
// With `raw` the division is left out (S is still reported).
// grid = batch*heads*ceil(n_max / 4096) (chunk fastest), block = 256.
// ---------------------------------------------------------------------------
constexpr int kNormChunk = 4096;

__global__ void __launch_bounds__(256) normalise_kernel(float* scores, const float* tile_sums,
                                                        float* head_sums, const int32_t* seqlens,
                                                        int heads, int n_max, int tiles_per_head,
                                                        int parts_per_tile, int chunks_per_head,
                                                        int raw) {
  __shared__ float red[8];
  const int p = blockIdx.x / chunks_per_head, chunk = blockIdx.x % chunks_per_head;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = seq_len_of(seqlens, p / heads, n_max);
  float* row = scores + (size_t)p * n_max;
  const int j0 = chunk * kNormChunk;
  const int j1 = min(j0 + kNormChunk, n_max);
  // a full chunk of valid scores is put on its way while the head sum is formed
  const bool vec = (reinterpret_cast<uintptr_t>(row) & 15u) == 0 && j0 + kNormChunk <= n;
  float4 v[4];
  if (vec && !raw) {
#pragma unroll
    for (int u = 0; u < 4; ++u) v[u] = reinterpret_cast<const float4*>(row + j0)[tid + 256 * u];
  }
  const int parts = ((n + kTileRows - 1) / kTileRows) * parts_per_tile;
  const float* mine = tile_sums + (size_t)p * tiles_per_head * parts_per_tile;
  float part = 0.f;                                        // fixed order: thread, warp tree, warp order
  for (int i = tid; i < parts; i += 256) part += mine[i];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
  if (lane == 0) red[warp] = part;
  __syncthreads();
  float S = 0.f;
#pragma unroll
  for (int w = 0; w < 8; ++w) S += red[w];
  if (chunk == 0 && tid == 0) head_sums[p] = S;
  const bool live = S > 0.f;
  if (raw) {                                               // only the padding is rewritten
    for (int j = max(j0, n) + tid; j < j1; j += 256) row[j] = 0.f;
  } else if (vec) {
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      float4 o;
      o.x = live ? __fdiv_rn(v[u].x, S) : 0.f;
      o.y = live ? __fdiv_rn(v[u].y, S) : 0.f;
      o.z = live ? __fdiv_rn(v[u].z, S) : 0.f;
      o.w = live ? __fdiv_rn(v[u].w, S) : 0.f;
      reinterpret_cast<float4*>(row + j0)[tid + 256 * u] = o;
    }
  } else {
    for (int j = j0 + tid; j < j1; j += 256) row[j] = (live && j < n) ? __fdiv_rn(row[j], S) : 0.f;
  }
}

}  // namespace curdkv
