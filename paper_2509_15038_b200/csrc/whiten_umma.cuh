// Whitened sketch: approximate leverage scores in the sense of Eq. (row
// leverage score).  Alg. 1's ||a_j G||^2 follows the row norms; the
// construction the paper's footnote points to first whitens the rows with the
// triangular factor of the matrix.  For every (sequence, head) and tensor
// A in {K, V}:
//   M = A^T A + lambda I            gram_umma_kernel (tensor cores, one pass over K, V)
//   M = L L^T,  W = L^{-T} G        whiten_factor_kernel (fp64, one CTA per matrix)
//   l_j = ||a_j W||^2               sketch_items_kernel (second pass, W staged per head)
// after which Alg. 1 (product and normalisation) run unchanged.
//
// Both streaming kernels walk "items": a head cut into `segments` runs of
// consecutive 128-row tiles, so that a CTA stays on one head long enough to
// amortise what it keeps per head (the Gram accumulators, the staged W).
#pragma once
#include "score_umma.cuh"

namespace curdkv {
namespace umma {

struct ItemArgs {
  const int32_t* seqlens;  // nullptr: every sequence has n_max rows
  int batch, heads, n_max, segments;
  uint32_t* status;
  unsigned long long wait_ns = kWaitLimitNs;   // limit of each pipeline wait
  // gram kernel
  float* partials;         // [batch*heads*segments][2][128][128]
  // sketch kernel
  const float* W;          // projections, fp32 [128][r] each:
                           //   whitened: [batch*heads][2 tensors]   (w_per_problem = 1, w_per_tensor = 1)
                           //   per-head G: [heads], shared by K, V  (w_per_problem = 0, w_per_tensor = 0)
  int w_per_problem, w_per_tensor;
  int r, tiles_per_head, score_mode;
  float* scores;
  float* tile_sums;        // [batch*heads][tiles_per_head][kPartsPerTile]
};

struct Item {
  int p, n, t_lo, t_hi;    // problem, valid rows, tiles [t_lo, t_hi)
};

__device__ __forceinline__ Item item_of(const ItemArgs& a, uint32_t item) {
  Item it;
  it.p = (int)(item / (uint32_t)a.segments);
  const int s = (int)(item % (uint32_t)a.segments);
  it.n = seq_len_of(a.seqlens, it.p / a.heads, a.n_max);
  const int tiles = (it.n + kTileRows - 1) / kTileRows;
  it.t_lo = (int)((long long)s * tiles / a.segments);
  it.t_hi = (int)((long long)(s + 1) * tiles / a.segments);
  return it;
}

// Instruction descriptor of the Gram product: A and B both MN-major (the
// contraction runs over the rows of the tile), bf16 in, fp32 out, M = N = 128.
__host__ __device__ constexpr uint32_t instr_desc_gram() {
  return instr_desc_bf16(128) | (1u << 15) | (1u << 16);
}
// Shared-memory descriptor of a 128-byte-swizzled tile read MN-major: the two
// 64-channel spans are kHalfBytes apart (leading offset), groups of 8 rows
// 1024 B apart (stride offset).
__device__ __forceinline__ uint64_t smem_desc_mn_sw128(uint32_t addr) {
  return (uint64_t)((addr & 0x3ffffu) >> 4) | ((uint64_t)(kHalfBytes >> 4) << 16) | (64ull << 32) |
         (1ull << 46) | (2ull << 61);
}

constexpr int kGramTmemCols = 512;                         // 2 stages x {K, V} x 128 columns
constexpr int kGramBar = kSlots * kSlotBytes;
constexpr int kGramDynamic = kGramBar + 256 + 1024;

// ---------------------------------------------------------------------------
// M_K = K^T K and M_V = V^T V of one item, fp32, written to partials[item].
// Persistent CTAs (one per SM), warp roles as in sketch_umma_kernel.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads, 1)
gram_umma_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                 const ItemArgs a) {
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
  const uint32_t bar0 = base + kGramBar;
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (kSlots + s); };
  auto acc_full_bar = [&](int s) { return bar0 + 8u * (2 * kSlots + s); };
  auto acc_empty_bar = [&](int s) { return bar0 + 8u * (2 * kSlots + 2 + s); };
  const uint32_t drain_bar = bar0 + 8u * (2 * kSlots + 4);
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(base_ptr + kGramBar + 8 * (2 * kSlots + 5));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    for (int s = 0; s < kSlots; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(acc_full_bar(s), 1); mbar_init(acc_empty_bar(s), 128); }
    mbar_init(drain_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(tmem_holder)),
                 "r"((uint32_t)kGramTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;
  const uint32_t items = (uint32_t)a.batch * (uint32_t)a.heads * (uint32_t)a.segments;
  const uint32_t first = blockIdx.x, stride = gridDim.x;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint64_t policy;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
      uint32_t it = 0;
      bool ok = true;
      for (uint32_t item = first; ok && item < items; item += stride) {
        const Item w = item_of(a, item);
        const int b = w.p / a.heads, h = w.p % a.heads;
        for (int t = w.t_lo; ok && t < w.t_hi; ++t) {
          for (int tensor = 0; tensor < 2; ++tensor, ++it) {
            const int slot = it % kSlots;
            const uint32_t phase = (it / kSlots) & 1u;
            if (!(ok = mbar_wait(empty_bar(slot), phase ^ 1u, abort_flag, a.status, a.wait_ns))) break;
            mbar_arrive_expect_tx(full_bar(slot), kSlotBytes);
            const uint32_t dst = base + slot * kSlotBytes;
            const CUtensorMap* map = tensor ? &map_v : &map_k;
            tma_load_4d(dst, map, full_bar(slot), 0, t * kTileRows, h, b, policy);
            tma_load_4d(dst + kHalfBytes, map, full_bar(slot), 64, t * kTileRows, h, b, policy);
          }
        }
      }
      if (!ok) {
        const uint32_t pending = it < (uint32_t)kSlots ? it : (uint32_t)kSlots;
        for (uint32_t q = it - pending; q < it; ++q) {
          unsigned long long t0 = global_ns();
          while (!mbar_try_wait(full_bar(q % kSlots), (q / kSlots) & 1u) &&
                 global_ns() - t0 < a.wait_ns) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc_gram();
      uint32_t it = 0, item_it = 0;
      bool ok = true;
      for (uint32_t item = first; ok && item < items; item += stride) {
        const Item w = item_of(a, item);
        if (w.t_lo >= w.t_hi) continue;
        const uint32_t acc = item_it & 1u, acc_phase = (item_it >> 1) & 1u;
        if (!(ok = mbar_wait(acc_empty_bar(acc), acc_phase ^ 1u, abort_flag, a.status, a.wait_ns))) break;
        tc_fence_after();
        for (int t = w.t_lo; ok && t < w.t_hi; ++t) {
          const int rows = min(kTileRows, w.n - t * kTileRows);
          const int groups = (rows + 15) >> 4;             // MMAs of 16 rows each
          for (int tensor = 0; tensor < 2; ++tensor, ++it) {
            const int slot = it % kSlots;
            if (!(ok = mbar_wait(full_bar(slot), (it / kSlots) & 1u, abort_flag, a.status, a.wait_ns))) break;
            tc_fence_after();
            const uint32_t tile = base + slot * kSlotBytes;
            if (rows < groups * 16) {
              // rows at or beyond the sequence length hold the caller's padding: clear the ones
              // the last 16-row MMA would read (whole 128-byte rows, so the swizzle does not matter)
              for (int j = rows; j < groups * 16; ++j)
                for (int half = 0; half < 2; ++half)
                  for (int c = 0; c < 8; ++c)
                    *reinterpret_cast<uint4*>(base_ptr + slot * kSlotBytes + half * kHalfBytes + j * 128 +
                                              c * 16) = make_uint4(0u, 0u, 0u, 0u);
              asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            }
            const uint32_t d_tmem = tmem_base + acc * 256u + tensor * 128u;
            // one descriptor per tile, stepped by 2048 bytes (128 units of 16 bytes) per 16 rows
            const uint64_t desc0 = smem_desc_mn_sw128(tile);
            if (groups == 8) {
              tc_mma_bf16(d_tmem, desc0, desc0, idesc, t > w.t_lo ? 1u : 0u);
#pragma unroll
              for (int g = 1; g < 8; ++g) tc_mma_bf16(d_tmem, desc0 + 128u * g, desc0 + 128u * g, idesc, 1u);
            } else {
              for (int g = 0; g < groups; ++g)
                tc_mma_bf16(d_tmem, desc0 + 128u * g, desc0 + 128u * g, idesc, (t > w.t_lo || g > 0) ? 1u : 0u);
            }
            tc_commit(empty_bar(slot));
          }
        }
        if (!ok) break;
        tc_commit(acc_full_bar(acc));
        ++item_it;
      }
      if (!ok) {
        tc_commit(drain_bar);
        unsigned long long t0 = global_ns();
        while (!mbar_try_wait(drain_bar, 0) && global_ns() - t0 < a.wait_ns) {}
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;                   // row of M this thread writes
    uint32_t item_it = 0;
    bool ok = true;
    for (uint32_t item = first; ok && item < items; item += stride) {
      const Item w = item_of(a, item);
      float* out = a.partials + (size_t)item * 2 * 128 * 128 + (size_t)row * 128;
      if (w.t_lo >= w.t_hi) {                              // nothing to add from this run of tiles
        for (int tensor = 0; tensor < 2; ++tensor)
          for (int c = 0; c < 128; c += 4)
            *reinterpret_cast<float4*>(out + tensor * 128 * 128 + c) = make_float4(0.f, 0.f, 0.f, 0.f);
        continue;
      }
      const uint32_t acc = item_it & 1u, acc_phase = (item_it >> 1) & 1u;
      ok = mbar_wait(acc_full_bar(acc), acc_phase, abort_flag, a.status, a.wait_ns);
      if (!(ok = __all_sync(0xffffffffu, ok))) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * 256u;
#pragma unroll 1
      for (int c0 = 0; c0 < 256; c0 += 32) {               // K columns 0-127, V columns 128-255
        float v[32];
        tmem_ld32(taddr + c0, v);
        tmem_ld_wait();
        float* dst = out + (c0 >> 7) * 128 * 128 + (c0 & 127);
#pragma unroll
        for (int c = 0; c < 32; c += 4)
          *reinterpret_cast<float4*>(dst + c) = make_float4(v[c], v[c + 1], v[c + 2], v[c + 3]);
      }
      tc_fence_before();
      mbar_arrive(acc_empty_bar(acc));
      ++item_it;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"((uint32_t)kGramTmemCols)
                 : "memory");
  }
}

// ---------------------------------------------------------------------------
// Sketch + norms + combine (Alg. 1 (sketch, row norms, product)) with a projection that changes
// from head to head (the whitened W of each head and tensor, or a caller's
// per-head G) instead of one shared G.  Same pipeline as sketch_umma_kernel;
// the epilogue warps restage [W_hi | W_lo] for K and for V at the start of
// every item and release the MMA issuer through g_ready.
// ---------------------------------------------------------------------------
template <int R>
struct ItemSmem {
  static constexpr int kN = 2 * R;
  static constexpr int kGHalf = kN * 128;                  // bytes per 64-channel span of W^T
  static constexpr int kGK = 0;
  static constexpr int kGV = 2 * kGHalf;
  static constexpr int kSlot0 = 4 * kGHalf;
  static constexpr int kRing = R <= 32 ? kSlots : 3;       // 64 columns: W takes 64 KB, ring of 3
  static constexpr int kBar = kSlot0 + kRing * kSlotBytes;
  static constexpr int kDynamic = kBar + 256 + 1024;
  static constexpr int kTmemCols = 4 * kN;
};

template <int R>
__global__ void __launch_bounds__(kThreads, 1)
sketch_items_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                    const ItemArgs a) {
  using L = ItemSmem<R>;
  constexpr int kRing = L::kRing;
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
  const uint32_t bar0 = base + L::kBar;
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (kRing + s); };
  auto acc_full_bar = [&](int s) { return bar0 + 8u * (2 * kRing + s); };
  auto acc_empty_bar = [&](int s) { return bar0 + 8u * (2 * kRing + 2 + s); };
  const uint32_t drain_bar = bar0 + 8u * (2 * kRing + 4);
  const uint32_t g_ready_bar = bar0 + 8u * (2 * kRing + 5);
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(base_ptr + L::kBar + 8 * (2 * kRing + 6));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    for (int s = 0; s < kRing; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(acc_full_bar(s), 1); mbar_init(acc_empty_bar(s), 128); }
    mbar_init(drain_bar, 1);
    mbar_init(g_ready_bar, 128);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(tmem_holder)),
                 "r"((uint32_t)L::kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;
  const uint32_t items = (uint32_t)a.batch * (uint32_t)a.heads * (uint32_t)a.segments;
  const uint32_t first = blockIdx.x, stride = gridDim.x;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint64_t policy;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
      uint32_t it = 0;
      bool ok = true;
      for (uint32_t item = first; ok && item < items; item += stride) {
        const Item w = item_of(a, item);
        const int b = w.p / a.heads, h = w.p % a.heads;
        for (int t = w.t_lo; ok && t < w.t_hi; ++t) {
          for (int tensor = 0; tensor < 2; ++tensor, ++it) {
            const int slot = it % kRing;
            const uint32_t phase = (it / kRing) & 1u;
            if (!(ok = mbar_wait(empty_bar(slot), phase ^ 1u, abort_flag, a.status, a.wait_ns))) break;
            mbar_arrive_expect_tx(full_bar(slot), kSlotBytes);
            const uint32_t dst = base + L::kSlot0 + slot * kSlotBytes;
            const CUtensorMap* map = tensor ? &map_v : &map_k;
            tma_load_4d(dst, map, full_bar(slot), 0, t * kTileRows, h, b, policy);
            tma_load_4d(dst + kHalfBytes, map, full_bar(slot), 64, t * kTileRows, h, b, policy);
          }
        }
      }
      if (!ok) {
        const uint32_t pending = it < (uint32_t)kRing ? it : (uint32_t)kRing;
        for (uint32_t q = it - pending; q < it; ++q) {
          unsigned long long t0 = global_ns();
          while (!mbar_try_wait(full_bar(q % kRing), (q / kRing) & 1u) &&
                 global_ns() - t0 < a.wait_ns) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc_bf16(L::kN);
      uint32_t it = 0, tile_it = 0, item_it = 0;
      bool ok = true;
      for (uint32_t item = first; ok && item < items; item += stride) {
        const Item w = item_of(a, item);
        if (w.t_lo >= w.t_hi) continue;
        if (!(ok = mbar_wait(g_ready_bar, item_it & 1u, abort_flag, a.status, a.wait_ns))) break;   // W staged
        ++item_it;
        for (int t = w.t_lo; ok && t < w.t_hi; ++t) {
          const uint32_t acc = tile_it & 1u, acc_phase = (tile_it >> 1) & 1u;
          if (!(ok = mbar_wait(acc_empty_bar(acc), acc_phase ^ 1u, abort_flag, a.status, a.wait_ns))) break;
          tc_fence_after();
          for (int tensor = 0; tensor < 2; ++tensor, ++it) {
            const int slot = it % kRing;
            if (!(ok = mbar_wait(full_bar(slot), (it / kRing) & 1u, abort_flag, a.status, a.wait_ns))) break;
            tc_fence_after();
            const uint32_t a_base = base + L::kSlot0 + slot * kSlotBytes;
            const uint32_t g_base = base + (tensor ? L::kGV : L::kGK);
            const uint32_t d_tmem = tmem_base + acc * (2 * L::kN) + tensor * L::kN;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
              const uint32_t koff = (k >> 2) * kHalfBytes + (k & 3) * 32;
              const uint32_t goff = (k >> 2) * L::kGHalf + (k & 3) * 32;
              tc_mma_bf16(d_tmem, smem_desc_sw128(a_base + koff), smem_desc_sw128(g_base + goff), idesc,
                          k > 0);
            }
            tc_commit(empty_bar(slot));
          }
          if (!ok) break;
          tc_commit(acc_full_bar(acc));
          ++tile_it;
        }
      }
      if (!ok) {
        tc_commit(drain_bar);
        unsigned long long t0 = global_ns();
        while (!mbar_try_wait(drain_bar, 0) && global_ns() - t0 < a.wait_ns) {}
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue
    const int quarter = warp & 3;
    const int etid = tid - 64;                             // 0..127 among the epilogue threads
    uint64_t keep;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(keep));
    uint32_t tile_it = 0;
    bool ok = true;
    for (uint32_t item = first; ok && item < items; item += stride) {
      const Item w = item_of(a, item);
      if (w.t_lo >= w.t_hi) continue;
      // every MMA of the previous item has retired (its last accumulator was handed over), so
      // the staged projections can be replaced: W^T = [W_hi | W_lo], swizzled K-major, per tensor
      for (int tensor = 0; tensor < 2; ++tensor) {
        const size_t which = (size_t)(a.w_per_problem ? w.p : w.p % a.heads) * (a.w_per_tensor ? 2 : 1) +
                             (a.w_per_tensor ? tensor : 0);
        const float* Wp = a.W + which * 128 * a.r;
        unsigned char* dstG = base_ptr + (tensor ? L::kGV : L::kGK);
        for (int i = etid; i < 128 * R; i += 128) {
          const int t = i / R, c = i % R;
          const float g = c < a.r ? __ldg(Wp + (size_t)t * a.r + c) : 0.f;
          const __nv_bfloat16 hi = __float2bfloat16_rn(g);
          const __nv_bfloat16 lo = __float2bfloat16_rn(g - __bfloat162float(hi));
          const int span = t >> 6, tt = t & 63;
          auto put = [&](int rowg, __nv_bfloat16 v) {
            const int chunk = (tt >> 3) ^ (rowg & 7);
            *reinterpret_cast<__nv_bfloat16*>(dstG + span * L::kGHalf + rowg * 128 + chunk * 16 +
                                              (tt & 7) * 2) = v;
          };
          put(c, hi);
          put(R + c, lo);
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      mbar_arrive(g_ready_bar);
      for (int t = w.t_lo; ok && t < w.t_hi; ++t) {
        const int row0 = t * kTileRows;
        const int j = row0 + quarter * 32 + lane;
        float s = 0.f;
        const uint32_t acc = tile_it & 1u, acc_phase = (tile_it >> 1) & 1u;
        ok = mbar_wait(acc_full_bar(acc), acc_phase, abort_flag, a.status, a.wait_ns);
        if (!(ok = __all_sync(0xffffffffu, ok))) break;
        tc_fence_after();
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * (2 * L::kN);
        const float lk = sketch_row_norm<R>(taddr);
        const float lv = sketch_row_norm<R>(taddr + L::kN);
        tc_fence_before();
        mbar_arrive(acc_empty_bar(acc));
        ++tile_it;
        if (j < w.n) s = combine_scores(lk, lv, a.score_mode);
        if (j < a.n_max)
          asm volatile("st.global.L2::cache_hint.f32 [%0], %1, %2;" ::"l"(a.scores + (size_t)w.p * a.n_max + j),
                       "f"(s), "l"(keep)
                       : "memory");
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (lane == 0)
          a.tile_sums[((size_t)w.p * a.tiles_per_head + t) * kPartsPerTile + quarter] = s;
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"((uint32_t)L::kTmemCols)
                 : "memory");
  }
}

}  // namespace umma
}  // namespace curdkv
