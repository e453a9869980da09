// Fused sketch + squared-norm + combine kernel on the 5th-gen tensor cores
// (Alg. 1 (sketch, row norms, product)) for d = 128 and r <= 64.
//
// Per 128-token tile and tensor (K, then V):  Y = A G  with A the bf16 tile
// [128 x 128] brought in by TMA (128-byte swizzle) and G held in shared memory
// for the whole kernel.  fp32 G is split G = G_hi + G_lo into two bf16 matrices
// (bf16 x bf16 products are exact in fp32, the residual of the split is
// ~2^-17 relative), and both halves ride in one MMA as the N = 2*R columns
// [G_hi | G_lo]; the epilogue adds the two column halves, squares and sums.
// Y never leaves TMEM.  One tcgen05.mma (M = 128, N = 2R, K = 16) per 16
// channels, fp32 accumulators double-buffered in TMEM.
//
// Persistent CTAs (one per SM), 6 warps:
//   warp 0      TMA producer (one lane): 32 KB tensor tiles into a 4-slot ring
//   warp 1      MMA issuer (one lane); owns the TMEM allocation
//   warps 2-5   epilogue: tcgen05.ld -> (hi+lo)^2 row sums -> lK*lV -> scores,
//               one partial sum per warp quarter for the head normaliser
// Every mbarrier wait is bounded; on expiry the kernel flags
// CURDKV_DEV_TIMEOUT, drains what it issued, frees TMEM and returns.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "select.cuh"

namespace curdkv {
namespace umma {

constexpr int kThreads = 192;
// The fused form adds a group of selection warps behind the six pipeline warps: whenever this CTA
// writes the last tile of a head, they normalise that head's scores and select its tokens (Alg. 1
// normalisation and selection steps) while the pipeline goes on streaming.
constexpr int kFusedSelThreads = 256;
constexpr int kFusedSelFirst = kThreads + 32;              // one publisher warp sits between the two groups
constexpr int kFusedThreads = kFusedSelFirst + kFusedSelThreads;
constexpr int kFusedListCap = 4096;                        // candidate list of the selection warps
constexpr int kFusedRuns = 32;                             // runs of tiles between the epilogue and the publisher
// Ring of tensor tiles.  Four 32 KB slots per SM keep HBM saturated; a deeper
// ring measurably lowers the achieved read bandwidth on B200.
constexpr int kSlots = 4;
constexpr int kHalfBytes = kTileRows * 128;       // 128 rows x 64 bf16 (one 128-byte swizzle span)
constexpr int kSlotBytes = 2 * kHalfBytes;        // d = 128 -> two spans
constexpr int kPartsPerTile = 4;                  // partial sums per tile (one per epilogue warp)
// Default limit of every device-side wait (the launchers pass it to the kernels as an argument).
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

struct Args {
  const float* G;          // [128][r]
  const int32_t* seqlens;  // nullptr: every sequence has n_max rows
  int batch, heads, n_max, r;
  int tiles_per_head;      // ceil(n_max / kTileRows): row stride of tile_sums
  int score_mode;
  float* scores;
  float* tile_sums;        // [batch*heads][tiles_per_head][kPartsPerTile]
  uint32_t* status;
  unsigned long long wait_ns = kWaitLimitNs;   // limit of each pipeline wait
  // fused selection only (sketch_umma_kernel<R, true>); pointers are those of this launch's first head
  float* head_sums = nullptr;          // [batch*heads]
  int32_t* head_done = nullptr;        // [batch*heads] tiles written so far, zero on entry
  int32_t* done_list = nullptr;        // [batch*heads] finished heads (index + 1) in the order they finished; zero on entry
  int32_t* queue_ctr = nullptr;        // [2] heads entered into done_list / tickets handed to selection groups; zero on entry
  int32_t* head_ready = nullptr;       // [batch*heads] or nullptr: set to 1 once a head's indices and count are written; zero on entry
  const int32_t* head_budgets = nullptr;
  int32_t* idx = nullptr;              // [batch*heads][budget]
  int32_t* counts = nullptr;
  int32_t* offsets = nullptr;          // or nullptr
  int budget = 0, num_sink = 0, window = 0, raw = 0;
  int first_head = 0, all_heads = 0;   // position of this launch's heads in the caller's batch
  // Tiles are dealt to the CTAs in chunks of this many consecutive tiles (1: tile t goes to CTA
  // t mod grid).  The fused kernel counts a head's tiles once per chunk instead of once per tile.
  int chunk_tiles = 1;
  // L2 policy of the K/V tile loads: 1 = evict-first (the tiles are read once), 0 = the default
  // policy.  Measured: on caches of many GB the default is ~0.5 % faster, on a 1 GB cache
  // evict-first is (the launcher picks by size).
  int evict_first = 1;
};

// The tiles of one CTA in the order every role walks them: chunks first, first + stride, ... of
// `chunk` consecutive tiles each.
struct TileWalk {
  uint32_t chunk_no, i, chunk, stride, total;
  __device__ __forceinline__ TileWalk(uint32_t first, uint32_t stride_, uint32_t chunk_, uint32_t total_)
      : chunk_no(first), i(0), chunk(chunk_), stride(stride_), total(total_) {}
  __device__ __forceinline__ bool valid() const { return chunk_no * chunk + i < total; }
  __device__ __forceinline__ uint32_t tile() const { return chunk_no * chunk + i; }
  __device__ __forceinline__ bool starts_chunk() const { return i == 0; }
  __device__ __forceinline__ void next() {
    if (++i == chunk || chunk_no * chunk + i >= total) {
      i = 0;
      chunk_no += stride;
    }
  }
};

// Ragged batches: the kernel walks only the tiles that hold valid rows.  Every
// CTA builds the exclusive prefix sums of the per-sequence tile counts in shared
// memory and maps a running tile number to (sequence, head, tile) by binary
// search, so all CTAs get the same number of real tiles.
constexpr int kMaxRaggedBatch = 8192;                      // sequences per launch with seqlens

template <int R, bool FUSED = false>
struct Smem {                                     // offsets from the 1024-aligned base
  static constexpr int kN = 2 * R;                // MMA N: [G_hi | G_lo]
  static constexpr int kGHalf = kN * 128;         // bytes per 64-channel span of G^T
  static constexpr int kG = 0;
  static constexpr int kSlot0 = 2 * kGHalf;
  static constexpr int kBar = kSlot0 + kSlots * kSlotBytes;
  static constexpr int kList = kBar + 256;        // (key, index) pairs of the selection warps
  static constexpr int kPrefix = kList + (FUSED ? kFusedListCap * 8 : 0);   // int32 [batch + 1], ragged launches only
  static constexpr int kFixed = kPrefix + 1024;   // + slack for manual alignment
  static constexpr int dynamic_bytes(int ragged_batch) {
    return kFixed + (ragged_batch > 0 ? (ragged_batch + 1) * 4 : 0);
  }
  static constexpr int kTmemCols = 4 * kN;        // 2 accumulator stages x {K, V} x N
};

// ---- PTX wrappers --------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Gives up when another role has aborted or after limit_ns;
// then raises the CTA's abort flag and the device status bit.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          uint32_t* status, unsigned long long limit_ns) {
  unsigned long long t0 = 0;
  for (uint32_t spin = 1;; ++spin) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spin & 0xffu) == 0) {
      if (*abort_flag) return false;
      const unsigned long long now = global_ns();
      if (t0 == 0) t0 = now;
      if (now - t0 > limit_ns) {
        *abort_flag = 1;
        flag_status(status, CURDKV_DEV_TIMEOUT);
        return false;
      }
    }
  }
}
// The bounded wait on its own, for tests of the failure path: every warp's first lane waits on a
// barrier that nothing ever completes.  The first wait to run out raises the abort flag and
// CURDKV_DEV_TIMEOUT; the others then leave through the abort path.  Returns after ~limit_ns.
__global__ void wait_selftest_kernel(uint32_t* status, unsigned long long limit_ns) {
  __shared__ alignas(8) unsigned long long never_completed;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&never_completed), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if ((threadIdx.x & 31) == 0) mbar_wait(smem_u32(&never_completed), 0, &abort_flag, status, limit_ns);
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar,
                                            int c0, int c1, int c2, int c3, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%3, %4, %5, %6}], [%2], %7;" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3),
      "l"(policy)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, bf16 inputs, fp32 accumulate, M = 128.
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                            uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t* u = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]),
        "=r"(u[7]), "=r"(u[8]), "=r"(u[9]), "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]),
        "=r"(u[14]), "=r"(u[15]), "=r"(u[16]), "=r"(u[17]), "=r"(u[18]), "=r"(u[19]), "=r"(u[20]),
        "=r"(u[21]), "=r"(u[22]), "=r"(u[23]), "=r"(u[24]), "=r"(u[25]), "=r"(u[26]), "=r"(u[27]),
        "=r"(u[28]), "=r"(u[29]), "=r"(u[30]), "=r"(u[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor of a K-major, 128-byte-swizzled operand:
// rows 128 B apart, 8-row groups 1024 B apart (stride offset 64 x 16 B),
// leading offset unused by swizzled K-major layouts (1), sm_100 version tag.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
  return (uint64_t)((addr & 0x3ffffu) >> 4) | (1ull << 16) | (64ull << 32) | (1ull << 46) |
         (2ull << 61);
}
// Instruction descriptor: fp32 accumulate, bf16 A and B, both K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t instr_desc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((128u >> 4) << 24);
}

// Sum over c < R of (hi_c + lo_c)^2 for this thread's row; hi at columns
// [col, col+R), lo at [col+R, col+2R).
template <int R>
__device__ __forceinline__ float sketch_row_norm(uint32_t taddr) {
  float acc = 0.f;
#pragma unroll
  for (int c0 = 0; c0 < R; c0 += 32) {
    float hi[32], lo[32];
    tmem_ld32(taddr + c0, hi);
    tmem_ld32(taddr + R + c0, lo);
    tmem_ld_wait();
#pragma unroll
    for (int c = 0; c < 32; ++c) {
      const float y = hi[c] + lo[c];
      acc = fmaf(y, y, acc);
    }
  }
  return acc;
}

// ---- fused selection ---------------------------------------------------------
// A "run" is a stretch of consecutive tiles of one head inside one chunk.  When the four epilogue
// warps have written a run's scores they arrive on the run's barrier; the publisher warp takes it
// from there (device-wide fence, count, hand-over), so no epilogue warp ever waits on a fence or on
// an atomic's round trip.
struct FusedSmem {
  SelectSmem sel;
  alignas(8) unsigned long long run_bar[kFusedRuns];
  int run_head[kFusedRuns], run_tiles[kFusedRuns], run_total[kFusedRuns];   // head, tiles in the run, tiles of the head
  int published;               // runs the publisher is done with
  int final_runs[4];           // runs each epilogue warp closed before it left its loop
  int producers_done;          // epilogue warps that have left their loop
  int current;                 // head the selection warps work on
};

// Finished heads go through one list in global memory that the selection groups of ALL CTAs serve:
// whichever CTA happens to write a head's last tile (a few CTAs do so far more often than the
// rest), the selections are spread evenly.  A lane of a publisher warp enters a head ...
__device__ __forceinline__ void fused_push(const Args& a, int p) {
  const int slot = atomicAdd(a.queue_ctr, 1);
  __threadfence();
  *(volatile int32_t*)(a.done_list + slot) = p + 1;
}

// ... and thread 0 of a selection group draws a ticket and waits (bounded) for that entry of the
// list.  Returns -1 when every head with rows has been handed out, or when the launch has failed.
// The CTAs of the launch are co-resident (cooperative launch), so the heads a ticket waits for are
// being streamed while it waits.
__device__ __forceinline__ int fused_pop(const Args& a, int nonempty_heads, volatile int* abort_flag) {
  const int ticket = atomicAdd(a.queue_ctr + 1, 1);
  if (ticket >= nonempty_heads) return -1;
  unsigned long long t0 = 0;
  for (uint32_t spin = 1;; ++spin) {
    const int v = *(volatile int32_t*)(a.done_list + ticket);
    if (v != 0) {
      __threadfence();                                     // the head's scores were written by other CTAs
      return v - 1;
    }
    __nanosleep(1000);
    if ((spin & 0xffu) == 0) {
      const unsigned long long now = global_ns();
      if (t0 == 0) t0 = now;
      // a launch that has timed out elsewhere never finishes its heads; the limit itself is a
      // second line of defence (the other roles' waits are bounded)
      if ((*(volatile uint32_t*)a.status & CURDKV_DEV_TIMEOUT) != 0 || now - t0 > 32ull * a.wait_ns) {
        flag_status(a.status, CURDKV_DEV_TIMEOUT);
        *abort_flag = 1;
        return -1;
      }
    }
  }
}

// Alg. 1 (normalisation and selection) for head p by the selection warps (group G of kFusedSelThreads threads): the head
// sum in the order normalise_kernel forms it, the division on the way into the leading-digit
// histogram, then the fixed-budget selection of select_fixed_kernel on the normalised scores.
template <class G>
__device__ __forceinline__ void fused_select_head(const Args& a, int p, const KeyList& list, SelectSmem& sm) {
  const int tid = G::tid();
  const int n = seq_len_of(a.seqlens, p / a.heads, a.n_max);
  const int tiles = (n + kTileRows - 1) / kTileRows;
  float* row = a.scores + (size_t)p * a.n_max;
  clear_hist<G>(sm.hist);
  const float S = head_sum_fixed_order<G>(a.tile_sums + (size_t)p * a.tiles_per_head * kPartsPerTile,
                                          tiles * kPartsPerTile, sm);
  if (tid == 0) a.head_sums[p] = S;

  int k = a.budget;
  if (a.head_budgets != nullptr) k = max(0, min(a.head_budgets[p], a.budget));
  const int k_eff = min(k, n);
  const ForcedSet F = forced_set(n, k_eff, a.num_sink, a.window);
  RowKeys keys = global_keys(row, n, F);
  keys.written_here = true;
  scale_row_and_histogram<G>(row, keys, a.n_max, tiles * kTileRows, S, a.raw != 0, sm.hist, nullptr);
  G::sync();
  select_fixed_row<G>(keys, F, k_eff, a.budget, nullptr, 0, list, true, a.idx + (size_t)p * a.budget, sm);
  if (tid == 0) {
    a.counts[p] = k_eff;
    if (a.offsets != nullptr) {                            // heads sit at multiples of `budget` rows
      const int gp = a.first_head + p;
      a.offsets[p] = gp * a.budget;
      if (gp == a.all_heads - 1) a.offsets[p + 1] = (gp + 1) * a.budget;
    }
  }
}

template <bool FUSED>
struct FusedState {
  FusedSmem s;
};
template <>
struct FusedState<false> {};

// ---------------------------------------------------------------------------
template <int R, bool FUSED = false>
__global__ void __launch_bounds__(FUSED ? kFusedThreads : kThreads, 1)
sketch_umma_kernel(const __grid_constant__ CUtensorMap map_k,
                   const __grid_constant__ CUtensorMap map_v, const Args a) {
  using L = Smem<R, FUSED>;
  __shared__ FusedState<FUSED> fused;
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
  const uint32_t bar0 = base + L::kBar;
  // barriers: full[kSlots], empty[kSlots], acc_full[2], acc_empty[2], drain
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (kSlots + s); };
  auto acc_full_bar = [&](int s) { return bar0 + 8u * (2 * kSlots + s); };
  auto acc_empty_bar = [&](int s) { return bar0 + 8u * (2 * kSlots + 2 + s); };
  const uint32_t drain_bar = bar0 + 8u * (2 * kSlots + 4);
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(base_ptr + L::kBar + 8 * (2 * kSlots + 5));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // ---- set-up: barriers, TMEM, G^T = [G_hi | G_lo] in swizzled K-major form
  if (tid == 0) {
    for (int s = 0; s < kSlots; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(acc_full_bar(s), 1); mbar_init(acc_empty_bar(s), 128); }
    mbar_init(drain_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if constexpr (FUSED) {
    if (tid < kFusedRuns) mbar_init(smem_u32(&fused.s.run_bar[tid]), 4);
    if (tid == 0) fused.s.producers_done = fused.s.published = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(tmem_holder)),
                 "r"((uint32_t)L::kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (a.seqlens != nullptr) {
    // exclusive prefix sums of heads * ceil(n_b / 128): a chunk of sequences per thread,
    // a scan over the chunk totals, then the running sums inside each chunk
    uint32_t* pre = reinterpret_cast<uint32_t*>(base_ptr + L::kPrefix);
    uint32_t* chunk_tot = reinterpret_cast<uint32_t*>(base_ptr + L::kSlot0);   // ring not in use yet
    const int per = (a.batch + kThreads - 1) / kThreads;
    const int b0 = min(tid * per, a.batch), b1 = min(b0 + per, a.batch);
    if (tid < kThreads) {                                  // the pipeline warps (all, unless fused)
      uint32_t sum = 0;
      for (int b = b0; b < b1; ++b)
        sum += (uint32_t)a.heads * (uint32_t)((seq_len_of(a.seqlens, b, a.n_max) + kTileRows - 1) / kTileRows);
      chunk_tot[tid] = sum;
    }
    __syncthreads();
    if (tid < kThreads) {
      uint32_t before = 0;
      for (int i = 0; i < tid; ++i) before += chunk_tot[i];
      for (int b = b0; b < b1; ++b) {
        pre[b] = before;
        before += (uint32_t)a.heads * (uint32_t)((seq_len_of(a.seqlens, b, a.n_max) + kTileRows - 1) / kTileRows);
      }
      if (tid == kThreads - 1) pre[a.batch] = before;
    }
    // made visible to every role by the barrier at the end of the set-up
  }
  for (int i = tid; i < 128 * R; i += (int)blockDim.x) {
    const int t = i / R, c = i % R;                        // channel t, sketch column c
    const float g = c < a.r ? __ldg(a.G + (size_t)t * a.r + c) : 0.f;
    const __nv_bfloat16 hi = __float2bfloat16_rn(g);
    const __nv_bfloat16 lo = __float2bfloat16_rn(g - __bfloat162float(hi));
    const int span = t >> 6, tt = t & 63;
    auto put = [&](int row, __nv_bfloat16 v) {             // row of G^T = sketch column
      const int chunk = (tt >> 3) ^ (row & 7);             // 128-byte swizzle on 16-byte chunks
      *reinterpret_cast<__nv_bfloat16*>(base_ptr + L::kG + span * L::kGHalf + row * 128 +
                                        chunk * 16 + (tt & 7) * 2) = v;
    };
    put(c, hi);
    put(R + c, lo);
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;
  if constexpr (FUSED) {
    // A gather launched as a programmatic dependent of this kernel may be scheduled from here on;
    // its CTAs find room as CTAs of this launch finish, and wait per head on head_ready.  (Without
    // such a dependent the instruction does nothing.)
    if (tid == 0 && a.head_ready != nullptr) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  }

  // ---- tile schedule: running tile number -> (problem p, first row, valid rows n)
  const uint32_t* prefix = reinterpret_cast<const uint32_t*>(base_ptr + L::kPrefix);
  uint32_t total_tiles;
  if (a.seqlens != nullptr) {
    total_tiles = prefix[a.batch];
  } else {
    total_tiles = (uint32_t)a.batch * (uint32_t)a.heads * (uint32_t)a.tiles_per_head;
  }
  const uint32_t first = blockIdx.x, stride = gridDim.x;
  auto locate = [&](uint32_t t, int& p, int& row0) -> int {
    if (a.seqlens == nullptr) {
      p = (int)(t / (uint32_t)a.tiles_per_head);
      row0 = (int)(t % (uint32_t)a.tiles_per_head) * kTileRows;
      return a.n_max;
    }
    int lo = 0, hi = a.batch;                              // last b with prefix[b] <= t
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (prefix[mid] <= t) lo = mid; else hi = mid;
    }
    const int n = seq_len_of(a.seqlens, lo, a.n_max);
    const uint32_t tiles_b = (uint32_t)((n + kTileRows - 1) / kTileRows);
    const uint32_t local = t - prefix[lo];
    p = lo * a.heads + (int)(local / tiles_b);
    row0 = (int)(local % tiles_b) * kTileRows;
    return n;
  };

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint64_t policy;
      if (a.evict_first) asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
      else asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(policy));
      uint32_t it = 0;
      bool ok = true;
      for (TileWalk w(first, stride, (uint32_t)a.chunk_tiles, total_tiles); ok && w.valid(); w.next()) {
        int p, row0;
        locate(w.tile(), p, row0);
        const int b = p / a.heads, h = p % a.heads;
        for (int tensor = 0; tensor < 2; ++tensor, ++it) {
          const int slot = it % kSlots;
          const uint32_t phase = (it / kSlots) & 1u;
          if (!(ok = mbar_wait(empty_bar(slot), phase ^ 1u, abort_flag, a.status, a.wait_ns))) break;
          mbar_arrive_expect_tx(full_bar(slot), kSlotBytes);
          const uint32_t dst = base + L::kSlot0 + slot * kSlotBytes;
          const CUtensorMap* map = tensor ? &map_v : &map_k;
          tma_load_4d(dst, map, full_bar(slot), 0, row0, h, b, policy);
          tma_load_4d(dst + kHalfBytes, map, full_bar(slot), 64, row0, h, b, policy);
        }
      }
      if (!ok) {
        // let the copies already issued land before the CTA gives up its shared memory
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
      constexpr uint32_t idesc = instr_desc_bf16(L::kN);
      uint32_t it = 0, tile_it = 0;
      bool ok = true;
      for (TileWalk w(first, stride, (uint32_t)a.chunk_tiles, total_tiles); ok && w.valid(); w.next()) {
        const uint32_t acc = tile_it & 1u, acc_phase = (tile_it >> 1) & 1u;
        if (!(ok = mbar_wait(acc_empty_bar(acc), acc_phase ^ 1u, abort_flag, a.status, a.wait_ns))) break;
        tc_fence_after();
        for (int tensor = 0; tensor < 2; ++tensor, ++it) {
          const int slot = it % kSlots;
          if (!(ok = mbar_wait(full_bar(slot), (it / kSlots) & 1u, abort_flag, a.status, a.wait_ns))) break;
          tc_fence_after();
          const uint32_t a_base = base + L::kSlot0 + slot * kSlotBytes;
          const uint32_t d_tmem = tmem_base + acc * (2 * L::kN) + tensor * L::kN;
#pragma unroll
          for (int k = 0; k < 8; ++k) {                    // 16 channels per MMA
            const uint32_t koff = (k >> 2) * kHalfBytes + (k & 3) * 32;
            const uint32_t goff = (k >> 2) * L::kGHalf + (k & 3) * 32;
            tc_mma_bf16(d_tmem, smem_desc_sw128(a_base + koff),
                        smem_desc_sw128(base + L::kG + goff), idesc, k > 0);
          }
          tc_commit(empty_bar(slot));                      // slot reusable once these MMAs retire
        }
        if (!ok) break;
        tc_commit(acc_full_bar(acc));
        ++tile_it;
      }
      if (!ok) {                                           // drain MMAs in flight before TMEM is freed
        tc_commit(drain_bar);
        unsigned long long t0 = global_ns();
        while (!mbar_try_wait(drain_bar, 0) && global_ns() - t0 < a.wait_ns) {}
      }
    }
  } else if (warp < kThreads / 32) {
    // ------------------------------------------------------------ epilogue
    const int quarter = warp & 3;                          // TMEM lanes this warp may read
    // scores are read again by the normaliser and the selection: ask L2 to keep them over
    // the K/V stream, which also defers their write-back into larger bursts
    uint64_t keep;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(keep));
    uint32_t tile_it = 0;
    bool ok = true;
    // fused: the run of tiles being written and how many runs this warp has closed
    int run_head = -1, run_len = 0, run_rows = 0, runs_closed = 0;
    auto close_run = [&]() {
      if constexpr (FUSED) {
        const int slot = runs_closed % kFusedRuns;
        if (lane == 0) {
          // the slot's previous run must have left the publisher (a run lasts microseconds, the
          // publisher needs a fraction of that: this never waits in practice)
          unsigned long long t0 = 0;
          for (uint32_t spin = 1; runs_closed - *(volatile int*)&fused.s.published >= kFusedRuns; ++spin) {
            if ((spin & 0xffu) == 0) {
              const unsigned long long now = global_ns();
              if (t0 == 0) t0 = now;
              if (*abort_flag || now - t0 > a.wait_ns) {
                *abort_flag = 1;
                flag_status(a.status, CURDKV_DEV_TIMEOUT);
                break;
              }
            }
          }
          if (quarter == 0) {
            fused.s.run_head[slot] = run_head;
            fused.s.run_tiles[slot] = run_len;
            fused.s.run_total[slot] = (run_rows + kTileRows - 1) / kTileRows;
          }
        }
        __syncwarp();                                      // every lane's stores before lane 0's arrival
        if (lane == 0 && !*abort_flag) mbar_arrive(smem_u32(&fused.s.run_bar[slot]));
        ++runs_closed;
        run_len = 0;
      }
    };
    for (TileWalk w(first, stride, (uint32_t)a.chunk_tiles, total_tiles); ok && w.valid(); w.next()) {
      int p, row0;
      const int n = locate(w.tile(), p, row0);
      if (FUSED && run_len > 0 && (p != run_head || w.starts_chunk())) close_run();
      const int j = row0 + quarter * 32 + lane;
      float s = 0.f;
      {
        const uint32_t acc = tile_it & 1u, acc_phase = (tile_it >> 1) & 1u;
        ok = mbar_wait(acc_full_bar(acc), acc_phase, abort_flag, a.status, a.wait_ns);
        if (!(ok = __all_sync(0xffffffffu, ok))) break;    // the TMEM loads need the whole warp
        tc_fence_after();
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * (2 * L::kN);
        const float lk = sketch_row_norm<R>(taddr);
        const float lv = sketch_row_norm<R>(taddr + L::kN);
        tc_fence_before();
        mbar_arrive(acc_empty_bar(acc));
        ++tile_it;
        if (j < n) s = combine_scores(lk, lv, a.score_mode);
      }
      if (j < a.n_max)
        asm volatile("st.global.L2::cache_hint.f32 [%0], %1, %2;" ::"l"(a.scores + (size_t)p * a.n_max + j),
                     "f"(s), "l"(keep)
                     : "memory");
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (lane == 0)
        a.tile_sums[((size_t)p * a.tiles_per_head + row0 / kTileRows) * kPartsPerTile + quarter] = s;
      run_head = p;
      run_rows = n;
      ++run_len;
    }
    if constexpr (FUSED) {
      if (ok && run_len > 0) close_run();
      if (lane == 0) {
        fused.s.final_runs[quarter] = runs_closed;
        __threadfence_block();
        atomicAdd(&fused.s.producers_done, 1);
      }
    }
  } else if (FUSED && warp == kThreads / 32) {
    // ------------------------------------------------------------ publisher
    // Takes the runs the epilogue warps have finished, in order, up to 32 at a time (a lane each):
    // one device-wide fence for the batch, then every lane adds its run's tiles to the head's
    // counter; the lane that completes a head hands it to the selection warps.
    if constexpr (FUSED) {
      uint32_t first_run = 0;
      unsigned long long t0 = 0;
      for (uint32_t spin = 1;; ++spin) {
        const uint32_t run = first_run + lane;
        const int slot = (int)(run % kFusedRuns);
        const bool done = mbar_try_wait(smem_u32(&fused.s.run_bar[slot]), (run / kFusedRuns) & 1u);
        const uint32_t ready = __ballot_sync(0xffffffffu, done);
        const int m = ready == 0xffffffffu ? 32 : __ffs(~ready) - 1;   // runs finish in order: a prefix
        if (m == 0) {
          int stop = 0;
          if (lane == 0) {
            if (*(volatile int*)&fused.s.producers_done == 4) {
              int total = fused.s.final_runs[0];
              for (int q = 1; q < 4; ++q) total = min(total, *(volatile int*)&fused.s.final_runs[q]);
              stop = (int)first_run >= total;
            }
            if ((spin & 0x3ffu) == 0) {
              const unsigned long long now = global_ns();
              if (t0 == 0) t0 = now;
              if (*abort_flag || now - t0 > 32ull * a.wait_ns) stop = 1;
            }
          }
          if (__shfl_sync(0xffffffffu, stop, 0)) break;
          __nanosleep(100);
          continue;
        }
        t0 = 0;
        __threadfence();                                   // the runs' scores (acquired through the barriers) first
        if (lane < m) {
          const int p = fused.s.run_head[slot], tiles = fused.s.run_tiles[slot];
          if (atomicAdd(a.head_done + p, tiles) + tiles == fused.s.run_total[slot]) {
            __threadfence();
            fused_push(a, p);
          }
        }
        __syncwarp();
        first_run += (uint32_t)m;
        if (lane == 0) *(volatile int*)&fused.s.published = (int)first_run;
      }
    }
  } else if constexpr (FUSED) {
    // ------------------------------------------------------------ selection (Alg. 1 (normalisation and selection))
    using G = WarpRange<kFusedSelFirst, kFusedSelThreads, 1>;
    const KeyList list{reinterpret_cast<uint2*>(base_ptr + L::kList), &fused.s.sel.list_count[0],
                       (uint32_t)kFusedListCap};
    // (the fused form is launched for batches without per-sequence lengths only: every head has
    // rows and gets finished exactly once)
    const int nonempty_heads = a.batch * a.heads;
    for (;;) {
      if (G::tid() == 0) fused.s.current = fused_pop(a, nonempty_heads, abort_flag);
      G::sync();
      const int p = fused.s.current;
      G::sync();
      if (p < 0) break;
      fused_select_head<G>(a, p, list, fused.s.sel);
      if (a.head_ready != nullptr) {
        G::sync();                                         // every thread's indices are written
        if (G::tid() == 0) {
          __threadfence();
          *(volatile int32_t*)(a.head_ready + p) = 1;
        }
      }
    }
  }

  // ---- teardown
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
