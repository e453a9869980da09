// Attention output O = softmax(scale * Q K^T) V of one cache (full or
// compressed), the quantity whose change under eviction Lemma 1 bounds.  Used by
// the eviction-loss evaluator; not a serving kernel (no causal mask: every
// query sees the whole cache, as in the question-after-context setting).
//
// One CTA per (problem, block of 128 queries), one pass over the keys with an
// online softmax on the tensor cores:
//   S = Q K_t^T per 128-key tile (tcgen05.mma, fp32 in TMEM, one buffer per group);
//   P = exp2(S - m) split into bf16 P_hi + P_lo, written back over S in TMEM;
//   O_g += P_hi V_t + P_lo V_t (A operand read from TMEM, V tile MN-major in
//   shared memory), row sums l_g.
// Keeping P in TMEM matters: an M = N = 128, K = 16 MMA with both operands in
// shared memory reads 8 KB per 64 cycles, all the 128 B/clk an SM has, so a P that
// went through shared memory (64 KB written and read again per tile, next to
// the 64 KB the TMA brings in) made shared memory the bound, not the tensor pipe.
// Warp 0 feeds the TMA ring, warp 1 issues the MMAs, and two groups of four
// softmax warps take alternate key tiles.  Each group runs its own online
// softmax (running maximum m_g, sum l_g, accumulator O_g in TMEM); the running
// maximum only moves when a tile exceeds it by more than 2^8, and then the group
// rescales its accumulator in TMEM, which after the first tiles is rare.  The
// two halves are merged at the end: O = (2^(m_0-m) O_0 + 2^(m_1-m) O_1) / (...).
// Bounded waits as in sketch_umma_kernel.  Keys at or beyond the problem's row
// count are masked by index; the value rows among them are cleared in shared
// memory so that padding can never leak NaNs through a zero weight.
#pragma once
#include "whiten_umma.cuh"

namespace curdkv {
namespace umma {

struct AttnArgs {
  const int32_t* rows;       // [problems] valid key rows of each problem
  const int32_t* row_start;  // [problems] first row inside the packed array, or nullptr
  const int32_t* extra_zero; // [problems] further keys with logit 0 and value 0 (Lemma 1), or nullptr
  int heads, m, packed;      // query rows per problem; packed: K, V are one [rows, d] array
  float scale;
  int split;                 // 1: weights as bf16 pairs hi + lo; 0: single bf16 weights
  float* O;                  // [problems][m][128]
  uint32_t* status;
  unsigned long long wait_ns = kWaitLimitNs;   // limit of each pipeline wait
};

constexpr int kAttnThreads = 320;                          // TMA, MMA, 2 x 4 softmax warps
constexpr int kAttnRing = 5;
constexpr int kAttnQ = 0;
constexpr int kAttnSlot0 = kSlotBytes;
constexpr int kAttnBar = kAttnSlot0 + kAttnRing * kSlotBytes;
constexpr int kAttnDynamic = kAttnBar + 256 + 1024;
// TMEM columns: S of group g at 128 g, overwritten in place by its P (bf16 pairs, see
// attn_p_column); O of group g at 256 + 128 g
constexpr int kAttnTmemCols = 512;
constexpr float kAttnMaxSlack = 8.f;                       // log2 units a tile may exceed the running maximum

// Where the weights of a tile sit inside the 128 columns its logits came in: the weights of keys
// 32c .. 32c+31 stay inside the columns of those keys' logits, P_hi (16 columns of bf16 pairs) at
// 32c and P_lo at 32c + 16, so that a softmax thread can turn the row over 32 keys at a time.
// Column of P_hi for the g-th group of 16 keys:
__host__ __device__ constexpr uint32_t attn_p_column(int g) { return 32u * (uint32_t)(g >> 1) + 8u * (uint32_t)(g & 1); }

// P V: A = P K-major, B = V tile MN-major (contraction over the keys)
__host__ __device__ constexpr uint32_t instr_desc_pv() { return instr_desc_bf16(128) | (1u << 16); }

// 32 consecutive fp32 columns of this thread's TMEM lane, written back.
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float (&v)[32]) {
  const uint32_t* u = reinterpret_cast<const uint32_t*>(v);
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
      "r"(u[0]), "r"(u[1]), "r"(u[2]), "r"(u[3]), "r"(u[4]), "r"(u[5]), "r"(u[6]), "r"(u[7]), "r"(u[8]),
      "r"(u[9]), "r"(u[10]), "r"(u[11]), "r"(u[12]), "r"(u[13]), "r"(u[14]), "r"(u[15]), "r"(u[16]),
      "r"(u[17]), "r"(u[18]), "r"(u[19]), "r"(u[20]), "r"(u[21]), "r"(u[22]), "r"(u[23]), "r"(u[24]),
      "r"(u[25]), "r"(u[26]), "r"(u[27]), "r"(u[28]), "r"(u[29]), "r"(u[30]), "r"(u[31])
      : "memory");
}
// 16 consecutive 32-bit columns of this thread's TMEM lane, written.
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&u)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
      "r"(u[0]), "r"(u[1]), "r"(u[2]), "r"(u[3]), "r"(u[4]), "r"(u[5]), "r"(u[6]), "r"(u[7]), "r"(u[8]),
      "r"(u[9]), "r"(u[10]), "r"(u[11]), "r"(u[12]), "r"(u[13]), "r"(u[14]), "r"(u[15])
      : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem], bf16 inputs, fp32 accumulate, M = 128: row i of A is TMEM lane
// i, its K = 16 elements sit in 8 consecutive 32-bit columns.
__device__ __forceinline__ void tc_mma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc,
                                               uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() {
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

// 2^x, relative error ~2^-22 (the weights are rounded to bf16 pairs afterwards)
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Packed fp32 pairs (one instruction for two lanes of arithmetic) and three-input max / min.
__device__ __forceinline__ uint64_t pack2(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t r, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(r));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ float min3(float a, float b, float c) {
  float d;
  asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// Two weights -> packed bf16 (hi) and packed bf16 of the remainders (lo).
__device__ __forceinline__ void split_bf16x2(float w0, float w1, uint32_t& hi, uint32_t& lo) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(w0, w1);
  hi = *reinterpret_cast<const uint32_t*>(&h);
  const float r0 = w0 - __uint_as_float(hi << 16), r1 = w1 - __uint_as_float(hi & 0xffff0000u);
  const __nv_bfloat162 l = __floats2bfloat162_rn(r0, r1);
  lo = *reinterpret_cast<const uint32_t*>(&l);
}

// SPLIT: the weights enter P V as bf16 pairs P_hi + P_lo (two products per tile, weights exact to
// 2^-17); without it as single bf16 values (one product, weights exact to 2^-9, and the row sums are
// taken over the rounded weights so that every row of P still sums to the normaliser it is divided by).
template <bool SPLIT>
__global__ void __launch_bounds__(kAttnThreads, 1)
attention_umma_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                      const __grid_constant__ CUtensorMap map_v, const AttnArgs a) {
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
  const uint32_t bar0 = base + kAttnBar;
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (kAttnRing + s); };
  auto s_full_bar = [&](int s) { return bar0 + 8u * (2 * kAttnRing + s); };
  auto p_ready_bar = [&](int s) { return bar0 + 8u * (2 * kAttnRing + 2 + s); };
  const uint32_t q_full_bar = bar0 + 8u * (2 * kAttnRing + 4);
  const uint32_t o_full_bar = bar0 + 8u * (2 * kAttnRing + 5);
  const uint32_t drain_bar = bar0 + 8u * (2 * kAttnRing + 6);
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(base_ptr + kAttnBar + 8 * (2 * kAttnRing + 7));
  __shared__ float xchg[2][kTileRows];                     // running maximum and row sum of the second group
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  const int q_blocks = (a.m + kTileRows - 1) / kTileRows;
  const int p = blockIdx.x / q_blocks, qb = blockIdx.x % q_blocks;
  const int b = p / a.heads, h = p % a.heads;
  const int n = max(a.rows[p], 0);
  const int T = (n + kTileRows - 1) / kTileRows;           // key tiles
  const int key0 = a.row_start != nullptr ? a.row_start[p] : 0;
  const int kh = a.packed ? 0 : h, kb = a.packed ? 0 : b;
  const int extra = a.extra_zero != nullptr ? max(a.extra_zero[p], 0) : 0;

  if (T == 0) {                                            // empty cache: define O = 0
    for (int e = tid; e < kTileRows * 128; e += kAttnThreads) {
      const int row = qb * kTileRows + e / 128;
      if (row < a.m) a.O[((size_t)p * a.m + row) * 128 + (e & 127)] = 0.f;
    }
    return;
  }

  if (tid == 0) {
    for (int s = 0; s < kAttnRing; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int s = 0; s < 2; ++s) {
      mbar_init(s_full_bar(s), 1);
      mbar_init(p_ready_bar(s), 128);
    }
    mbar_init(q_full_bar, 1);
    mbar_init(o_full_bar, 1);
    mbar_init(drain_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(tmem_holder)),
                 "r"((uint32_t)kAttnTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;

  // Tiles go through the ring in the order the MMA issuer consumes them:
  //   K_0, K_1, then for every t: V_t, K_{t+2} (if any).
  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint64_t pol_keep;
      asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));
      mbar_arrive_expect_tx(q_full_bar, kSlotBytes);
      tma_load_4d(base + kAttnQ, &map_q, q_full_bar, 0, qb * kTileRows, h, b, pol_keep);
      tma_load_4d(base + kAttnQ + kHalfBytes, &map_q, q_full_bar, 64, qb * kTileRows, h, b, pol_keep);
      uint32_t it = 0;
      bool ok = true;
      auto load = [&](const CUtensorMap* map, int t) {
        const int slot = it % kAttnRing;
        const uint32_t phase = (it / kAttnRing) & 1u;
        if (!(ok = mbar_wait(empty_bar(slot), phase ^ 1u, abort_flag, a.status, a.wait_ns))) return;
        mbar_arrive_expect_tx(full_bar(slot), kSlotBytes);
        const uint32_t dst = base + kAttnSlot0 + slot * kSlotBytes;
        // the key tiles of a problem are read by all of its query blocks: no evict-first
        tma_load_4d(dst, map, full_bar(slot), 0, key0 + t * kTileRows, kh, kb, pol_keep);
        tma_load_4d(dst + kHalfBytes, map, full_bar(slot), 64, key0 + t * kTileRows, kh, kb, pol_keep);
        ++it;
      };
      load(&map_k, 0);
      if (ok && T > 1) load(&map_k, 1);
      for (int t = 0; ok && t < T; ++t) {
        load(&map_v, t);
        if (ok && t + 2 < T) load(&map_k, t + 2);
      }
      if (!ok) {
        const uint32_t pending = it < (uint32_t)kAttnRing ? it : (uint32_t)kAttnRing;
        for (uint32_t q = it - pending; q < it; ++q) {
          unsigned long long t0 = global_ns();
          while (!mbar_try_wait(full_bar(q % kAttnRing), (q / kAttnRing) & 1u) &&
                 global_ns() - t0 < a.wait_ns) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_s = instr_desc_bf16(128);
      constexpr uint32_t idesc_pv = instr_desc_pv();
      uint32_t it = 0;
      bool ok = mbar_wait(q_full_bar, 0, abort_flag, a.status, a.wait_ns);
      tc_fence_after();
      // The issuing thread shares its scheduler with two softmax warps, so what it executes per
      // MMA counts: descriptors are formed once per tile and stepped by constants (the address
      // field counts 16-byte units and cannot carry out of its 14 bits inside shared memory).
      const uint64_t q_desc = smem_desc_sw128(base + kAttnQ);
      auto issue_s = [&](uint32_t buf) {                   // S[buf] = Q K^T for the next K tile of the ring
        const int slot = it % kAttnRing;
        if (!(ok = mbar_wait(full_bar(slot), (it / kAttnRing) & 1u, abort_flag, a.status, a.wait_ns))) return;
        tc_fence_after();
        const uint64_t k_desc = smem_desc_sw128(base + kAttnSlot0 + slot * kSlotBytes);
        const uint32_t d_tmem = tmem_base + buf * 128u;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          constexpr uint32_t kHalfUnits = kHalfBytes >> 4;
          const uint32_t off = (uint32_t)(k >> 2) * kHalfUnits + (uint32_t)(k & 3) * 2u;   // 16-byte units
          tc_mma_bf16(d_tmem, q_desc + off, k_desc + off, idesc_s, k > 0);
        }
        tc_commit(empty_bar(slot));
        tc_commit(s_full_bar(buf));
        ++it;
      };
      // A group's S buffer is taken over by its P; S_{t+2} goes into it right behind P_t V_t (the
      // tensor pipe runs the MMAs of one thread in order, so the product has read P by then).
      if (ok) issue_s(0);                                  // tile 0
      if (ok && T > 1) issue_s(1);                         // tile 1
      for (int t = 0; ok && t < T; ++t) {
        const int slot = it % kAttnRing;
        if (!(ok = mbar_wait(full_bar(slot), (it / kAttnRing) & 1u, abort_flag, a.status, a.wait_ns))) break;
        const int rows = min(kTileRows, n - t * kTileRows);
        const int groups = (rows + 15) >> 4;
        if (rows < groups * 16) {                          // clear the padding rows the last MMA reads
          for (int j = rows; j < groups * 16; ++j)
            for (int half = 0; half < 2; ++half)
              for (int c = 0; c < 8; ++c)
                *reinterpret_cast<uint4*>(base_ptr + kAttnSlot0 + slot * kSlotBytes + half * kHalfBytes +
                                          j * 128 + c * 16) = make_uint4(0u, 0u, 0u, 0u);
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }
        const uint32_t buf = (uint32_t)t & 1u;             // the group that owns this tile, its P and O
        if (!(ok = mbar_wait(p_ready_bar(buf), (uint32_t)(t >> 1) & 1u, abort_flag, a.status, a.wait_ns))) break;
        tc_fence_after();
        const uint64_t v_desc = smem_desc_mn_sw128(base + kAttnSlot0 + slot * kSlotBytes);
        const uint32_t o_tmem = tmem_base + 256u + buf * 128u;
#pragma unroll
        for (int part = 0; part < (SPLIT ? 2 : 1); ++part) {   // P_hi, then P_lo
          const uint32_t p_tmem = tmem_base + buf * 128u + part * 16u;
          // 16 keys per MMA: 8 columns of P (attn_p_column), 2048 bytes (128 units) of the V tile
          if (groups == 8) {
            tc_mma_bf16_ts(o_tmem, p_tmem, v_desc, idesc_pv, (t > 1 || part > 0) ? 1u : 0u);
#pragma unroll
            for (int g = 1; g < 8; ++g)
              tc_mma_bf16_ts(o_tmem, p_tmem + attn_p_column(g), v_desc + 128u * g, idesc_pv, 1u);
          } else {
            for (int g = 0; g < groups; ++g)
              tc_mma_bf16_ts(o_tmem, p_tmem + attn_p_column(g), v_desc + 128u * g, idesc_pv,
                             (t > 1 || part > 0 || g > 0) ? 1u : 0u);
          }
        }
        tc_commit(empty_bar(slot));
        ++it;
        if (t + 2 < T) issue_s(buf);
      }
      if (ok) tc_commit(o_full_bar);
      if (!ok) {
        tc_commit(drain_bar);
        unsigned long long t0 = global_ns();
        while (!mbar_try_wait(drain_bar, 0) && global_ns() - t0 < a.wait_ns) {}
      }
    }
  } else {
    // ------------------------------------------------------------ softmax + epilogue
    const int group = (warp - 2) >> 2;                     // takes the jobs of its parity
    const int quarter = warp & 3;
    const int r = quarter * 32 + lane;                     // query row inside the block = TMEM lane
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
    constexpr float kLog2e = 1.4426950408889634f;
    const float sc = a.scale * kLog2e;                     // logits in units of log2
    // running maximum (log2 units) and row sum of this group's tiles; Lemma 1's zero keys (logit 0,
    // weight 2^0 each) are booked by the first group
    float top = (extra > 0 && group == 0) ? 0.f : -INFINITY;
    float sum = (extra > 0 && group == 0) ? (float)extra : 0.f;
    bool has_o = false, ok = true;                         // has_o: O_group holds at least one product
    const uint32_t s_addr = lane_addr + group * 128u, o_addr = lane_addr + 256u + group * 128u;
    for (int t = group; ok && t < T; t += 2) {
      ok = mbar_wait(s_full_bar(group), (uint32_t)(t >> 1) & 1u, abort_flag, a.status, a.wait_ns);
      if (!(ok = __all_sync(0xffffffffu, ok))) break;
      tc_fence_after();
      const int valid = n - t * kTileRows;                 // keys of this tile that exist
      // First pass over the row: its maximum.  The row is read from TMEM 64 columns at a time here
      // and again below (a thread that held all 128 logits left the compiler no room).
      float tile_top = -INFINITY;
      if (valid >= kTileRows) {
        // max_c (v_c * sc) = sc * max_c v_c or sc * min_c v_c; four independent chains
        float ext[4];
#pragma unroll
        for (int c0 = 0; c0 < 128; c0 += 64) {
          float v[64];
          tmem_ld32(s_addr + c0, *reinterpret_cast<float(*)[32]>(v));
          tmem_ld32(s_addr + c0 + 32, *reinterpret_cast<float(*)[32]>(v + 32));
          tmem_ld_wait();
          if (c0 == 0) { ext[0] = v[0]; ext[1] = v[1]; ext[2] = v[2]; ext[3] = v[3]; }
          if (sc >= 0.f) {
#pragma unroll
            for (int c = 0; c < 64; c += 8)
#pragma unroll
              for (int j = 0; j < 4; ++j) ext[j] = max3(ext[j], v[c + 2 * j], v[c + 2 * j + 1]);
          } else {
#pragma unroll
            for (int c = 0; c < 64; c += 8)
#pragma unroll
              for (int j = 0; j < 4; ++j) ext[j] = min3(ext[j], v[c + 2 * j], v[c + 2 * j + 1]);
          }
        }
        tile_top = (sc >= 0.f ? fmaxf(fmaxf(ext[0], ext[1]), fmaxf(ext[2], ext[3]))
                              : fminf(fminf(ext[0], ext[1]), fminf(ext[2], ext[3]))) * sc;
      } else {
#pragma unroll
        for (int c0 = 0; c0 < 128; c0 += 64) {
          float v[64];
          tmem_ld32(s_addr + c0, *reinterpret_cast<float(*)[32]>(v));
          tmem_ld32(s_addr + c0 + 32, *reinterpret_cast<float(*)[32]>(v + 32));
          tmem_ld_wait();
#pragma unroll
          for (int c = 0; c < 64; ++c)
            if (c0 + c < valid) tile_top = fmaxf(tile_top, v[c] * sc);
        }
      }
      // move the running maximum only when the tile exceeds it by more than the slack
      const bool move = tile_top > top + kAttnMaxSlack || top == -INFINITY;
      const float new_top = move ? fmaxf(top, tile_top) : top;
      const float alpha = move ? fast_exp2(top - new_top) : 1.f;      // 0 when top was -inf
      // (this group's previous product has retired: S of this tile was issued behind it)
      if (has_o && __any_sync(0xffffffffu, move)) {        // rescale O_group in TMEM
#pragma unroll 1
        for (int c0 = 0; c0 < 128; c0 += 32) {
          float o[32];
          tmem_ld32(o_addr + c0, o);
          tmem_ld_wait();
#pragma unroll
          for (int c = 0; c < 32; ++c) o[c] *= alpha;
          tmem_st32(o_addr + c0, o);
        }
        tmem_st_wait();
      }
      sum *= alpha;
      top = new_top;
      // Second pass: the weights of 64 keys take the place of those keys' logits.
      if (valid >= kTileRows) {
        // full tile: the arithmetic runs on packed pairs of keys
        const uint64_t sc2 = pack2(sc, sc), ntop2 = pack2(-top, -top);
        uint64_t part[4] = {0ull, 0ull, 0ull, 0ull};       // eight partial row sums
#pragma unroll
        for (int c0 = 0; c0 < 128; c0 += 64) {
          float v[64];
          tmem_ld32(s_addr + c0, *reinterpret_cast<float(*)[32]>(v));
          tmem_ld32(s_addr + c0 + 32, *reinterpret_cast<float(*)[32]>(v + 32));
          tmem_ld_wait();
#pragma unroll
          for (int c1 = 0; c1 < 64; c1 += 32) {            // 32 keys -> 16 columns of P_hi and of P_lo
            uint32_t hi[16], lo[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              const int c = c1 + 2 * e;
              float x0, x1;
              unpack2(fma2(pack2(v[c], v[c + 1]), sc2, ntop2), x0, x1);
              const uint64_t w2 = pack2(fast_exp2(x0), fast_exp2(x1));
              float w0, w1;
              unpack2(w2, w0, w1);
              const __nv_bfloat162 h = __floats2bfloat162_rn(w0, w1);
              hi[e] = *reinterpret_cast<const uint32_t*>(&h);
              const uint64_t h2 = pack2(__uint_as_float(hi[e] << 16), __uint_as_float(hi[e] & 0xffff0000u));
              if (SPLIT) {
                part[e & 3] = add2(part[e & 3], w2);       // equals the bf16 pairs to 2^-17
                float r0, r1;
                unpack2(sub2(w2, h2), r0, r1);
                const __nv_bfloat162 q = __floats2bfloat162_rn(r0, r1);
                lo[e] = *reinterpret_cast<const uint32_t*>(&q);
              } else {
                part[e & 3] = add2(part[e & 3], h2);       // the weights the product really uses
              }
            }
            tmem_st16(s_addr + (uint32_t)(c0 + c1), hi);
            if (SPLIT) tmem_st16(s_addr + (uint32_t)(c0 + c1) + 16u, lo);
          }
        }
        float p0, p1;
        unpack2(add2(add2(part[0], part[1]), add2(part[2], part[3])), p0, p1);
        sum += p0 + p1;
      } else {
        // last tile of the cache: keys beyond its end are masked by index
#pragma unroll
        for (int c0 = 0; c0 < 128; c0 += 64) {
          float v[64];
          tmem_ld32(s_addr + c0, *reinterpret_cast<float(*)[32]>(v));
          tmem_ld32(s_addr + c0 + 32, *reinterpret_cast<float(*)[32]>(v + 32));
          tmem_ld_wait();
#pragma unroll
          for (int c1 = 0; c1 < 64; c1 += 32) {
            uint32_t hi[16], lo[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              const int c = c1 + 2 * e;
              const float w0 = c0 + c < valid ? fast_exp2(fmaf(v[c], sc, -top)) : 0.f;
              const float w1 = c0 + c + 1 < valid ? fast_exp2(fmaf(v[c + 1], sc, -top)) : 0.f;
              split_bf16x2(w0, w1, hi[e], lo[e]);
              sum += SPLIT ? w0 + w1 : __uint_as_float(hi[e] << 16) + __uint_as_float(hi[e] & 0xffff0000u);
            }
            tmem_st16(s_addr + (uint32_t)(c0 + c1), hi);
            if (SPLIT) tmem_st16(s_addr + (uint32_t)(c0 + c1) + 16u, lo);
          }
        }
      }
      tmem_st_wait();
      tc_fence_before();
      mbar_arrive(p_ready_bar(group));
      has_o = true;
    }
    // the second group hands its statistics to the first, which merges the two accumulators
    if (group == 1) {
      xchg[0][r] = has_o ? top : -INFINITY;
      xchg[1][r] = has_o ? sum : 0.f;
    }
    asm volatile("bar.sync 1, 256;" ::: "memory");         // reached by all eight warps, aborted or not
    if (group == 0) {
      const float top1 = xchg[0][r], sum1 = xchg[1][r];
      const float m = fmaxf(top, top1);                    // group 0 always owns tile 0: m is finite
      const float w0 = fast_exp2(top - m), w1 = top1 == -INFINITY ? 0.f : fast_exp2(top1 - m);
      const float denom = w0 * sum + w1 * sum1;
      if (ok) {
        ok = mbar_wait(o_full_bar, 0, abort_flag, a.status, a.wait_ns);
        ok = __all_sync(0xffffffffu, ok);
      }
      if (ok) {
        tc_fence_after();
        const int row = qb * kTileRows + r;
        const float i0 = denom > 0.f ? w0 / denom : 0.f, i1 = denom > 0.f ? w1 / denom : 0.f;
        const bool both = T > 1;                           // O_1 exists only if the second group had a tile
        float* out = a.O + ((size_t)p * a.m + row) * 128;
#pragma unroll 1
        for (int c0 = 0; c0 < 128; c0 += 32) {
          float v[32], u[32];
          tmem_ld32(lane_addr + 256u + c0, v);
          if (both) tmem_ld32(lane_addr + 384u + c0, u);
          tmem_ld_wait();
          if (row < a.m) {
#pragma unroll
            for (int c = 0; c < 32; c += 4) {
              float4 o;
              o.x = v[c] * i0 + (both ? u[c] * i1 : 0.f);
              o.y = v[c + 1] * i0 + (both ? u[c + 1] * i1 : 0.f);
              o.z = v[c + 2] * i0 + (both ? u[c + 2] * i1 : 0.f);
              o.w = v[c + 3] * i0 + (both ? u[c + 3] * i1 : 0.f);
              *reinterpret_cast<float4*>(out + c0 + c) = o;
            }
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                 "r"((uint32_t)kAttnTmemCols)
                 : "memory");
  }
}

// ||O - O'||_F and ||O||_F per problem.  grid = problems, block = 256; fixed summation order.
__global__ void __launch_bounds__(256) frob_diff_kernel(const float* O, const float* Oc, int elems,
                                                        float* loss, float* ref_norm) {
  __shared__ double red[2][8];
  const int p = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* x = O + (size_t)p * elems;
  const float* y = Oc + (size_t)p * elems;
  double d2 = 0.0, r2 = 0.0;
  for (int e = tid; e < elems; e += 256) {
    const double u = x[e], w = (double)x[e] - (double)y[e];
    d2 += w * w;
    r2 += u * u;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    d2 += __shfl_xor_sync(0xffffffffu, d2, o);
    r2 += __shfl_xor_sync(0xffffffffu, r2, o);
  }
  if (lane == 0) { red[0][warp] = d2; red[1][warp] = r2; }
  __syncthreads();
  if (tid == 0) {
    double s0 = 0.0, s1 = 0.0;
    for (int w = 0; w < 8; ++w) { s0 += red[0][w]; s1 += red[1][w]; }
    loss[p] = (float)sqrt(s0);
    if (ref_norm != nullptr) ref_norm[p] = (float)sqrt(s1);
  }
}

}  // namespace umma
}  // namespace curdkv
