// Whitening factors of the leverage-score sketch: for one (sequence, head) and
// one tensor, sums the partial Gram matrices of its segments in a fixed order,
// adds the ridge, factors M = L L^T and solves L^T W = G, all in fp64 (the Gram
// matrix squares the conditioning of K or V).  Writes W as fp32 [128][r].
//
// One CTA of 256 threads per matrix, two CTAs per SM.  Three things of similar size bound the
// kernel (measured on B200 by leaving each out in turn): the chain of dependent steps, the
// shared-memory loads of the published columns and the fp64 pipe.  So each thread holds a large
// register tile (few warps repeat the per-step loads and bookkeeping), the steps are chained as
// tightly as the hardware allows, and two matrices per SM fill each other's gaps.
//  * Factorisation.  Warp w owns two adjacent columns out of every 16 of the lower triangle; lane
//    l holds their rows l + 32u in registers (40 values per thread: the blocks on or below the
//    diagonal).  A finished pair of columns of L is written to shared memory (packed lower
//    triangle) by its warp, which then arrives, without waiting, on a named barrier; the other
//    warps wait on that barrier before they apply the pair to their columns.  The warp that owns
//    the next pair updates, factors (inside the warp, by shuffles) and publishes it first and
//    updates its other columns afterwards, so the chain pair -> next pair is one warp's short path
//    and the bulk of the rank-2 update runs behind it.  (A hand-over through a hardware barrier
//    costs about 90 cycles here, through an mbarrier about 220, which is why columns go in pairs
//    and over barriers.)
//  * Back substitution, 32 right-hand sides at a time.  Lane l holds the rows l + 32u of the
//    solution, warp w their columns 4w .. 4w + 3, so a warp solves its columns without the
//    others: the finished row i is broadcast by shuffles.
#pragma once
#include "common.cuh"

namespace curdkv {

constexpr int kFactorThreads = 256;
constexpr int kFactorWarps = kFactorThreads / 32;
constexpr int kFactorD = 128;
constexpr int kFactorPass = 32;                            // right-hand sides per back-substitution pass
// dynamic shared memory: L (packed lower triangle, by columns), one pass of solved rows, 1 / L[i][i]
constexpr size_t kFactorOffW = (size_t)kFactorD * (kFactorD + 1) / 2 * sizeof(double);
constexpr size_t kFactorOffInv = kFactorOffW + (size_t)kFactorD * kFactorPass * sizeof(double);
constexpr size_t kFactorSmemBytes = kFactorOffInv + kFactorD * sizeof(double);   // >= two staging areas

struct FactorArgs {
  const float* partials;   // [batch*heads*segments][2][128][128]
  const float* G;          // [128][r]
  float* W;                // [batch*heads][2][128][r]
  int segments, r;         // r <= 64
  double ridge;
  uint32_t* status;
};

// Copies what the factorisation reads of one stored 128 x 128 fp32 matrix into shared memory: rows
// 0 .. 63 (32 KB), then columns 64 .. 127 of rows 64 .. 127 (16 KB).  Whole CTA; one cp.async group.
constexpr int kFactorStageBytes = 48 * 1024;
static_assert(2 * kFactorStageBytes <= kFactorSmemBytes, "two staging areas must fit");
__device__ __forceinline__ void stage_partial(const float* src, unsigned char* stage, int tid) {
  const uint32_t dst = static_cast<uint32_t>(__cvta_generic_to_shared(stage));
  const unsigned char* g = reinterpret_cast<const unsigned char*>(src);
  for (int q = tid; q < 2048; q += kFactorThreads)
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + 16u * q), "l"(g + 16 * q) : "memory");
  for (int q = tid; q < 1024; q += kFactorThreads) {
    const int row = 64 + (q >> 4), chunk = q & 15;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + 32768u + 16u * q),
                 "l"(g + (row * kFactorD + 64) * 4 + 16 * chunk)
                 : "memory");
  }
  asm volatile("cp.async.commit_group;" ::: "memory");
}

// "Column pair p is in shared memory": hardware barrier 1 + p mod 8, on which the pair's warp only
// arrives and the seven others wait.  Every warp executes exactly one of the two per pair, in
// pair order, so a barrier is never reused before its previous round has completed.
__device__ __forceinline__ void pair_arrive(int p) {
  asm volatile("bar.arrive %0, %1;" ::"r"(1 + (p & 7)), "r"(kFactorThreads) : "memory");
}
__device__ __forceinline__ void pair_wait(int p) {
  asm volatile("bar.sync %0, %1;" ::"r"(1 + (p & 7)), "r"(kFactorThreads) : "memory");
}

// Column k of the packed triangle holds rows k .. 127; the returned offset already has k
// subtracted, so that row i of column k is element tri_base(k) + i.
__device__ __forceinline__ int tri_base(int k) { return k * (kFactorD - 1) - ((k * (k - 1)) >> 1); }

// m[u][c] is the element (l + 32u, column_of(w, c)) of the matrix being eliminated: a warp owns
// the two adjacent columns 2w, 2w + 1 of every group of 16, and only the blocks on or below the
// diagonal (u >= c / 4) are held.  Elements above the diagonal (inside the diagonal blocks) and
// columns that have already been published are dead: they are updated along with the rest, with
// whatever the loads return for them, and never read.
__device__ __forceinline__ int column_of(int w, int c) { return 16 * (c >> 1) + 2 * w + (c & 1); }

// The warp that owns the columns kA = 2p and kB = kA + 1 (its register columns 2P and 2P + 1)
// finishes both and writes them to shared memory: column kA is scaled by the inverse root of its
// pivot, applied to column kB, and column kB scaled in turn; all of it stays inside the warp.
template <int P>
__device__ __forceinline__ void publish_pair(const double (&m)[4][16], int p, double* Lt, double* invd, int l,
                                             bool& bad) {
  constexpr int U = P / 2, CA = 2 * P, CB = 2 * P + 1;
  const int kA = 2 * p, kB = kA + 1;
  double pivA = __shfl_sync(0xffffffffu, m[U][CA], kA & 31);
  if (!(pivA > 0.0)) { pivA = 1e-300; bad = true; }
  const double rsA = rsqrt(pivA);
  double la[4], lb[4];
#pragma unroll
  for (int u = U; u < 4; ++u) la[u] = m[u][CA] * rsA;
  const double lBA = __shfl_sync(0xffffffffu, la[U], kB & 31);   // L[kB][kA]
#pragma unroll
  for (int u = U; u < 4; ++u) lb[u] = m[u][CB] - la[u] * lBA;
  double pivB = __shfl_sync(0xffffffffu, lb[U], kB & 31);
  if (!(pivB > 0.0)) { pivB = 1e-300; bad = true; }
  const double rsB = rsqrt(pivB);
  double* colA = Lt + tri_base(kA);
  double* colB = Lt + tri_base(kB);
#pragma unroll
  for (int u = U; u < 4; ++u) {
    const int i = l + 32 * u;
    if (i >= kA) colA[i] = la[u];
    if (i >= kB) colB[i] = lb[u] * rsB;
  }
  if (l == (kA & 31)) invd[kA] = rsA;                      // 1 / L[k][k]
  if (l == (kB & 31)) invd[kB] = rsB;
  pair_arrive(p);
}

// m[.][C] -= L[.][kA] L[j][kA] + L[.][kB] L[j][kB] for this warp's column j = column_of(w, C).
template <int C>
__device__ __forceinline__ void apply_pair(double (&m)[4][16], const double (&liA)[4], const double (&liB)[4],
                                           const double* colA, const double* colB, int w) {
  const int j = column_of(w, C);
  const double ljA = colA[j], ljB = colB[j];               // one value each for the whole warp
#pragma unroll
  for (int u = C / 4; u < 4; ++u) m[u][C] = fma(-liB[u], ljB, fma(-liA[u], ljA, m[u][C]));
}
template <int C>
__device__ __forceinline__ void apply_pair_from(double (&m)[4][16], const double (&liA)[4],
                                                const double (&liB)[4], const double* colA, const double* colB,
                                                int w) {
  if constexpr (C < 16) {
    apply_pair<C>(m, liA, liB, colA, colB, w);
    apply_pair_from<C + 1>(m, liA, liB, colA, colB, w);
  }
}

// Elimination by the column pairs p = 8*KH .. 8*KH + 7 (columns 16*KH .. 16*KH + 15): only the
// register columns c >= 2*KH and the row blocks u >= KH / 2 still change, so the steps are
// compiled for exactly those.  Loads of rows or columns before the pair stay inside the packed
// triangle (they reach at most 31 elements back) and only feed dead elements.
template <int KH>
__device__ __forceinline__ void cholesky_pairs(double (&m)[4][16], double* Lt, double* invd, int w, int l,
                                               bool& bad) {
  constexpr int U0 = KH / 2;
#pragma unroll 1
  for (int pt = 0; pt < 8; ++pt) {
    const int p = 8 * KH + pt, kA = 2 * p;
    if (pt != w) pair_wait(p);                             // its own pair needs no waiting for
    const double* colA = Lt + tri_base(kA);
    const double* colB = colA + (kFactorD - 1 - kA);       // tri_base(kA + 1)
    double liA[4], liB[4];
#pragma unroll
    for (int u = U0; u < 4; ++u) {
      liA[u] = colA[l + 32 * u];
      liB[u] = colB[l + 32 * u];
    }
    // the owner of the next pair brings it up to date and publishes it before anything else
    if (pt + 1 == w) {
      apply_pair<2 * KH>(m, liA, liB, colA, colB, w);
      apply_pair<2 * KH + 1>(m, liA, liB, colA, colB, w);
      publish_pair<KH>(m, p + 1, Lt, invd, l, bad);
    } else if (pt == 7 && w == 0) {
      if constexpr (KH + 1 < 8) {
        apply_pair<2 * KH + 2>(m, liA, liB, colA, colB, w);
        apply_pair<2 * KH + 3>(m, liA, liB, colA, colB, w);
        publish_pair<KH + 1>(m, p + 1, Lt, invd, l, bad);
      }
    }
    // (the owner applies the pair once more to the columns it has just published: dead registers)
    apply_pair_from<2 * KH>(m, liA, liB, colA, colB, w);
  }
}

// Back-substitution steps i = 32*IU + 31 .. 32*IU of one pass: only the rows of the blocks
// u <= IU are still open.  x[u][c] is the element (l + 32u, column 4w + c of the pass) of the
// right-hand side / solution; tb[u] = tri_base(l + 32u).  A warp solves its four columns on its
// own: the finished row i is broadcast from the lane that holds it by shuffles, so the chain of
// 128 dependent steps never leaves the warp.
template <int IU>
__device__ __forceinline__ void backsub_steps(double (&x)[4][4], const int (&tb)[4],
                                              const double* __restrict__ Lt, double* __restrict__ Wt,
                                              const double* __restrict__ invd, int w, int l) {
#pragma unroll 2
  for (int it = 31; it >= 0; --it) {
    const int i = 32 * IU + it;
    const double dinv = invd[i];                           // 1 / L[i][i]
    double wv[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) wv[c] = __shfl_sync(0xffffffffu, x[IU][c] * dinv, it);   // W[i][4w + c]
#pragma unroll
    for (int u = IU; u >= 0; --u) {                        // block IU first: the next step waits for it
      double lv = Lt[tb[u] + i];                           // L[i][row]; finished rows read a neighbour: masked
      if (u == IU && l >= it) lv = 0.0;
#pragma unroll
      for (int c = 0; c < 4; ++c) x[u][c] -= lv * wv[c];
    }
    if (l == it) {
      double* dst = Wt + i * kFactorPass + 4 * w;
      *reinterpret_cast<double2*>(dst) = make_double2(wv[0], wv[1]);
      *reinterpret_cast<double2*>(dst + 2) = make_double2(wv[2], wv[3]);
    }
  }
}

// grid = batch*heads*2, block = 256, dynamic shared memory = kFactorSmemBytes.
__global__ void __launch_bounds__(kFactorThreads, 2) whiten_factor_kernel(const FactorArgs a) {
  extern __shared__ __align__(16) unsigned char fsm[];
  constexpr int D = kFactorD;
  double* Lt = reinterpret_cast<double*>(fsm);                       // packed: L[i][k] at tri_base(k) + i
  double* Wt = reinterpret_cast<double*>(fsm + kFactorOffW);         // Wt[i*32 + c] = W[i][32*pass + c]
  double* invd = reinterpret_cast<double*>(fsm + kFactorOffInv);     // 1 / L[i][i]
  __shared__ double red[kFactorWarps];
  const int tid = threadIdx.x, w = tid >> 5, l = tid & 31;
  const int p = blockIdx.x >> 1, tensor = blockIdx.x & 1;
  const int r = a.r;

  // ---- M = sum of the segments' partial Gram matrices (segment order).  Element (i, j), i >= j,
  // is taken from row j of the stored matrix, so that a warp reads along a row; the part of a
  // diagonal block above the diagonal mirrors the part below it.  The rows 0 .. 63 and the lower
  // right quadrant of a stored matrix (all that this needs) are staged in shared memory by
  // asynchronous copies, two segments in flight.
  double m[4][16];
#pragma unroll
  for (int v = 0; v < 16; ++v)
#pragma unroll
    for (int u = v / 4; u < 4; ++u) m[u][v] = 0.0;
  const float* first = a.partials + (((size_t)p * a.segments) * 2 + tensor) * D * D;
  stage_partial(first, fsm, tid);
  if (a.segments > 1) stage_partial(first + 2 * D * D, fsm + kFactorStageBytes, tid);
  for (int g = 0; g < a.segments; ++g) {
    if (g + 1 < a.segments) asm volatile("cp.async.wait_group 1;" ::: "memory");
    else asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    const float* top = reinterpret_cast<const float*>(fsm + (g & 1) * kFactorStageBytes);
    const float* quad = top + 64 * D;
#pragma unroll
    for (int v = 0; v < 16; ++v) {
#pragma unroll
      for (int u = v / 4; u < 4; ++u) {
        const int i = l + 32 * u, j = column_of(w, v);
        const int lo = min(i, j), hi = max(i, j);
        m[u][v] += (double)(v < 8 ? top[lo * D + hi] : quad[(lo - 64) * 64 + (hi - 64)]);
      }
    }
    __syncthreads();
    if (g + 2 < a.segments)
      stage_partial(first + (size_t)(g + 2) * 2 * D * D, fsm + (g & 1) * kFactorStageBytes, tid);
  }
  double tr = 0.0;
#pragma unroll
  for (int v = 0; v < 16; ++v)
    if (l + 32 * (v / 4) == column_of(w, v)) tr += m[v / 4][v];   // the diagonal sits in the blocks u = v / 4
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) tr += __shfl_xor_sync(0xffffffffu, tr, o);
  if (l == 0) red[w] = tr;
  __syncthreads();
  double trace = 0.0;
#pragma unroll
  for (int q = 0; q < kFactorWarps; ++q) trace += red[q];
  float* out = a.W + ((size_t)p * 2 + tensor) * D * r;
  if (!(trace > 0.0)) {                                    // no valid rows (or all zero): nothing to whiten
    for (int e = tid; e < D * r; e += kFactorThreads) out[e] = 0.f;
    return;
  }
  const double lambda = a.ridge * trace / D;
#pragma unroll
  for (int v = 0; v < 16; ++v)
    if (l + 32 * (v / 4) == column_of(w, v)) m[v / 4][v] += lambda;

  // ---- Cholesky by outer products: column k of L is published as soon as columns 0 .. k-1 have
  // been applied to it, and every thread subtracts L_ik L_jk from its elements right of it
  bool bad = false;
  if (w == 0) publish_pair<0>(m, 0, Lt, invd, l, bad);
  cholesky_pairs<0>(m, Lt, invd, w, l, bad);
  cholesky_pairs<1>(m, Lt, invd, w, l, bad);
  cholesky_pairs<2>(m, Lt, invd, w, l, bad);
  cholesky_pairs<3>(m, Lt, invd, w, l, bad);
  cholesky_pairs<4>(m, Lt, invd, w, l, bad);
  cholesky_pairs<5>(m, Lt, invd, w, l, bad);
  cholesky_pairs<6>(m, Lt, invd, w, l, bad);
  cholesky_pairs<7>(m, Lt, invd, w, l, bad);
  if (bad && l == 0) flag_status(a.status, CURDKV_DEV_NOT_SPD);

  // ---- back substitution L^T W = G, last row first, 32 columns of G per pass
  int tb[4];
#pragma unroll
  for (int u = 0; u < 4; ++u) tb[u] = tri_base(l + 32 * u);
  const int passes = (r + kFactorPass - 1) / kFactorPass;
  for (int pass = 0; pass < passes; ++pass) {
    double x[4][4];
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int col = kFactorPass * pass + 4 * w + c;
        x[u][c] = col < r ? (double)__ldg(a.G + (size_t)(l + 32 * u) * r + col) : 0.0;
      }
    __syncthreads();                                       // L complete; Wt of the previous pass stored
    backsub_steps<3>(x, tb, Lt, Wt, invd, w, l);
    backsub_steps<2>(x, tb, Lt, Wt, invd, w, l);
    backsub_steps<1>(x, tb, Lt, Wt, invd, w, l);
    backsub_steps<0>(x, tb, Lt, Wt, invd, w, l);
    __syncthreads();
    const int width = min(kFactorPass, r - kFactorPass * pass);
    for (int e = tid; e < D * width; e += kFactorThreads) {
      const int i = e / width, cc = e % width;
      out[(size_t)i * r + kFactorPass * pass + cc] = (float)Wt[i * kFactorPass + cc];
    }
  }
}

}  // namespace curdkv
