// Whitening factors of the leverage-score sketch: for one (sequence, head) and
// one tensor, sums the partial Gram matrices of its segments in a fixed order,
// adds the ridge, factors M = L L^T and solves L^T W = G, all in fp64 (the Gram
// matrix squares the conditioning of K or V).  Writes W as fp32 [128][r].
//
// One CTA of 256 threads per matrix, two CTAs per SM.  The kernel is bound by
// instruction issue and by the chain of 2 x 128 dependent steps, so each thread
// holds a large register tile (few warps repeat the per-step bookkeeping) and no
// CTA-wide barrier sits inside the two sequential loops: both run as a dataflow
// over shared memory.
//  * Factorisation.  Warp w owns the columns w, w + 8, ... of the lower triangle;
//    lane l holds their rows l + 32u in registers (40 values per thread: the
//    32 x 8 blocks on or below the diagonal).  Column k of L is written to shared
//    memory (packed lower triangle) by its warp, which then arrives on the
//    column's own mbarrier; every warp waits for that mbarrier before it applies
//    column k to its columns.  The warp that owns column k + 1 updates and
//    publishes that column first and its other columns afterwards, so the chain
//    column k -> column k + 1 is one warp's short path and the bulk of the
//    rank-1 update runs behind it.
//  * Back substitution, 32 right-hand sides at a time.  Lane l holds the rows
//    l + 32u of the solution, warp w their columns 4w .. 4w + 3.  Row i is
//    published through shared memory and a per-row mbarrier in the same way: the
//    lane that holds row i - 1 finishes it first, in every warp.
// Every wait is bounded: on expiry the CTA stops waiting, finishes (with a wrong
// result) and raises the time-out bit of the device status word.
#pragma once
#include "common.cuh"
#include "score_umma.cuh"

namespace curdkv {

constexpr int kFactorThreads = 256;
constexpr int kFactorWarps = kFactorThreads / 32;
constexpr int kFactorD = 128;
constexpr int kFactorPass = 32;                            // right-hand sides per back-substitution pass
// dynamic shared memory: L (packed lower triangle, by columns), one pass of solved rows, 1 / L[i][i],
// one mbarrier per column and per row, abort flag
constexpr size_t kFactorOffW = (size_t)kFactorD * (kFactorD + 1) / 2 * sizeof(double);
constexpr size_t kFactorOffInv = kFactorOffW + (size_t)kFactorD * kFactorPass * sizeof(double);
constexpr size_t kFactorOffColBar = kFactorOffInv + kFactorD * sizeof(double);
constexpr size_t kFactorOffRowBar = kFactorOffColBar + kFactorD * sizeof(uint64_t);
constexpr size_t kFactorOffAbort = kFactorOffRowBar + kFactorD * sizeof(uint64_t);
constexpr size_t kFactorSmemBytes = kFactorOffAbort + 16;

struct FactorArgs {
  const float* partials;   // [batch*heads*segments][2][128][128]
  const float* G;          // [128][r]
  float* W;                // [batch*heads][2][128][r]
  int segments, r;         // r <= 64
  double ridge;
  uint32_t* status;
};

struct FactorSync {
  uint32_t col_bar, row_bar;                               // shared-memory addresses of the mbarrier arrays
  volatile int* abort_flag;
  uint32_t* status;
  __device__ __forceinline__ void wait_col(int k) const {
    umma::mbar_wait(col_bar + 8u * (uint32_t)k, 0u, abort_flag, status);
  }
  // called by a whole warp after its stores: one arrival per warp
  __device__ __forceinline__ void publish_col(int k) const {
    __syncwarp();
    if ((threadIdx.x & 31) == 0) umma::mbar_arrive(col_bar + 8u * (uint32_t)k);
  }
  __device__ __forceinline__ void wait_row(int i, uint32_t pass) const {
    umma::mbar_wait(row_bar + 8u * (uint32_t)i, pass, abort_flag, status);
  }
  // called by the one lane of a warp that holds row i, after it has stored its part of the row
  __device__ __forceinline__ void publish_row_part(int i) const { umma::mbar_arrive(row_bar + 8u * (uint32_t)i); }
};

// Column k of the packed triangle holds rows k .. 127; the returned offset already has k
// subtracted, so that row i of column k is element tri_base(k) + i.
__device__ __forceinline__ int tri_base(int k) { return k * (kFactorD - 1) - ((k * (k - 1)) >> 1); }

// piv^(-1/2): fp32 seed and two Newton steps; out-of-range pivots take the library routine.
__device__ __forceinline__ double pivot_rsqrt(double piv) {
  if (piv > 1e-30 && piv < 1e30) {
    double y = (double)rsqrtf((float)piv);
    const double h = 0.5 * piv;
    y = y * fma(-(h * y), y, 1.5);
    return y * fma(-(h * y), y, 1.5);
  }
  return rsqrt(piv);
}

// m[u][v] is the element (l + 32u, w + 8v) of the matrix being eliminated; only the blocks on or
// below the diagonal (u >= v / 4) are held.
//
// The warp that owns column k = w + 8V scales it by the inverse root of its pivot and writes the
// rows k .. 127 (column k of L) to shared memory.
template <int V>
__device__ __forceinline__ void publish_column(const double (&m)[4][16], int k, double* Lt, double* invd,
                                               const FactorSync& sync, int l, bool& bad) {
  constexpr int U = V / 4;
  double piv = __shfl_sync(0xffffffffu, m[U][V], k & 31);
  if (!(piv > 0.0)) { piv = 1e-300; bad = true; }
  const double rs = pivot_rsqrt(piv);
  double* col = Lt + tri_base(k);
#pragma unroll
  for (int u = U; u < 4; ++u) {
    const int i = l + 32 * u;
    if (i >= k) col[i] = m[u][V] * rs;
  }
  if (l == (k & 31)) invd[k] = rs;                         // 1 / L[k][k]
  sync.publish_col(k);
}

// m[.][V] -= L[.][k] L[j][k] for this warp's column j = w + 8V.  MASK: the column may be finished
// (j <= k), in which case nothing is subtracted.
template <int V, bool MASK>
__device__ __forceinline__ void apply_column(double (&m)[4][16], const double (&li)[4], const double* col, int k,
                                             int w) {
  const int j = w + 8 * V;
  double lj = col[j];                                      // one value for the whole warp
  if (MASK && j <= k) lj = 0.0;
#pragma unroll
  for (int u = V / 4; u < 4; ++u) m[u][V] -= li[u] * lj;
}
template <int V>
__device__ __forceinline__ void apply_from(double (&m)[4][16], const double (&li)[4], const double* col, int k,
                                           int w) {
  if constexpr (V < 16) {
    apply_column<V, false>(m, li, col, k, w);
    apply_from<V + 1>(m, li, col, k, w);
  }
}

// Elimination steps k = 16*KH .. 16*KH + 15: only the columns v >= 2*KH and the row blocks
// u >= KH / 2 still change, so the steps are compiled for exactly those.
template <int KH>
__device__ __forceinline__ void cholesky_steps(double (&m)[4][16], double* Lt, double* invd,
                                               const FactorSync& sync, int w, int l, bool& bad) {
  constexpr int D = kFactorD, V0 = 2 * KH, U0 = KH / 2;
#pragma unroll 1
  for (int kt = 0; kt < 16; ++kt) {
    const int k = 16 * KH + kt;
    sync.wait_col(k);
    const double* col = Lt + tri_base(k);
    double li[4];
#pragma unroll
    for (int u = U0; u < 4; ++u) li[u] = col[l + 32 * u];  // rows above k read a neighbouring column: masked
    if (l + 32 * U0 <= k) li[U0] = 0.0;                    // rows up to k are finished
    // the owner of column k + 1 brings it up to date and publishes it before anything else
    const int kn = k + 1, vn = kn >> 3;                    // vn is V0, V0 + 1 or (last step) V0 + 2
    const bool owner_next = kn < D && (kn & 7) == w;
    if (owner_next) {
      if (vn == V0) {
        apply_column<V0, true>(m, li, col, k, w);
        publish_column<V0>(m, kn, Lt, invd, sync, l, bad);
      } else if (vn == V0 + 1) {
        apply_column<V0 + 1, true>(m, li, col, k, w);
        publish_column<V0 + 1>(m, kn, Lt, invd, sync, l, bad);
      } else if constexpr (V0 + 2 < 16) {
        apply_column<V0 + 2, false>(m, li, col, k, w);
        publish_column<V0 + 2>(m, kn, Lt, invd, sync, l, bad);
      }
    }
    // (the owner applies column k to the column it has just published once more: those registers are dead)
    apply_column<V0, true>(m, li, col, k, w);
    apply_column<V0 + 1, true>(m, li, col, k, w);
    apply_from<V0 + 2>(m, li, col, k, w);
  }
}

// Back-substitution steps i = 32*IU + 31 .. 32*IU of one pass: only the rows of the blocks
// u <= IU are still open.  x[u][c] is the element (l + 32u, column 4w + c of the pass) of the
// right-hand side / solution; tb[u] = tri_base(l + 32u).  Row i - 1 sits in one lane of every
// warp: that lane finishes and publishes its four columns before the warp does anything else.
template <int IU>
__device__ __forceinline__ void backsub_steps(double (&x)[4][4], const int (&tb)[4], const double* Lt,
                                              double* Wt, const double* invd, const FactorSync& sync,
                                              uint32_t pass, int w, int l) {
#pragma unroll 1
  for (int it = 31; it >= 0; --it) {
    const int i = 32 * IU + it;
    sync.wait_row(i, pass);
    const double2 w01 = *reinterpret_cast<const double2*>(Wt + i * kFactorPass + 4 * w);
    const double2 w23 = *reinterpret_cast<const double2*>(Wt + i * kFactorPass + 4 * w + 2);
    const double wv[4] = {w01.x, w01.y, w23.x, w23.y};
    const int in = i - 1;
    if (in >= 0 && l == (in & 31)) {
      const double lv = Lt[tri_base(in) + i], dinv = invd[in];   // L[i][i-1], 1 / L[i-1][i-1]
      double o[4];
      if (it > 0) {
#pragma unroll
        for (int c = 0; c < 4; ++c) o[c] = (x[IU][c] - lv * wv[c]) * dinv;
      } else if constexpr (IU > 0) {
#pragma unroll
        for (int c = 0; c < 4; ++c) o[c] = (x[IU - 1][c] - lv * wv[c]) * dinv;
      }
      double* dst = Wt + in * kFactorPass + 4 * w;
      *reinterpret_cast<double2*>(dst) = make_double2(o[0], o[1]);
      *reinterpret_cast<double2*>(dst + 2) = make_double2(o[2], o[3]);
      sync.publish_row_part(in);
    }
#pragma unroll
    for (int u = 0; u <= IU; ++u) {                        // (a row just published is dead in x)
      if (u < IU || l < it) {
        const double lv = Lt[tb[u] + i];                   // L[i][row]
#pragma unroll
        for (int c = 0; c < 4; ++c) x[u][c] -= lv * wv[c];
      }
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
  volatile int* abort_flag = reinterpret_cast<volatile int*>(fsm + kFactorOffAbort);
  __shared__ double red[kFactorWarps];
  const int tid = threadIdx.x, w = tid >> 5, l = tid & 31;
  const int p = blockIdx.x >> 1, tensor = blockIdx.x & 1;
  const int r = a.r;
  const FactorSync sync{umma::smem_u32(fsm + kFactorOffColBar), umma::smem_u32(fsm + kFactorOffRowBar),
                        abort_flag, a.status};
  if (tid < D) {                                           // one arrival: the owning warp's
    umma::mbar_init(sync.col_bar + 8u * (uint32_t)tid, 1);
    umma::mbar_init(sync.row_bar + 8u * (uint32_t)tid, kFactorWarps);   // a row is spread over all warps
  }
  if (tid == 0) *abort_flag = 0;
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");

  // ---- M = sum of the segments' partial Gram matrices (segment order).  Element (i, j), i >= j,
  // is taken from row j of the stored matrix, so that a warp reads along a row; the part of a
  // diagonal block above the diagonal mirrors the part below it.
  double m[4][16];
#pragma unroll
  for (int v = 0; v < 16; ++v)
#pragma unroll
    for (int u = v / 4; u < 4; ++u) m[u][v] = 0.0;
  for (int g = 0; g < a.segments; ++g) {
    const float* src = a.partials + (((size_t)p * a.segments + g) * 2 + tensor) * D * D;
#pragma unroll
    for (int v = 0; v < 16; ++v) {
#pragma unroll
      for (int u = v / 4; u < 4; ++u) {
        const int i = l + 32 * u, j = w + 8 * v;
        m[u][v] += (double)__ldg(src + min(i, j) * D + max(i, j));
      }
    }
  }
  double tr = 0.0;
#pragma unroll
  for (int v = 0; v < 16; ++v)
    if (l + 32 * (v / 4) == w + 8 * v) tr += m[v / 4][v];  // diagonal elements sit in the blocks u = v / 4
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
    if (l + 32 * (v / 4) == w + 8 * v) m[v / 4][v] += lambda;

  // ---- Cholesky by outer products: column k of L is published as soon as columns 0 .. k-1 have
  // been applied to it, and every thread subtracts L_ik L_jk from its elements right of it
  bool bad = false;
  if (w == 0) publish_column<0>(m, 0, Lt, invd, sync, l, bad);
  cholesky_steps<0>(m, Lt, invd, sync, w, l, bad);
  cholesky_steps<1>(m, Lt, invd, sync, w, l, bad);
  cholesky_steps<2>(m, Lt, invd, sync, w, l, bad);
  cholesky_steps<3>(m, Lt, invd, sync, w, l, bad);
  cholesky_steps<4>(m, Lt, invd, sync, w, l, bad);
  cholesky_steps<5>(m, Lt, invd, sync, w, l, bad);
  cholesky_steps<6>(m, Lt, invd, sync, w, l, bad);
  cholesky_steps<7>(m, Lt, invd, sync, w, l, bad);
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
    if (l == 31) {                                         // row 127 has nothing to subtract
      const double dinv = invd[D - 1];
      double* dst = Wt + (D - 1) * kFactorPass + 4 * w;
      *reinterpret_cast<double2*>(dst) = make_double2(x[3][0] * dinv, x[3][1] * dinv);
      *reinterpret_cast<double2*>(dst + 2) = make_double2(x[3][2] * dinv, x[3][3] * dinv);
      sync.publish_row_part(D - 1);
    }
    backsub_steps<3>(x, tb, Lt, Wt, invd, sync, (uint32_t)pass, w, l);
    backsub_steps<2>(x, tb, Lt, Wt, invd, sync, (uint32_t)pass, w, l);
    backsub_steps<1>(x, tb, Lt, Wt, invd, sync, (uint32_t)pass, w, l);
    backsub_steps<0>(x, tb, Lt, Wt, invd, sync, (uint32_t)pass, w, l);
    __syncthreads();
    const int width = min(kFactorPass, r - kFactorPass * pass);
    for (int e = tid; e < D * width; e += kFactorThreads) {
      const int i = e / width, cc = e % width;
      out[(size_t)i * r + kFactorPass * pass + cc] = (float)Wt[i * kFactorPass + cc];
    }
  }
}

}  // namespace curdkv
