// Whitening factors of the leverage-score sketch: for one (sequence, head) and
// one tensor, sums the partial Gram matrices of its segments in a fixed order,
// adds the ridge, factors M = L L^T and solves L^T W = G, all in fp64 (the Gram
// matrix squares the conditioning of K or V).  Writes W as fp32 [128][r].
//
// One CTA of 1024 threads per matrix, and no CTA-wide barrier inside the two
// sequential loops: both run as a dataflow over shared memory.
//  * Factorisation.  Warp w owns the columns w, w + 32, w + 64, w + 96 of the
//    lower triangle; lane l holds their rows l + 32u in registers (ten values per
//    thread, blocks on or below the diagonal).  Column k is published (unscaled,
//    pivot included) to shared memory by its warp, which then arrives on the
//    column's own mbarrier; every warp waits for that mbarrier before it applies
//    column k to its columns.  The warp that owns column k + 1 updates and
//    publishes that column first and its other columns afterwards, so the chain
//    column k -> column k + 1 is one warp's short path and the bulk of the
//    rank-1 update runs behind it.
//  * Back substitution.  Warp w owns the rows w + 32u of the solution, lane l its
//    column l (and l + 32 when r > 32).  Row i is published through shared memory
//    and a per-row mbarrier in the same way, the owner of row i - 1 going first.
// Every wait is bounded: on expiry the CTA stops waiting, finishes (with a wrong
// result) and raises the time-out bit of the device status word.
#pragma once
#include "common.cuh"
#include "score_umma.cuh"

namespace curdkv {

constexpr int kFactorThreads = 1024;
constexpr int kFactorD = 128;
constexpr int kFactorWCols = 64;                           // r <= 64
// dynamic shared memory: published columns, solved rows, 1 / L[i][i], two mbarriers per index, abort flag
constexpr size_t kFactorOffW = (size_t)kFactorD * kFactorD * sizeof(double);
constexpr size_t kFactorOffInv = kFactorOffW + (size_t)kFactorD * kFactorWCols * sizeof(double);
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
  __device__ __forceinline__ void publish_col(int k) const { umma::mbar_arrive(col_bar + 8u * (uint32_t)k); }
  __device__ __forceinline__ void wait_row(int i) const {
    umma::mbar_wait(row_bar + 8u * (uint32_t)i, 0u, abort_flag, status);
  }
  __device__ __forceinline__ void publish_row(int i) const { umma::mbar_arrive(row_bar + 8u * (uint32_t)i); }
};

// 1 / piv: fp32 seed and two Newton steps; out-of-range pivots take the exact division.
__device__ __forceinline__ double pivot_reciprocal(double piv) {
  if (piv > 1e-30 && piv < 1e30) {
    double inv = (double)(1.0f / (float)piv);
    inv = inv * (2.0 - piv * inv);
    return inv * (2.0 - piv * inv);
  }
  return 1.0 / piv;
}

// The warp that owns column k = w + 32V writes it to shared memory twice: as it is (pivot
// included; this becomes the factor) and divided by the pivot (the multipliers of step k, kept
// only until every warp has passed that step: a ring of 64 columns is enough, because a column
// is published only after all earlier ones, and each of the 32 warps publishes one column out
// of any 32 consecutive ones after it has applied every column before it).
template <int V>
__device__ __forceinline__ void publish_column(const double (&m)[4][4], int k, double* Lt, double* ring,
                                               const FactorSync& sync, int l, bool& bad) {
  constexpr int D = kFactorD;
  double piv = __shfl_sync(0xffffffffu, m[V][V], k & 31);
  if (!(piv > 0.0)) { piv = 1e-300; bad = true; }
  const double inv = pivot_reciprocal(piv);
  double* scaled = ring + (k & 63) * D;
#pragma unroll
  for (int u = V; u < 4; ++u) {
    Lt[k * D + l + 32 * u] = m[u][V];
    scaled[l + 32 * u] = m[u][V] * inv;
  }
  sync.publish_col(k);
}

// Elimination steps k = 32*KU .. 32*KU + 31: only the blocks u >= v >= KU still change, so the
// phase is compiled for exactly those (no selects on the block index, no work on finished blocks).
// m[u][v] is the element (l + 32u, w + 32v); only u >= v is held.
template <int KU>
__device__ __forceinline__ void cholesky_phase(double (&m)[4][4], double* Lt, double* ring,
                                               const FactorSync& sync, int w, int l, bool& bad) {
  constexpr int D = kFactorD;
#pragma unroll 1
  for (int kt = 0; kt < 32; ++kt) {
    const int k = 32 * KU + kt;
    sync.wait_col(k);
    const double* scaled = ring + (k & 63) * D;
    double li[4], lj[4];
#pragma unroll
    for (int u = KU; u < 4; ++u) {
      li[u] = Lt[k * D + l + 32 * u];                      // m_ik of this lane's rows
      lj[u] = scaled[w + 32 * u];                          // m_jk / m_kk of this warp's columns
    }
    if (l <= kt) li[KU] = 0.0;                             // rows and columns up to k are finished
    if (w <= kt) lj[KU] = 0.0;
    // the owner of column k + 1 brings it up to date and publishes it before anything else
    const int kn = k + 1;
    const bool owner_next = kn < D && (kn & 31) == w;
    const bool next_block = kt == 31;                      // column k + 1 opens the next block
    if (owner_next) {
      if (!next_block) {
#pragma unroll
        for (int u = KU; u < 4; ++u) m[u][KU] -= li[u] * lj[KU];
        publish_column<KU>(m, kn, Lt, ring, sync, l, bad);
      } else if constexpr (KU < 3) {
#pragma unroll
        for (int u = KU + 1; u < 4; ++u) m[u][KU + 1] -= li[u] * lj[KU + 1];
        publish_column<KU + 1>(m, kn, Lt, ring, sync, l, bad);
      }
    }
#pragma unroll
    for (int v = KU; v < 4; ++v) {
      if (!(owner_next && v == (next_block ? KU + 1 : KU))) {
#pragma unroll
        for (int u = v; u < 4; ++u) m[u][v] -= li[u] * lj[v];
      }
    }
  }
}

// Back-substitution steps i = 32*IU + 31 .. 32*IU: only rows of blocks u <= IU are still open.
// x[u][c] is the element (w + 32u, l + 32c) of the right-hand side / solution.
template <int IU, int WCOLS>
__device__ __forceinline__ void backsub_phase(double (&x)[4][2], const double* Lt, double* Wt,
                                              const double* invd, const FactorSync& sync, int w, int l) {
  constexpr int D = kFactorD;
#pragma unroll 1
  for (int it = 31; it >= 0; --it) {
    const int i = 32 * IU + it;
    sync.wait_row(i);
    double wv[2];
#pragma unroll
    for (int c = 0; c < WCOLS; ++c) wv[c] = Wt[i * kFactorWCols + l + 32 * c];
    // the owner of row i - 1 finishes and publishes it before anything else
    const int in = i - 1, un = in >> 5;
    const bool owner_next = in >= 0 && (in & 31) == w;
    if (owner_next) {
#pragma unroll
      for (int u = 0; u <= IU; ++u) {
        if (u == un) {
          const double lv = Lt[in * D + i], dinv = invd[in];   // L[i][i-1], 1 / L[i-1][i-1]
#pragma unroll
          for (int c = 0; c < WCOLS; ++c) {
            x[u][c] = (x[u][c] - lv * wv[c]) * dinv;
            Wt[in * kFactorWCols + l + 32 * c] = x[u][c];
          }
        }
      }
      sync.publish_row(in);
    }
#pragma unroll
    for (int u = 0; u <= IU; ++u) {
      const int row = w + 32 * u;
      if ((u < IU || w < it) && !(owner_next && u == un)) {
        const double lv = Lt[row * D + i];                 // L[i][row]
#pragma unroll
        for (int c = 0; c < WCOLS; ++c) x[u][c] -= lv * wv[c];
      }
    }
  }
}

template <int WCOLS>
__device__ __forceinline__ void backsub_all(double (&x)[4][2], const double* Lt, double* Wt, const double* invd,
                                            const FactorSync& sync, int w, int l) {
  backsub_phase<3, WCOLS>(x, Lt, Wt, invd, sync, w, l);
  backsub_phase<2, WCOLS>(x, Lt, Wt, invd, sync, w, l);
  backsub_phase<1, WCOLS>(x, Lt, Wt, invd, sync, w, l);
  backsub_phase<0, WCOLS>(x, Lt, Wt, invd, sync, w, l);
}

// grid = batch*heads*2, block = 1024, dynamic shared memory = kFactorSmemBytes.
__global__ void __launch_bounds__(kFactorThreads, 1) whiten_factor_kernel(const FactorArgs a) {
  extern __shared__ __align__(16) unsigned char fsm[];
  constexpr int D = kFactorD;
  double* Lt = reinterpret_cast<double*>(fsm);                       // Lt[k*D + i] = L[i][k], i >= k
  // Wt[i*64 + c] = W[i][c]; during the factorisation, the ring of scaled columns
  double* Wt = reinterpret_cast<double*>(fsm + kFactorOffW);
  double* invd = reinterpret_cast<double*>(fsm + kFactorOffInv);     // 1 / L[i][i]
  volatile int* abort_flag = reinterpret_cast<volatile int*>(fsm + kFactorOffAbort);
  __shared__ double red[kFactorThreads / 32];
  __shared__ double s_trace;
  const int tid = threadIdx.x, w = tid >> 5, l = tid & 31;
  const int p = blockIdx.x >> 1, tensor = blockIdx.x & 1;
  const int r = a.r;
  const FactorSync sync{umma::smem_u32(fsm + kFactorOffColBar), umma::smem_u32(fsm + kFactorOffRowBar),
                        abort_flag, a.status};
  if (tid < D) {                                           // every lane of the owning warp arrives
    umma::mbar_init(sync.col_bar + 8u * (uint32_t)tid, 32);
    umma::mbar_init(sync.row_bar + 8u * (uint32_t)tid, 32);
  }
  if (tid == 0) *abort_flag = 0;
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");

  // ---- M = sum of the segments' partial Gram matrices (segment order).  Element (i, j), i >= j,
  // is taken from row j of the stored matrix, so that a warp reads along a row; the part of a
  // diagonal block above the diagonal mirrors the part below it.
  double m[4][4];
  double tr = 0.0;
#pragma unroll
  for (int v = 0; v < 4; ++v) {
#pragma unroll
    for (int u = v; u < 4; ++u) {
      const int i = l + 32 * u, j = w + 32 * v;
      const int hi = max(i, j), lo = min(i, j);
      double s = 0.0;
      for (int g = 0; g < a.segments; ++g)
        s += (double)__ldg(a.partials + (((size_t)p * a.segments + g) * 2 + tensor) * D * D + lo * D + hi);
      m[u][v] = s;
      if (i == j) tr += s;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) tr += __shfl_xor_sync(0xffffffffu, tr, o);
  if (l == 0) red[w] = tr;
  __syncthreads();
  if (tid == 0) {
    double t = 0.0;
    for (int q = 0; q < kFactorThreads / 32; ++q) t += red[q];
    s_trace = t;
  }
  __syncthreads();
  float* out = a.W + ((size_t)p * 2 + tensor) * D * r;
  if (!(s_trace > 0.0)) {                                  // no valid rows (or all zero): nothing to whiten
    for (int e = tid; e < D * r; e += kFactorThreads) out[e] = 0.f;
    return;
  }
  const double lambda = a.ridge * s_trace / D;
  if (l == w) {
#pragma unroll
    for (int u = 0; u < 4; ++u) m[u][u] += lambda;
  }

  // ---- Cholesky by outer products: column k is published unscaled (pivot included) and every
  // thread updates its elements below and right of it: m_ij -= m_ik m_jk / m_kk
  bool bad = false;
  if (w == 0) publish_column<0>(m, 0, Lt, Wt, sync, l, bad);
  cholesky_phase<0>(m, Lt, Wt, sync, w, l, bad);
  cholesky_phase<1>(m, Lt, Wt, sync, w, l, bad);
  cholesky_phase<2>(m, Lt, Wt, sync, w, l, bad);
  cholesky_phase<3>(m, Lt, Wt, sync, w, l, bad);
  if (bad && l == 0) flag_status(a.status, CURDKV_DEV_NOT_SPD);
  __syncthreads();
  // scale the published columns: L[i][k] = m_ik / sqrt(m_kk), L[k][k] = sqrt(m_kk)
  double piv = 0.0;
  if (tid < D) {
    piv = Lt[tid * D + tid];
    piv = piv > 0.0 ? piv : 1e-300;
    invd[tid] = rsqrt(piv);                                // 1 / L[k][k]
  }
  __syncthreads();
  for (int e = tid; e < D * D; e += kFactorThreads) {
    const int k = e / D, i = e % D;
    if (i > k) Lt[e] *= invd[k];
  }
  if (tid < D) Lt[tid * D + tid] = sqrt(piv);

  // ---- back substitution L^T W = G, last row first
  double x[4][2];
#pragma unroll
  for (int u = 0; u < 4; ++u)
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      const int col = l + 32 * c;
      x[u][c] = col < r ? (double)__ldg(a.G + (size_t)(w + 32 * u) * r + col) : 0.0;
    }
  __syncthreads();
  if (w == 31) {                                           // row 127 has nothing to subtract
    const double dinv = invd[D - 1];
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      x[3][c] *= dinv;
      Wt[(D - 1) * kFactorWCols + l + 32 * c] = x[3][c];
    }
    sync.publish_row(D - 1);
  }
  if (r > 32) backsub_all<2>(x, Lt, Wt, invd, sync, w, l);
  else backsub_all<1>(x, Lt, Wt, invd, sync, w, l);
  __syncthreads();
  for (int e = tid; e < D * r; e += kFactorThreads) out[e] = (float)Wt[(e / r) * kFactorWCols + e % r];
}

}  // namespace curdkv
