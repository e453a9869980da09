// Whitening factors of the leverage-score sketch: for one (sequence, head) and
// one tensor, sums the partial Gram matrices of its segments in a fixed order,
// adds the ridge, factors M = L L^T and solves L^T W = G, all in fp64 (the Gram
// matrix squares the conditioning of K or V).  Writes W as fp32 [128][r].
//
// One CTA of 1024 threads per matrix.  The matrix lives in registers, spread
// 2-D cyclically: thread (ti, tj) = (tid / 32, tid % 32) owns the elements
// (ti + 32u, tj + 32v), u, v < 4.  Each elimination step publishes one column
// through shared memory and costs one barrier; the published columns are the
// (unscaled) factor, which the back substitution then reads from shared memory.
#pragma once
#include "common.cuh"

namespace curdkv {

constexpr int kFactorThreads = 1024;
constexpr int kFactorD = 128;
constexpr size_t kFactorSmemBytes = ((size_t)kFactorD * kFactorD + 2 * 64) * sizeof(double);

struct FactorArgs {
  const float* partials;   // [batch*heads*segments][2][128][128]
  const float* G;          // [128][r]
  float* W;                // [batch*heads][2][128][r]
  int segments, r;         // r <= 64
  double ridge;
  uint32_t* status;
};

// Elimination steps k = 32*KU .. 32*KU + 31: only the blocks u, v >= KU still change, so the
// phase is compiled for exactly those (no selects on the block index, no work on finished blocks).
template <int KU>
__device__ __forceinline__ void cholesky_phase(double (&m)[4][4], double* Lt, int ti, int tj, bool& bad) {
  constexpr int D = kFactorD;
#pragma unroll 1
  for (int kt = 0; kt < 32; ++kt) {
    const int k = 32 * KU + kt;
    if (tj == kt) {                                        // owners publish column k, pivot included
#pragma unroll
      for (int u = KU; u < 4; ++u) Lt[k * D + ti + 32 * u] = m[u][KU];
    }
    __syncthreads();
    double piv = Lt[k * D + k];
    if (!(piv > 0.0)) { piv = 1e-300; bad = true; }
    // 1 / piv: fp32 seed and two Newton steps; out-of-range pivots take the exact division
    double inv;
    if (piv > 1e-30 && piv < 1e30) {
      inv = (double)(1.0f / (float)piv);
      inv = inv * (2.0 - piv * inv);
      inv = inv * (2.0 - piv * inv);
    } else {
      inv = 1.0 / piv;
    }
    double li[4], lj[4];
#pragma unroll
    for (int u = KU; u < 4; ++u) {
      li[u] = Lt[k * D + ti + 32 * u] * inv;
      lj[u] = Lt[k * D + tj + 32 * u];
    }
    if (ti <= kt) li[KU] = 0.0;                            // rows and columns up to k are finished
    if (tj <= kt) lj[KU] = 0.0;
#pragma unroll
    for (int u = KU; u < 4; ++u)
#pragma unroll
      for (int v = KU; v < 4; ++v) m[u][v] -= li[u] * lj[v];
  }
}

// Back-substitution steps i = 32*IU + 31 .. 32*IU: only rows of blocks u <= IU are still open.
template <int IU, int WCOLS>
__device__ __forceinline__ void backsub_phase(double (&x)[4][2], const double* Lt, double* wrow, int ti,
                                              int tj) {
  constexpr int D = kFactorD;
#pragma unroll 1
  for (int it = 31; it >= 0; --it) {
    const int i = 32 * IU + it;
    double* wr = wrow + (i & 1) * 64;
    if (ti == it) {
      const double inv = 1.0 / Lt[i * D + i];
#pragma unroll
      for (int w = 0; w < WCOLS; ++w) {
        x[IU][w] *= inv;                                   // W[i][c]
        wr[tj + 32 * w] = x[IU][w];
      }
    }
    __syncthreads();
    double wv[2];
#pragma unroll
    for (int w = 0; w < WCOLS; ++w) wv[w] = wr[tj + 32 * w];
#pragma unroll
    for (int u = 0; u <= IU; ++u) {
      const int row = ti + 32 * u;
      if (u < IU || ti < it) {
        const double l = Lt[row * D + i];                  // L[i][row]
#pragma unroll
        for (int w = 0; w < WCOLS; ++w) x[u][w] -= l * wv[w];
      }
    }
  }
}

template <int WCOLS>
__device__ __forceinline__ void backsub_all(double (&x)[4][2], const double* Lt, double* wrow, int ti, int tj) {
  backsub_phase<3, WCOLS>(x, Lt, wrow, ti, tj);
  backsub_phase<2, WCOLS>(x, Lt, wrow, ti, tj);
  backsub_phase<1, WCOLS>(x, Lt, wrow, ti, tj);
  backsub_phase<0, WCOLS>(x, Lt, wrow, ti, tj);
}

// grid = batch*heads*2, block = 1024, dynamic shared memory = kFactorSmemBytes.
__global__ void __launch_bounds__(kFactorThreads, 1) whiten_factor_kernel(const FactorArgs a) {
  extern __shared__ double fsm[];
  constexpr int D = kFactorD;
  double* Lt = fsm;                    // Lt[k*D + i] = L[i][k]
  double* wrow = fsm + D * D;          // two rows of up to 64 solved values
  __shared__ double red[kFactorThreads / 32];
  __shared__ double s_trace;
  const int tid = threadIdx.x, ti = tid >> 5, tj = tid & 31;
  const int p = blockIdx.x >> 1, tensor = blockIdx.x & 1;
  const int r = a.r;

  // ---- M = sum of the segments' partial Gram matrices (segment order); both (i, j) and (j, i)
  // are read from the lower triangle so that the matrix is symmetric to the last bit
  double m[4][4];
  double tr = 0.0;
#pragma unroll
  for (int u = 0; u < 4; ++u) {
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      const int i = ti + 32 * u, j = tj + 32 * v;
      const int hi = max(i, j), lo = min(i, j);
      double s = 0.0;
      for (int g = 0; g < a.segments; ++g)
        s += (double)__ldg(a.partials + (((size_t)p * a.segments + g) * 2 + tensor) * D * D + hi * D + lo);
      m[u][v] = s;
      if (i == j) tr += s;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) tr += __shfl_xor_sync(0xffffffffu, tr, o);
  if (tj == 0) red[ti] = tr;
  __syncthreads();
  if (tid == 0) {
    double t = 0.0;
    for (int w = 0; w < kFactorThreads / 32; ++w) t += red[w];
    s_trace = t;
  }
  __syncthreads();
  float* out = a.W + ((size_t)p * 2 + tensor) * D * r;
  if (!(s_trace > 0.0)) {                                  // no valid rows (or all zero): nothing to whiten
    for (int e = tid; e < D * r; e += kFactorThreads) out[e] = 0.f;
    return;
  }
  const double lambda = a.ridge * s_trace / D;
#pragma unroll
  for (int u = 0; u < 4; ++u)
    if (ti == tj) m[u][u] += lambda;

  // ---- Cholesky by outer products: step k publishes column k (unscaled, pivot included) and
  // every thread updates its elements below and right of it: m_ij -= m_ik m_jk / m_kk
  bool bad = false;
  cholesky_phase<0>(m, Lt, ti, tj, bad);
  cholesky_phase<1>(m, Lt, ti, tj, bad);
  cholesky_phase<2>(m, Lt, ti, tj, bad);
  cholesky_phase<3>(m, Lt, ti, tj, bad);
  if (bad && tid == 0) flag_status(a.status, CURDKV_DEV_NOT_SPD);
  __syncthreads();
  // scale the published columns: L[i][k] = m_ik / sqrt(m_kk), L[k][k] = sqrt(m_kk)
  for (int e = tid; e < D * D; e += kFactorThreads) {
    const int k = e / D, i = e % D;
    const double piv = Lt[k * D + k];
    if (i > k) Lt[e] *= rsqrt(piv > 0.0 ? piv : 1e-300);
  }
  __syncthreads();
  if (tid < D) {
    const double piv = Lt[tid * D + tid];
    Lt[tid * D + tid] = sqrt(piv > 0.0 ? piv : 1e-300);
  }

  // ---- back substitution L^T W = G, last row first.  x[u][w] holds row ti + 32u, column tj + 32w.
  double x[4][2];
#pragma unroll
  for (int u = 0; u < 4; ++u)
#pragma unroll
    for (int w = 0; w < 2; ++w) {
      const int c = tj + 32 * w;
      x[u][w] = c < r ? (double)__ldg(a.G + (size_t)(ti + 32 * u) * r + c) : 0.0;
    }
  __syncthreads();
  if (r > 32) backsub_all<2>(x, Lt, wrow, ti, tj);
  else backsub_all<1>(x, Lt, wrow, ti, tj);
#pragma unroll
  for (int u = 0; u < 4; ++u)
#pragma unroll
    for (int w = 0; w < 2; ++w) {
      const int c = tj + 32 * w;
      if (c < r) out[(size_t)(ti + 32 * u) * r + c] = (float)x[u][w];
    }
}

}  // namespace curdkv
