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
#pragma unroll 1
  for (int k = 0; k < D; ++k) {
    const int ku = k >> 5, kt = k & 31;
    if (tj == kt) {
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        double c = 0.0;
#pragma unroll
        for (int v = 0; v < 4; ++v)
          if (v == ku) c = m[u][v];
        Lt[k * D + ti + 32 * u] = c;
      }
    }
    __syncthreads();
    double piv = Lt[k * D + k];
    if (!(piv > 0.0)) { piv = 1e-300; bad = true; }
    // 1 / piv: fp32 seed and two Newton steps (an fp64 division in every thread and step would
    // cost as much as the update itself); out-of-range pivots take the exact division
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
    for (int u = 0; u < 4; ++u) {
      li[u] = ti + 32 * u > k ? Lt[k * D + ti + 32 * u] * inv : 0.0;
      lj[u] = tj + 32 * u > k ? Lt[k * D + tj + 32 * u] : 0.0;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
      for (int v = 0; v < 4; ++v) m[u][v] -= li[u] * lj[v];
  }
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
#pragma unroll 1
  for (int i = D - 1; i >= 0; --i) {
    const int iu = i >> 5, it = i & 31;
    double* wr = wrow + (i & 1) * 64;
    if (ti == it) {
      const double inv = 1.0 / Lt[i * D + i];
#pragma unroll
      for (int w = 0; w < 2; ++w) {
        double v = 0.0;
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (u == iu) v = x[u][w];
        v *= inv;
        wr[tj + 32 * w] = v;
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (u == iu) x[u][w] = v;                        // W[i][c]
      }
    }
    __syncthreads();
    const double w0 = wr[tj], w1 = wr[tj + 32];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int row = ti + 32 * u;
      if (row < i) {
        const double l = Lt[row * D + i];                  // L[i][row]
        x[u][0] -= l * w0;
        x[u][1] -= l * w1;
      }
    }
  }
#pragma unroll
  for (int u = 0; u < 4; ++u)
#pragma unroll
    for (int w = 0; w < 2; ++w) {
      const int c = tj + 32 * w;
      if (c < r) out[(size_t)(ti + 32 * u) * r + c] = (float)x[u][w];
    }
}

}  // namespace curdkv
