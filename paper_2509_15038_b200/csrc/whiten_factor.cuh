// Whitening factors of the leverage-score sketch: for one (sequence, head) and
// one tensor, sums the partial Gram matrices of its segments in a fixed order,
// adds the ridge, factors M = L L^T and solves L^T W = G, all in fp64 (the Gram
// matrix squares the conditioning of K or V).  Writes W as fp32 [128][r].
#pragma once
#include "common.cuh"

namespace curdkv {

constexpr int kFactorThreads = 256;
constexpr int kFactorD = 128;

struct FactorArgs {
  const float* partials;   // [batch*heads*segments][2][128][128]
  const float* G;          // [128][r]
  float* W;                // [batch*heads][2][128][r]
  int segments, r;
  double ridge;
  uint32_t* status;
};

// Dynamic shared memory: A fp64 [128][129] (lower triangle used, padded rows),
// X fp64 [128][r].  grid = batch*heads*2, block = 256.
__global__ void __launch_bounds__(kFactorThreads) whiten_factor_kernel(const FactorArgs a) {
  extern __shared__ double fsm[];
  constexpr int D = kFactorD, LD = D + 1;
  double* A = fsm;
  double* X = fsm + D * LD;
  __shared__ double red[kFactorThreads / 32];
  __shared__ double s_lambda, s_trace;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int p = blockIdx.x >> 1, tensor = blockIdx.x & 1;
  const int r = a.r;

  // ---- M = sum of the segments' partial Gram matrices (segment order), lower triangle
  double tr = 0.0;
  for (int e = tid; e < D * D; e += kFactorThreads) {
    const int i = e / D, j = e % D;
    if (j > i) continue;
    double m = 0.0;
    for (int s = 0; s < a.segments; ++s)
      m += (double)a.partials[(((size_t)p * a.segments + s) * 2 + tensor) * D * D + e];
    A[i * LD + j] = m;
    if (i == j) tr += m;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) tr += __shfl_xor_sync(0xffffffffu, tr, o);
  if (lane == 0) red[warp] = tr;
  __syncthreads();
  if (tid == 0) {
    double t = 0.0;
    for (int w = 0; w < kFactorThreads / 32; ++w) t += red[w];
    s_lambda = a.ridge * t / D;
    s_trace = t;
  }
  __syncthreads();
  float* out = a.W + ((size_t)p * 2 + tensor) * D * r;
  if (!(s_trace > 0.0)) {                                  // no valid rows (or all zero): nothing to whiten
    for (int e = tid; e < D * r; e += kFactorThreads) out[e] = 0.f;
    return;
  }
  if (tid < D) A[tid * LD + tid] += s_lambda;
  for (int e = tid; e < D * r; e += kFactorThreads) X[e] = (double)a.G[e];
  __syncthreads();

  // ---- Cholesky by outer products.  Column k is final once step k-1 is done, so the trailing
  // update reads it unscaled: A[i][j] -= A[i][k] A[j][k] / A[k][k]; L[i][k] = A[i][k] / sqrt(A[k][k])
  // is formed afterwards.
  for (int k = 0; k < D - 1; ++k) {
    double piv = A[k * LD + k];
    if (!(piv > 0.0)) piv = 1e-300;
    const double inv = 1.0 / piv;
    for (int i = k + 1 + (tid >> 4); i < D; i += kFactorThreads / 16) {   // rows k+1 .. D-1
      const double lik = A[i * LD + k] * inv;
      for (int j = k + 1 + (tid & 15); j <= i; j += 16) A[i * LD + j] -= lik * A[j * LD + k];
    }
    __syncthreads();
  }
  bool bad = false;
  for (int k = tid; k < D; k += kFactorThreads) bad |= !(A[k * LD + k] > 0.0);
  if (bad) flag_status(a.status, CURDKV_DEV_NOT_SPD);
  __syncthreads();
  // X rows are scaled as they are solved; keep the pivots' square roots on the diagonal of A
  for (int e = tid; e < D * D; e += kFactorThreads) {
    const int i = e / D, j = e % D;
    if (j < i) {
      const double piv = A[j * LD + j];
      A[i * LD + j] *= rsqrt(piv > 0.0 ? piv : 1e-300);
    }
  }
  __syncthreads();
  if (tid < D) {
    const double piv = A[tid * LD + tid];
    A[tid * LD + tid] = sqrt(piv > 0.0 ? piv : 1e-300);
  }
  __syncthreads();

  // ---- back substitution L^T W = G, row D-1 first: W[i] = X[i] / L[i][i], then
  // X[m] -= L[i][m] W[i] for every m < i
  for (int i = D - 1; i >= 0; --i) {
    const double inv = 1.0 / A[i * LD + i];
    for (int c = lane; c < r; c += 32) {
      const double wic = X[i * r + c] * inv;
      for (int m = warp; m < i; m += kFactorThreads / 32) X[m * r + c] -= A[i * LD + m] * wic;
    }
    __syncthreads();
    if (tid < r) X[i * r + tid] *= inv;
    // row i is not read again by later steps (they touch rows < i and read row i' < i)
  }
  __syncthreads();
  for (int e = tid; e < D * r; e += kFactorThreads) out[e] = (float)X[e];
}

}  // namespace curdkv
