// Sparse GGT (appendix "Sparse GGT", algorithm "Detailed Sparse GGT Implementation"): the
// m x m stage of the step when the preconditioner is ((sum_i c_i c_i^T)^(1/2) + eps I)^-1.
//
// The listing eigendecomposes the matrix S of scalar products of the window rows, forms
// U_m = G^T V Sigma^+ (d x m, dense) and returns
//     u = x / eps + U_m [(Sigma + eps I)^-1 - I / eps] U_m^T x,       x = a_t[I_t].
// x is row i of the window, so U_m^T x = Sigma V^T e_i and the expression collapses to a
// linear combination of the window rows,
//     u = G^T w,   w = V diag(1 / (sigma_j + eps)) V^T e_i   over the sigma_j > 0,
// which is what the linear-combination kernel already computes from a weight vector: U_m is
// never formed and x / eps never added and cancelled.  Components whose eigenvalue is at most
// m 2^-48 times the largest (empty rows of a window that is not full, dependent rows) are
// left out: G^T v_j = 0 for them.
//
// The eigendecomposition is a cyclic Jacobi method with the round-robin ordering: in each of
// the m - 1 rounds of a sweep, m / 2 disjoint rotations are applied at once, first to the
// columns of A and V, then to the rows of A.  One thread block, A and V in shared memory
// (which bounds m), fp64.  The loop ends when the off-diagonal part is below 1e-15 of the
// matrix in Frobenius norm, or after kGgtMaxSweeps sweeps with the numeric status raised.
#pragma once

#include "efcp_common.cuh"

namespace efcp {

constexpr int kGgtMaxM = 112;  // two (m x m) fp64 matrices in one SM's shared memory
constexpr int kGgtThreads = 1024;
constexpr int kGgtMaxSweeps = 30;

__host__ __device__ inline int ggt_even(int m) { return (m + 1) & ~1; }
__host__ __device__ inline int ggt_ld(int m) { return ggt_even(m) | 1; }  // odd: no bank pattern
__host__ __device__ inline size_t ggt_smem_bytes(int m) {
  return size_t(2) * ggt_even(m) * ggt_ld(m) * 8 + size_t(ggt_even(m) / 2) * 16;
}

// players p, q of pair j in round r of the circle method on n (even) players
__device__ __forceinline__ void ggt_pair(int n, int r, int j, int* p, int* q) {
  const int c = n - 1;
  if (j == 0) {
    *p = c;
    *q = r % c;
  } else {
    *p = (r + j) % c;
    *q = (r - j + c) % c;
  }
}

__global__ void __launch_bounds__(kGgtThreads) k_ggt_weights(
    const double* __restrict__ S, int m, int slot, double eps, double* __restrict__ w,
    float* __restrict__ wf, Scalars* sc) {
  extern __shared__ __align__(16) unsigned char ggt_smraw[];
  const int n = ggt_even(m), ld = ggt_ld(m), half = n >> 1;
  double* A = reinterpret_cast<double*>(ggt_smraw);
  double* V = A + size_t(n) * ld;
  double2* cs = reinterpret_cast<double2*>(V + size_t(n) * ld);
  __shared__ double red[32];
  const int tid = threadIdx.x;
  // A = S (an odd m gets a zero row and column, which no rotation touches), V = I
  double fro2 = 0.0;
  for (int e = tid; e < n * n; e += kGgtThreads) {
    const int r = e / n, c = e % n;
    const double a = (r < m && c < m) ? S[int64_t(r) * m + c] : 0.0;
    A[r * ld + c] = a;
    V[r * ld + c] = r == c ? 1.0 : 0.0;
    fro2 += a * a;
  }
  fro2 = block_sum(fro2, red);  // ends with a barrier
  bool converged = fro2 == 0.0;
  double off2 = 0.0;
  for (int sweep = 0; sweep < kGgtMaxSweeps && !converged; ++sweep) {
    for (int r = 0; r < n - 1; ++r) {
      // rotation angles of this round's pairs
      if (tid < half) {
        int p, q;
        ggt_pair(n, r, tid, &p, &q);
        const double apq = A[p * ld + q], app = A[p * ld + p], aqq = A[q * ld + q];
        double c = 1.0, s = 0.0;
        if (fabs(apq) > 1e-300 && fabs(apq) > 1e-19 * (fabs(app) + fabs(aqq))) {
          const double theta = (aqq - app) / (2.0 * apq);
          const double t = (theta >= 0.0 ? 1.0 : -1.0) / (fabs(theta) + sqrt(theta * theta + 1.0));
          c = 1.0 / sqrt(t * t + 1.0);
          s = t * c;
        }
        cs[tid] = make_double2(c, s);
      }
      __syncthreads();
      // columns p, q of A and of V
      for (int e = tid; e < n * half; e += kGgtThreads) {
        const int row = e / half, j = e % half;
        const double2 g = cs[j];
        if (g.y != 0.0) {
          int p, q;
          ggt_pair(n, r, j, &p, &q);
          const double ap = A[row * ld + p], aq = A[row * ld + q];
          A[row * ld + p] = g.x * ap - g.y * aq;
          A[row * ld + q] = g.y * ap + g.x * aq;
          const double vp = V[row * ld + p], vq = V[row * ld + q];
          V[row * ld + p] = g.x * vp - g.y * vq;
          V[row * ld + q] = g.y * vp + g.x * vq;
        }
      }
      __syncthreads();
      // rows p, q of A
      for (int e = tid; e < half * n; e += kGgtThreads) {
        const int j = e / n, col = e % n;
        const double2 g = cs[j];
        if (g.y != 0.0) {
          int p, q;
          ggt_pair(n, r, j, &p, &q);
          const double ap = A[p * ld + col], aq = A[q * ld + col];
          A[p * ld + col] = g.x * ap - g.y * aq;
          A[q * ld + col] = g.y * ap + g.x * aq;
        }
      }
      __syncthreads();
    }
    off2 = 0.0;
    for (int e = tid; e < n * n; e += kGgtThreads) {
      const int r = e / n, c = e % n;
      if (r != c) off2 += A[r * ld + c] * A[r * ld + c];
    }
    off2 = block_sum(off2, red);
    converged = off2 <= 1e-30 * fro2;
  }
  // w = V diag(f) V^T e_slot, f_j = 1 / (sqrt(lambda_j) + eps) above the rank tolerance
  double lmax = 0.0;
  bool bad = false;
  for (int j = tid; j < m; j += kGgtThreads) {
    const double l = A[j * ld + j];
    bad |= !(fabs(l) <= 1.79e308);
    lmax = fmax(lmax, l);
  }
  // block maximum through the sum helper's buffer: warp maxima, then the first warp
  for (int o = 16; o > 0; o >>= 1) lmax = fmax(lmax, __shfl_xor_sync(0xFFFFFFFFu, lmax, o));
  if ((tid & 31) == 0) red[tid >> 5] = lmax;
  __syncthreads();
  lmax = red[0];
  for (int i = 1; i < kGgtThreads / 32; ++i) lmax = fmax(lmax, red[i]);
  const double thr = double(m) * 3.5527136788005009e-15 * lmax;  // m 2^-48 lambda_max
  if (tid < m) {
    double acc = 0.0;
    for (int j = 0; j < m; ++j) {
      const double l = A[j * ld + j];
      const double f = l > thr ? 1.0 / (sqrt(l) + eps) : 0.0;
      acc += V[tid * ld + j] * f * V[slot * ld + j];
    }
    w[tid] = acc;
    wf[tid] = float(acc);
    bad |= !(fabs(acc) <= 3.4e38);
  }
  if (bad) atomicOr(&sc->status, kStNonFinite);
  if (tid == 0) {
    sc->resid = fro2 > 0.0 ? sqrt(off2 / fro2) : 0.0;
    if (!converged) atomicOr(&sc->status, kStPivot);
  }
}

}  // namespace efcp
