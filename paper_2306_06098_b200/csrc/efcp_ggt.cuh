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
// the m - 1 rounds of a sweep, m / 2 disjoint rotations are applied at once: to A from both
// sides in 2 x 2 blocks (upper triangle of blocks, mirrored), to the columns of V.  One thread block, A and V in shared memory
// (which bounds m), fp64.  The loop ends when the off-diagonal part is below 1e-15 of the
// matrix in Frobenius norm, or after kGgtMaxSweeps sweeps with the numeric status raised.
// The iteration starts from the previous step's eigenvectors (S changes in one row and column
// per step), which takes it from about ten sweeps to a few.
#pragma once

#include "efcp_common.cuh"

namespace efcp {

constexpr int kGgtMaxM = 112;  // two (m x m) fp64 matrices in one SM's shared memory
constexpr int kGgtThreads = 1024;
constexpr int kGgtMaxSweeps = 30;

__host__ __device__ inline int ggt_even(int m) { return (m + 1) & ~1; }
__host__ __device__ inline int ggt_ld(int m) { return ggt_even(m) | 1; }  // odd: no bank pattern
__host__ __device__ inline size_t ggt_smem_bytes(int m) {
  return size_t(2) * ggt_even(m) * ggt_ld(m) * 8 + size_t(ggt_even(m) / 2) * 24;
}

// 1 / x and 1 / sqrt(x) to fp64 accuracy from the fp32 hardware approximations and Newton
// steps (fused multiply-adds only: the rotation angles sit on the critical path of a round,
// where an fp64 division or square root costs a long dependent chain).  x within fp32 range.
__device__ __forceinline__ double ggt_rcp(double x) {
  double r = double(__frcp_rn(float(x)));
  r = fma(r, fma(-x, r, 1.0), r);
  r = fma(r, fma(-x, r, 1.0), r);
  return fma(r, fma(-x, r, 1.0), r);
}
__device__ __forceinline__ double ggt_rsqrt(double x) {
  double y = double(rsqrtf(float(x)));
  const double h = 0.5 * x;
  y = y * fma(-h * y, y, 1.5);
  y = y * fma(-h * y, y, 1.5);
  return y * fma(-h * y, y, 1.5);
}

// c, s of the Jacobi rotation that annihilates a_pq (c = 1, s = 0: nothing to do)
__device__ __forceinline__ double2 ggt_rotation(double app, double aqq, double apq) {
  const double mag = fabs(apq);
  if (!(mag > 1e-300) || !(mag > 1e-19 * (fabs(app) + fabs(aqq)))) return make_double2(1.0, 0.0);
  const double diff = aqq - app;
  double t;
  if (mag > 1e-30 && mag < 1e30 && fabs(diff) < 1e8 * mag) {
    const double theta = 0.5 * diff * ggt_rcp(apq);
    const double x = fma(theta, theta, 1.0);  // in [1, 1e16]
    const double root = x * ggt_rsqrt(x);
    t = (theta >= 0.0 ? 1.0 : -1.0) * ggt_rcp(fabs(theta) + root);
  } else {  // far from the fp32 range, or a rotation by almost nothing: the plain formulas
    const double theta = diff / (2.0 * apq);
    t = (theta >= 0.0 ? 1.0 : -1.0) / (fabs(theta) + sqrt(theta * theta + 1.0));
  }
  const double c = ggt_rsqrt(fma(t, t, 1.0));
  return make_double2(c, t * c);
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
    float* __restrict__ wf, Scalars* sc, double* __restrict__ Vg, double* Tg) {
  extern __shared__ __align__(16) unsigned char ggt_smraw[];
  const int n = ggt_even(m), ld = ggt_ld(m), half = n >> 1;
  double* A = reinterpret_cast<double*>(ggt_smraw);
  double* V = A + size_t(n) * ld;
  double2* cs = reinterpret_cast<double2*>(V + size_t(n) * ld);
  __shared__ double red[32];
  const int tid = threadIdx.x;
  // thread layouts without divisions: (row, pair) with 64 pair lanes for the column phase,
  // (pair, column) with 128 column lanes for the row phase and for whole-matrix passes
  const int px = tid & 63, py = tid >> 6;    // 16 rows at a time
  const int cx = tid & 127, cy = tid >> 7;   // 8 rows or pairs at a time
  int2* pq = reinterpret_cast<int2*>(cs + half);
  // A = S, V = the eigenvectors of the previous step's S (Vg, m x m; the identity at first).
  // An odd m gets a zero row and column, which no rotation touches.
  double fro2 = 0.0;
  for (int r = cy; r < n; r += 8) {
    if (cx < n) {
      const bool in = r < m && cx < m;
      const double a = in ? S[int64_t(r) * m + cx] : 0.0;
      A[r * ld + cx] = a;
      V[r * ld + cx] = in ? Vg[int64_t(r) * m + cx] : (r == cx ? 1.0 : 0.0);
      fro2 += a * a;
    }
  }
  fro2 = block_sum(fro2, red);  // ends with a barrier
  // warm start: S changed in one row and column only, so V^T S V is close to diagonal and a
  // few sweeps finish the job.  T = S V goes through global scratch, then A = V^T T (upper
  // triangle, mirrored, so that A is exactly symmetric).
  for (int r = cy; r < n; r += 8) {
    if (cx < n) {
      double acc = 0.0;
      for (int k = 0; k < n; ++k) acc = fma(A[r * ld + k], V[k * ld + cx], acc);
      Tg[r * n + cx] = acc;
    }
  }
  __syncthreads();
  for (int r = cy; r < n; r += 8) {
    if (cx < n && cx >= r) {
      double acc = 0.0;
      for (int k = 0; k < n; ++k) acc = fma(V[k * ld + r], Tg[k * n + cx], acc);
      A[r * ld + cx] = acc;
    }
  }
  __syncthreads();
  for (int r = cy; r < n; r += 8)
    if (cx < r) A[r * ld + cx] = A[cx * ld + r];
  __syncthreads();
  // A is symmetric: a round updates it in 2 x 2 blocks (pair i's rows, pair j's columns),
  // one block per i <= j with its mirror image.  This thread's blocks, found once:
  int bi[2], bj[2];
#pragma unroll
  for (int sl = 0; sl < 2; ++sl) {
    int rem = tid + sl * kGgtThreads, i = 0;
    while (i < half && rem >= half - i) {
      rem -= half - i;
      ++i;
    }
    bi[sl] = i < half ? i : -1;
    bj[sl] = i + rem;
  }
  bool converged = fro2 == 0.0;
  double off2 = 0.0;
  for (int sweep = 0; sweep < kGgtMaxSweeps && !converged; ++sweep) {
    for (int r = 0; r < n - 1; ++r) {
      // this round's pairs and their rotation angles
      if (tid < half) {
        int p, q;
        ggt_pair(n, r, tid, &p, &q);
        cs[tid] = ggt_rotation(A[p * ld + p], A[q * ld + q], A[p * ld + q]);
        pq[tid] = make_int2(p, q);
      }
      __syncthreads();
      // A <- J^T A J
#pragma unroll
      for (int sl = 0; sl < 2; ++sl) {
        if (bi[sl] < 0) continue;
        const double2 gi = cs[bi[sl]], gj = cs[bj[sl]];
        if (gi.y == 0.0 && gj.y == 0.0) continue;
        const int2 ri = pq[bi[sl]], cj = pq[bj[sl]];
        const double a = A[ri.x * ld + cj.x], bq = A[ri.x * ld + cj.y];
        const double c = A[ri.y * ld + cj.x], d = A[ri.y * ld + cj.y];
        // rows of pair i, then columns of pair j
        const double a1 = gi.x * a - gi.y * c, b1 = gi.x * bq - gi.y * d;
        const double c1 = gi.y * a + gi.x * c, d1 = gi.y * bq + gi.x * d;
        const double a2 = gj.x * a1 - gj.y * b1, d2 = gj.y * c1 + gj.x * d1;
        double b2 = gj.y * a1 + gj.x * b1, c2 = gj.x * c1 - gj.y * d1;
        if (bi[sl] == bj[sl]) b2 = c2 = 0.0;  // the entry this rotation annihilates
        A[ri.x * ld + cj.x] = a2;
        A[ri.x * ld + cj.y] = b2;
        A[ri.y * ld + cj.x] = c2;
        A[ri.y * ld + cj.y] = d2;
        A[cj.x * ld + ri.x] = a2;
        A[cj.y * ld + ri.x] = b2;
        A[cj.x * ld + ri.y] = c2;
        A[cj.y * ld + ri.y] = d2;
      }
      // V <- V J
      if (px < half) {
        const double2 g = cs[px];
        if (g.y != 0.0) {
          const int2 ix = pq[px];
          for (int row = py; row < n; row += 16) {
            double* v = V + row * ld;
            const double vp = v[ix.x], vq = v[ix.y];
            v[ix.x] = g.x * vp - g.y * vq;
            v[ix.y] = g.y * vp + g.x * vq;
          }
        }
      }
      __syncthreads();
    }
    off2 = 0.0;
    for (int r = cy; r < n; r += 8)
      if (cx < n && cx != r) off2 += A[r * ld + cx] * A[r * ld + cx];
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
  // the eigenvectors start the next step's iteration; after a failure it starts afresh
  const bool keep = converged && __syncthreads_or(bad) == 0;
  for (int r = cy; r < m; r += 8)
    if (cx < m) Vg[int64_t(r) * m + cx] = keep ? V[r * ld + cx] : (r == cx ? 1.0 : 0.0);
  if (bad) atomicOr(&sc->status, kStNonFinite);
  if (tid == 0) {
    sc->resid = fro2 > 0.0 ? sqrt(off2 / fro2) : 0.0;
    if (!converged) atomicOr(&sc->status, kStPivot);
  }
}

}  // namespace efcp
