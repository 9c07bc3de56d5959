// The m x m stage: coefficients of Eq. (2) from the scalar products (Section 2.1).
//
// With A = m*lambda*I + S the Woodbury identity gives
//     F^-1 x = x/lambda - G^T coef,   coef = (1/lambda) A^-1 (G x).
// For x = row i of G (the compressed accumulator just inserted) G x = S e_i = (A - m lambda I) e_i,
// hence coef = e_i/lambda - m A^-1 e_i and the x/lambda term cancels exactly:
//     u = G^T w,   w = m A^-1 e_i.
// So only column i of A^-1 is needed, and the update is a pure linear combination of the
// window rows with no large cancelling terms.
//
// A changes by one row/column per step (the ring slot that was replaced).  B = A^-1 is kept
// explicitly in fp64 and updated in O(m^2):
//   1. remove slot i:  C = B - b b^T / beta          (b = B[:, i], beta = B[i][i]; row/col i -> 0)
//   2. border with the new row: z = C a' (a' = new column without entry i),
//      s = (m lambda + delta_i) - a'^T z   (Schur complement, > 0),
//      B' = C + z z^T / s,  B'[:, i] = B'[i, :] = -z/s,  B'[i][i] = 1/s.
// Then w = m B'[:, i], followed by one step of iterative refinement against A itself
// (r = m e_i - A w, w += B' r), which squares whatever error B has accumulated.
//
// When the right-hand side is the whole accumulator a = xi + c (xi: the error buffer after
// the step, zero on the support of c), the c part is treated as above and the xi part
// literally: F^-1 xi = xi/lambda - G^T A^-1 (G xi)/lambda.  Together
//     u = xi/lambda + G^T w,   w = A^-1 (m e_i - q/lambda),   q = G xi,
// one product with B' and the same refinement step against A.
// All kernels are BLAS-2 shaped and L2 resident (8 MB at m = 1024): no tensor cores.
#pragma once

#include "efcp_common.cuh"

namespace efcp {

__global__ void __launch_bounds__(256) k_init_identity(double* __restrict__ B, int m, double diag) {
  const int64_t n = int64_t(m) * m;
  for (int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; i < n;
       i += int64_t(gridDim.x) * blockDim.x)
    B[i] = (i / m == i % m) ? diag : 0.0;
}

// y = M x (M m x m row-major fp64), one warp per row, fixed summation order.
__global__ void __launch_bounds__(256) k_gemv(const double* __restrict__ M,
                                               const double* __restrict__ x,
                                               double* __restrict__ y, int m) {
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= m) return;
  const double* Mr = M + int64_t(row) * m;
  double acc = 0.0;
  for (int c = lane; c < m; c += 32) acc += Mr[c] * x[c];
  acc = warp_sum(acc);
  if (lane == 0) y[row] = acc;
}

// Scalars of the remove-and-border update; one block.
//   in : y = B a', Brow = old row `slot` of B, delta (delta[slot] = |c_t|^2), aprime
//   out: bold = copy of the old row, z, w (column `slot` of the new inverse times m),
//        sc->schur, sc->beta
__global__ void __launch_bounds__(1024) k_border_scalars(
    const double* __restrict__ y, const double* __restrict__ Brow, const double* __restrict__ delta,
    const double* __restrict__ aprime, int m, int slot, double mlambda, double* __restrict__ bold,
    double* __restrict__ z, double* __restrict__ w, Scalars* sc) {
  __shared__ double sm[32];
  const double t = y[slot];
  const double beta = Brow[slot];
  const double tb = t / beta;
  double part = 0.0;
  for (int r = threadIdx.x; r < m; r += blockDim.x) {
    const double b = Brow[r];
    const double zr = r == slot ? 0.0 : y[r] - b * tb;
    bold[r] = b;
    z[r] = zr;
    part += aprime[r] * zr;
  }
  const double dot = block_sum(part, sm);
  const double s = (mlambda + delta[slot]) - dot;
  const double inv = 1.0 / s;
  for (int r = threadIdx.x; r < m; r += blockDim.x)
    w[r] = r == slot ? double(m) * inv : -double(m) * z[r] * inv;
  if (threadIdx.x == 0) {
    sc->schur = s;
    sc->beta = beta;
    if (!(s > 0.0) || !(beta > 0.0) || !isfinite(s) || !isfinite(beta))
      atomicOr(&sc->status, kStPivot);
  }
}

// B <- B - b b^T / beta + z z^T / s off row/column `slot`; row/column `slot` <- -z/s, 1/s.
// The expression is evaluated identically for (r, c) and (c, r): B stays exactly symmetric.
__global__ void __launch_bounds__(256) k_rank2(double* __restrict__ B, const double* __restrict__ bold,
                                                const double* __restrict__ z, const Scalars* sc,
                                                int m, int slot) {
  const double invs = 1.0 / sc->schur, invb = 1.0 / sc->beta;
  const int64_t n = int64_t(m) * m;
  for (int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; i < n;
       i += int64_t(gridDim.x) * blockDim.x) {
    const int r = int(i / m), c = int(i % m);
    double v;
    if (r == slot || c == slot) {
      v = (r == c) ? invs : -z[r == slot ? c : r] * invs;
    } else {
      const double up = (z[r] * z[c]) * invs;
      const double dn = (bold[r] * bold[c]) * invb;
      v = B[i] + (up - dn);
    }
    B[i] = v;
  }
}

// res = rhs - (m lambda I + S) w with rhs = m e_slot when `rhs` is null; one warp per row.
__global__ void __launch_bounds__(256) k_residual(const double* __restrict__ S,
                                                   const double* __restrict__ w,
                                                   double* __restrict__ res, int m, int slot,
                                                   double mlambda, const double* __restrict__ rhs) {
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= m) return;
  const double* Sr = S + int64_t(row) * m;
  double acc = 0.0;
  for (int c = lane; c < m; c += 32) acc += Sr[c] * w[c];
  acc = warp_sum(acc);
  if (lane == 0) {
    const double b = rhs ? rhs[row] : (row == slot ? double(m) : 0.0);
    res[row] = b - (mlambda * w[row] + acc);
  }
}

// w += dw ; wf = float(w) ; sc->resid = max |res| / m.  One block.
__global__ void __launch_bounds__(1024) k_refine_finish(double* __restrict__ w,
                                                         const double* __restrict__ dw,
                                                         const double* __restrict__ res,
                                                         float* __restrict__ wf, int m,
                                                         Scalars* sc) {
  __shared__ double sm[32];
  double mx = 0.0;
  for (int r = threadIdx.x; r < m; r += blockDim.x) {
    const double v = w[r] + dw[r];
    w[r] = v;
    wf[r] = float(v);
    mx = fmax(mx, fabs(res[r]));
  }
  // max-reduce through the sum tree shape: use shuffles directly
  for (int o = 16; o > 0; o >>= 1) mx = fmax(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
  if ((threadIdx.x & 31) == 0) sm[threadIdx.x >> 5] = mx;
  __syncthreads();
  if (threadIdx.x == 0) {
    double v = 0.0;
    for (int i = 0; i < (blockDim.x >> 5); ++i) v = fmax(v, sm[i]);
    sc->resid = v / double(m);
  }
}

}  // namespace efcp
