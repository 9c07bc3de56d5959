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
// All of it is BLAS-2 shaped and L2 resident (8 MB at m = 1024): no tensor cores.
//
// One cooperative kernel runs the stage as phases separated by grid-wide barriers (it used
// to be eight launches):
//   0  partial[p][r] = sum of the scalar-product kernel's per-slab sums over the slabs
//      p, p + P, ... in increasing order
//   1  delta[r] = sum over p in order (and q, rhs for x = a); with a coordinate-sharded state
//      this is the shard's part of delta, to be summed over the shards before phase 2
//   2  S row/column i := delta; a' ; the old row i of B is set aside
//   3  y = B a'
//   4  every block forms z, the Schur complement and w for itself; B <- B'; the residual
//      m e_i - A w
//   5  (x = a only) w = B' rhs      6  (x = a only) residual rhs - A w
//   7  dw = B' residual; the largest residual entry is recorded
// The linear-combination kernel adds dw to w when it loads the weights.
#pragma once

#include "efcp_common.cuh"

namespace efcp {

constexpr int kMxmThreads = 256;
constexpr int kMxmPhases = 8;

__global__ void __launch_bounds__(256) k_init_identity(double* __restrict__ B, int m, double diag) {
  const int64_t n = int64_t(m) * m;
  for (int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; i < n;
       i += int64_t(gridDim.x) * blockDim.x)
    B[i] = (i / m == i % m) ? diag : 0.0;
}

struct MxmArgs {
  const double* slab_part;  // [n_slabs][stride] from the scalar-product kernel
  double* partial;          // [parts][stride]
  int n_slabs, parts, m, slot;
  int acc;                  // x = a: stride is 2 m, the second half sums to q = G xi
  int fuse12;               // nothing is exchanged between phases 1 and 2: phase 1 does both
  double mlambda, lambda;
  double* S;
  double* B;
  // m-vectors
  double* delta;
  double* aprime;
  double* y;
  double* bold;
  double* w;
  double* res;
  double* dw;
  double* rhs;
  Scalars* sc;
  unsigned int* bar;
  int phase_begin, phase_end;
};

// y[row] = sum_c M[row][c] x[c] for the rows this warp owns (fixed summation order)
__device__ __forceinline__ void gemv_rows(const double* __restrict__ M, const double* x,
                                          double* __restrict__ y, int m, int gwarp, int nwarps,
                                          int lane) {
  for (int row = gwarp; row < m; row += nwarps) {
    const double* Mr = M + int64_t(row) * m;
    double acc = 0.0;
    for (int c = lane; c < m; c += 32) acc += Mr[c] * x[c];
    acc = warp_sum(acc);
    if (lane == 0) y[row] = acc;
  }
}

// dynamic shared memory: 3 m doubles (z, old row of B, w)
__host__ __device__ inline size_t mxm_smem_bytes(int m) { return size_t(m) * 24; }

__global__ void __launch_bounds__(kMxmThreads) k_mxm(const MxmArgs A) {
  extern __shared__ __align__(16) unsigned char mxm_smraw[];
  double* zs = reinterpret_cast<double*>(mxm_smraw);
  double* bs = zs + A.m;
  double* ws = bs + A.m;
  __shared__ double red[32];
  const int tid = threadIdx.x, lane = tid & 31;
  const int m = A.m, slot = A.slot;
  const int stride = A.acc ? 2 * m : m;
  const int64_t gthread = int64_t(blockIdx.x) * kMxmThreads + tid;
  const int64_t nthreads = int64_t(gridDim.x) * kMxmThreads;
  const int gwarp = int(gthread >> 5), nwarps = int(nthreads >> 5);
  unsigned int barriers = 0;
  for (int phase = A.phase_begin; phase < A.phase_end; ++phase) {
    if (!A.acc && (phase == 5 || phase == 6)) continue;
    if (A.fuse12 && phase == 2) continue;
    if (phase > A.phase_begin) {
      if (!grid_barrier(A.bar, ++barriers)) {
        if (tid == 0) atomicOr(&A.sc->status, kStTimeout);
        break;
      }
    }
    if (phase == 0) {
      const int64_t tasks = int64_t(A.parts) * stride;
      for (int64_t t = gthread; t < tasks; t += nthreads) {
        const int p = int(t / stride), r = int(t % stride);
        double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
        int s = p;
        const int step = A.parts;
        for (; s + 3 * step < A.n_slabs; s += 4 * step) {
          a0 += A.slab_part[int64_t(s) * stride + r];
          a1 += A.slab_part[int64_t(s + step) * stride + r];
          a2 += A.slab_part[int64_t(s + 2 * step) * stride + r];
          a3 += A.slab_part[int64_t(s + 3 * step) * stride + r];
        }
        for (; s < A.n_slabs; s += step) a0 += A.slab_part[int64_t(s) * stride + r];
        A.partial[t] = (a0 + a1) + (a2 + a3);
      }
    } else if (phase == 1 || phase == 2) {
      for (int64_t r = gthread; r < m; r += nthreads) {
        if (phase == 1) {
          double s = 0.0;
          for (int p = 0; p < A.parts; ++p) s += A.partial[int64_t(p) * stride + r];
          A.delta[r] = s;
          if (A.acc) {
            double q = 0.0;
            for (int p = 0; p < A.parts; ++p) q += A.partial[int64_t(p) * stride + m + r];
            A.rhs[r] = q;  // G xi for now; phase 2 turns it into the right-hand side
          }
        }
        if (phase == 2 || A.fuse12) {
          // Section 2.1: S_{i,:} = S_{:,i} = G g
          const double s = A.delta[r];
          A.S[int64_t(slot) * m + r] = s;
          A.S[int64_t(r) * m + slot] = s;
          A.aprime[r] = r == slot ? 0.0 : s;
          A.bold[r] = A.B[int64_t(slot) * m + r];
          if (A.acc) A.rhs[r] = (r == slot ? double(m) : 0.0) - A.rhs[r] / A.lambda;
        }
      }
    } else if (phase == 3) {
      gemv_rows(A.B, A.aprime, A.y, m, gwarp, nwarps, lane);
    } else if (phase == 4) {
      // z, the Schur complement and w, the same arithmetic in every block
      const double t = A.y[slot];
      const double beta = A.bold[slot];
      const double tb = t / beta;
      double part = 0.0;
      for (int r = tid; r < m; r += kMxmThreads) {
        const double b = A.bold[r];
        const double zr = r == slot ? 0.0 : A.y[r] - b * tb;
        bs[r] = b;
        zs[r] = zr;
        part += A.aprime[r] * zr;
      }
      const double dot = block_sum(part, red);
      const double s = (A.mlambda + A.delta[slot]) - dot;
      const double invs = 1.0 / s, invb = 1.0 / beta;
      for (int r = tid; r < m; r += kMxmThreads) {
        const double wr = r == slot ? double(m) * invs : -double(m) * zs[r] * invs;
        ws[r] = wr;
        if (blockIdx.x == 0) A.w[r] = wr;
      }
      if (blockIdx.x == 0 && tid == 0) {
        A.sc->schur = s;
        A.sc->beta = beta;
        if (!(s > 0.0) || !(beta > 0.0) || !isfinite(s) || !isfinite(beta))
          atomicOr(&A.sc->status, kStPivot);
      }
      __syncthreads();
      // B <- B - b b^T / beta + z z^T / s off row/column i; row/column i <- -z/s, 1/s.  The
      // expression is evaluated identically for (r, c) and (c, r): B stays exactly symmetric.
      for (int r = gwarp; r < m; r += nwarps) {
        double* Br = A.B + int64_t(r) * m;
        const double zr = zs[r], br = bs[r];
        for (int c = lane; c < m; c += 32) {
          double v;
          if (r == slot || c == slot) {
            v = (r == c) ? invs : -zs[r == slot ? c : r] * invs;
          } else {
            const double up = (zr * zs[c]) * invs;
            const double dn = (br * bs[c]) * invb;
            v = Br[c] + (up - dn);
          }
          Br[c] = v;
        }
      }
      if (!A.acc) {  // res = m e_i - (m lambda I + S) w
        for (int row = gwarp; row < m; row += nwarps) {
          const double* Sr = A.S + int64_t(row) * m;
          double acc = 0.0;
          for (int c = lane; c < m; c += 32) acc += Sr[c] * ws[c];
          acc = warp_sum(acc);
          if (lane == 0)
            A.res[row] = (row == slot ? double(m) : 0.0) - (A.mlambda * ws[row] + acc);
        }
      }
    } else if (phase == 5) {
      // x = a: w = B' rhs replaces the column of B'
      gemv_rows(A.B, A.rhs, A.w, m, gwarp, nwarps, lane);
    } else if (phase == 6) {
      for (int row = gwarp; row < m; row += nwarps) {
        const double* Sr = A.S + int64_t(row) * m;
        double acc = 0.0;
        for (int c = lane; c < m; c += 32) acc += Sr[c] * A.w[c];
        acc = warp_sum(acc);
        if (lane == 0) A.res[row] = A.rhs[row] - (A.mlambda * A.w[row] + acc);
      }
    } else {
      gemv_rows(A.B, A.res, A.dw, m, gwarp, nwarps, lane);
      if (blockIdx.x == 0) {  // sc->resid = max |res| / m
        double mx = 0.0;
        for (int r = tid; r < m; r += kMxmThreads) mx = fmax(mx, fabs(A.res[r]));
        for (int o = 16; o > 0; o >>= 1) mx = fmax(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
        if (lane == 0) red[tid >> 5] = mx;
        __syncthreads();
        if (tid == 0) {
          double v = 0.0;
          for (int i = 0; i < kMxmThreads / 32; ++i) v = fmax(v, red[i]);
          A.sc->resid = v / double(m);
        }
      }
    }
  }
  grid_exit(A.bar);
}

}  // namespace efcp
