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
// the m - 1 rounds of a sweep, m / 2 disjoint rotations are applied at once to A from both
// sides, in 2 x 2 blocks; only the upper triangle of A is kept.  One thread block, A in shared
// memory (which bounds m), fp64.  The eigenvector matrix V = J_1 J_2 ... J_K is not formed
// either - updating it costs more shared-memory traffic than A itself, and only w is wanted:
// z = V^T e_i is carried along as a vector through the rotations, every rotation is logged
// (global memory), and w = V (f * z) applies the log backwards to a vector.  The loop ends
// when the off-diagonal part is below 1e-13 of the matrix in Frobenius norm, or after
// kGgtMaxSweeps sweeps with the numeric status raised.
#pragma once

#include "efcp_common.cuh"

namespace efcp {

constexpr int kGgtMaxM = 160;  // an (m x m) fp64 matrix in one SM's shared memory
constexpr int kGgtThreads = 1024;
constexpr int kGgtMaxSweeps = 30;
constexpr int kGgtStage = 8;   // rounds of the rotation log applied per stage

__host__ __device__ inline int ggt_even(int m) { return (m + 1) & ~1; }
// 2 x 2 blocks of the upper triangle of A one thread handles per round
__host__ __device__ inline int ggt_slots(int m) {
  const int h = ggt_even(m) / 2;
  return (h * (h + 1) / 2 + kGgtThreads - 1) / kGgtThreads;
}
__host__ __device__ inline int ggt_ld(int m) { return ggt_even(m) | 1; }  // odd: no bank pattern
__host__ __device__ inline size_t ggt_smem_bytes(int m) {
  const size_t n = ggt_even(m);
  // A, z, g, (c, s), a stage of the rotation log, (p, q)
  return n * ggt_ld(m) * 8 + 2 * n * 8 + (n / 2) * 16 * (1 + kGgtStage) + (n / 2) * 8;
}
// rotations one step can log: (c, s) pairs
__host__ __device__ inline int64_t ggt_log_entries(int m) {
  const int64_t n = ggt_even(m);
  return int64_t(kGgtMaxSweeps) * (n - 1) * (n / 2);
}

// 1 / sqrt(x) to fp64 accuracy from the fp32 hardware approximation and Newton steps (fused
// multiply-adds only).  x within fp32 range.
template <int STEPS>
__device__ __forceinline__ double ggt_rsqrt(double x) {
  double y = double(rsqrtf(float(x)));
  const double h = 0.5 * x;
#pragma unroll
  for (int i = 0; i < STEPS; ++i) y = y * fma(-h * y, y, 1.5);
  return y;
}

// c, s of the Jacobi rotation that annihilates a_pq (c = 1, s = 0: nothing to do).  The
// tangent t only steers the convergence: it is computed in fp32 (about 1e-7 accurate, so a
// rotation leaves 1e-7 of a_pq behind, which costs nothing before the last sweeps and at most
// one sweep there).  c = 1 / sqrt(1 + t^2) and s = t c are accurate to fp64 rounding (1 + t^2
// lies in [1, 2]; three Newton steps from the fp32 estimate): that keeps the transformation
// orthogonal.  The rotation angles sit on the critical path of a round - the rest of the
// thread block waits for them - hence no fp64 division or square root here.
__device__ __forceinline__ double2 ggt_rotation(double app, double aqq, double apq) {
  const double mag = fabs(apq);
  if (!(mag > 1e-300) || !(mag > 1e-19 * (fabs(app) + fabs(aqq)))) return make_double2(1.0, 0.0);
  const double diff = aqq - app;
  double t;
  if (mag > 1e-30 && mag < 1e30 && fabs(diff) < 1e8 * mag) {
    const float theta = 0.5f * float(diff) * __frcp_rn(float(apq));  // |theta| < 1e8
    const float root = sqrtf(fmaf(theta, theta, 1.0f));
    t = double(copysignf(__frcp_rn(fabsf(theta) + root), theta));
  } else {  // far from the fp32 range, or a rotation by almost nothing: the plain formulas
    const double theta = diff / (2.0 * apq);
    t = (theta >= 0.0 ? 1.0 : -1.0) / (fabs(theta) + sqrt(theta * theta + 1.0));
  }
  const double c = ggt_rsqrt<3>(fma(t, t, 1.0));
  return make_double2(c, t * c);
}

// position of the symmetric matrix's entry (r, c) in its upper triangle
__device__ __forceinline__ int ggt_at(int r, int c, int ld) {
  return r <= c ? r * ld + c : c * ld + r;
}

// players p, q of pair j in round r (0 <= r < n - 1) of the circle method on n (even) players
__device__ __forceinline__ void ggt_pair(int n, int r, int j, int* p, int* q) {
  const int c = n - 1;
  if (j == 0) {
    *p = c;
    *q = r;
  } else {  // (r + j) mod c and (r - j) mod c; both arguments lie in [0, 2 c)
    const int a = r + j, b = r - j + c;
    *p = a >= c ? a - c : a;
    *q = b >= c ? b - c : b;
  }
}

template <int SLOTS>  // 2 x 2 blocks per thread: ggt_slots(m) <= SLOTS
__global__ void __launch_bounds__(kGgtThreads) k_ggt_weights(
    const double* __restrict__ S, int m, int slot, double eps, double* __restrict__ w,
    float* __restrict__ wf, Scalars* sc, double2* __restrict__ rot) {
  extern __shared__ __align__(16) unsigned char ggt_smraw[];
  const int n = ggt_even(m), ld = ggt_ld(m), half = n >> 1;
  double* A = reinterpret_cast<double*>(ggt_smraw);
  double* z = A + size_t(n) * ld;  // n is even: everything behind A stays 16-byte aligned
  double* gv = z + n;
  double2* cs = reinterpret_cast<double2*>(gv + n);
  double2* stage = cs + half;
  int2* pq = reinterpret_cast<int2*>(stage + kGgtStage * half);
  __shared__ double red[32];
  const int tid = threadIdx.x;
  const int cx = tid & 255, cy = tid >> 8;  // whole-matrix passes: 256 column lanes, 4 rows
  // A = S (an odd m gets a zero row and column, which no rotation touches), z = e_slot
  double fro2 = 0.0;
  for (int r = cy; r < n; r += 4) {
    if (cx < n) {
      const double a = (r < m && cx < m) ? S[int64_t(r) * m + cx] : 0.0;
      A[r * ld + cx] = a;
      fro2 += a * a;
    }
  }
  if (tid < n) z[tid] = tid == slot ? 1.0 : 0.0;
  fro2 = block_sum(fro2, red);  // ends with a barrier
  // A is symmetric: a round updates it in 2 x 2 blocks (pair i's rows, pair j's columns),
  // one block per i <= j.  This thread's blocks, found once:
  int bi[SLOTS], bj[SLOTS];
#pragma unroll
  for (int sl = 0; sl < SLOTS; ++sl) {
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
  int rounds = 0;  // rotations logged so far: rounds * half
  for (int sweep = 0; sweep < kGgtMaxSweeps && !converged; ++sweep) {
    for (int r = 0; r < n - 1; ++r, ++rounds) {
      // this round's pairs and their rotations
      if (tid < half) {
        int p, q;
        ggt_pair(n, r, tid, &p, &q);
        const double2 g = ggt_rotation(A[p * ld + p], A[q * ld + q], A[ggt_at(p, q, ld)]);
        cs[tid] = g;
        pq[tid] = make_int2(p, q);
        rot[int64_t(rounds) * half + tid] = g;
      }
      __syncthreads();
      // z <- J^T z (off the critical path: the warps below are waiting for the rotations)
      if (tid >= kGgtThreads - half) {
        const int j = kGgtThreads - 1 - tid;
        const double2 g = cs[j];
        const int2 ix = pq[j];
        const double zp = z[ix.x], zq = z[ix.y];
        z[ix.x] = g.x * zp - g.y * zq;
        z[ix.y] = g.y * zp + g.x * zq;
      }
      // A <- J^T A J
#pragma unroll
      for (int sl = 0; sl < SLOTS; ++sl) {
        if (bi[sl] < 0) continue;
        const double2 gi = cs[bi[sl]], gj = cs[bj[sl]];
        if (gi.y == 0.0 && gj.y == 0.0) continue;
        const int2 ri = pq[bi[sl]], cj = pq[bj[sl]];
        // only the upper triangle of A is kept up to date
        const int ia = ggt_at(ri.x, cj.x, ld), ib = ggt_at(ri.x, cj.y, ld);
        const int ic = ggt_at(ri.y, cj.x, ld), id = ggt_at(ri.y, cj.y, ld);
        const double a = A[ia], bq = A[ib], c = A[ic], d = A[id];
        // rows of pair i, then columns of pair j
        const double a1 = gi.x * a - gi.y * c, b1 = gi.x * bq - gi.y * d;
        const double c1 = gi.y * a + gi.x * c, d1 = gi.y * bq + gi.x * d;
        const double a2 = gj.x * a1 - gj.y * b1, d2 = gj.y * c1 + gj.x * d1;
        double b2 = gj.y * a1 + gj.x * b1, c2 = gj.x * c1 - gj.y * d1;
        if (bi[sl] == bj[sl]) b2 = c2 = 0.0;  // the entry this rotation annihilates (ib == ic)
        A[ia] = a2;
        A[ib] = b2;
        A[ic] = c2;
        A[id] = d2;
      }
      __syncthreads();
    }
    off2 = 0.0;
    for (int r = cy; r < n; r += 4)
      if (cx < n && cx > r) off2 += 2.0 * A[r * ld + cx] * A[r * ld + cx];
    off2 = block_sum(off2, red);
    converged = off2 <= 1e-26 * fro2;
  }
  // g = f * z, f_j = 1 / (sqrt(lambda_j) + eps) above the rank tolerance
  double lmax = 0.0;
  bool bad = false;
  for (int j = tid; j < m; j += kGgtThreads) {
    const double l = A[j * ld + j];
    bad |= !(fabs(l) <= 1.79e308);
    lmax = fmax(lmax, l);
  }
  for (int o = 16; o > 0; o >>= 1) lmax = fmax(lmax, __shfl_xor_sync(0xFFFFFFFFu, lmax, o));
  if ((tid & 31) == 0) red[tid >> 5] = lmax;
  __syncthreads();
  lmax = red[0];
  for (int i = 1; i < kGgtThreads / 32; ++i) lmax = fmax(lmax, red[i]);
  const double thr = double(m) * 3.5527136788005009e-15 * lmax;  // m 2^-48 lambda_max
  if (tid < n) {
    const double l = tid < m ? A[tid * ld + tid] : 0.0;
    gv[tid] = l > thr ? z[tid] / (sqrt(l) + eps) : 0.0;
  }
  __syncthreads();
  // w = V g = J_1 (J_2 (... (J_K g))): the log is walked backwards, kGgtStage rounds at a
  // time: all threads fetch a stage (the next one while the current one is applied), one warp
  // applies it to g
  {
    const int per = kGgtStage * half;  // entries of a stage, at most kGgtThreads
    auto fetch = [&](int hi) {  // rounds hi - kGgtStage .. hi - 1, entry `tid`
      const int64_t e = int64_t(hi - kGgtStage) * half + tid;
      return (tid < per && e >= 0) ? rot[e] : make_double2(1.0, 0.0);
    };
    double2 nxt = fetch(rounds);
    for (int hi = rounds; hi > 0; hi -= kGgtStage) {
      if (tid < per) stage[tid] = nxt;
      __syncthreads();
      nxt = fetch(hi - kGgtStage);
      if (tid < 32) {
        for (int a = kGgtStage - 1; a >= 0; --a) {
          const int rd = hi - kGgtStage + a;
          if (rd < 0) break;
          for (int j = tid; j < half; j += 32) {
            const double2 g = stage[a * half + j];
            if (g.y != 0.0) {
              int p, q;
              ggt_pair(n, rd % (n - 1), j, &p, &q);
              const double gp = gv[p], gq = gv[q];
              gv[p] = g.x * gp + g.y * gq;
              gv[q] = g.x * gq - g.y * gp;
            }
          }
          __syncwarp();
        }
      }
      __syncthreads();
    }
  }
  if (tid < m) {
    const double acc = gv[tid];
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
