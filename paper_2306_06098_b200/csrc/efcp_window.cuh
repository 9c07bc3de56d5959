// Sparse ring-buffer window G = (I, V) and its two primitives (Section 3.1, "Sparse
// Scalar Products" and "Sparse LCG"; Appendix "CUDA Kernels").
//
// Layout: I (int32) and V (fp32) are m x k row-major, one row per ring slot, every row
// sorted by ascending index.  The coordinate range [0, d) is cut into slabs of W
// coordinates; offs[s * m + r] is the position inside row r of its first entry with
// index >= s * W (offs has n_slabs + 1 slab rows), so the entries of row r that fall in
// slab s are the contiguous range [offs[s][r], offs[s+1][r]).
//
// Both primitives are slab-major: a block owns a slab, keeps the dense slab of the
// right-hand side (SP) or of the output (LCG) in shared memory, and streams the
// matching segment of every row past it.  The window is read exactly once per
// primitive, fully coalesced, and no gather or scatter ever leaves the SM.  This
// replaces the paper's block-wise Top-k (which fixes the segment boundaries by
// construction) with a small table written when a row is inserted, so Top-k can stay
// global.
#pragma once

#include "efcp_common.cuh"

namespace efcp {

// offs[s][slot] = lower_bound(row, s * W) for s = 0..n_slabs.
__global__ void __launch_bounds__(256) k_build_offsets(const int32_t* __restrict__ row_idx,
                                                        int64_t k, int W, int n_slabs, int m,
                                                        int slot, int32_t* __restrict__ offs) {
  const int s = blockIdx.x * blockDim.x + threadIdx.x;
  if (s > n_slabs) return;
  const int64_t target = int64_t(s) * W;
  int64_t lo = 0, hi = k;
  while (lo < hi) {
    const int64_t mid = (lo + hi) >> 1;
    if (int64_t(row_idx[mid]) < target) lo = mid + 1; else hi = mid;
  }
  offs[int64_t(s) * m + slot] = int32_t(lo);
}

// Shared-memory layout of the slab kernels: float slab[W]; double/float per-row
// scratch; int32 seg[2 * m] (segment begin / end of every row in the current slab).
__host__ __device__ inline size_t slab_smem_bytes(int W, int m) {
  return size_t(W) * 4 + size_t(m) * 8 + size_t(m) * 8;
}

// Scalar products of every window row with the newest row (x = dens(c_t)):
//   partial[block][r] = sum over this block's slabs of <row_r, x> restricted to the slab
// accumulated in fp64 (every fp32 x fp32 product is exact in fp64).
__global__ void __launch_bounds__(1024, 1) k_sp_rows(
    const int32_t* __restrict__ I, const float* __restrict__ V, const int32_t* __restrict__ offs,
    int64_t k, int m, int W, int n_slabs, int slot, double* __restrict__ partial) {
  extern __shared__ __align__(16) unsigned char smraw[];
  float* xs = reinterpret_cast<float*>(smraw);
  double* ds = reinterpret_cast<double*>(smraw + size_t(W) * 4);
  int32_t* seg = reinterpret_cast<int32_t*>(smraw + size_t(W) * 4 + size_t(m) * 8);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  for (int r = tid; r < m; r += blockDim.x) ds[r] = 0.0;
  const int32_t* Inew = I + int64_t(slot) * k;
  const float* Vnew = V + int64_t(slot) * k;
  for (int s = blockIdx.x; s < n_slabs; s += gridDim.x) {
    __syncthreads();
    float4* xs4 = reinterpret_cast<float4*>(xs);
    for (int i = tid; i < (W >> 2); i += blockDim.x) xs4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int r = tid; r < m; r += blockDim.x) {
      seg[r] = offs[int64_t(s) * m + r];
      seg[m + r] = offs[int64_t(s + 1) * m + r];
    }
    __syncthreads();
    const int base = s * W;
    {
      const int b = seg[slot], e = seg[m + slot];
      for (int j = b + tid; j < e; j += blockDim.x) xs[Inew[j] - base] = Vnew[j];
    }
    __syncthreads();
    for (int r = warp; r < m; r += nwarps) {
      const int b = seg[r], e = seg[m + r];
      if (b >= e) continue;
      const int32_t* Ir = I + int64_t(r) * k;
      const float* Vr = V + int64_t(r) * k;
      double acc = 0.0;
      for (int j = b + lane; j < e; j += 128) {
        const int j1 = j + 32, j2 = j + 64, j3 = j + 96;
        const int i0 = __ldcs(Ir + j);
        const float v0 = __ldcs(Vr + j);
        const int i1 = j1 < e ? __ldcs(Ir + j1) : base;
        const float v1 = j1 < e ? __ldcs(Vr + j1) : 0.f;
        const int i2 = j2 < e ? __ldcs(Ir + j2) : base;
        const float v2 = j2 < e ? __ldcs(Vr + j2) : 0.f;
        const int i3 = j3 < e ? __ldcs(Ir + j3) : base;
        const float v3 = j3 < e ? __ldcs(Vr + j3) : 0.f;
        acc += double(v0) * double(xs[i0 - base]);
        acc += double(v1) * double(xs[i1 - base]);
        acc += double(v2) * double(xs[i2 - base]);
        acc += double(v3) * double(xs[i3 - base]);
      }
      acc = warp_sum(acc);
      if (lane == 0) ds[r] += acc;
    }
  }
  __syncthreads();
  for (int r = tid; r < m; r += blockDim.x) partial[int64_t(blockIdx.x) * m + r] = ds[r];
}

// delta[r] = sum of the per-block partials in block order; S row/column `slot` := delta
// (Section 2.1: S_{i,:} = S_{:,i} = G g); aprime = delta with entry `slot` cleared.
__global__ void __launch_bounds__(128) k_sp_finish(const double* __restrict__ partial, int nparts,
                                                    int m, int slot, double* __restrict__ delta,
                                                    double* __restrict__ S,
                                                    double* __restrict__ aprime) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= m) return;
  double s = 0.0;
  for (int p = 0; p < nparts; ++p) s += partial[int64_t(p) * m + r];
  delta[r] = s;
  S[int64_t(slot) * m + r] = s;
  S[int64_t(r) * m + slot] = s;
  aprime[r] = r == slot ? 0.0 : s;
}

// Linear combination of the window rows, u = sum_r w_r row_r, one slab at a time in a
// shared-memory accumulator (Eq. (2) in the form that has no x/lambda term, see
// efcp_mxm.cuh).  Every element of u is written exactly once.
template <bool VEC>
__global__ void __launch_bounds__(1024, 1) k_lcg(
    const int32_t* __restrict__ I, const float* __restrict__ V, const int32_t* __restrict__ offs,
    int64_t k, int m, int W, int n_slabs, const float* __restrict__ wf, float* __restrict__ u,
    int64_t d) {
  extern __shared__ __align__(16) unsigned char smraw[];
  float* acc = reinterpret_cast<float*>(smraw);
  float* wc = reinterpret_cast<float*>(smraw + size_t(W) * 4);
  int32_t* seg = reinterpret_cast<int32_t*>(smraw + size_t(W) * 4 + size_t(m) * 8);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  for (int r = tid; r < m; r += blockDim.x) wc[r] = wf[r];
  for (int s = blockIdx.x; s < n_slabs; s += gridDim.x) {
    __syncthreads();
    float4* acc4 = reinterpret_cast<float4*>(acc);
    for (int i = tid; i < (W >> 2); i += blockDim.x) acc4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int r = tid; r < m; r += blockDim.x) {
      seg[r] = offs[int64_t(s) * m + r];
      seg[m + r] = offs[int64_t(s + 1) * m + r];
    }
    __syncthreads();
    const int base = s * W;
    for (int r = warp; r < m; r += nwarps) {
      const int b = seg[r], e = seg[m + r];
      const float c = wc[r];
      if (b >= e || c == 0.f) continue;
      const int32_t* Ir = I + int64_t(r) * k;
      const float* Vr = V + int64_t(r) * k;
      for (int j = b + lane; j < e; j += 128) {
        const int j1 = j + 32, j2 = j + 64, j3 = j + 96;
        const int i0 = __ldcs(Ir + j);
        const float v0 = __ldcs(Vr + j);
        const int i1 = j1 < e ? __ldcs(Ir + j1) : -1;
        const float v1 = j1 < e ? __ldcs(Vr + j1) : 0.f;
        const int i2 = j2 < e ? __ldcs(Ir + j2) : -1;
        const float v2 = j2 < e ? __ldcs(Vr + j2) : 0.f;
        const int i3 = j3 < e ? __ldcs(Ir + j3) : -1;
        const float v3 = j3 < e ? __ldcs(Vr + j3) : 0.f;
        atomicAdd(&acc[i0 - base], c * v0);
        if (i1 >= 0) atomicAdd(&acc[i1 - base], c * v1);
        if (i2 >= 0) atomicAdd(&acc[i2 - base], c * v2);
        if (i3 >= 0) atomicAdd(&acc[i3 - base], c * v3);
      }
    }
    __syncthreads();
    const int64_t gbase = int64_t(s) * W;
    const int n = int(min(int64_t(W), d - gbase));
    if (VEC) {
      float4* u4 = reinterpret_cast<float4*>(u + gbase);
      const int nv = n >> 2;
      for (int i = tid; i < nv; i += blockDim.x) __stcs(u4 + i, acc4[i]);
      for (int i = (nv << 2) + tid; i < n; i += blockDim.x) u[gbase + i] = acc[i];
    } else {
      for (int i = tid; i < n; i += blockDim.x) u[gbase + i] = acc[i];
    }
  }
}

}  // namespace efcp
