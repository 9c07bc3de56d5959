// The parameter update around the preconditioner: theta <- (1 - gamma eta) theta - eta s u
// (last line of the loop of Algorithm 1 with the decoupled weight decay of Section 2), s the
// factor that clips |u|_2 to a constant (hyper-parameter appendix), 1 without clipping.
// Two streaming kernels: the squared norm of u (fp64, fixed summation order) and the update
// itself (12 bytes per coordinate: theta read and written, u read).
#pragma once

#include "efcp_common.cuh"

namespace efcp {

constexpr int kUpdThreads = 256;
constexpr int kUpdMaxBlocks = 2048;  // partial sums the norm kernel may write

// part[b] = sum of u_j^2 over block b's grid-stride share of [0, d); the grid is fixed per
// handle, so the order of the summation is too
template <bool VEC>
__global__ void __launch_bounds__(kUpdThreads) k_update_sumsq(const float* __restrict__ u,
                                                              int64_t d,
                                                              double* __restrict__ part) {
  __shared__ double sm[32];
  double acc = 0.0;
  const int64_t tid = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t nth = int64_t(gridDim.x) * blockDim.x;
  if (VEC) {
    const float4* u4 = reinterpret_cast<const float4*>(u);
    const int64_t nv = d >> 2;
    for (int64_t v = tid; v < nv; v += 2 * nth) {
      const float4 a = u4[v];
      const bool more = v + nth < nv;
      const float4 b = more ? u4[v + nth] : make_float4(0.f, 0.f, 0.f, 0.f);
      acc += double(a.x) * double(a.x);
      acc += double(a.y) * double(a.y);
      acc += double(a.z) * double(a.z);
      acc += double(a.w) * double(a.w);
      acc += double(b.x) * double(b.x);
      acc += double(b.y) * double(b.y);
      acc += double(b.z) * double(b.z);
      acc += double(b.w) * double(b.w);
    }
    for (int64_t j = (nv << 2) + tid; j < d; j += nth) acc += double(u[j]) * double(u[j]);
  } else {
    for (int64_t j = tid; j < d; j += nth) acc += double(u[j]) * double(u[j]);
  }
  acc = block_sum(acc, sm);
  if (threadIdx.x == 0) part[blockIdx.x] = acc;
}

// out = part[0] + ... + part[n-1], one block, fixed order
__global__ void __launch_bounds__(256) k_sum_parts(const double* __restrict__ part, int n,
                                                    double* __restrict__ out) {
  __shared__ double sm[32];
  double acc = 0.0;
  for (int i = threadIdx.x; i < n; i += blockDim.x) acc += part[i];
  acc = block_sum(acc, sm);
  if (threadIdx.x == 0) *out = acc;
}

// the factor eta s of the update, rounded once to fp32; norm2 is |u|^2 on the device
__device__ __forceinline__ float update_step(double eta, double clip, const double* norm2) {
  double s = 1.0;
  if (clip > 0.0) {
    const double nrm = sqrt(*norm2);
    if (nrm > clip) s = clip / nrm;
  }
  return float(eta * s);
}

template <bool VEC>
__global__ void __launch_bounds__(kUpdThreads) k_apply_update(float* __restrict__ theta,
                                                              const float* __restrict__ u,
                                                              int64_t n, float decay, double eta,
                                                              double clip,
                                                              const double* __restrict__ norm2) {
  const float step = -update_step(eta, clip, norm2);
  const int64_t tid = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  const int64_t nth = int64_t(gridDim.x) * blockDim.x;
  if (VEC) {
    float4* t4 = reinterpret_cast<float4*>(theta);
    const float4* u4 = reinterpret_cast<const float4*>(u);
    const int64_t nv = n >> 2;
    for (int64_t v = tid; v < nv; v += nth) {
      float4 t = t4[v];
      const float4 x = __ldcs(u4 + v);
      t.x = __fmaf_rn(step, x.x, __fmul_rn(decay, t.x));
      t.y = __fmaf_rn(step, x.y, __fmul_rn(decay, t.y));
      t.z = __fmaf_rn(step, x.z, __fmul_rn(decay, t.z));
      t.w = __fmaf_rn(step, x.w, __fmul_rn(decay, t.w));
      t4[v] = t;
    }
    for (int64_t j = (nv << 2) + tid; j < n; j += nth)
      theta[j] = __fmaf_rn(step, u[j], __fmul_rn(decay, theta[j]));
  } else {
    for (int64_t j = tid; j < n; j += nth)
      theta[j] = __fmaf_rn(step, u[j], __fmul_rn(decay, theta[j]));
  }
}

}  // namespace efcp
