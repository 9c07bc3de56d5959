// Shared declarations of the EFCP CUDA library (device-side constants, the
// device scalar block, block-level primitives).  sm_100a only.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace efcp {

// Radix-select digit layout over the 31-bit magnitude key (IEEE bits, sign cleared):
// 12 + 10 + 9 bits, most significant first.
constexpr int kBits1 = 12, kBins1 = 1 << kBits1, kShift1 = 31 - kBits1;          // 19
constexpr int kBits2 = 10, kBins2 = 1 << kBits2, kShift2 = kShift1 - kBits2;     // 9
constexpr int kBits3 = 9, kBins3 = 1 << kBits3;

// A chunk is the unit of the ordered compactions: 256 threads x 8 consecutive elements.
constexpr int kChunk = 2048;
constexpr int kChunkThreads = 256;
constexpr int kPerThread = kChunk / kChunkThreads;

// Sticky device status bits.
constexpr uint32_t kStNonFinite = 1u;  // gradient or accumulator entry was Inf/NaN
constexpr uint32_t kStPivot = 2u;      // non-positive pivot / Schur complement in the m x m update
constexpr uint32_t kStCount = 4u;      // selection count mismatch (internal)
constexpr uint32_t kStTimeout = 8u;    // a bounded wait expired

// Scalars that live on the device so that no step needs a host round trip.
struct Scalars {
  uint32_t b1, k1;  // threshold bin of digit 1, entries still to take from it
  uint32_t b2, k2;  // same for digit 2
  uint32_t T;       // exact threshold key
  uint32_t n_eq;    // how many entries with key == T are kept (lowest indices first)
  int32_t n_cand;   // candidates: entries whose digit 1 is >= b1
  int32_t n_sel;    // entries selected (must equal k)
  uint32_t status;  // sticky status bits
  uint32_t have_prev;  // b1 holds the previous step's threshold bin
  uint32_t spec_ok;    // this step's speculative candidate buckets cover the threshold bin
  uint32_t guess;      // the bin from which this step's error-feedback kernel set entries aside
  double schur;     // Schur complement of the bordered inverse (1 / B_ii)
  double beta;      // B_ii before the row was replaced
  double resid;     // max-norm residual of the m x m solve, relative to m
};

__device__ __forceinline__ uint32_t mag_key(float v) { return __float_as_uint(v) & 0x7FFFFFFFu; }

// bfloat16 (the upper half of an IEEE fp32) as raw bits: the optional value format of the
// window (Section 3.1, "Format for V").
struct bf16raw {
  uint16_t bits;
};
// fp32 -> bfloat16, round to nearest, ties to even; NaN stays a (quiet) NaN.
__device__ __forceinline__ uint16_t bf16_bits_rn(float v) {
  uint32_t b = __float_as_uint(v);
  if ((b & 0x7FFFFFFFu) > 0x7F800000u) return uint16_t((b | 0x00400000u) >> 16);
  b += 0x7FFFu + ((b >> 16) & 1u);
  return uint16_t(b >> 16);
}
__device__ __forceinline__ float bf16_to_float(uint16_t bits) {
  return __uint_as_float(uint32_t(bits) << 16);
}
// streaming load of one window value of either format
__device__ __forceinline__ float load_value(const float* p) { return __ldcs(p); }
__device__ __forceinline__ float load_value(const bf16raw* p) {
  return bf16_to_float(__ldcs(reinterpret_cast<const uint16_t*>(p)));
}
// the same through the ordinary cached path (short pieces whose sectors are touched again)
__device__ __forceinline__ float load_value_cached(const float* p) { return *p; }
__device__ __forceinline__ float load_value_cached(const bf16raw* p) {
  return bf16_to_float(*reinterpret_cast<const uint16_t*>(p));
}

// Exclusive prefix sum over the threads of a block (blockDim.x a multiple of 32,
// at most 1024).  sm needs 33 entries.  *total receives the block sum.
template <typename T>
__device__ __forceinline__ T block_excl_scan(T v, T* total, T* sm) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
  T inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    T n = __shfl_up_sync(0xFFFFFFFFu, inc, o);
    if (lane >= o) inc += n;
  }
  if (lane == 31) sm[wid] = inc;
  __syncthreads();
  if (wid == 0) {
    T w = lane < nw ? sm[lane] : T(0);
    T winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      T n = __shfl_up_sync(0xFFFFFFFFu, winc, o);
      if (lane >= o) winc += n;
    }
    sm[lane] = winc - w;
    if (lane == 31) sm[32] = winc;
  }
  __syncthreads();
  T res = sm[wid] + inc - v;
  *total = sm[32];
  __syncthreads();
  return res;
}

__device__ __forceinline__ uint64_t now_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

// Barrier across all thread blocks of a kernel that was launched cooperatively (every block
// resident).  bar[0] counts arrivals, bar[1] exits; both are zero between launches: the
// n-th barrier of a launch (n = 1, 2, ...) completes when bar[0] reaches n * gridDim.x, and
// grid_exit(), called by every block as its last action, lets the last block out clear both
// words for the next launch.  The wait is bounded (kGridWaitNs): if it runs out the call
// returns false for the whole block, which must then return from the kernel at once; the
// caller raises the sticky time-out status.
constexpr uint64_t kGridWaitNs = 2000000000ull;  // 2 s
__device__ __forceinline__ bool grid_barrier(unsigned int* bar, unsigned int n) {
  __syncthreads();
  bool ok = true;
  if (threadIdx.x == 0) {
    const unsigned int target = n * gridDim.x;
    __threadfence();  // this block's writes before the arrival
    atomicAdd(&bar[0], 1u);
    const uint64_t t0 = now_ns();
    unsigned int it = 0;
    for (;;) {
      unsigned int seen;
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(&bar[0]) : "memory");
      if (seen >= target) break;
      if ((++it & 1023u) == 0u && now_ns() - t0 > kGridWaitNs) {
        ok = false;
        break;
      }
    }
    __threadfence();
  }
  return __syncthreads_and(ok) != 0;
}
__device__ __forceinline__ void grid_exit(unsigned int* bar) {
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    if (atomicAdd(&bar[1], 1u) == gridDim.x - 1u) {  // everyone else has left
      bar[0] = 0u;
      __threadfence();
      bar[1] = 0u;
    }
  }
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}

// Deterministic block sum of doubles (fixed tree).  sm needs 32 entries.
__device__ __forceinline__ double block_sum(double v, double* sm) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
  v = warp_sum(v);
  if (lane == 0) sm[wid] = v;
  __syncthreads();
  double r = 0.0;
  if (wid == 0) {
    r = lane < nw ? sm[lane] : 0.0;
    r = warp_sum(r);
    if (lane == 0) sm[0] = r;
  }
  __syncthreads();
  r = sm[0];
  __syncthreads();
  return r;
}

}  // namespace efcp
