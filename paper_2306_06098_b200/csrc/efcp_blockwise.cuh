// Block-wise Top-k (Section 3.1, "Sparsity Pattern"): the accumulator is cut into blocks of B
// coordinates and every block keeps exactly its ceil(len * k / d) entries of largest
// magnitude (ties to the lower index).  One thread block handles one block of coordinates
// start to finish - a = xi + g, the exact selection, xi = a - c - so the accumulator is read
// and written once and nothing but the selection leaves the SM.
//
// The selection needs the count-th largest magnitude key T of the block.  T moves little from
// step to step, so while a is formed the kernel sets aside (in any order) the keys at or
// above (last step's T of this block) - kBlkMargin; when between `count` and kBlkThreads keys
// qualify, T is found by a 31-step bisection in which every thread holds one key and a step
// is one __syncthreads_count.  Otherwise (first step, a jump of the threshold) the bisection
// runs over all keys of the block.  Either way T is exact, and the output is written in
// index order from per-thread counts and one block scan.
#pragma once

#include "efcp_common.cuh"

namespace efcp {

constexpr int kBlkThreads = 512;
constexpr int kBlkMax = 16384;                  // largest block (coordinates) the kernel holds
constexpr int kBlkEpt = kBlkMax / kBlkThreads;  // elements per thread at most
constexpr uint32_t kBlkMargin = 1u << 20;       // key distance below the old threshold (1/8 binade)

// padded position in shared memory: consecutive threads' chunks never share a bank
__host__ __device__ __forceinline__ int blk_pad(int i) { return i + (i >> 5); }

// entries block-wise Top-k keeps in a block of `len` coordinates at density k/d
__host__ __device__ inline int64_t block_count(int64_t len, int64_t k, int64_t d) {
  return (len * k + d - 1) / d;
}

template <bool VEC>
__global__ void __launch_bounds__(kBlkThreads) k_ef_block_select(
    float* __restrict__ e, const float* __restrict__ g, int64_t d, int64_t k_req, int B,
    int n_blocks, uint32_t* __restrict__ blk_T, int32_t* __restrict__ sel_idx,
    float* __restrict__ sel_val, Scalars* sc, int values_bf16) {
  extern __shared__ __align__(16) unsigned char smraw[];
  float* as = reinterpret_cast<float*>(smraw);  // blk_pad(B) floats
  __shared__ uint32_t ckey[kBlkThreads];
  __shared__ int sm[33];
  __shared__ int s_nc;  // candidate keys set aside for the current block
  const int tid = threadIdx.x;
  const int64_t c_full = block_count(B, k_req, d);
  bool bad = false;
  if (tid == 0) s_nc = 0;
  for (int b = blockIdx.x; b < n_blocks; b += gridDim.x) {
    const int64_t b0 = int64_t(b) * B;
    const int len = int(min(int64_t(B), d - b0));
    const int count = int(block_count(len, k_req, d));
    const uint32_t told = blk_T[b];
    const uint32_t lower = told > kBlkMargin ? told - kBlkMargin : 0u;
    auto note = [&](float x) {  // non-finite check; candidate keys go to ckey, unordered
      const uint32_t key = mag_key(x);
      bad |= key >= 0x7F800000u;
      if (told != 0u && key >= lower) {
        const int slot = atomicAdd(&s_nc, 1);
        if (slot < kBlkThreads) ckey[slot] = key;
      }
    };
    __syncthreads();  // the previous block's shared data is no longer in use
    // ---- a = xi + g, kept in shared memory and written back as the new xi
    if (VEC && (len & 3) == 0) {
      float4* e4 = reinterpret_cast<float4*>(e + b0);
      const float4* g4 = reinterpret_cast<const float4*>(g + b0);
      for (int v = tid; v < (len >> 2); v += kBlkThreads) {
        float4 x = e4[v];
        const float4 y = __ldcs(g4 + v);
        x.x = __fadd_rn(x.x, y.x); x.y = __fadd_rn(x.y, y.y);
        x.z = __fadd_rn(x.z, y.z); x.w = __fadd_rn(x.w, y.w);
        e4[v] = x;
        const int p = blk_pad(4 * v);  // 4 v .. 4 v + 3 lie in one group of 32
        as[p] = x.x; as[p + 1] = x.y; as[p + 2] = x.z; as[p + 3] = x.w;
        note(x.x); note(x.y); note(x.z); note(x.w);
      }
    } else {
      for (int i = tid; i < len; i += kBlkThreads) {
        const float x = __fadd_rn(e[b0 + i], g[b0 + i]);
        e[b0 + i] = x;
        as[blk_pad(i)] = x;
        note(x);
      }
    }
    __syncthreads();
    // this thread's chunk of the block, in index order
    const int ept = (len + kBlkThreads - 1) / kBlkThreads;
    const int lo = min(len, tid * ept), hi = min(len, lo + ept);
    // ---- the count-th largest key T
    const int n_cand = s_nc;
    uint32_t T = 0u;
    if (told != 0u && n_cand >= count && n_cand <= kBlkThreads) {
      const bool have = tid < n_cand;
      const uint32_t key = have ? ckey[tid] : 0u;
      for (int bit = 30; bit >= 0; --bit) {
        const uint32_t cand = T | (1u << bit);
        if (__syncthreads_count(have && key >= cand) >= count) T = cand;
      }
    } else {
      for (int bit = 30; bit >= 0; --bit) {
        const uint32_t cand = T | (1u << bit);
        int c = 0;
        for (int i = lo; i < hi; ++i) c += mag_key(as[blk_pad(i)]) >= cand ? 1 : 0;
        int total;
        (void)block_excl_scan<int>(c, &total, sm);
        if (total >= count) T = cand;
      }
    }
    // ---- keep every key above T and the first (count - #above) keys equal to T
    int gt = 0, eq = 0;
    for (int i = lo; i < hi; ++i) {
      const uint32_t key = mag_key(as[blk_pad(i)]);
      gt += key > T ? 1 : 0;
      eq += key == T ? 1 : 0;
    }
    // one scan for both counts (each at most 16384: 15 bits)
    int tot;
    const int before = block_excl_scan<int>((gt << 16) | eq, &tot, sm);
    const int n_gt = tot >> 16, n_eq_all = tot & 0xFFFF;
    const int gt_before = before >> 16, eq_before = before & 0xFFFF;
    const int need_eq = count - n_gt;
    const int my_eq = max(0, min(eq, need_eq - eq_before));
    int out = gt_before + max(0, min(eq_before, need_eq));
    const int n_sel = n_gt + max(0, min(n_eq_all, need_eq));
    if (tid == 0) s_nc = 0;  // every thread has read it (barriers above); next block starts at 0
    if (tid == 0) {
      blk_T[b] = T;
      if (n_sel != count || need_eq < 0 || need_eq > n_eq_all) atomicOr(&sc->status, kStCount);
    }
    const int64_t row_off = int64_t(b) * c_full;
    int eq_left = my_eq;
    for (int i = lo; i < hi && gt + my_eq > 0; ++i) {  // most chunks keep nothing
      const float v = as[blk_pad(i)];
      const uint32_t key = mag_key(v);
      bool take = key > T;
      if (key == T && eq_left > 0) {
        take = true;
        --eq_left;
      }
      if (take) {
        const int64_t o = row_off + out++;
        sel_idx[o] = int32_t(b0 + i);
        if (values_bf16) {
          const float r = bf16_to_float(bf16_bits_rn(v));
          sel_val[o] = r;
          e[b0 + i] = __fsub_rn(v, r);
        } else {
          sel_val[o] = v;
          e[b0 + i] = 0.0f;
        }
      }
    }
  }
  if (bad) atomicOr(&sc->status, kStNonFinite);
}

}  // namespace efcp
