// Error feedback and the building blocks of the exact global Top-k (Algorithm 1: the
// error-feedback, compression and error-update statements; Section 3.1).
//
// Selection is a most-significant-digit radix select on the 31-bit magnitude key
// (12 + 10 + 9 bits).  Ties at the threshold key are taken in index order, so the result is
// the unique "first k of a sort by (|a| descending, index ascending)".
//
// Two users:
//   * a step: k_ef_spec (below) forms a = xi + g, histograms digit 1 and leaves the
//     speculative buckets; everything after it is the cooperative kernel of efcp_select.cuh;
//   * efcp_topk_static, the stand-alone selection on a caller's vector: the chain of small
//     kernels in this file (k_pick, k_count_chunks, k_scan_counts, k_compact_cand, k_hist3,
//     k_count_sel, k_scan_sel), which compacts the candidates into a dense list first.
#pragma once

#include "efcp_common.cuh"

namespace efcp {

// Speculation.  The threshold of the selection moves little from one step to the next, so
// the kernel that forms a = xi + g already sets aside, chunk by chunk, every entry at or
// above a guessed bin of digit 1 (the previous step's threshold bin minus kSpecMargin).
// Once the true threshold bin is known the guess is judged: if it was not above the bin
// and did not let in too many entries, the buckets are the candidates and the accumulator is
// not read again; otherwise (first step, threshold fell by more than the margin) they are
// rebuilt with the exact bin.  Both routes give the same exact selection.
constexpr int kSpecMargin = 1;

__device__ __forceinline__ uint32_t spec_guess(const Scalars* sc, int enable) {
  if (!enable || !sc->have_prev) return uint32_t(kBins1);  // nothing is set aside
  return sc->b1 > uint32_t(kSpecMargin) ? sc->b1 - kSpecMargin : 0u;
}

// a = xi + g in place over xi, histogram of digit 1, non-finite detection, and the
// speculative buckets: chunk ch gets its entries with digit 1 >= guess, in index order, at
// bk_off / bk_val [ch * kChunk ...) (offset inside the chunk, value); cnt[ch] = how many.
template <bool VEC>
__global__ void __launch_bounds__(kChunkThreads, 8) k_ef_spec(
    float* __restrict__ e, const float* __restrict__ g, int64_t d, uint32_t* __restrict__ hist1,
    Scalars* sc, int32_t* __restrict__ cnt, uint16_t* __restrict__ bk_off,
    float* __restrict__ bk_val, int n_chunks, int enable) {
  __shared__ uint32_t h[kBins1];
  __shared__ int sm[33];
  for (int i = threadIdx.x; i < kBins1; i += blockDim.x) h[i] = 0u;
  const uint32_t guess = spec_guess(sc, enable);
  if (blockIdx.x == 0 && threadIdx.x == 0) sc->guess = guess;  // for the selection kernel
  __syncthreads();
  bool bad = false;
  for (int ch = blockIdx.x; ch < n_chunks; ch += gridDim.x) {
    const int local = threadIdx.x * kPerThread;
    const int64_t base = int64_t(ch) * kChunk + local;
    float a[kPerThread];
    bool ok[kPerThread];
    if (VEC && base + kPerThread <= d) {
      float4* e4 = reinterpret_cast<float4*>(e + base);
      const float4* g4 = reinterpret_cast<const float4*>(g + base);
      float4 e0 = e4[0], e1 = e4[1];
      const float4 g0 = __ldcs(g4), g1 = __ldcs(g4 + 1);
      e0.x = __fadd_rn(e0.x, g0.x); e0.y = __fadd_rn(e0.y, g0.y);
      e0.z = __fadd_rn(e0.z, g0.z); e0.w = __fadd_rn(e0.w, g0.w);
      e1.x = __fadd_rn(e1.x, g1.x); e1.y = __fadd_rn(e1.y, g1.y);
      e1.z = __fadd_rn(e1.z, g1.z); e1.w = __fadd_rn(e1.w, g1.w);
      e4[0] = e0; e4[1] = e1;
      a[0] = e0.x; a[1] = e0.y; a[2] = e0.z; a[3] = e0.w;
      a[4] = e1.x; a[5] = e1.y; a[6] = e1.z; a[7] = e1.w;
#pragma unroll
      for (int q = 0; q < kPerThread; ++q) ok[q] = true;
    } else {
#pragma unroll
      for (int q = 0; q < kPerThread; ++q) {
        ok[q] = base + q < d;
        a[q] = 0.f;
        if (ok[q]) {
          a[q] = __fadd_rn(e[base + q], g[base + q]);
          e[base + q] = a[q];
        }
      }
    }
    int c = 0;
#pragma unroll
    for (int q = 0; q < kPerThread; ++q) {
      const uint32_t key = mag_key(a[q]);
      if (ok[q]) {
        atomicAdd(&h[key >> kShift1], 1u);
        bad |= key >= 0x7F800000u;
      }
      ok[q] = ok[q] && (key >> kShift1) >= guess;
      c += ok[q] ? 1 : 0;
    }
    int total;
    int pos = block_excl_scan<int>(c, &total, sm);
    if (total) {
      uint16_t* bo = bk_off + int64_t(ch) * kChunk;
      float* bv = bk_val + int64_t(ch) * kChunk;
#pragma unroll
      for (int q = 0; q < kPerThread; ++q) {
        if (ok[q]) {
          bo[pos] = uint16_t(local + q);
          bv[pos] = a[q];
          ++pos;
        }
      }
    }
    if (threadIdx.x == 0) cnt[ch] = total;
  }
  __syncthreads();
  for (int i = threadIdx.x; i < kBins1; i += blockDim.x) {
    const uint32_t c = h[i];
    if (c) atomicAdd(&hist1[i], c);
  }
  if (bad) atomicOr(&sc->status, kStNonFinite);
}

// Finds the threshold bin of one digit: the bin b with count(bins > b) < k_rem <=
// count(bins >= b).  Clears the histogram for the next step.  One block of 1024.
// At level 1, `spec` >= 0 also judges the speculation of k_ef_spec (spec = its `enable`):
// sc->spec_ok = the guessed bin is not above the threshold bin and lets in at most
// `spec_limit` entries.
template <int NB, int LEVEL>
__global__ void __launch_bounds__(1024) k_pick(uint32_t* __restrict__ hist, Scalars* sc,
                                                uint32_t k_total, int spec = -1,
                                                uint32_t spec_limit = 0) {
  __shared__ uint32_t h[NB];
  __shared__ uint32_t sm[33];
  for (int i = threadIdx.x; i < NB; i += blockDim.x) {
    h[i] = hist[i];
    hist[i] = 0u;
  }
  uint32_t guess = NB;
  if (LEVEL == 1 && spec >= 0) guess = spec_guess(sc, spec);  // before b1 is overwritten
  __syncthreads();
  const uint32_t k_rem = LEVEL == 1 ? k_total : (LEVEL == 2 ? sc->k1 : sc->k2);
  constexpr int P = (NB + 1023) / 1024;
  uint32_t mine = 0;
#pragma unroll
  for (int p = 0; p < P; ++p) {
    const int pos = threadIdx.x * P + p;  // position counted from the highest bin
    if (pos < NB) mine += h[NB - 1 - pos];
  }
  uint32_t total;
  uint32_t above = block_excl_scan<uint32_t>(mine, &total, sm);
#pragma unroll
  for (int p = 0; p < P; ++p) {
    const int pos = threadIdx.x * P + p;
    if (pos < NB) {
      const uint32_t bin = NB - 1 - pos;
      const uint32_t c = h[bin];
      if (above < k_rem && above + c >= k_rem) {
        if (LEVEL == 1) { sc->b1 = bin; sc->k1 = k_rem - above; }
        if (LEVEL == 2) { sc->b2 = bin; sc->k2 = k_rem - above; }
        if (LEVEL == 3) {
          sc->T = (sc->b1 << kShift1) | (sc->b2 << kShift2) | bin;
          sc->n_eq = k_rem - above;
        }
      }
      above += c;
    }
  }
  if (threadIdx.x == 0 && total < k_rem) atomicOr(&sc->status, kStCount);
  if (LEVEL == 1 && spec >= 0) {
    uint32_t let_in = 0;
#pragma unroll
    for (int p = 0; p < P; ++p) {
      const int pos = threadIdx.x * P + p;
      if (pos < NB && uint32_t(NB - 1 - pos) >= guess) let_in += h[NB - 1 - pos];
    }
    uint32_t n_spec;
    (void)block_excl_scan<uint32_t>(let_in, &n_spec, sm);
    if (threadIdx.x == 0) {  // after the scan's barriers every thread has written b1
      sc->spec_ok = (guess < uint32_t(NB) && guess <= sc->b1 && n_spec <= spec_limit) ? 1u : 0u;
      sc->have_prev = 1u;
    }
  }
}

__device__ __forceinline__ void load_chunk8(const float* __restrict__ a, int64_t base, int64_t n,
                                            float (&v)[kPerThread], bool (&ok)[kPerThread]) {
  if (base + kPerThread <= n) {
    const float4 x0 = *reinterpret_cast<const float4*>(a + base);
    const float4 x1 = *reinterpret_cast<const float4*>(a + base + 4);
    v[0] = x0.x; v[1] = x0.y; v[2] = x0.z; v[3] = x0.w;
    v[4] = x1.x; v[5] = x1.y; v[6] = x1.z; v[7] = x1.w;
#pragma unroll
    for (int q = 0; q < kPerThread; ++q) ok[q] = true;
  } else {
#pragma unroll
    for (int q = 0; q < kPerThread; ++q) {
      ok[q] = base + q < n;
      v[q] = ok[q] ? a[base + q] : 0.f;
    }
  }
}

// Per chunk of the accumulator: how many entries have digit 1 >= b1.  Blocks stride over
// the chunks.
__global__ void __launch_bounds__(kChunkThreads) k_count_chunks(const float* __restrict__ a,
                                                                 int64_t d, const Scalars* sc,
                                                                 int32_t* __restrict__ cnt,
                                                                 int n_chunks) {
  __shared__ int sm[33];
  if (sc->spec_ok) return;  // (never set for the stand-alone selection)
  const uint32_t b1 = sc->b1;
  for (int ch = blockIdx.x; ch < n_chunks; ch += gridDim.x) {
    const int64_t base = int64_t(ch) * kChunk + threadIdx.x * kPerThread;
    float v[kPerThread];
    bool ok[kPerThread];
    load_chunk8(a, base, d, v, ok);
    int c = 0;
#pragma unroll
    for (int q = 0; q < kPerThread; ++q) c += (ok[q] && (mag_key(v[q]) >> kShift1) >= b1) ? 1 : 0;
    int total;
    (void)block_excl_scan<int>(c, &total, sm);
    if (threadIdx.x == 0) cnt[ch] = total;
  }
}

// In-place exclusive scan of n chunk counts by one block; cnt[n] and *total_out get the sum.
// Tiles of 16384 counts: every thread scans 16 consecutive counts (vector loads), the
// thread sums are scanned across the block.
__global__ void __launch_bounds__(1024) k_scan_counts(int32_t* __restrict__ cnt, int n,
                                                       int32_t* total_out) {
  __shared__ int sm[33];
  constexpr int kPer = 16;  // counts per thread and tile
  int carry = 0;
  for (int base = 0; base < n; base += 1024 * kPer) {
    const int lo = base + int(threadIdx.x) * kPer;
    int v[kPer];
    if (lo + kPer <= n) {
      const int4* p = reinterpret_cast<const int4*>(cnt + lo);  // cnt is 256-byte aligned
#pragma unroll
      for (int q = 0; q < kPer / 4; ++q) {
        const int4 x = p[q];
        v[4 * q] = x.x; v[4 * q + 1] = x.y; v[4 * q + 2] = x.z; v[4 * q + 3] = x.w;
      }
    } else {
#pragma unroll
      for (int q = 0; q < kPer; ++q) v[q] = lo + q < n ? cnt[lo + q] : 0;
    }
    int mine = 0;
#pragma unroll
    for (int q = 0; q < kPer; ++q) mine += v[q];
    int total;
    int run = carry + block_excl_scan<int>(mine, &total, sm);
#pragma unroll
    for (int q = 0; q < kPer; ++q) {
      const int x = v[q];
      v[q] = run;
      run += x;
    }
    if (lo + kPer <= n) {
      int4* p = reinterpret_cast<int4*>(cnt + lo);
#pragma unroll
      for (int q = 0; q < kPer / 4; ++q) p[q] = make_int4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
    } else {
#pragma unroll
      for (int q = 0; q < kPer; ++q)
        if (lo + q < n) cnt[lo + q] = v[q];
    }
    carry += total;
  }
  if (threadIdx.x == 0) {
    cnt[n] = carry;
    *total_out = carry;
  }
}

// Ordered compaction of the candidates (digit 1 >= b1) and histogram of digit 2 over
// the entries inside the threshold bin.
__global__ void __launch_bounds__(kChunkThreads, 8) k_compact_cand(
    const float* __restrict__ a, int64_t d, const Scalars* sc, const int32_t* __restrict__ off,
    int32_t* __restrict__ cand_idx, float* __restrict__ cand_val, uint32_t* __restrict__ hist2,
    int n_chunks) {
  __shared__ uint32_t h[kBins2];
  __shared__ int sm[33];
  if (sc->spec_ok) return;  // (never set for the stand-alone selection)
  for (int i = threadIdx.x; i < kBins2; i += blockDim.x) h[i] = 0u;
  __syncthreads();
  const uint32_t b1 = sc->b1;
  for (int ch = blockIdx.x; ch < n_chunks; ch += gridDim.x) {
    const int64_t base = int64_t(ch) * kChunk + threadIdx.x * kPerThread;
    float v[kPerThread];
    bool ok[kPerThread];
    const int off0 = off[ch], off1 = off[ch + 1];  // in flight together with the chunk
    load_chunk8(a, base, d, v, ok);
    if (off1 == off0) continue;  // no candidate in this chunk (block-uniform)
    int c = 0;
#pragma unroll
    for (int q = 0; q < kPerThread; ++q) {
      ok[q] = ok[q] && (mag_key(v[q]) >> kShift1) >= b1;
      c += ok[q] ? 1 : 0;
    }
    int total;
    int pos = off0 + block_excl_scan<int>(c, &total, sm);
#pragma unroll
    for (int q = 0; q < kPerThread; ++q) {
      if (ok[q]) {
        cand_idx[pos] = int32_t(base + q);
        cand_val[pos] = v[q];
        ++pos;
        const uint32_t key = mag_key(v[q]);
        if ((key >> kShift1) == b1) atomicAdd(&h[(key >> kShift2) & (kBins2 - 1)], 1u);
      }
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < kBins2; i += blockDim.x) {
    const uint32_t cc = h[i];
    if (cc) atomicAdd(&hist2[i], cc);
  }
}

// Histogram of digit 3 over the candidates whose digits 1 and 2 match the threshold.
__global__ void __launch_bounds__(256) k_hist3(const float* __restrict__ cand_val,
                                                const Scalars* sc, uint32_t* __restrict__ hist3) {
  __shared__ uint32_t h[kBins3];
  for (int i = threadIdx.x; i < kBins3; i += blockDim.x) h[i] = 0u;
  __syncthreads();
  const int n = sc->n_cand;
  const uint32_t prefix = (sc->b1 << kBits2) | sc->b2;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    const uint32_t key = mag_key(cand_val[i]);
    if ((key >> kShift2) == prefix) atomicAdd(&h[key & (kBins3 - 1)], 1u);
  }
  __syncthreads();
  for (int i = threadIdx.x; i < kBins3; i += blockDim.x) {
    const uint32_t c = h[i];
    if (c) atomicAdd(&hist3[i], c);
  }
}

// Per candidate chunk: entries above the threshold key and entries equal to it.
__global__ void __launch_bounds__(kChunkThreads) k_count_sel(const float* __restrict__ cand_val,
                                                              const Scalars* sc,
                                                              int32_t* __restrict__ cnt_gt,
                                                              int32_t* __restrict__ cnt_eq) {
  __shared__ int sm[33];
  const int n = sc->n_cand;
  const uint32_t T = sc->T;
  const int n_cc = (n + kChunk - 1) / kChunk;
  for (int c = blockIdx.x; c < n_cc; c += gridDim.x) {
    const int64_t base = int64_t(c) * kChunk + threadIdx.x * kPerThread;
    float v[kPerThread];
    bool ok[kPerThread];
    load_chunk8(cand_val, base, n, v, ok);
    int packed = 0;  // gt in the low half, eq in the high half (each <= 2048)
#pragma unroll
    for (int q = 0; q < kPerThread; ++q) {
      const uint32_t key = mag_key(v[q]);
      packed += (ok[q] && key > T) ? 1 : 0;
      packed += (ok[q] && key == T) ? (1 << 16) : 0;
    }
    int total;
    (void)block_excl_scan<int>(packed, &total, sm);
    if (threadIdx.x == 0) {
      cnt_gt[c] = total & 0xFFFF;
      cnt_eq[c] = total >> 16;
    }
  }
}

// Exclusive scans of both per-chunk counts (one block) and the count check.
__global__ void __launch_bounds__(1024) k_scan_sel(int32_t* __restrict__ cnt_gt,
                                                    int32_t* __restrict__ cnt_eq, Scalars* sc,
                                                    uint32_t k_total) {
  __shared__ int sm[33];
  const int n_cc = (sc->n_cand + kChunk - 1) / kChunk;
  int carry_gt = 0, carry_eq = 0;
  for (int base = 0; base < n_cc; base += 1024) {
    const int i = base + threadIdx.x;
    const int g = i < n_cc ? cnt_gt[i] : 0;
    const int q = i < n_cc ? cnt_eq[i] : 0;
    int tg, tq;
    const int eg = block_excl_scan<int>(g, &tg, sm);
    const int eq = block_excl_scan<int>(q, &tq, sm);
    if (i < n_cc) {
      cnt_gt[i] = carry_gt + eg;
      cnt_eq[i] = carry_eq + eq;
    }
    carry_gt += tg;
    carry_eq += tq;
  }
  if (threadIdx.x == 0) {
    const uint32_t n_eq = sc->n_eq;
    sc->n_sel = carry_gt + int32_t(n_eq);
    if (uint32_t(carry_gt) + n_eq != k_total || uint32_t(carry_eq) < n_eq)
      atomicOr(&sc->status, kStCount);
  }
}

}  // namespace efcp
