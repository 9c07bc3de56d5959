// Block-wise Top-k (Section 3.1, "Sparsity Pattern"): the accumulator is cut into blocks of B
// coordinates and every block keeps exactly its ceil(len * k / d) entries of largest
// magnitude (ties to the lower index).  One thread block handles one block of coordinates
// start to finish - a = xi + g, the exact selection, xi = a - c - so the error buffer is read
// once and written once and nothing but the selection leaves the SM.
//
// Data movement.  A block of xi and of g is one contiguous piece of 4 B bytes each: two bulk
// copies (cp.async.bulk, global -> shared, completion counted on an mbarrier) bring them in,
// a is formed in place over xi's copy, the kept coordinates are overwritten there with their
// new xi value (+0, or the bfloat16 rounding residue), and one bulk copy (shared -> global)
// writes the block of xi back.  xi has two buffers: as soon as a is formed, the loads of the
// thread block's next block start, so they run under the selection of the current one.
// Unaligned gradients and a ragged last block use plain loads and stores.
//
// Selection.  It needs the count-th largest magnitude key T of the block.  T moves little
// from step to step, so while a is formed every warp - it owns a contiguous range of the
// block and walks it 32 coordinates at a time - sets aside, in index order, the keys at or
// above (last step's T of this block) - margin together with their positions.  When
// between `count` and kBlkThreads keys qualify, every thread takes one of them and T is found
// by bisection, a step being one __syncthreads_count: log2(margin) + 1 steps when T lies
// within 2 margin above the lower bound (one more count tells), else 31.  All kept coordinates
// are among the candidates, so the output - in index order - is ranked from warp votes over
// them and the block is not read again.  Otherwise (first step, a jump of the threshold, a
// crowded range) the bisection and the ranking run over all keys of the block.  Either way T
// and the selection are exact.
//
// The wait on the mbarrier is bounded (a poll count and a wall-clock limit).  If it runs out
// the thread block raises the sticky time-out status, starts no further copy, gives the loads
// it had started a second bounded wait to land (so that nothing is written into shared memory
// the block has already given up), lets its stores finish and returns.  The step's result is
// then undefined and the handle reports EFCP_ETIMEOUT.
#pragma once

#include "efcp_common.cuh"

namespace efcp {

constexpr int kBlkThreads = 512;           // threads of the largest variant of the kernel
constexpr int kBlkMax = 16384;             // largest block (coordinates) the kernel holds
// log2 of the key distance below the old threshold from which keys are set aside: kept per
// block and moved by one per step so that the candidates number 1.25 to 2 times the kept
// entries (2^20 is 1/8 binade)
constexpr int kBlkMarginInit = 20, kBlkMarginMin = 12, kBlkMarginMax = 22;
constexpr uint32_t kBlkSpin = 1u << 22;    // polls before the wait for a bulk load gives up
constexpr uint64_t kBlkWaitNs = 1000000000ull;  // and the wall-clock limit of that wait: 1 s
constexpr int kBlkWarpCap = 256;           // candidates one warp can set aside per block

// dynamic shared memory of k_ef_block_select: two blocks of xi and one of g
__host__ __device__ inline size_t block_select_smem(int B) { return size_t(B) * 12; }

// threads per thread block for blocks of B coordinates keeping `count` each: a warp per 512
// coordinates, and room for one candidate per thread with spares
__host__ __device__ inline int block_select_threads(int B, int64_t count) {
  int nt = 128;
  while (nt < kBlkThreads && (nt * 16 < B || nt < 3 * count)) nt *= 2;
  return nt;
}

// entries block-wise Top-k keeps in a block of `len` coordinates at density k/d
__host__ __device__ inline int64_t block_count(int64_t len, int64_t k, int64_t d) {
  return (len * k + d - 1) / d;
}

__device__ __forceinline__ uint32_t blk_smem_u32(const void* p) {
  return uint32_t(__cvta_generic_to_shared(p));
}

// one poll of the mbarrier's phase with the given parity
__device__ __forceinline__ bool blk_mbar_try(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(blk_smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0u;
}

__device__ __forceinline__ uint64_t blk_now_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

// polls the mbarrier's phase until it completes, kBlkSpin polls were made or kBlkWaitNs went by
__device__ __forceinline__ bool blk_mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
  const uint64_t t0 = blk_now_ns();
  for (uint32_t it = 0; it < kBlkSpin; ++it) {
    if (blk_mbar_try(bar, parity)) return true;
    if ((it & 255u) == 255u && blk_now_ns() - t0 > kBlkWaitNs) break;
  }
  return false;
}

// barrier 1 for the first `nthr` threads of the block (whole warps); returns how many of them
// passed a true predicate
__device__ __forceinline__ int blk_bar_count(int nthr, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.u32 p, %2, 0;\n"
      "bar.red.popc.u32 %0, 1, %1, p;\n"
      "}\n"
      : "=r"(r)
      : "r"(nthr), "r"(uint32_t(pred))
      : "memory");
  return int(r);
}

// global -> shared bulk copy of `bytes` (multiple of 16, both ends 16-byte aligned) whose
// completion is counted on `bar`
__device__ __forceinline__ void blk_bulk_g2s(void* sdst, const void* gsrc, uint32_t bytes,
                                             uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      :
      : "r"(blk_smem_u32(sdst)), "l"(gsrc), "r"(bytes), "r"(blk_smem_u32(bar))
      : "memory");
}

template <bool ALIGNED, int NT>
__global__ void __launch_bounds__(NT) k_ef_block_select(
    float* __restrict__ e, const float* __restrict__ g, int64_t d, int64_t k_req, int B,
    int n_blocks, uint32_t* __restrict__ blk_T, int32_t* __restrict__ sel_idx,
    float* __restrict__ sel_val, Scalars* sc, int values_bf16, int drop_loads) {
  // drop_loads (failure-detection test only): the mbarrier is armed but the copies are not
  // issued, so nothing is in flight and the bounded wait below runs out
  constexpr int NW = NT / 32;
  extern __shared__ __align__(128) unsigned char blk_smraw[];
  float* ebuf0 = reinterpret_cast<float*>(blk_smraw);  // two buffers for xi / a / the new xi
  float* gbuf = ebuf0 + 2 * B;
  __shared__ uint16_t wpos[NW][kBlkWarpCap];  // per warp: positions in the block of
                                                     // its candidates, in index order
  __shared__ int wcnt[NW];                    // candidates each warp met
  __shared__ int wtot[NW];  // per warp: (#keys > T) << 16 | #keys == T
  __shared__ int sm[33];
  __shared__ __align__(8) uint64_t mbar;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const unsigned lt = (1u << lane) - 1u;
  const int64_t c_full = block_count(B, k_req, d);
  uint32_t kmax = 0u;  // largest key this thread met: the non-finite check
  uint32_t phase = 0;
  // blocks that move by bulk copies: aligned gradient, length a multiple of 4
  auto is_bulk = [&](int bn) {
    return ALIGNED && (int(min(int64_t(B), d - int64_t(bn) * B)) & 3) == 0;
  };
  // thread 0: start the loads of block bn into eb and gbuf, counted on mbar
  auto issue_loads = [&](int bn, float* eb) {
    const int64_t bn0 = int64_t(bn) * B;
    const uint32_t bytes = uint32_t(min(int64_t(B), d - bn0)) * 4u;
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(
                     blk_smem_u32(&mbar)),
                 "r"(2u * bytes)
                 : "memory");
    if (drop_loads) return;
    blk_bulk_g2s(eb, e + bn0, bytes, &mbar);
    blk_bulk_g2s(gbuf, g + bn0, bytes, &mbar);
  };
  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(blk_smem_u32(&mbar)) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (int(blockIdx.x) < n_blocks && is_bulk(blockIdx.x)) issue_loads(blockIdx.x, ebuf0);
  }
  __syncthreads();
  int n = 0;
  for (int b = blockIdx.x; b < n_blocks; b += gridDim.x, ++n) {
    float* ebuf = ebuf0 + (n & 1) * B;
    const int64_t b0 = int64_t(b) * B;
    const int len = int(min(int64_t(B), d - b0));
    const int count = int(block_count(len, k_req, d));
    const uint32_t told = blk_T[b];
    int mexp = int(blk_T[n_blocks + b]);  // log2 of this block's margin below told
    uint32_t margin = 1u << mexp;
    // candidates are of use with a previous threshold and one key per thread; no key reaches
    // 0xFFFFFFFF, so otherwise nothing is set aside
    const bool guess = told != 0u && count <= NT;
    uint32_t lower = !guess ? 0xFFFFFFFFu : (told > margin ? told - margin : 0u);
    const bool bulk = is_bulk(b);
    // ---- the block of xi and of g: started one block ahead, or fetched here
    if (bulk) {
      // one thread polls, the rest wait at the barrier below
      bool landed = tid != 0 || blk_mbar_wait_bounded(&mbar, phase);
      if (!__syncthreads_and(landed)) {  // one verdict for the whole thread block
        if (tid == 0) {
          atomicOr(&sc->status, kStTimeout);
          // no further loads are started; the ones in flight (this block's two) may still
          // land in shared memory: give them a second bounded wait before the block leaves
          (void)blk_mbar_wait_bounded(&mbar, phase);
        }
        __syncthreads();
        break;
      }
      phase ^= 1u;
    } else {
      // the copy engine must have read this buffer's last contents before it is refilled
      if (tid == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
      __syncthreads();
      for (int i = tid; i < len; i += NT) {
        ebuf[i] = e[b0 + i];
        gbuf[i] = g[b0 + i];
      }
      __syncthreads();
    }
    // warp w owns [wlo, whi): a multiple of 32 coordinates except at the block's end
    const int per_warp = (((len + NW - 1) / NW) + 31) & ~31;
    const int wlo = min(len, warp * per_warp), whi = min(len, wlo + per_warp);
    // ---- a = xi + g in place; candidates' positions to the warp's list, in index order
    int wn = 0;
    auto set_aside = [&](bool cand, int i) {
      const unsigned cb = __ballot_sync(0xFFFFFFFFu, cand);
      if (cb) {
        const int p = wn + __popc(cb & lt);
        if (cand && p < kBlkWarpCap) wpos[warp][p] = uint16_t(i);
        wn += __popc(cb);
      }
    };
    for (int i0 = wlo; i0 < whi; i0 += 128) {
      float x[4], y[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {  // loads first: they need not wait for the stores below
        const int i = i0 + 32 * q + lane;
        x[q] = i < whi ? ebuf[i] : 0.f;
        y[q] = i < whi ? gbuf[i] : 0.f;
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int i = i0 + 32 * q + lane;
        const float a = __fadd_rn(x[q], y[q]);
        if (i < whi) ebuf[i] = a;
        const uint32_t key = mag_key(a);
        kmax = max(kmax, key);
        set_aside(i < whi && key >= lower, i);
      }
    }
    if (lane == 0) wcnt[warp] = wn;
    __syncthreads();
    // gbuf is free again, and so is the other xi buffer once its write-back has been read:
    // the next block's loads run under this block's selection
    if (tid == 0 && b + int(gridDim.x) < n_blocks && is_bulk(b + gridDim.x)) {
      asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
      issue_loads(b + gridDim.x, ebuf0 + ((n + 1) & 1) * B);
    }
    // the candidate lists end to end are one list in index order; thread `tid` takes its
    // tid-th entry.  Too few candidates (T fell below the margin) or too many: the keys are
    // read once more with the margin 8 times wider or narrower, twice at most.
    int n_cand, my_w, my_p;
    bool usable;
    for (int attempt = 0;; ++attempt) {
      n_cand = 0;
      my_w = -1;
      my_p = 0;
      bool crowded = false;
#pragma unroll
      for (int w = 0; w < NW; ++w) {
        const int c = wcnt[w];
        crowded |= c > kBlkWarpCap;
        if (tid >= n_cand && tid < n_cand + c) {
          my_w = w;
          my_p = tid - n_cand;
        }
        n_cand += c;
      }
      usable = !crowded && n_cand >= count && n_cand <= NT;
      if (usable || !guess || attempt == 2) break;
      mexp = n_cand < count ? min(mexp + 3, kBlkMarginMax) : max(mexp - 3, kBlkMarginMin);
      margin = 1u << mexp;
      lower = told > margin ? told - margin : 0u;
      __syncthreads();  // every thread has read the counts
      wn = 0;
      for (int i0 = wlo; i0 < whi; i0 += 32) {
        const int i = i0 + lane;
        const uint32_t key = i < whi ? mag_key(ebuf[i]) : 0u;
        set_aside(i < whi && key >= lower, i);
      }
      if (lane == 0) wcnt[warp] = wn;
      __syncthreads();
    }
    const int64_t row_off = int64_t(b) * c_full;
    uint32_t T = 0u;
    if (usable) {
      // ---- T and the selection from the candidates alone, by the warps that hold some; the
      // others go on to the barrier before the write-back
      const int nthr = (n_cand + 31) & ~31;  // they meet at barrier 1
      if (tid < nthr) {
        const bool have = my_w >= 0;
        const int pos = have ? int(wpos[my_w][my_p]) : 0;
        const uint32_t key = have ? mag_key(ebuf[pos]) : 0u;
        // the largest T with #(key >= T) >= count, by bisection upward from a base for which
        // that holds: `lower` when fewer than count keys lie 2 margin above it, else 0
        const uint32_t hi = lower + 2u * margin;
        const bool window = blk_bar_count(nthr, have && key >= hi) < count;
        T = window ? lower : 0u;
        for (int bit = window ? mexp : 30; bit >= 0; --bit) {
          const uint32_t cand = T + (1u << bit);
          if (blk_bar_count(nthr, have && key >= cand) >= count) T = cand;
        }
        const bool is_gt = have && key > T, is_eq = have && key == T;
        const unsigned gtb = __ballot_sync(0xFFFFFFFFu, is_gt);
        const unsigned eqb = __ballot_sync(0xFFFFFFFFu, is_eq);
        if (lane == 0) wtot[warp] = (__popc(gtb) << 16) | __popc(eqb);
        (void)blk_bar_count(nthr, false);
        int gt_before = 0, eq_before = 0, n_gt = 0;
        for (int w = 0; w < (nthr >> 5); ++w) {
          const int t = wtot[w];
          if (w < warp) {
            gt_before += t >> 16;
            eq_before += t & 0xFFFF;
          }
          n_gt += t >> 16;
        }
        const int need_eq = count - n_gt;  // in [1, #equal keys] by the choice of T
        const int eq_rank = eq_before + __popc(eqb & lt);  // among the block's keys equal to T
        if (is_gt || (is_eq && eq_rank < need_eq)) {
          // kept before me: every larger key, and the equal ones up to need_eq
          const int64_t o = row_off + gt_before + __popc(gtb & lt) + min(eq_rank, need_eq);
          const float v = ebuf[pos];
          sel_idx[o] = int32_t(b0 + pos);
          if (values_bf16) {
            const float r = bf16_to_float(bf16_bits_rn(v));
            sel_val[o] = r;
            ebuf[pos] = __fsub_rn(v, r);
          } else {
            sel_val[o] = v;
            ebuf[pos] = 0.0f;
          }
        }
        if (tid == 0) {
          blk_T[b] = T;
          if (need_eq < 1) atomicOr(&sc->status, kStCount);
        }
      }
      // the margin follows the data: the spare candidates are kept between 4 and 16 standard
      // deviations of the number of keys above a fixed threshold (few risk a miss, many cost
      // time)
      const int spare = n_cand - count, sd = int(sqrtf(float(count))) + 1;
      if (spare < 4 * sd) mexp = min(mexp + 1, kBlkMarginMax);
      else if (spare > 16 * sd) mexp = max(mexp - 1, kBlkMarginMin);
    } else {
      mexp = kBlkMarginInit;
      // ---- T and the selection from all keys of the block
      for (int bit = 30; bit >= 0; --bit) {
        const uint32_t cand = T | (1u << bit);
        int c = 0;
        for (int i = tid; i < len; i += NT) c += mag_key(ebuf[i]) >= cand ? 1 : 0;
        int total;
        (void)block_excl_scan<int>(c, &total, sm);
        if (total >= count) T = cand;
      }
      // keep every key above T and the first (count - #above) keys equal to T, in index order
      int gt_w = 0, eq_w = 0;
      unsigned groups = 0;  // bit j: the j-th 32 coordinates of the range hold a key >= T
      for (int i0 = wlo, j = 0; i0 < whi; i0 += 32, ++j) {
        const int i = i0 + lane;
        const uint32_t key = i < whi ? mag_key(ebuf[i]) : 0u;
        const unsigned gtb = __ballot_sync(0xFFFFFFFFu, i < whi && key > T);
        const unsigned eqb = __ballot_sync(0xFFFFFFFFu, i < whi && key == T);
        gt_w += __popc(gtb);
        eq_w += __popc(eqb);
        groups |= (gtb | eqb) ? 1u << j : 0u;
      }
      if (lane == 0) wtot[warp] = (gt_w << 16) | eq_w;  // each count is at most 1024
      __syncthreads();
      int gt_before = 0, eq_before = 0, n_gt = 0, n_eq_all = 0;
#pragma unroll
      for (int w = 0; w < NW; ++w) {
        const int t = wtot[w];
        if (w < warp) {
          gt_before += t >> 16;
          eq_before += t & 0xFFFF;
        }
        n_gt += t >> 16;
        n_eq_all += t & 0xFFFF;
      }
      const int need_eq = count - n_gt;
      if (tid == 0 && (need_eq < 0 || need_eq > n_eq_all)) atomicOr(&sc->status, kStCount);
      const int eq_base = max(0, min(eq_before, need_eq));  // equal keys kept by earlier warps
      int gt_run = 0, eq_run = 0;
      for (; groups; groups &= groups - 1u) {  // most groups of 32 keep nothing
        const int i = wlo + 32 * (__ffs(groups) - 1) + lane;
        const float v = i < whi ? ebuf[i] : 0.f;
        const uint32_t key = mag_key(v);
        const bool is_gt = i < whi && key > T, is_eq = i < whi && key == T;
        const unsigned gtb = __ballot_sync(0xFFFFFFFFu, is_gt);
        const unsigned eqb = __ballot_sync(0xFFFFFFFFu, is_eq);
        const int eq_rank = eq_before + eq_run + __popc(eqb & lt);  // among the block's equals
        if (is_gt || (is_eq && eq_rank < need_eq)) {
          const int eq_kept = max(0, min(eq_rank, need_eq)) - eq_base;  // before me, this warp
          const int64_t o = row_off + gt_before + eq_base + gt_run + __popc(gtb & lt) + eq_kept;
          sel_idx[o] = int32_t(b0 + i);
          if (values_bf16) {
            const float r = bf16_to_float(bf16_bits_rn(v));
            sel_val[o] = r;
            ebuf[i] = __fsub_rn(v, r);
          } else {
            sel_val[o] = v;
            ebuf[i] = 0.0f;
          }
        }
        gt_run += __popc(gtb);
        eq_run += __popc(eqb);
      }
    }
    if (tid == 0) {
      if (!usable) blk_T[b] = T;
      blk_T[n_blocks + b] = uint32_t(mexp);
    }
    // every thread's writes to ebuf become visible to the copy engine, then the barrier
    if (bulk) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();
    // ---- the block of the new xi goes back
    if (bulk) {
      if (tid == 0) {
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(e + b0),
                     "r"(blk_smem_u32(ebuf)), "r"(uint32_t(len) * 4u)
                     : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
      }
    } else {
      for (int i = tid; i < len; i += NT) e[b0 + i] = ebuf[i];
    }
  }
  if (tid == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");  // stores have landed
  if (kmax >= 0x7F800000u) atomicOr(&sc->status, kStNonFinite);
}

}  // namespace efcp
