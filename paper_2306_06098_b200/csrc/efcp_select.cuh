// Selection and ring insert in one cooperative kernel (Algorithm 1: compression and error
// update; Section 3.1 "Sparsity format for G": the row replaces ring slot (t-1) mod m).
//
// The kernel that forms a = xi + g (k_ef_spec) leaves the digit-1 histogram of the magnitude
// keys and, chunk by chunk, buckets of the entries at or above a guessed bin.  Everything
// between that and the scalar products used to be fourteen small launches; here it is a
// sequence of phases of one kernel, separated by grid-wide barriers:
//
//   0  threshold bin of digit 1 from the histogram (every block computes it for itself);
//      if the guess of k_ef_spec was too high or let in too much, the buckets are rebuilt
//      from a with the exact bin (one more read of a; first step, threshold jumps);
//      histogram of digit 2 over the bucket entries inside the threshold bin
//   1  threshold bin of digit 2; histogram of digit 3
//   2  exact threshold key T; per chunk, the entries above T and equal to T
//   3  positions from the chunk counts; the kept (index, value) pairs are written in ascending
//      index order, keys equal to T are kept in index order until k is reached; kept
//      coordinates of xi become a - c
//   4  where the new row crosses the slab boundaries (offset table, slab weights)
//   5  slabs ordered heavy first; the row goes into the ring slot, every slab segment in the
//      bank-interleaved order the slab kernels want
//
// A warp works on a group of kSelGroup consecutive chunks at a time: their buckets, each a
// few dozen entries at the benchmark's densities, are walked as one list in index order, so
// that a warp has many independent loads in flight instead of a short dependent chain per
// chunk.  Groups are owned by blocks in contiguous runs, so that a block can rank its own
// groups from the totals of the blocks before it.  A launch runs the phases [phase_begin,
// phase_end); a caller that has to exchange something between two phases (histograms summed
// over the shards of a coordinate-sharded state) launches the ranges one after the other.
// The buckets are the candidate list: nothing is compacted in between.
#pragma once

#include "efcp_common.cuh"
#include "efcp_topk.cuh"
#include "efcp_window.cuh"

namespace efcp {

constexpr int kSelThreads = 256;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kSelPhases = 6;
constexpr int kSelGroup = 8;  // chunks whose buckets a warp walks as one list

// dynamic shared memory: the larger of one histogram of digit 1 and the staging of phase 5
constexpr size_t kSelLayoutBytes =
    size_t(kSelWarps) * kLayoutWarpBytes;
constexpr size_t kSelSmemBytes = kSelLayoutBytes > size_t(kBins1) * 4 ? kSelLayoutBytes
                                                                      : size_t(kBins1) * 4;

struct SelectArgs {
  // the accumulator a (in place over xi) and what k_ef_spec left
  float* e;
  int64_t d;
  uint32_t* hist1;
  uint32_t* hist2;
  uint32_t* hist3;
  Scalars* sc;
  int32_t* cnt;       // candidates per chunk (the fill of its bucket)
  uint16_t* bk_off;   // buckets: offset inside the chunk, value
  float* bk_val;
  int n_chunks;
  uint32_t k_total;   // entries to keep (over all shards)
  uint32_t spec_limit;
  // ranking
  int32_t* cnt_gt;    // per group of chunks: entries above T, then their exclusive prefix
  int32_t* cnt_eq;    // same for the entries equal to T
  int32_t* blk_tot;   // per block: totals of its chunks (gt, then eq at + gridDim.x)
  // a coordinate-sharded state: totals of every shard (gt, eq pairs, shard order = coordinate
  // order), filled between phases 2 and 3; nullptr for an unsharded state
  uint32_t* shard_tot;
  int shard, n_shards;
  // the selection
  int32_t* sel_idx;
  float* sel_val;
  int64_t row_cap;    // entries a window row can hold
  int values_bf16;
  // the ring slot
  int W, n_slabs, m, slot;
  int32_t* offs;
  int64_t* colsum;
  int32_t* order;
  int32_t* row_idx;
  uint16_t* row_rel;
  float* row_val;
  bf16raw* row_v16;
  int* slab_ctr;
  float* vmax;
  unsigned int* bar;
  int phase_begin, phase_end;
};

// The bin b of a histogram of NB bins (in shared memory) with
//   count(bins > b) < k_rem <= count(bins >= b),
// found by every thread block for itself.  res[0] = b, res[1] = k_rem - count(bins > b),
// res[2] = 1 when the histogram holds fewer than k_rem entries.
template <int NB>
__device__ __forceinline__ void pick_bin(const uint32_t* h, uint32_t k_rem, uint32_t* res,
                                         uint32_t* sm) {
  constexpr int P = NB / kSelThreads;
  static_assert(NB % kSelThreads == 0, "bins per thread");
  uint32_t mine = 0;
#pragma unroll
  for (int p = 0; p < P; ++p) mine += h[NB - 1 - (threadIdx.x * P + p)];
  if (threadIdx.x == 0) res[0] = res[1] = 0u;  // stays when the histogram is short of k_rem
  uint32_t total;
  uint32_t above = block_excl_scan<uint32_t>(mine, &total, sm);
  if (threadIdx.x == 0) res[2] = total < k_rem ? 1u : 0u;
#pragma unroll
  for (int p = 0; p < P; ++p) {
    const uint32_t bin = NB - 1 - (threadIdx.x * P + p);
    const uint32_t c = h[bin];
    if (above < k_rem && above + c >= k_rem) {
      res[0] = bin;
      res[1] = k_rem - above;
    }
    above += c;
  }
  __syncthreads();
}

__device__ __forceinline__ void flush_hist(const uint32_t* h, uint32_t* __restrict__ g, int nb) {
  __syncthreads();
  for (int i = threadIdx.x; i < nb; i += blockDim.x) {
    const uint32_t c = h[i];
    if (c) atomicAdd(&g[i], c);
  }
}

// The buckets of the chunks [ch0, ch0 + kSelGroup) as one list in index order: calls
// f(on, value, chunk, position in the chunk's bucket) for every entry, 32 entries per
// call (`on` is false for the lanes past the end of the list, so f may vote).  The loads of
// kSelAhead calls are issued together: the passes over the buckets are chains of dependent
// global loads otherwise.
constexpr int kSelAhead = 4;
template <typename F>
__device__ __forceinline__ void walk_group(const SelectArgs& A, int ch0, int lane, F&& f) {
  const int nch = min(kSelGroup, A.n_chunks - ch0);
  const int mine = lane < nch ? A.cnt[ch0 + lane] : 0;
  int pre[kSelGroup + 1];  // exclusive prefix of the bucket fills, the same in every lane
  pre[0] = 0;
#pragma unroll
  for (int q = 0; q < kSelGroup; ++q) pre[q + 1] = pre[q] + __shfl_sync(0xFFFFFFFFu, mine, q);
  const int total = pre[kSelGroup];
  for (int f0 = 0; f0 < total; f0 += 32 * kSelAhead) {
    bool on[kSelAhead];
    int ch[kSelAhead], i[kSelAhead];
    float v[kSelAhead];
#pragma unroll
    for (int u = 0; u < kSelAhead; ++u) {
      const int fl = f0 + 32 * u + lane;
      on[u] = fl < total;
      int t = 0, base = 0;
#pragma unroll
      for (int q = 1; q < kSelGroup; ++q) {
        const bool past = fl >= pre[q];
        t += past ? 1 : 0;
        base = past ? pre[q] : base;
      }
      ch[u] = ch0 + (on[u] ? t : 0);
      i[u] = on[u] ? fl - base : 0;
      v[u] = on[u] ? A.bk_val[int64_t(ch[u]) * kChunk + i[u]] : 0.f;
    }
#pragma unroll
    for (int u = 0; u < kSelAhead; ++u) {
      if (f0 + 32 * u >= total) break;  // warp-uniform
      f(on[u], v[u], ch[u], i[u]);
    }
  }
}

__global__ void __launch_bounds__(kSelThreads) k_select_insert(const SelectArgs A) {
  extern __shared__ __align__(16) unsigned char sel_smraw[];
  uint32_t* hs = reinterpret_cast<uint32_t*>(sel_smraw);
  __shared__ uint32_t sm[33];
  __shared__ uint32_t res[4];
  __shared__ int s_tot[2];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const unsigned lt = (1u << lane) - 1u;
  // the groups of chunks this block owns
  const int n_groups = (A.n_chunks + kSelGroup - 1) / kSelGroup;
  const int per_block = (n_groups + int(gridDim.x) - 1) / int(gridDim.x);
  const int gr_lo = min(n_groups, int(blockIdx.x) * per_block);
  const int gr_hi = min(n_groups, gr_lo + per_block);
  const int ch_lo = gr_lo * kSelGroup, ch_hi = min(A.n_chunks, gr_hi * kSelGroup);
  unsigned int barriers = 0;
  for (int phase = A.phase_begin; phase < A.phase_end; ++phase) {
    if (phase > A.phase_begin) {
      if (!grid_barrier(A.bar, ++barriers)) {
        if (tid == 0) atomicOr(&A.sc->status, kStTimeout);
        break;
      }
    }
    if (phase == 0) {
      // ---- digit 1: threshold bin, verdict on the speculation, digit-2 histogram
      for (int i = tid; i < kBins1; i += kSelThreads) hs[i] = A.hist1[i];
      const uint32_t guess = A.sc->guess;
      __syncthreads();
      pick_bin<kBins1>(hs, A.k_total, res, sm);
      const uint32_t b1 = res[0], k1 = res[1];
      uint32_t let_in = 0;
      for (int i = tid; i < kBins1; i += kSelThreads) let_in += uint32_t(i) >= guess ? hs[i] : 0u;
      uint32_t n_spec;
      (void)block_excl_scan<uint32_t>(let_in, &n_spec, sm);
      const bool spec_ok = guess < uint32_t(kBins1) && guess <= b1 && n_spec <= A.spec_limit;
      if (blockIdx.x == 0 && tid == 0) {
        A.sc->b1 = b1;
        A.sc->k1 = k1;
        A.sc->spec_ok = spec_ok ? 1u : 0u;
        A.sc->have_prev = 1u;
        if (res[2]) atomicOr(&A.sc->status, kStCount);
      }
      __syncthreads();  // hs is reused below
      if (!spec_ok) {
        // the buckets again, from a, with the exact bin: chunk by chunk, in index order
        for (int ch = ch_lo; ch < ch_hi; ++ch) {
          const int local = tid * kPerThread;
          const int64_t base = int64_t(ch) * kChunk + local;
          float v[kPerThread];
          bool ok[kPerThread];
          load_chunk8(A.e, base, A.d, v, ok);
          int c = 0;
#pragma unroll
          for (int q = 0; q < kPerThread; ++q) {
            ok[q] = ok[q] && (mag_key(v[q]) >> kShift1) >= b1;
            c += ok[q] ? 1 : 0;
          }
          int total;
          int pos = block_excl_scan<int>(c, &total, reinterpret_cast<int*>(sm));
          uint16_t* bo = A.bk_off + int64_t(ch) * kChunk;
          float* bv = A.bk_val + int64_t(ch) * kChunk;
#pragma unroll
          for (int q = 0; q < kPerThread; ++q) {
            if (ok[q]) {
              bo[pos] = uint16_t(local + q);
              bv[pos] = v[q];
              ++pos;
            }
          }
          if (tid == 0) A.cnt[ch] = total;
        }
        __syncthreads();  // the block reads its own buckets next
      }
      for (int i = tid; i < kBins2; i += kSelThreads) hs[i] = 0u;
      __syncthreads();
      for (int gr = gr_lo + warp; gr < gr_hi; gr += kSelWarps)
        walk_group(A, gr * kSelGroup, lane, [&](bool on, float v, int, int) {
          const uint32_t key = mag_key(v);
          if (on && (key >> kShift1) == b1) atomicAdd(&hs[(key >> kShift2) & (kBins2 - 1)], 1u);
        });
      flush_hist(hs, A.hist2, kBins2);
    } else if (phase == 1) {
      // ---- digit 2: threshold bin, digit-3 histogram
      for (int i = tid; i < kBins2; i += kSelThreads) hs[i] = A.hist2[i];
      const uint32_t b1 = A.sc->b1, k1 = A.sc->k1;
      __syncthreads();
      pick_bin<kBins2>(hs, k1, res, sm);
      const uint32_t b2 = res[0], k2 = res[1];
      if (blockIdx.x == 0) {
        if (tid == 0) {
          A.sc->b2 = b2;
          A.sc->k2 = k2;
          if (res[2]) atomicOr(&A.sc->status, kStCount);
        }
        for (int i = tid; i < kBins1; i += kSelThreads) A.hist1[i] = 0u;  // for the next step
      }
      __syncthreads();
      for (int i = tid; i < kBins3; i += kSelThreads) hs[i] = 0u;
      __syncthreads();
      const uint32_t prefix = (b1 << kBits2) | b2;
      for (int gr = gr_lo + warp; gr < gr_hi; gr += kSelWarps)
        walk_group(A, gr * kSelGroup, lane, [&](bool on, float v, int, int) {
          const uint32_t key = mag_key(v);
          if (on && (key >> kShift2) == prefix) atomicAdd(&hs[key & (kBins3 - 1)], 1u);
        });
      flush_hist(hs, A.hist3, kBins3);
    } else if (phase == 2) {
      // ---- digit 3: the exact threshold key; per chunk, entries above it and equal to it
      for (int i = tid; i < kBins3; i += kSelThreads) hs[i] = A.hist3[i];
      const uint32_t b1 = A.sc->b1, b2 = A.sc->b2, k2 = A.sc->k2;
      if (tid < 2) s_tot[tid] = 0;
      __syncthreads();
      pick_bin<kBins3>(hs, k2, res, sm);
      const uint32_t T = (b1 << kShift1) | (b2 << kShift2) | res[0];
      if (blockIdx.x == 0) {
        if (tid == 0) {
          A.sc->T = T;
          A.sc->n_eq = res[1];
          if (res[2]) atomicOr(&A.sc->status, kStCount);
        }
        for (int i = tid; i < kBins2; i += kSelThreads) A.hist2[i] = 0u;
      }
      int w_gt = 0, w_eq = 0;
      for (int gr = gr_lo + warp; gr < gr_hi; gr += kSelWarps) {
        int gt = 0, eq = 0;
        walk_group(A, gr * kSelGroup, lane, [&](bool on, float v, int, int) {
          const uint32_t key = mag_key(v);
          gt += __popc(__ballot_sync(0xFFFFFFFFu, on && key > T));
          eq += __popc(__ballot_sync(0xFFFFFFFFu, on && key == T));
        });
        if (lane == 0) {
          A.cnt_gt[gr] = gt;
          A.cnt_eq[gr] = eq;
        }
        w_gt += gt;
        w_eq += eq;
      }
      if (lane == 0) {
        atomicAdd(&s_tot[0], w_gt);
        atomicAdd(&s_tot[1], w_eq);
      }
      __syncthreads();
      if (tid == 0) {
        A.blk_tot[blockIdx.x] = s_tot[0];
        A.blk_tot[gridDim.x + blockIdx.x] = s_tot[1];
        if (A.shard_tot) {
          atomicAdd(&A.shard_tot[2 * A.shard], uint32_t(s_tot[0]));
          atomicAdd(&A.shard_tot[2 * A.shard + 1], uint32_t(s_tot[1]));
        }
      }
    } else if (phase == 3) {
      // ---- positions, the kept pairs in ascending index order, xi = a - c
      const uint32_t T = A.sc->T;
      int64_t n_eq = int64_t(A.sc->n_eq);  // equal keys to keep, lowest indices first
      // totals of the blocks before this one (and of all blocks)
      int bg = 0, be = 0, ag = 0, ae = 0;
      for (int b = tid; b < int(gridDim.x); b += kSelThreads) {
        const int g = A.blk_tot[b], q = A.blk_tot[gridDim.x + b];
        ag += g;
        ae += q;
        if (b < int(blockIdx.x)) {
          bg += g;
          be += q;
        }
      }
      int tot;
      int* smi = reinterpret_cast<int*>(sm);
      (void)block_excl_scan<int>(bg, &tot, smi);
      const int base_gt = tot;
      (void)block_excl_scan<int>(be, &tot, smi);
      int64_t base_eq = tot;
      (void)block_excl_scan<int>(ag, &tot, smi);
      const int all_gt = tot;
      (void)block_excl_scan<int>(ae, &tot, smi);
      const int all_eq = tot;
      int64_t out_base = 0;  // kept entries of this shard start at 0 of its own row
      if (A.shard_tot) {
        // equal keys on shards of lower coordinates are served first
        uint64_t gt_all = 0, eq_before = 0, eq_all = 0;
        for (int r = 0; r < A.n_shards; ++r) {
          gt_all += A.shard_tot[2 * r];
          eq_all += A.shard_tot[2 * r + 1];
          if (r < A.shard) eq_before += A.shard_tot[2 * r + 1];
        }
        if (blockIdx.x == 0 && tid == 0 &&
            (gt_all + uint64_t(n_eq) != uint64_t(A.k_total) || eq_all < uint64_t(n_eq)))
          atomicOr(&A.sc->status, kStCount);
        n_eq = max(int64_t(0), min(int64_t(all_eq), n_eq - int64_t(eq_before)));
      } else if (blockIdx.x == 0 && tid == 0 &&
                 (uint32_t(all_gt) + uint32_t(n_eq) != A.k_total || int64_t(all_eq) < n_eq)) {
        atomicOr(&A.sc->status, kStCount);
      }
      const int64_t n_sel = int64_t(all_gt) + n_eq;
      if (blockIdx.x == 0) {
        if (tid == 0) {
          A.sc->n_sel = int32_t(min(n_sel, A.row_cap));
          if (n_sel > A.row_cap) atomicOr(&A.sc->status, kStCount);
        }
        for (int i = tid; i < kBins3; i += kSelThreads) A.hist3[i] = 0u;
      }
      // exclusive prefix of this block's group counts, in place
      int run_gt = base_gt;
      int64_t run_eq = base_eq;
      for (int c0 = gr_lo; c0 < gr_hi; c0 += kSelThreads) {
        const int gr = c0 + tid;
        const int g = gr < gr_hi ? A.cnt_gt[gr] : 0;
        const int q = gr < gr_hi ? A.cnt_eq[gr] : 0;
        int tg, tq;
        const int eg = block_excl_scan<int>(g, &tg, smi);
        const int eq = block_excl_scan<int>(q, &tq, smi);
        if (gr < gr_hi) {
          A.cnt_gt[gr] = run_gt + eg;
          A.cnt_eq[gr] = int32_t(min(run_eq + eq, int64_t(0x7FFFFFFF)));
        }
        run_gt += tg;
        run_eq += tq;
      }
      __syncthreads();
      for (int gr = gr_lo + warp; gr < gr_hi; gr += kSelWarps) {
        const int64_t eq_before_group = A.cnt_eq[gr];
        int64_t pos0 = out_base + A.cnt_gt[gr] + min(eq_before_group, n_eq);
        int64_t eq_run = eq_before_group;
        walk_group(A, gr * kSelGroup, lane, [&](bool on, float v, int ch, int i) {
          const uint32_t key = mag_key(v);
          const bool is_gt = on && key > T, is_eq = on && key == T;
          const unsigned eqb = __ballot_sync(0xFFFFFFFFu, is_eq);
          const bool keep = is_gt || (is_eq && eq_run + __popc(eqb & lt) < n_eq);
          const unsigned kb = __ballot_sync(0xFFFFFFFFu, keep);
          const int64_t pos = pos0 + __popc(kb & lt);
          if (keep && pos < A.row_cap) {
            const int64_t j = int64_t(ch) * kChunk + A.bk_off[int64_t(ch) * kChunk + i];
            A.sel_idx[pos] = int32_t(j);
            if (A.values_bf16) {  // c holds the rounded value, the residue stays in xi (exact)
              const float r = bf16_to_float(bf16_bits_rn(v));
              A.sel_val[pos] = r;
              A.e[j] = __fsub_rn(v, r);
            } else {
              A.sel_val[pos] = v;
              A.e[j] = 0.0f;
            }
          }
          pos0 += __popc(kb);
          eq_run += __popc(eqb);
        });
      }
    } else if (phase == 4) {
      // ---- the new row's offset in every slab; slab weights
      // an unsharded row always holds row_cap entries; a shard keeps what phase 3 counted
      const int64_t n_sel = A.shard_tot ? int64_t(A.sc->n_sel) : A.row_cap;
      row_offsets(A.sel_idx, n_sel, A.W, A.n_slabs, A.m, A.slot, A.offs, A.colsum,
                  int64_t(blockIdx.x) * kSelThreads + tid, int64_t(gridDim.x) * kSelThreads);
      if (A.vmax)  // the insert below takes maxima into these
        for (int64_t s2 = int64_t(blockIdx.x) * kSelThreads + tid; s2 < A.n_slabs;
             s2 += int64_t(gridDim.x) * kSelThreads)
          A.vmax[s2 * A.m + A.slot] = 0.f;
    } else {
      // ---- slabs heavy first (one block), and the row into its ring slot
      if (blockIdx.x == gridDim.x - 1) {
        slab_order_block(A.colsum, A.n_slabs, A.order, reinterpret_cast<int*>(sel_smraw),
                         reinterpret_cast<int*>(sm));
        if (tid < 16) A.slab_ctr[tid] = 0;  // work counters of the slab kernels' launches
        __syncthreads();
      }
      layout_row_slabs(A.sel_idx, A.sel_val, A.W, A.n_slabs, A.m, A.slot, A.offs, A.row_idx,
                       A.row_rel, A.row_val, A.row_v16, A.vmax,
                       sel_smraw + size_t(warp) * kLayoutWarpBytes,
                       int(blockIdx.x) * kSelWarps + warp, int(gridDim.x) * kSelWarps);
    }
  }
  grid_exit(A.bar);
}

}  // namespace efcp
