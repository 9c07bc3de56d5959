// Sparse ring-buffer window G = (I, V) and its two primitives (Section 3.1, "Sparse
// Scalar Products" and "Sparse LCG"; Appendix "CUDA Kernels").
//
// Layout: I (int32) and V (fp32) are m x k row-major, one row per ring slot.  The
// coordinate range [0, d) is cut into slabs of W coordinates (W a multiple of 32);
// offs[s * m + r] is the number of entries of row r with index < s * W (offs has
// n_slabs + 1 slab rows), so the entries of row r that fall in slab s are the contiguous
// range [offs[s][r], offs[s+1][r]) of the row: its segment in that slab.
//
// Both primitives are slab-major: a block owns a slab, keeps the dense slab of the
// right-hand side (SP) or of the output (LCG) in shared memory, and streams the
// matching segment of every row past it.  The window is read exactly once per
// primitive, fully coalesced, and no gather or scatter ever leaves the SM.  This
// replaces the paper's block-wise Top-k (which fixes the segment boundaries by
// construction) with a small table written when a row is inserted, so Top-k can stay
// global.
//
// Indices as the kernels read them.  Inside slab s an index is s * W plus an offset below
// W <= 65536, and a segment lies in one slab, so next to I the window keeps R (uint16,
// m x k, same positions): the slab-relative offsets.  SP and LCG stream R and V, 6 bytes per
// entry instead of 8, and use the offset directly as the shared-memory address; I is only
// written (at insert) and read back by efcp_get_row / efcp_get_window.
//
// Order inside a segment.  A warp takes 32 consecutive entries of a segment at a time and
// uses their indices as shared-memory addresses, so what matters for speed is how many
// of the 32 fall into the same bank (index mod 32).  Neither primitive depends on the
// order of the entries inside a segment, so the insert kernel stores every chunk of 512
// entries (counted from the segment start) sorted by (occurrence number of the entry's
// bank, bank): the first entry of every bank, then the second of every bank, and so on.
// Every aligned group of 32 then holds mostly distinct banks.  efcp_get_row returns rows
// in ascending index order again.
#pragma once

#include "efcp_common.cuh"

namespace efcp {

constexpr int kLayoutChunk = 512;   // entries permuted together (a multiple of 32)
constexpr int kLayoutLevels = 64;   // occurrence levels with precomputed ranks (more: slow path)
// shared memory of one warp of the insert: indices, values, occurrence numbers of a chunk,
// per-bank counts, per-level bank masks and level starts
constexpr int kLayoutWarpBytes = kLayoutChunk * 10 + 32 * 4 + kLayoutLevels * 6;

// offs[s][slot] for the new row from its ascending index list of n entries: entry `pos`
// starts every slab between its predecessor's slab (exclusive) and its own (inclusive); the
// last entry also closes all slabs behind it.  One thread per entry, no searches (`first`
// and `stride` spread the entries over the calling threads).  colsum[s] = sum over the rows
// of offs[s][.] is kept up to date (one writer per s), so that colsum[s + 1] - colsum[s] is
// the number of window entries in slab s.  An empty row (n == 0: a shard of the coordinates
// that keeps nothing this step) has offset 0 everywhere.
__device__ __forceinline__ void row_offsets(const int32_t* __restrict__ idx, int64_t n, int W,
                                            int n_slabs, int m, int slot,
                                            int32_t* __restrict__ offs,
                                            int64_t* __restrict__ colsum, int64_t first,
                                            int64_t stride) {
  auto put = [&](int s, int32_t v) {
    int32_t* p = offs + int64_t(s) * m + slot;
    colsum[s] += int64_t(v) - int64_t(*p);
    *p = v;
  };
  if (n == 0) {
    for (int64_t s = first; s <= n_slabs; s += stride) put(int(s), 0);
    return;
  }
  for (int64_t pos = first; pos < n; pos += stride) {
    const int s1 = idx[pos] / W;
    const int s0 = pos > 0 ? idx[pos - 1] / W : -1;
    for (int s = s0 + 1; s <= s1; ++s) put(s, int32_t(pos));
    if (pos == n - 1)
      for (int s = s1 + 1; s <= n_slabs; ++s) put(s, int32_t(n));
  }
}

// order[] = the slabs, heaviest first up to a factor 2^(1/4): a counting sort on the top
// bits of the slab weight colsum[s + 1] - colsum[s].  The slab kernels hand out slabs in
// this order, so the heavy slabs are never the last ones a block starts.  The order inside
// a weight class is arbitrary; no result depends on it.  Called by all threads of one
// block; cnt: kOrderBins ints of shared memory, sm: 33.
constexpr int kOrderBins = 1024;
__device__ __forceinline__ void slab_order_block(const int64_t* __restrict__ colsum, int n_slabs,
                                                 int32_t* __restrict__ order, int* cnt, int* sm) {
  for (int i = threadIdx.x; i < kOrderBins; i += blockDim.x) cnt[i] = 0;
  __syncthreads();
  auto bin_of = [&](int s) {
    const float w = float(colsum[s + 1] - colsum[s]);           // >= 0
    const int key = int(__float_as_uint(w) >> 21);               // exponent and 2 mantissa bits
    return kOrderBins - 1 - min(key, kOrderBins - 1);            // heavy slabs first
  };
  for (int s = threadIdx.x; s < n_slabs; s += blockDim.x) atomicAdd(&cnt[bin_of(s)], 1);
  __syncthreads();
  int carry = 0;
  for (int b0 = 0; b0 < kOrderBins; b0 += blockDim.x) {  // exclusive prefix of the bin counts
    const int b = b0 + threadIdx.x;
    const int mine = b < kOrderBins ? cnt[b] : 0;
    int total;
    const int start = block_excl_scan<int>(mine, &total, sm);
    if (b < kOrderBins) cnt[b] = carry + start;
    carry += total;
  }
  __syncthreads();
  for (int s = threadIdx.x; s < n_slabs; s += blockDim.x) order[atomicAdd(&cnt[bin_of(s)], 1)] = s;
  __syncthreads();
}

// Insert of the new row: from the ascending (index, value) list of the selection,
//   ring slot <- the row, every segment [offs[s][slot], offs[s+1][slot]) in the
//   bank-interleaved order described above.  One warp handles one chunk at a time; a slab's
//   chunks are shared by `wps` warps (1, 2, 4 or 8: as many as there are warps to go round),
//   warp `gwarp` of `nwarps` taking the (slab, part) pairs gwarp, gwarp + nwarps, ...
//   smraw: this warp's kLayoutWarpBytes of shared memory.  vmax[s][slot] must be
//   zero on entry; it receives the largest magnitude of the segment.
__device__ __forceinline__ void layout_row_slabs(
    const int32_t* __restrict__ src_idx, const float* __restrict__ src_val, int W, int n_slabs,
    int m, int slot, const int32_t* __restrict__ offs, int32_t* __restrict__ dst_idx,
    uint16_t* __restrict__ dst_rel, float* __restrict__ dst_val, bf16raw* __restrict__ dst_v16,
    float* __restrict__ vmax, unsigned char* smraw, int gwarp, int nwarps) {
  const int lane = threadIdx.x & 31;
  int32_t* ci = reinterpret_cast<int32_t*>(smraw);
  float* cv = reinterpret_cast<float*>(smraw + kLayoutChunk * 4);
  uint16_t* cq = reinterpret_cast<uint16_t*>(smraw + kLayoutChunk * 8);
  int* cnt = reinterpret_cast<int*>(smraw + kLayoutChunk * 10);
  uint32_t* lvl_mask = reinterpret_cast<uint32_t*>(smraw + kLayoutChunk * 10 + 128);
  uint16_t* lvl_start = reinterpret_cast<uint16_t*>(smraw + kLayoutChunk * 10 + 128 +
                                                    kLayoutLevels * 4);
  int wps = 1;
  while (wps < 8 && int64_t(n_slabs) * wps * 2 <= nwarps) wps *= 2;
  for (int64_t t = gwarp; t < int64_t(n_slabs) * wps; t += nwarps) {
    const int s = int(t / wps), part = int(t % wps);
    float vm = 0.f;  // largest magnitude this thread staged (for the fixed-point LCG's bound)
    const int seg_b = offs[int64_t(s) * m + slot];
    const int seg_e = offs[int64_t(s + 1) * m + slot];
    for (int c0 = seg_b + part * kLayoutChunk; c0 < seg_e; c0 += wps * kLayoutChunk) {
      const int n = min(kLayoutChunk, seg_e - c0);
      cnt[lane] = 0;
      __syncwarp();
      // stage the chunk (all loads in flight together), then number every entry within its
      // bank in ascending index order
      for (int a = lane; a < n; a += 32) {
        ci[a] = src_idx[c0 + a];
        cv[a] = src_val[c0 + a];
        vm = fmaxf(vm, fabsf(cv[a]));
      }
      __syncwarp();
      for (int a0 = 0; a0 < n; a0 += 32) {
        const int a = a0 + lane;
        const bool on = a < n;
        const int bank = on ? (ci[a] & 31) : 0;
        const unsigned same = __match_any_sync(0xFFFFFFFFu, on ? bank : 32 + lane);
        const int before = on ? cnt[bank] : 0;
        __syncwarp();
        if (on) {
          cq[a] = uint16_t(before + __popc(same & ((1u << lane) - 1u)));
          if ((same & ((1u << lane) - 1u)) == 0u) cnt[bank] = before + __popc(same);
        }
        __syncwarp();
      }
      // position in the (occurrence, bank) order: level q (the q-th entry of every bank that
      // has one) starts where the levels below it end, and inside it the banks go in order.
      // Levels and their bank masks are tabulated when there are at most kLayoutLevels.
      const int my_cnt = cnt[lane];
      int maxc = my_cnt;
      for (int o = 16; o > 0; o >>= 1) maxc = max(maxc, __shfl_xor_sync(0xFFFFFFFFu, maxc, o));
      const bool tabulated = maxc <= kLayoutLevels;
      if (tabulated) {
        int start = 0;
        for (int q = 0; q < maxc; ++q) {
          const unsigned mk = __ballot_sync(0xFFFFFFFFu, my_cnt > q);
          if (lane == 0) {
            lvl_mask[q] = mk;
            lvl_start[q] = uint16_t(start);
          }
          start += __popc(mk);
        }
        __syncwarp();
      }
      for (int a0 = 0; a0 < n; a0 += 32) {
        const int a = a0 + lane;
        if (a < n) {
          const int idx = ci[a], bank = idx & 31, q = cq[a];
          int pos = 0;
          if (tabulated) {
            pos = int(lvl_start[q]) + __popc(lvl_mask[q] & ((1u << bank) - 1u));
          } else {
#pragma unroll 8
            for (int bb = 0; bb < 32; ++bb) {
              const int c = cnt[bb];
              pos += min(c, q) + ((bb < bank && c > q) ? 1 : 0);
            }
          }
          dst_idx[c0 + pos] = idx;
          dst_rel[c0 + pos] = uint16_t(idx - s * W);
          dst_val[c0 + pos] = cv[a];
          if (dst_v16) dst_v16[c0 + pos].bits = bf16_bits_rn(cv[a]);  // exact: already rounded
        }
      }
      __syncwarp();
    }
    if (vmax != nullptr) {  // max |value| of the row's segment in this slab (0 when empty)
      for (int o = 16; o > 0; o >>= 1) vm = fmaxf(vm, __shfl_xor_sync(0xFFFFFFFFu, vm, o));
      // non-negative floats order like their bit patterns
      if (lane == 0 && vm > 0.f)
        atomicMax(reinterpret_cast<int*>(vmax + int64_t(s) * m + slot), __float_as_int(vm));
    }
  }
}

// vmax[s][r] = max |V| over row r's segment in slab s, for every slab and row (after a state
// import; a step keeps the table up to date when it inserts the row).
__global__ void __launch_bounds__(256) k_vmax_all(const float* __restrict__ V,
                                                  const int32_t* __restrict__ offs, int64_t k,
                                                  int m, float* __restrict__ vmax) {
  const int s = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int r = warp; r < m; r += 8) {
    const int b = offs[int64_t(s) * m + r], e = offs[int64_t(s + 1) * m + r];
    float vm = 0.f;
    for (int j = b + lane; j < e; j += 32) vm = fmaxf(vm, fabsf(V[int64_t(r) * k + j]));
    for (int o = 16; o > 0; o >>= 1) vm = fmaxf(vm, __shfl_xor_sync(0xFFFFFFFFu, vm, o));
    if (lane == 0) vmax[int64_t(s) * m + r] = vm;
  }
}

// Shared-memory layout of the slab kernels: float slab[W]; double/float per-row
// scratch; int32 seg[2 * m] (segment begin / end of every row in the current slab).
__host__ __device__ inline size_t slab_smem_bytes(int W, int m) {
  return size_t(W) * 4 + size_t(m) * 8 + size_t(m) * 8 + size_t(W) / 8;  // + bit mask (SP, x = a)
}

#ifndef EFCP_SLAB_THREADS
#define EFCP_SLAB_THREADS 1024
#endif
#ifndef EFCP_SLAB_BLOCKS
#define EFCP_SLAB_BLOCKS 1
#endif
constexpr int kSlabBlocksPerSM = EFCP_SLAB_BLOCKS;  // resident blocks of a slab kernel per SM
#ifndef EFCP_DEPTH
#define EFCP_DEPTH 12
#endif
constexpr int kSlabThreads = EFCP_SLAB_THREADS;  // threads of a slab-kernel block (one block per SM)
constexpr int kDepth = EFCP_DEPTH;               // groups of 32 entries a warp loads per pass

// Asks L2 for the lines of entries [b, e) of a row's index and value streams (at most 16
// lines of each; longer segments are covered at their start only).  Issued one row ahead
// of use, so that the loads of the next row find their data in L2 instead of waiting for
// HBM.
template <typename VT>
__device__ __forceinline__ void prefetch_segment(const uint16_t* Rr, const VT* Vr, int b, int e,
                                                 int lane) {
  const int half = lane & 15;
  const char* p = (lane < 16) ? reinterpret_cast<const char*>(Rr + b)
                              : reinterpret_cast<const char*>(Vr + b);
  const int bytes = (e - b) * (lane < 16 ? 2 : int(sizeof(VT)));
  if (half * 128 < bytes) asm volatile("prefetch.global.L2 [%0];" ::"l"(p + half * 128));
}

// The last pass over a segment: N groups of 32 entries (1 <= N <= kDepth), only the last of
// which can be incomplete.  `use(q, index, value)` consumes entry q of this lane; a lane
// without an entry in the last group gets (pad, 0).
template <int N, typename VT, typename F>
__device__ __forceinline__ void tail_pass(const uint16_t* pi, const VT* pv, bool last_on, int pad,
                                          F&& use) {
  int ii[N];
  float vv[N];
#pragma unroll
  for (int q = 0; q < N - 1; ++q) {
    ii[q] = __ldcs(pi + 32 * q);
    vv[q] = load_value(pv + 32 * q);
  }
  ii[N - 1] = last_on ? int(__ldcs(pi + 32 * (N - 1))) : pad;
  vv[N - 1] = last_on ? load_value(pv + 32 * (N - 1)) : 0.f;
#pragma unroll
  for (int q = 0; q < N; ++q) use(q, ii[q], vv[q]);
}

template <typename VT, typename F>
__device__ __forceinline__ void tail_dispatch(int groups, const uint16_t* pi, const VT* pv,
                                              bool last_on, int pad, F&& use) {
  static_assert(kDepth <= 16, "tail_dispatch covers up to 16 groups");
  switch (groups) {
#define EFCP_TAIL_CASE(N) \
    case N: if (N <= kDepth) tail_pass<(N <= kDepth ? N : 1)>(pi, pv, last_on, pad, use); break;
    EFCP_TAIL_CASE(1) EFCP_TAIL_CASE(2) EFCP_TAIL_CASE(3) EFCP_TAIL_CASE(4)
    EFCP_TAIL_CASE(5) EFCP_TAIL_CASE(6) EFCP_TAIL_CASE(7) EFCP_TAIL_CASE(8)
    EFCP_TAIL_CASE(9) EFCP_TAIL_CASE(10) EFCP_TAIL_CASE(11) EFCP_TAIL_CASE(12)
    EFCP_TAIL_CASE(13) EFCP_TAIL_CASE(14) EFCP_TAIL_CASE(15) EFCP_TAIL_CASE(16)
#undef EFCP_TAIL_CASE
    default: break;
  }
}

// Short segments.  When a row has only a group or two of entries per slab (low densities,
// small d), the burst above is one short dependent chain per row - offsets, loads, use,
// reduction - and a warp walks its rows one latency after the other.  This walk keeps kRing
// passes of kShort groups in flight per warp instead, across row boundaries: the loads of the
// pass kRing ahead are issued when a pass is consumed.
//   skip(r)   rows the caller does not want read (a zero weight);
//   empty(r)  called for every row that is skipped or has no entry in this slab;
//   use(p)    consumes a pass: p.ii[q] / p.vv[q] are entry q of this lane (index PAD and value 0
//             past the segment's end), p.row the row, p.last whether the row ends here.
constexpr int kShort = 2;  // groups of 32 entries per pass
constexpr int kRing = 4;   // passes in flight per warp
constexpr int kShortSegment = 96;  // entries per row and slab below which this walk is used

struct ShortPass {
  int ii[kShort];
  float vv[kShort];
  int row;
  bool last;
};

template <int PAD, typename VT, typename Skip, typename Empty, typename Use>
__device__ __forceinline__ void walk_short_segments(const uint16_t* __restrict__ R,
                                                    const VT* __restrict__ V, int64_t k,
                                                    const int32_t* seg, int m, int warp,
                                                    int nwarps, int lane, Skip&& skip,
                                                    Empty&& empty, Use&& use) {
  int r = warp - nwarps;  // row of the next pass to load
  int j = 0, e = 0;  // its next unread position and the end of its segment
  const uint16_t* Rr = R;
  const VT* Vr = V;
  auto next_row = [&]() {
    for (r += nwarps; r < m; r += nwarps) {
      j = seg[r];
      e = seg[m + r];
      if (j < e && !skip(r)) {
        Rr = R + int64_t(r) * k;
        Vr = V + int64_t(r) * k;
        return true;
      }
      empty(r);
    }
    return false;
  };
  auto load = [&](ShortPass& p) {
    p.row = r;
    const int left = e - j - lane;  // this lane has entry q of the pass when 32 q < left
#pragma unroll
    for (int q = 0; q < kShort; ++q) {
      const bool on = 32 * q < left;
      p.ii[q] = on ? int(Rr[j + lane + 32 * q]) : PAD;
      p.vv[q] = on ? load_value_cached(Vr + j + lane + 32 * q) : 0.f;
    }
    j += 32 * kShort;
    p.last = j >= e;
  };
  ShortPass buf[kRing];
  bool have[kRing];
  bool more = next_row();
#pragma unroll
  for (int i = 0; i < kRing; ++i) {
    have[i] = more;
    if (more) {
      load(buf[i]);
      if (buf[i].last) more = next_row();
    }
  }
  for (bool going = have[0]; going;) {
#pragma unroll
    for (int i = 0; i < kRing; ++i) {
      if (!have[i]) {
        going = false;
        break;
      }
      use(buf[i]);
      have[i] = more;
      if (more) {
        load(buf[i]);
        if (buf[i].last) more = next_row();
      }
    }
  }
}

// Shared -> global bulk copy (TMA, untiled form): both addresses 16-byte aligned, size a
// multiple of 16.  Used where the method leaves a large contiguous piece to move: a
// finished slab of the update.  The fence makes the accumulator's generic-proxy writes
// visible to the copy engine; wait_read returns when the engine has read shared memory
// (the global writes may still be in flight; they complete before the kernel ends).
__device__ __forceinline__ void bulk_store_fence() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void bulk_s2g(void* gdst, const void* ssrc, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst),
               "r"(uint32_t(__cvta_generic_to_shared(ssrc))), "r"(bytes)
               : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void bulk_store_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}

// Slab scheduling of the two slab kernels.  Slabs differ in weight (the kept entries
// cluster where the gradient is large), so blocks do not take a fixed share: block b starts
// with slab b and then draws the next unprocessed slab from a counter in global memory
// (cleared by the insert earlier in the step).  The draw for the next slab is issued at
// the start of the current one, so its latency is hidden.  Results do not depend on which
// block processes which slab, nor on the order the slabs are handed out in: LCG slabs are disjoint outputs, and SP writes one partial
// sum per (slab, row) that is reduced afterwards in slab order.

// Scalar products of every window row with the newest row c_t:
//   slab_part[s][r] = <row_r, c_t> restricted to slab s                      (both modes)
// and, when the right-hand side is the whole accumulator a_t = xi_t + c_t (ACC):
//   slab_part[s][m + r] = <row_r, xi_t> restricted to slab s,
// accumulated in fp64 (every fp32 x fp32 product is exact in fp64).  In ACC mode the slab in
// shared memory holds a_t (xi_t with the kept coordinates, which are zero in xi_t, filled
// in from c_t) and a bit mask says which coordinates belong to c_t, so that one gather
// serves both sums.  `stride` is the row length of slab_part (m or 2 m).
// VT is the format of the streamed values: float, or bf16raw (same values, half the bytes);
// Vf is the fp32 copy, used for the new row only.
// SHORT selects the ring walk for short segments (a variant of its own: the two walks have
// different register needs).
template <bool ACC, typename VT, bool SHORT = false>
__global__ void __launch_bounds__(kSlabThreads, kSlabBlocksPerSM) k_sp_rows(
    const uint16_t* __restrict__ R, const VT* __restrict__ V, const float* __restrict__ Vf,
    const int32_t* __restrict__ offs,
    int64_t k, int m, int W, int n_slabs, int slot, double* __restrict__ slab_part, int* ctr,
    const int32_t* __restrict__ order, const float* __restrict__ e, int64_t d) {
  extern __shared__ __align__(16) unsigned char smraw[];
  float* xs = reinterpret_cast<float*>(smraw);
  int32_t* seg = reinterpret_cast<int32_t*>(smraw + size_t(W) * 4 + size_t(m) * 8);
  uint32_t* mask = reinterpret_cast<uint32_t*>(smraw + size_t(W) * 4 + size_t(m) * 16);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const uint16_t* Rnew = R + int64_t(slot) * k;
  const float* Vnew = Vf + int64_t(slot) * k;
  const int stride = ACC ? 2 * m : m;
  __shared__ int s_next;
  for (int t = blockIdx.x; t < n_slabs;) {  // t: position in the hand-out order
    const int s = order[t];
    const int base = s * W;
    __syncthreads();
    if (tid == 0) s_next = int(gridDim.x) + atomicAdd(ctr, 1);
    if (ACC) {
      const int n = int(min(int64_t(W), d - base));
      for (int i = tid; i < W; i += blockDim.x) xs[i] = i < n ? e[int64_t(base) + i] : 0.f;
      for (int i = tid; i < (W >> 5); i += blockDim.x) mask[i] = 0u;
    } else {
      float4* xs4 = reinterpret_cast<float4*>(xs);
      for (int i = tid; i < (W >> 2); i += blockDim.x) xs4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    for (int r = tid; r < m; r += blockDim.x) {
      seg[r] = offs[int64_t(s) * m + r];
      seg[m + r] = offs[int64_t(s + 1) * m + r];
    }
    __syncthreads();
    {
      const int b = seg[slot], e2 = seg[m + slot];
      for (int j = b + tid; j < e2; j += blockDim.x) {
        const int i = Rnew[j];
        xs[i] = Vnew[j];
        if (ACC) atomicOr(&mask[i >> 5], 1u << (i & 31));
      }
    }
    __syncthreads();
    double* out = slab_part + int64_t(s) * stride;
    if constexpr (SHORT) {
      double acc = 0.0, acc2 = 0.0;  // <row, c> (two chains), or with ACC <row, c> and <row, xi>
      walk_short_segments<0>(
          R, V, k, seg, m, warp, nwarps, lane, [](int) { return false; },
          [&](int r) {
            if (lane == 0) {
              out[r] = 0.0;
              if (ACC) out[m + r] = 0.0;
            }
          },
          [&](const ShortPass& p) {
#pragma unroll
            for (int q = 0; q < kShort; ++q) {
              const int i = p.ii[q];
              const double pr = double(p.vv[q]) * double(xs[i]);
              if (ACC) {
                const bool in_c = (mask[i >> 5] >> (i & 31)) & 1u;
                acc += in_c ? pr : 0.0;
                acc2 += in_c ? 0.0 : pr;
              } else if (q & 1) {
                acc2 += pr;
              } else {
                acc += pr;
              }
            }
            if (p.last) {
              if (ACC) {
                acc = warp_sum(acc);
                acc2 = warp_sum(acc2);
                if (lane == 0) {
                  out[p.row] = acc;
                  out[m + p.row] = acc2;
                }
              } else {
                acc = warp_sum(acc + acc2);
                if (lane == 0) out[p.row] = acc;
              }
              acc = 0.0;
              acc2 = 0.0;
            }
          });
    } else {
    for (int r = warp; r < m; r += nwarps) {
      const int b = seg[r], e2 = seg[m + r];
      if (b >= e2) {
        if (lane == 0) {
          out[r] = 0.0;
          if (ACC) out[m + r] = 0.0;
        }
        continue;
      }
      const uint16_t* Rr = R + int64_t(r) * k;
      const VT* Vr = V + int64_t(r) * k;
      if (r + nwarps < m) {
        const int rn = r + nwarps;
        prefetch_segment(R + int64_t(rn) * k, V + int64_t(rn) * k, seg[rn], seg[m + rn], lane);
      }
      double acc = 0.0, acc2 = 0.0;  // COMPRESSED: two chains of <row, c>; ACC: <row, c>, <row, xi>
      auto use = [&](int q, int i, float v) {
        const double p = double(v) * double(xs[i]);
        if (ACC) {
          const bool in_c = (mask[i >> 5] >> (i & 31)) & 1u;
          acc += in_c ? p : 0.0;
          acc2 += in_c ? 0.0 : p;
        } else if (q & 1) {
          acc2 += p;
        } else {
          acc += p;
        }
      };
      // kDepth groups of 32 entries per pass: all loads of a pass are issued before the
      // first use.  Full passes need no bounds checks and address every load by a
      // constant offset from one pointer pair.
      int j0 = b + lane;
      for (; j0 + 32 * (kDepth - 1) < e2 - 31 + lane; j0 += 32 * kDepth) {
        const uint16_t* pi = Rr + j0;
        const VT* pv = Vr + j0;
        int ii[kDepth];
        float vv[kDepth];
#pragma unroll
        for (int q = 0; q < kDepth; ++q) {
          ii[q] = __ldcs(pi + 32 * q);
          vv[q] = load_value(pv + 32 * q);
        }
#pragma unroll
        for (int q = 0; q < kDepth; ++q) use(q, ii[q], vv[q]);
      }
      const int rem = e2 - (j0 - lane);  // entries left for the last pass (warp-uniform)
      if (rem > 0) {
        const int groups = (rem + 31) >> 5;
        tail_dispatch(groups, Rr + j0, Vr + j0, j0 + 32 * (groups - 1) < e2, 0,
                      [&](int q, int i, float v) { use(q, i, v); });
      }
      if (ACC) {
        acc = warp_sum(acc);
        acc2 = warp_sum(acc2);
        if (lane == 0) {
          out[r] = acc;
          out[m + r] = acc2;
        }
      } else {
        acc = warp_sum(acc + acc2);
        if (lane == 0) out[r] = acc;
      }
    }
    }  // burst walk
    t = s_next;
  }
}

// Linear combination of the window rows, u = sum_r w_r row_r, one slab at a time in a
// shared-memory accumulator (Eq. (2) in the form that has no x/lambda term, see
// efcp_mxm.cuh).  Every element of u is written exactly once.
// With ACC (x = a_t) the accumulator of a slab starts from xi_t / lambda instead of zero.
// The parameter update fused into the write-out of the linear combination (theta == nullptr:
// off, u is written instead): theta <- decay theta + neg_step u.
struct LcgApply {
  float* theta;
  float decay, neg_step;
};

// FIXED: the accumulator of a slab holds int32 fixed-point sums.  An fp32 atomicAdd on shared
// memory is a compare-and-swap loop, the integer one is a single operation of less than half
// the cost.  Per slab, bound = sum_r |w_r| max|V_r in the slab| is an upper bound of every
// partial sum of every coordinate, so with scale = 2^e, bound * scale < 2^30, nothing can
// overflow; each product is rounded to a multiple of q = 1 / scale (error at most q / 2, random
// in sign), which over the slab's n entries adds up to a variance of n q^2 / 12.  The slab is
// accepted if that is below (1e-5 |u_slab|)^2 - ten times inside the tolerance of the update,
// slab by slab and therefore for the whole vector - and otherwise accumulated again with fp32
// atomics (its 2.5 MB of entries are still in L2).  Integer sums do not depend on the order of
// the adds: the accepted slabs of u are reproducible bit for bit.
template <bool VEC, bool ACC, typename VT, bool FIXED = false, bool SHORT = false>
__global__ void __launch_bounds__(kSlabThreads, kSlabBlocksPerSM) k_lcg(
    const uint16_t* __restrict__ R, const VT* __restrict__ V, const int32_t* __restrict__ offs,
    int64_t k, int m, int W, int n_slabs, const double* __restrict__ w64,
    const double* __restrict__ dw64, double* __restrict__ w_out, float* __restrict__ u,
    int64_t d, int* ctr, const int32_t* __restrict__ order, int slab0,
    const float* __restrict__ xi,
    float inv_lambda, LcgApply ap, const float* __restrict__ vmax = nullptr,
    unsigned long long* __restrict__ redo_count = nullptr, double fixed_tol2 = 1e-10) {
  static_assert(!(FIXED && ACC), "the fixed-point accumulator starts from zero");
  extern __shared__ __align__(16) unsigned char smraw[];
  __shared__ double red[32];
  float* acc = reinterpret_cast<float*>(smraw);
  float* wc = reinterpret_cast<float*>(smraw + size_t(W) * 4);
  int32_t* seg = reinterpret_cast<int32_t*>(smraw + size_t(W) * 4 + size_t(m) * 8);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  // the weights: the m x m stage's solution plus its refinement step (dw64 == nullptr: none)
  for (int r = tid; r < m; r += blockDim.x) {
    const double v = w64[r] + (dw64 ? dw64[r] : 0.0);
    wc[r] = float(v);
    if (blockIdx.x == 0) w_out[r] = v;
  }
  float4* acc4 = reinterpret_cast<float4*>(acc);
  for (int i = tid; i < (W >> 2); i += blockDim.x) acc4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  __shared__ int s_next;
  for (int t = blockIdx.x; t < n_slabs;) {  // t: position in the hand-out order
    // order == nullptr: this launch covers the slabs slab0 .. slab0 + n_slabs - 1 in their
    // natural order (the host entry point launches ranges so that finished ranges can leave)
    const int s = order ? order[t] : slab0 + t;
    __syncthreads();
    if (tid == 0) s_next = int(gridDim.x) + atomicAdd(ctr, 1);
    for (int r = tid; r < m; r += blockDim.x) {
      seg[r] = offs[int64_t(s) * m + r];
      seg[m + r] = offs[int64_t(s + 1) * m + r];
    }
    const int base = s * W;
    if (ACC) {
      const int n = int(min(int64_t(W), d - base));
      for (int i = tid; i < n; i += blockDim.x) acc[i] = xi[int64_t(base) + i] * inv_lambda;
    }
    __syncthreads();
    // every row's segment of this slab, scaled by the row's weight, into the accumulator
    auto accumulate = [&](auto add) {
      if constexpr (SHORT) {
        walk_short_segments<-1>(
            R, V, k, seg, m, warp, nwarps, lane, [&](int r) { return wc[r] == 0.f; },
            [](int) {},
            [&](const ShortPass& p) {
              const float c = wc[p.row];
#pragma unroll
              for (int q = 0; q < kShort; ++q)
                if (p.ii[q] >= 0) add(p.ii[q], c * p.vv[q]);
            });
      } else {
      for (int r = warp; r < m; r += nwarps) {
        const int b = seg[r], e = seg[m + r];
        const float c = wc[r];
        if (b >= e || c == 0.f) continue;
        const uint16_t* Rr = R + int64_t(r) * k;
        const VT* Vr = V + int64_t(r) * k;
        if (r + nwarps < m) {
          const int rn = r + nwarps;
          prefetch_segment(R + int64_t(rn) * k, V + int64_t(rn) * k, seg[rn], seg[m + rn], lane);
        }
        int j0 = b + lane;
        for (; j0 + 32 * (kDepth - 1) < e - 31 + lane; j0 += 32 * kDepth) {  // full passes
          const uint16_t* pi = Rr + j0;
          const VT* pv = Vr + j0;
          int ii[kDepth];
          float vv[kDepth];
  #pragma unroll
          for (int q = 0; q < kDepth; ++q) {
            ii[q] = __ldcs(pi + 32 * q);
            vv[q] = load_value(pv + 32 * q);
          }
  #pragma unroll
          for (int q = 0; q < kDepth; ++q) add(ii[q], c * vv[q]);
        }
        const int rem = e - (j0 - lane);  // entries left for the last pass (warp-uniform)
        if (rem > 0) {
          const int groups = (rem + 31) >> 5;
          tail_dispatch(groups, Rr + j0, Vr + j0, j0 + 32 * (groups - 1) < e, -1,
                        [&](int, int i, float v) {
                          if (i >= 0) add(i, c * v);
                        });
        }
      }
      }  // burst walk
    };
    const int64_t gbase = int64_t(s) * W;
    const int n = int(min(int64_t(W), d - gbase));
    bool by_float = true;
    if (FIXED) {
      double part = 0.0, cnt = 0.0;
      for (int r = tid; r < m; r += blockDim.x) {
        part += double(fabsf(wc[r])) * double(vmax[int64_t(s) * m + r]);
        cnt += double(seg[m + r] - seg[r]);
      }
      const double bound = block_sum(part, red);
      const double n_entries = block_sum(cnt, red);
      if (bound > 0.0 && bound < 1e30) {
        int ex;
        (void)frexp(bound, &ex);  // bound < 2^ex
        ex = max(ex, -90);
        const float scale = ldexpf(1.0f, 30 - ex);
        int* acci = reinterpret_cast<int*>(acc);
        accumulate([&](int i, float t) { atomicAdd(acci + i, __float2int_rn(t * scale)); });
        __syncthreads();
        const float q = ldexpf(1.0f, ex - 30);
        double nrm2 = 0.0;
        for (int i = tid; i < n; i += blockDim.x) {
          const float v = float(acci[i]) * q;
          acc[i] = v;
          nrm2 += double(v) * double(v);
        }
        nrm2 = block_sum(nrm2, red);
        by_float = !(n_entries * double(q) * double(q) / 12.0 <= fixed_tol2 * nrm2);
        if (by_float) {  // too coarse for this slab: start over
          if (tid == 0 && redo_count) atomicAdd(redo_count, 1ULL);
          for (int i = tid; i < (W >> 2); i += blockDim.x) acc4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
          __syncthreads();
        }
      }
    }
    if (by_float) accumulate([&](int i, float t) { atomicAdd(&acc[i], t); });
    if (VEC) bulk_store_fence();  // every thread's adds, before the barrier that orders them
    __syncthreads();
    // write the slab out and clear it for the next one
    if (ap.theta != nullptr) {
      // the parameter update takes the finished slab of u straight from shared memory:
      // theta <- decay theta + (-eta) u; u itself is not written
      float* th = ap.theta + gbase;
      if ((reinterpret_cast<uintptr_t>(th) & 15) == 0 && (n & 3) == 0) {
        float4* th4 = reinterpret_cast<float4*>(th);
        for (int i = tid; i < (n >> 2); i += blockDim.x) {
          float4 t4 = th4[i];
          const float4 a4 = acc4[i];
          t4.x = __fmaf_rn(ap.neg_step, a4.x, __fmul_rn(ap.decay, t4.x));
          t4.y = __fmaf_rn(ap.neg_step, a4.y, __fmul_rn(ap.decay, t4.y));
          t4.z = __fmaf_rn(ap.neg_step, a4.z, __fmul_rn(ap.decay, t4.z));
          t4.w = __fmaf_rn(ap.neg_step, a4.w, __fmul_rn(ap.decay, t4.w));
          th4[i] = t4;
          acc4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
      } else {
        for (int i = tid; i < n; i += blockDim.x) {
          th[i] = __fmaf_rn(ap.neg_step, acc[i], __fmul_rn(ap.decay, th[i]));
          acc[i] = 0.f;
        }
      }
    } else if (VEC && (n & 3) == 0) {
      // the slab is one contiguous, 16-byte aligned piece of u: a single bulk copy (the
      // copy engine reads shared memory itself) instead of a load and a store per thread
      if (tid == 0) {
        bulk_s2g(u + gbase, acc, uint32_t(n) * 4u);
        bulk_store_wait_read();  // the engine has read the accumulator: it can be cleared
      }
      __syncthreads();
      for (int i = tid; i < (n >> 2); i += blockDim.x) acc4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    } else if (VEC) {
      float4* u4 = reinterpret_cast<float4*>(u + gbase);
      const int nv = n >> 2;
      for (int i = tid; i < nv; i += blockDim.x) {
        __stcs(u4 + i, acc4[i]);
        acc4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      }
      for (int i = (nv << 2) + tid; i < n; i += blockDim.x) {
        u[gbase + i] = acc[i];
        acc[i] = 0.f;
      }
    } else {
      for (int i = tid; i < n; i += blockDim.x) {
        u[gbase + i] = acc[i];
        acc[i] = 0.f;
      }
    }
    t = s_next;
  }
}

// ---- consistency checks of the window's derived structures (efcp_validate, EFCP_DEBUG_CHECKS)

// One block per (slab, row) for the rows [row0, row_end): offsets monotone and ending at the row
// length (full_rows: every row holds exactly k entries), entries inside the slab, R == I - s W.
__global__ void __launch_bounds__(128) k_validate_rows(
    const int32_t* __restrict__ I, const uint16_t* __restrict__ R, const int32_t* __restrict__ offs,
    int64_t k, int64_t d, int m, int W, int n_slabs, int row0, int row_end, int full_rows,
    unsigned long long* __restrict__ bad) {
  const int s = blockIdx.x, r = row0 + blockIdx.y;
  if (r >= row_end) return;
  const int b = offs[int64_t(s) * m + r], e = offs[int64_t(s + 1) * m + r];
  unsigned long long v = 0;
  if (threadIdx.x == 0) {
    if (b > e || b < 0 || e > k) ++v;
    if (s == 0 && b != 0) ++v;
    if (s == n_slabs - 1 && full_rows && e != k) ++v;  // (a shard's rows vary in length)
  }
  const int64_t lo = int64_t(s) * W, hi = lo + W < d ? lo + W : d;
  for (int j = b + threadIdx.x; j < e && j < k; j += blockDim.x) {
    const int64_t idx = I[int64_t(r) * k + j];
    if (idx < lo || idx >= hi) ++v;
    else if (int64_t(R[int64_t(r) * k + j]) != idx - lo) ++v;
  }
  if (v) atomicAdd(bad, v);
}

// colsum[s] == sum over rows of offs[s][r]
__global__ void __launch_bounds__(256) k_validate_colsum(const int32_t* __restrict__ offs,
                                                          const int64_t* __restrict__ colsum,
                                                          int m, int n_slabs,
                                                          unsigned long long* __restrict__ bad) {
  __shared__ double sm[32];
  const int s = blockIdx.x;
  double acc = 0.0;  // exact: sums stay far below 2^53
  for (int r = threadIdx.x; r < m; r += blockDim.x) acc += double(offs[int64_t(s) * m + r]);
  acc = block_sum(acc, sm);
  if (threadIdx.x == 0 && int64_t(acc) != colsum[s]) atomicAdd(bad, 1ull);
}

// EFCP_DEBUG_CHECKS: a step's consistency checks found violations -> sticky internal error.
__global__ void k_fold_bad(const unsigned long long* __restrict__ bad, Scalars* sc) {
  if (*bad != 0ull) atomicOr(&sc->status, kStCount);
}

}  // namespace efcp
