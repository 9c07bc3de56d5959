// Host side of the EFCP C ABI (see include/efcp.h): handle, allocation, and the kernel
// sequence of one step.  Everything a step computes runs in the kernels of this
// directory; there is no CPU fallback.
#include "efcp.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <utility>
#include <vector>

#include "efcp_common.cuh"
#include "efcp_blockwise.cuh"
#include "efcp_update.cuh"
#include "efcp_ggt.cuh"
#include "efcp_mxm.cuh"
#include "efcp_topk.cuh"
#include "efcp_window.cuh"
#include "efcp_select.cuh"

using namespace efcp;

struct efcp_ctx {
  int64_t d = 0, k = 0;  // k: entries per window row
  int64_t k_req = 0;     // the k of the create call (block-wise Top-k keeps a little more)
  int block = 0, n_blocks = 0;  // block-wise Top-k: block length in coordinates, number of blocks
  int blk_resident = 1;         // thread blocks of the block-wise kernel one SM holds
  double2* ggt_rot = nullptr;   // Sparse GGT: the rotations of one step's eigendecomposition
  float* vmax = nullptr;        // fixed-point LCG: max |V| per (slab, row)
  unsigned long long* lcg_redo = nullptr;  // slabs the fixed-point LCG redid in fp32
  double lcg_tol2 = 1e-10;      // its acceptance bound, squared: (1e-5)^2
  double* upd_norm = nullptr;   // [0]: |u|^2 of the last efcp_update_norm, then its partial sums
  int64_t norm_t = -1;          // step count at that call
  int blk_threads = kBlkThreads;  // threads per thread block of the block-wise kernel
  uint32_t* blk_T = nullptr;    // per block: last step's threshold key
  int32_t m = 0;
  float lambda = 0.f;
  uint32_t flags = 0;
  int device = 0;
  int num_sms = 0;
  int64_t t = 0;
  int W = 0, n_slabs = 0, n_chunks = 0;
  int grid_slab = 0;  // blocks of the slab kernels (SP partials are per block)
  // state
  float* e = nullptr;
  int32_t* I = nullptr;
  uint16_t* R = nullptr;  // slab-relative copy of I, the index stream SP and LCG read
  bf16raw* V16 = nullptr; // EFCP_VALUES_BF16: the value stream SP and LCG read (V holds the same values)
  float* V = nullptr;
  int32_t* offs = nullptr;
  double* S = nullptr;
  double* B = nullptr;
  // scratch
  uint32_t* hist = nullptr;  // kBins1 + kBins2 + kBins3
  int32_t* chunk_off = nullptr;
  uint16_t* bk_off = nullptr;  // speculative candidate buckets, one of kChunk entries per chunk
  float* bk_val = nullptr;
  bool spec = true;            // EFCP_NO_SPEC=1 forces the two-pass candidate path
  int32_t* sel_idx = nullptr;  // the selection of the current step, ascending (k entries)
  float* sel_val = nullptr;
  int32_t* sel_gt = nullptr;
  int32_t* sel_eq = nullptr;
  Scalars* sc = nullptr;
  double* slab_part = nullptr;  // SP: one partial sum per (slab, row)
  double* partial = nullptr;    // SP: kSpParts x m sums of slab partials
  double* vecs = nullptr;  // 10 m-vectors: delta, aprime, y, bold, z, w, res, dw, rhs, final w
  int32_t* blk_tot = nullptr;   // selection kernel: per-block totals
  unsigned int* bar = nullptr;  // grid barriers of the two cooperative kernels (2 words each)
  int sel_grid = 0, mxm_grid = 0;  // their grids: every block resident
  // a coordinate shard of a larger state (efcp_create_shard); otherwise d_global == d etc.
  int64_t d_global = 0, k_global = 0;
  int shard = 0, n_shards = 1;
  uint32_t* shard_tot = nullptr;  // per shard: entries above / at the threshold key
  int next_phase = 0;             // of efcp_shard_phase
  bool is_shard = false;
  bool split_phases = false;      // EFCP_SPLIT_PHASES=1: one launch per phase (profiling)
  int short_rows = 0;             // rows have few entries per slab: the slab kernels' ring walk
  float* wf = nullptr;
  int* slab_ctr = nullptr;   // work counters of the slab kernels (SP, LCG)
  int64_t* colsum = nullptr; // n_slabs + 1 column sums of offs
  int32_t* order = nullptr;  // n_slabs slabs, heavy first
  float* stage_g = nullptr;  // efcp_step_host staging
  float* stage_u = nullptr;
  cudaStream_t copy_stream = nullptr;    // efcp_step_host: device-to-host copies of finished ranges
  cudaEvent_t host_ev[4] = {nullptr, nullptr, nullptr, nullptr};
  int last_cuda = 0;
  int launches = 0;
  unsigned long long* dbg_bad = nullptr;  // EFCP_DEBUG_CHECKS: violations found after a step
  int hook_drop_loads = 0;  // efcp_test_hook: the block-wise kernel arms its wait, copies nothing
  // stage timing (efcp_profile_*): 5 events per recorded step
  std::vector<cudaEvent_t> prof_ev;
  int prof_cap = 0, prof_n = 0;
  bool prof_on = false;
  std::vector<void*> allocs;
  // where the device memory comes from: cudaMalloc per buffer (ws_base == nullptr), or pieces
  // of one caller-supplied workspace; ws_measure only adds the sizes up
  unsigned char* ws_base = nullptr;
  int64_t ws_cap = 0, ws_used = 0;
  bool ws_measure = false;
};

namespace {

constexpr int kSpParts = 32;  // second-level partial sums of the scalar products
constexpr int kMaxCoopBlocks = 1024;  // largest grid of the cooperative kernels
constexpr int kHostRanges = 4;  // efcp_step_host: ranges of slabs that leave for the host one by one
static_assert(kHostRanges == sizeof(efcp_ctx::host_ev) / sizeof(cudaEvent_t), "one event per range");

struct Sizes {
  int W, n_slabs, n_chunks, grid_slab;
};

int pick_slab_width(int64_t d, int m, int num_sms) {
  int W = (40960 / kSlabBlocksPerSM) & ~31;  // 160 KB of the 227 KB a block may use
  if (const char* env = getenv("EFCP_SLAB_W")) {
    const int v = atoi(env);
    if (v >= 256 && v <= 49152 && (v & 31) == 0) return v;
  }
  // shared memory: W*4 + 16*m must stay under the 227 KB per-block limit
  while (slab_smem_bytes(W, m) * kSlabBlocksPerSM > 220 * 1024 && W > 1024) W >>= 1;
  // at least one slab per SM (the slab kernels run one block per SM and rebalance by
  // drawing slabs from a counter), but no slab narrower than 2048 coordinates: below that
  // a row's segment is a handful of entries and the per-row bookkeeping dominates
  while (W / 2 >= 2048 && (d + W - 1) / W < int64_t(num_sms)) W = (W / 2) & ~31;
  return W;
}

inline int64_t align256(int64_t b) { return (b + 255) & ~int64_t(255); }
constexpr int64_t align256c(int64_t b) { return (b + 255) & ~int64_t(255); }

Sizes compute_sizes(int64_t d, int32_t m, int num_sms) {
  Sizes z;
  z.W = pick_slab_width(d, m, num_sms);
  z.n_slabs = int((d + z.W - 1) / z.W);
  z.n_chunks = int((d + kChunk - 1) / kChunk);
  z.grid_slab = z.n_slabs < num_sms * kSlabBlocksPerSM ? z.n_slabs : num_sms * kSlabBlocksPerSM;
  return z;
}

bool valid_args(int64_t d, int32_t m, int64_t k) {
  return d >= 1 && m >= 1 && m <= 4096 && k >= 1 && k <= d && d < (int64_t(1) << 31);
}

__global__ void k_init_rows(int32_t* __restrict__ I, int64_t k, int64_t total) {
  for (int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
       i += int64_t(gridDim.x) * blockDim.x)
    I[i] = int32_t(i % k);
}

#define EFCP_CUDA(call)                         \
  do {                                          \
    cudaError_t err__ = (call);                 \
    if (err__ != cudaSuccess) {                 \
      ctx->last_cuda = int(err__);              \
      return EFCP_ECUDA;                        \
    }                                           \
  } while (0)

#define EFCP_LAUNCHED()                         \
  do {                                          \
    ++ctx->launches;                            \
    cudaError_t err__ = cudaGetLastError();     \
    if (err__ != cudaSuccess) {                 \
      ctx->last_cuda = int(err__);              \
      return EFCP_ECUDA;                        \
    }                                           \
  } while (0)

template <typename T>
int dev_alloc(efcp_ctx* ctx, T** p, int64_t bytes) {
  const int64_t need = align256(bytes);
  if (ctx->ws_measure) {
    ctx->ws_used += need;
    *p = nullptr;
    return EFCP_OK;
  }
  if (ctx->ws_base) {
    if (ctx->ws_used + need > ctx->ws_cap) return EFCP_ENOMEM;
    *p = reinterpret_cast<T*>(ctx->ws_base + ctx->ws_used);
    ctx->ws_used += need;
    return EFCP_OK;
  }
  void* q = nullptr;
  cudaError_t err = cudaMalloc(&q, size_t(need));
  if (err != cudaSuccess) {
    ctx->last_cuda = int(err);
    (void)cudaGetLastError();
    return EFCP_ENOMEM;
  }
  ctx->allocs.push_back(q);
  *p = static_cast<T*>(q);
  return EFCP_OK;
}

int status_to_code(uint32_t st) {
  if (st & kStCount) return EFCP_EINTERNAL;
  if (st & kStTimeout) return EFCP_ETIMEOUT;
  if (st & (kStNonFinite | kStPivot)) return EFCP_ENUMERIC;
  return EFCP_OK;
}

int sync_status(efcp_ctx* ctx) {
  EFCP_CUDA(cudaSetDevice(ctx->device));
  EFCP_CUDA(cudaDeviceSynchronize());
  Scalars h;
  EFCP_CUDA(cudaMemcpy(&h, ctx->sc, sizeof(h), cudaMemcpyDeviceToHost));
  return status_to_code(h.status);
}

void free_all(efcp_ctx* ctx) {
  for (void* p : ctx->allocs) cudaFree(p);
  ctx->allocs.clear();
  for (cudaEvent_t ev : ctx->prof_ev) cudaEventDestroy(ev);
  ctx->prof_ev.clear();
  for (cudaEvent_t& ev : ctx->host_ev) {
    if (ev) cudaEventDestroy(ev);
    ev = nullptr;
  }
  if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
  ctx->copy_stream = nullptr;
}

inline void prof_mark(efcp_ctx* ctx, int which, cudaStream_t st) {
  if (ctx->prof_on && ctx->prof_n < ctx->prof_cap)
    cudaEventRecord(ctx->prof_ev[size_t(ctx->prof_n) * 5 + which], st);
}

// calls f with the instantiation of the block-wise kernel for `threads` threads per block
template <typename F>
bool for_block_kernel(int threads, bool aligned, F f) {
  if (aligned) {
    if (threads == 128) return f(k_ef_block_select<true, 128>);
    if (threads == 256) return f(k_ef_block_select<true, 256>);
    return f(k_ef_block_select<true, 512>);
  }
  if (threads == 128) return f(k_ef_block_select<false, 128>);
  if (threads == 256) return f(k_ef_block_select<false, 256>);
  return f(k_ef_block_select<false, 512>);
}

}  // namespace

extern "C" {

const char* efcp_strerror(int code) {
  switch (code) {
    case EFCP_OK: return "ok";
    case EFCP_EINVAL: return "invalid argument";
    case EFCP_ENOMEM: return "out of memory";
    case EFCP_ECUDA: return "CUDA runtime error (see efcp_last_cuda_error)";
    case EFCP_ENUMERIC: return "non-finite input or non-positive pivot in the m x m update";
    case EFCP_ETIMEOUT: return "bounded device-side wait expired";
    case EFCP_EINTERNAL: return "internal consistency check failed";
    case EFCP_ETOOBIG: return "size exceeds the fixed scratch capacity of the allocation-free entry point";
    default: return "unknown error code";
  }
}

int64_t efcp_state_bytes(int64_t d, int32_t m, int64_t k) {
  return efcp_workspace_bytes(d, m, k, EFCP_RHS_COMPRESSED, 0);
}

int efcp_create(efcp_ctx** out, int64_t d, int32_t m, int64_t k, float lambda) {
  return efcp_create_ex(out, d, m, k, lambda, EFCP_RHS_COMPRESSED);
}

int efcp_create_ex(efcp_ctx** out, int64_t d, int32_t m, int64_t k, float lambda,
                   uint32_t flags) {
  return efcp_create_blockwise(out, d, m, k, lambda, flags, 0);
}

int64_t efcp_row_length(efcp_ctx* ctx) { return ctx ? ctx->k : -1; }

}  // extern "C"

namespace {

// Checks the arguments of a create call and fills in everything of the handle that follows
// from them and from the SM count (no device memory yet).
int configure(efcp_ctx* ctx, int64_t d, int32_t m, int64_t k, float lambda, uint32_t flags,
              int32_t block, int num_sms) {
  if (!valid_args(d, m, k) || !(lambda > 0.f) || !std::isfinite(lambda)) return EFCP_EINVAL;
  if (flags & ~(EFCP_RHS_ACCUMULATOR | EFCP_VALUES_BF16 | EFCP_PRECOND_GGT | EFCP_LCG_FP32 |
                EFCP_DEBUG_CHECKS))
    return EFCP_EINVAL;
  if ((flags & EFCP_RHS_ACCUMULATOR) && (flags & EFCP_VALUES_BF16)) return EFCP_EINVAL;
  // EFCP_LCG=fp32 / fixed in the environment overrides the flag (testing)
  if (const char* env = getenv("EFCP_LCG")) {
    if (!std::strcmp(env, "fp32")) flags |= EFCP_LCG_FP32;
    if (!std::strcmp(env, "fixed")) flags &= ~EFCP_LCG_FP32;
  }
  if ((flags & EFCP_PRECOND_GGT) && ((flags & EFCP_RHS_ACCUMULATOR) || m > kGgtMaxM))
    return EFCP_EINVAL;
  if (block != 0 && (block < 32 || block > kBlkMax || (block & 31))) return EFCP_EINVAL;
  const int64_t k_req = k;
  int n_blocks = 0;
  if (block) {  // the row length is the sum of the per-block counts
    n_blocks = int((d + block - 1) / block);
    const int64_t last = d - int64_t(n_blocks - 1) * block;
    k = int64_t(n_blocks - 1) * block_count(block, k_req, d) + block_count(last, k_req, d);
  }
  ctx->num_sms = num_sms;
  ctx->d = d; ctx->m = m; ctx->k = k; ctx->lambda = lambda; ctx->flags = flags;
  ctx->k_req = k_req; ctx->block = block; ctx->n_blocks = n_blocks;
  ctx->d_global = d; ctx->k_global = k; ctx->shard = 0; ctx->n_shards = 1;
  const Sizes z = compute_sizes(d, m, ctx->num_sms);
  ctx->W = z.W; ctx->n_slabs = z.n_slabs; ctx->n_chunks = z.n_chunks;
  ctx->grid_slab = z.grid_slab;
  ctx->short_rows = k / z.n_slabs < kShortSegment ? 1 : 0;
  if (const char* env = getenv("EFCP_NO_SPEC")) ctx->spec = atoi(env) == 0;
  if (const char* env = getenv("EFCP_SPLIT_PHASES")) ctx->split_phases = atoi(env) != 0;
  // EFCP_LCG_FIXED_TOL: relative error a slab of the fixed-point LCG may have before it is redone
  // in fp32 (default 1e-5; 0 sends every slab through the fallback, which a parity test does)
  if (const char* env = getenv("EFCP_LCG_FIXED_TOL")) {
    const double tol = atof(env);
    if (tol >= 0.0 && tol <= 1e-4) ctx->lcg_tol2 = tol * tol;
  }
  return EFCP_OK;
}

// Every device buffer of a configured handle, in one fixed order (efcp_workspace_bytes runs
// the same list with an arena that only adds up the sizes).
int alloc_all(efcp_ctx* ctx) {
  const int64_t d = ctx->d, k = ctx->k;
  const int m = ctx->m, n_slabs = ctx->n_slabs, n_chunks = ctx->n_chunks;
  const uint32_t flags = ctx->flags;
  const int64_t mk = int64_t(m) * k;
  const bool lcg_fixed = !(flags & EFCP_LCG_FP32) && !(flags & EFCP_RHS_ACCUMULATOR);
  const int64_t sums = (flags & EFCP_RHS_ACCUMULATOR) ? 2 : 1;
  int rc = EFCP_OK;
#define EFCP_ALLOC(field, bytes) \
  if ((rc = dev_alloc(ctx, &ctx->field, (bytes)))) return rc
  EFCP_ALLOC(e, d * 4);
  EFCP_ALLOC(I, mk * 4);
  EFCP_ALLOC(R, mk * 2);
  if (flags & EFCP_VALUES_BF16) EFCP_ALLOC(V16, mk * 2);
  EFCP_ALLOC(V, mk * 4);
  EFCP_ALLOC(offs, int64_t(n_slabs + 1) * m * 4);
  EFCP_ALLOC(S, int64_t(m) * m * 8);
  EFCP_ALLOC(B, int64_t(m) * m * 8);
  EFCP_ALLOC(hist, (kBins1 + kBins2 + kBins3) * 4);
  EFCP_ALLOC(chunk_off, int64_t(n_chunks + 1) * 4);
  EFCP_ALLOC(sel_gt, int64_t(n_chunks + 1) * 4);
  EFCP_ALLOC(sel_eq, int64_t(n_chunks + 1) * 4);
  EFCP_ALLOC(bk_off, int64_t(n_chunks) * kChunk * 2);
  EFCP_ALLOC(bk_val, int64_t(n_chunks) * kChunk * 4);
  EFCP_ALLOC(sel_idx, k * 4);
  EFCP_ALLOC(sel_val, k * 4);
  EFCP_ALLOC(sc, sizeof(Scalars));
  EFCP_ALLOC(slab_part, int64_t(n_slabs) * m * 8 * sums);
  EFCP_ALLOC(upd_norm, int64_t(kUpdMaxBlocks + 1) * 8);
  if (lcg_fixed) {
    EFCP_ALLOC(vmax, int64_t(n_slabs) * m * 4);
    EFCP_ALLOC(lcg_redo, 8);
  }
  if (flags & EFCP_PRECOND_GGT) EFCP_ALLOC(ggt_rot, ggt_log_entries(m) * 16);
  EFCP_ALLOC(partial, int64_t(kSpParts) * m * 8 * sums);
  EFCP_ALLOC(vecs, int64_t(10) * m * 8);
  EFCP_ALLOC(blk_tot, int64_t(2) * kMaxCoopBlocks * 4);
  EFCP_ALLOC(bar, 64);
  EFCP_ALLOC(wf, int64_t(m) * 4);
  EFCP_ALLOC(slab_ctr, 256);
  // block-wise Top-k, per block: last step's threshold key, then log2 of the candidate margin
  if (ctx->block) EFCP_ALLOC(blk_T, int64_t(ctx->n_blocks) * 8);
  EFCP_ALLOC(colsum, int64_t(n_slabs + 1) * 8);
  EFCP_ALLOC(order, int64_t(n_slabs) * 4);
  EFCP_ALLOC(dbg_bad, 8);
  if (ctx->is_shard) EFCP_ALLOC(shard_tot, int64_t(ctx->n_shards) * 8);
#undef EFCP_ALLOC
  return EFCP_OK;
}

// Initial contents (empty window, xi = 0, B = I / (m lambda)) and kernel attributes.
bool init_state(efcp_ctx* ctx) {
  const int64_t d = ctx->d, k = ctx->k;
  const int m = ctx->m, n_slabs = ctx->n_slabs;
  const int64_t mk = int64_t(m) * k;
  bool ok = true;
  ok &= cudaMemset(ctx->e, 0, size_t(d) * 4) == cudaSuccess;
  ok &= cudaMemset(ctx->V, 0, size_t(mk) * 4) == cudaSuccess;
  ok &= cudaMemset(ctx->R, 0, size_t(mk) * 2) == cudaSuccess;
  if (ctx->V16) ok &= cudaMemset(ctx->V16, 0, size_t(mk) * 2) == cudaSuccess;
  ok &= cudaMemset(ctx->offs, 0, size_t(n_slabs + 1) * m * 4) == cudaSuccess;
  ok &= cudaMemset(ctx->S, 0, size_t(m) * m * 8) == cudaSuccess;
  ok &= cudaMemset(ctx->colsum, 0, size_t(n_slabs + 1) * 8) == cudaSuccess;
  ok &= cudaMemset(ctx->hist, 0, (kBins1 + kBins2 + kBins3) * 4) == cudaSuccess;
  ok &= cudaMemset(ctx->sc, 0, sizeof(Scalars)) == cudaSuccess;
  ok &= cudaMemset(ctx->vecs, 0, size_t(10) * m * 8) == cudaSuccess;
  ok &= cudaMemset(ctx->bar, 0, 64) == cudaSuccess;
  ok &= cudaMemset(ctx->blk_tot, 0, size_t(2) * kMaxCoopBlocks * 4) == cudaSuccess;
  ok &= cudaMemset(ctx->wf, 0, size_t(m) * 4) == cudaSuccess;
  // a step that gives up (EFCP_ETIMEOUT) leaves the selection buffers as they were; the
  // kernels after it must still find indices inside [0, d)
  ok &= cudaMemset(ctx->sel_idx, 0, size_t(k) * 4) == cudaSuccess;
  ok &= cudaMemset(ctx->sel_val, 0, size_t(k) * 4) == cudaSuccess;
  ok &= cudaMemset(ctx->dbg_bad, 0, 8) == cudaSuccess;
  if (ctx->shard_tot)
    ok &= cudaMemset(ctx->shard_tot, 0, size_t(ctx->n_shards) * 8) == cudaSuccess;
  if (ctx->vmax) {
    ok &= cudaMemset(ctx->vmax, 0, size_t(n_slabs) * m * 4) == cudaSuccess;
    ok &= cudaMemset(ctx->lcg_redo, 0, 8) == cudaSuccess;
  }
  if (ctx->blk_T) ok &= cudaMemset(ctx->blk_T, 0, size_t(ctx->n_blocks) * 8) == cudaSuccess;
  k_init_rows<<<ctx->num_sms * 4, 256>>>(ctx->I, k, mk);
  k_init_identity<<<ctx->num_sms * 2, 256>>>(ctx->B, m,
                                             1.0 / (double(m) * double(ctx->lambda)));
  const size_t smem = slab_smem_bytes(ctx->W, m);
  const auto attr = cudaFuncAttributeMaxDynamicSharedMemorySize;
  if (ctx->block) {
    const int bs = int(block_select_smem(ctx->block));
    ctx->blk_threads = block_select_threads(ctx->block, block_count(ctx->block, ctx->k_req, d));
    ok &= for_block_kernel(ctx->blk_threads, true, [&](auto kern) {
      int resident = 0;
      bool good = cudaFuncSetAttribute(kern, attr, bs) == cudaSuccess;
      good &= cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, kern, ctx->blk_threads,
                                                            bs) == cudaSuccess;
      ctx->blk_resident = resident > 0 ? resident : 1;
      return good;
    });
    ok &= for_block_kernel(ctx->blk_threads, false, [&](auto kern) {
      return cudaFuncSetAttribute(kern, attr, bs) == cudaSuccess;
    });
  }
  {
    // the cooperative kernels: as many blocks as are resident together, at most 2 (m x m)
    // or 4 (selection: its passes are latency bound) per SM; a grid-wide barrier costs in
    // proportion to the number of blocks
    int occ = 0;
    ok &= cudaFuncSetAttribute(k_mxm, attr, int(mxm_smem_bytes(m))) == cudaSuccess;
    ok &= cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_mxm, kMxmThreads,
                                                        mxm_smem_bytes(m)) == cudaSuccess;
    ok &= occ >= 1;
    ctx->mxm_grid = std::min(kMaxCoopBlocks, ctx->num_sms * std::min(occ, 2));
    occ = 0;
    ok &= cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_select_insert, kSelThreads,
                                                        kSelSmemBytes) == cudaSuccess;
    ok &= occ >= 1;
    // a warp per group of chunk buckets, per (slab, part) of the insert, four row entries per
    // thread in the offsets phase; at least one block per SM
    const int64_t n_groups = (ctx->n_chunks + kSelGroup - 1) / kSelGroup;
    const int64_t want = std::max<int64_t>({(n_groups + kSelWarps - 1) / kSelWarps,
                                            (int64_t(n_slabs) * 2 + kSelWarps - 1) / kSelWarps,
                                            (k + 4 * kSelThreads - 1) / (4 * kSelThreads),
                                            int64_t(ctx->num_sms)});
    ctx->sel_grid = int(std::min<int64_t>({int64_t(kMaxCoopBlocks),
                                           int64_t(ctx->num_sms) * std::min(occ, 4), want}));
  }
  if (ctx->flags & EFCP_PRECOND_GGT)
    ok &= cudaFuncSetAttribute(ggt_slots(m) <= 2 ? k_ggt_weights<2> : k_ggt_weights<4>, attr,
                               int(ggt_smem_bytes(m))) == cudaSuccess;
  auto big_smem = [&](auto kern) {
    return cudaFuncSetAttribute(kern, attr, int(smem)) == cudaSuccess;
  };
  ok &= big_smem(k_sp_rows<false, float, false>) && big_smem(k_sp_rows<false, float, true>);
  ok &= big_smem(k_sp_rows<true, float, false>) && big_smem(k_sp_rows<true, float, true>);
  ok &= big_smem(k_sp_rows<false, bf16raw, false>) && big_smem(k_sp_rows<false, bf16raw, true>);
#define EFCP_LCG_ATTR(VEC, ACC, VT, FIXED)                         \
  ok &= big_smem(k_lcg<VEC, ACC, VT, FIXED, false>) && big_smem(k_lcg<VEC, ACC, VT, FIXED, true>)
  EFCP_LCG_ATTR(true, false, float, false);
  EFCP_LCG_ATTR(false, false, float, false);
  EFCP_LCG_ATTR(true, true, float, false);
  EFCP_LCG_ATTR(false, true, float, false);
  EFCP_LCG_ATTR(true, false, bf16raw, false);
  EFCP_LCG_ATTR(false, false, bf16raw, false);
  EFCP_LCG_ATTR(true, false, float, true);
  EFCP_LCG_ATTR(false, false, float, true);
  EFCP_LCG_ATTR(true, false, bf16raw, true);
  EFCP_LCG_ATTR(false, false, bf16raw, true);
#undef EFCP_LCG_ATTR
  ok &= cudaDeviceSynchronize() == cudaSuccess;
  return ok;
}

int current_sm_count(int* device) {
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) {
    (void)cudaGetLastError();
    return 0;
  }
  if (device) *device = dev;
  return n;
}

// what efcp_create_shard adds to a create call
struct ShardSpec {
  int64_t d_global, k_global;
  int shard, n_shards;
};

int create_impl(efcp_ctx** out, int64_t d, int32_t m, int64_t k, float lambda, uint32_t flags,
                int32_t block, void* workspace, int64_t workspace_bytes, bool own_memory,
                const ShardSpec* shard = nullptr) {
  if (!out) return EFCP_EINVAL;
  *out = nullptr;
  if (!own_memory && (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) ||
                      workspace_bytes < 0))
    return EFCP_EINVAL;
  efcp_ctx* ctx = new (std::nothrow) efcp_ctx();
  if (!ctx) return EFCP_ENOMEM;
  auto fail = [&](int code) {
    free_all(ctx);
    delete ctx;
    return code;
  };
  const int sms = current_sm_count(&ctx->device);
  if (sms < 1) return fail(EFCP_ECUDA);
  int rc = configure(ctx, d, m, k, lambda, flags, block, sms);
  if (rc != EFCP_OK) return fail(rc);
  if (shard) {
    ctx->d_global = shard->d_global; ctx->k_global = shard->k_global;
    ctx->shard = shard->shard; ctx->n_shards = shard->n_shards;
    ctx->is_shard = true;
  }
  if (!own_memory) {
    ctx->ws_base = static_cast<unsigned char*>(workspace);
    ctx->ws_cap = workspace_bytes;
  }
  if ((rc = alloc_all(ctx)) != EFCP_OK) return fail(rc);
  if (!init_state(ctx)) {
    ctx->last_cuda = int(cudaGetLastError());
    return fail(EFCP_ECUDA);
  }
  *out = ctx;
  return EFCP_OK;
}

}  // namespace

extern "C" {

int efcp_create_blockwise(efcp_ctx** out, int64_t d, int32_t m, int64_t k, float lambda,
                          uint32_t flags, int32_t block) {
  return create_impl(out, d, m, k, lambda, flags, block, nullptr, 0, true);
}

int64_t efcp_workspace_bytes(int64_t d, int32_t m, int64_t k, uint32_t flags, int32_t block) {
  efcp_ctx tmp;
  tmp.ws_measure = true;
  int sms = current_sm_count(nullptr);
  if (sms < 1) sms = 148;  // no device: the SM count of a B200
  if (configure(&tmp, d, m, k, 1.0f, flags, block, sms) != EFCP_OK) return -1;
  if (alloc_all(&tmp) != EFCP_OK) return -1;
  return tmp.ws_used;
}

int efcp_create_in(efcp_ctx** out, int64_t d, int32_t m, int64_t k, float lambda, uint32_t flags,
                   int32_t block, void* workspace, int64_t workspace_bytes) {
  return create_impl(out, d, m, k, lambda, flags, block, workspace, workspace_bytes, false);
}

int efcp_destroy(efcp_ctx* ctx) {
  if (!ctx) return EFCP_EINVAL;
  cudaSetDevice(ctx->device);
  cudaDeviceSynchronize();
  free_all(ctx);
  delete ctx;
  return EFCP_OK;
}

}  // extern "C"

namespace {

// The m-vectors of the m x m stage inside ctx->vecs.
struct Vecs {
  double *delta, *aprime, *y, *bold, *z, *w, *res, *dw, *rhs, *wfin;
};
Vecs vecs_of(efcp_ctx* ctx) {
  double* v = ctx->vecs;
  const int m = ctx->m;
  return Vecs{v, v + m, v + 2 * m, v + 3 * m, v + 4 * m, v + 5 * m, v + 6 * m, v + 7 * m,
              v + 8 * m, v + 9 * m};
}

// a = xi + g with the digit-1 histogram and the speculative candidate buckets, or, with
// block-wise Top-k, the whole selection.
int launch_ef(efcp_ctx* ctx, const float* grad, cudaStream_t st) {
  const int64_t d = ctx->d;
  if (ctx->block) {
    const size_t bs = block_select_smem(ctx->block);
    const int grid = std::min(ctx->n_blocks, ctx->num_sms * ctx->blk_resident);
    for_block_kernel(ctx->blk_threads, (reinterpret_cast<uintptr_t>(grad) & 15) == 0,
                     [&](auto kern) {
                       kern<<<grid, ctx->blk_threads, bs, st>>>(
                           ctx->e, grad, d, ctx->k_req, ctx->block, ctx->n_blocks, ctx->blk_T,
                           ctx->sel_idx, ctx->sel_val, ctx->sc, ctx->V16 ? 1 : 0,
                           ctx->hook_drop_loads);
                       return true;
                     });
  } else {
    const int chunk_grid = ctx->n_chunks < ctx->num_sms * 8 ? ctx->n_chunks : ctx->num_sms * 8;
    const int spec = ctx->spec ? 1 : 0;
    if ((reinterpret_cast<uintptr_t>(grad) & 15) == 0)
      k_ef_spec<true><<<chunk_grid, kChunkThreads, 0, st>>>(ctx->e, grad, d, ctx->hist, ctx->sc,
                                                            ctx->chunk_off, ctx->bk_off,
                                                            ctx->bk_val, ctx->n_chunks, spec);
    else
      k_ef_spec<false><<<chunk_grid, kChunkThreads, 0, st>>>(ctx->e, grad, d, ctx->hist, ctx->sc,
                                                             ctx->chunk_off, ctx->bk_off,
                                                             ctx->bk_val, ctx->n_chunks, spec);
  }
  EFCP_LAUNCHED();
  return EFCP_OK;
}

// Phases [pb, pe) of the selection / ring-insert kernel for ring slot `slot`.
int launch_select(efcp_ctx* ctx, int slot, int pb, int pe, cudaStream_t st) {
  const int64_t k = ctx->k;
  SelectArgs sa{};
  sa.e = ctx->e; sa.d = ctx->d;
  sa.hist1 = ctx->hist; sa.hist2 = ctx->hist + kBins1; sa.hist3 = ctx->hist + kBins1 + kBins2;
  sa.sc = ctx->sc;
  sa.cnt = ctx->chunk_off; sa.bk_off = ctx->bk_off; sa.bk_val = ctx->bk_val;
  sa.n_chunks = ctx->n_chunks;
  sa.k_total = uint32_t(ctx->k_global);
  sa.spec_limit = uint32_t(std::min<int64_t>(ctx->d_global, 3 * ctx->k_global + 65536));
  sa.cnt_gt = ctx->sel_gt; sa.cnt_eq = ctx->sel_eq; sa.blk_tot = ctx->blk_tot;
  sa.shard_tot = ctx->shard_tot; sa.shard = ctx->shard; sa.n_shards = ctx->n_shards;
  sa.sel_idx = ctx->sel_idx; sa.sel_val = ctx->sel_val;
  sa.row_cap = k;
  sa.values_bf16 = ctx->V16 ? 1 : 0;
  sa.W = ctx->W; sa.n_slabs = ctx->n_slabs; sa.m = ctx->m; sa.slot = slot;
  sa.offs = ctx->offs; sa.colsum = ctx->colsum; sa.order = ctx->order;
  sa.row_idx = ctx->I + int64_t(slot) * k; sa.row_rel = ctx->R + int64_t(slot) * k;
  sa.row_val = ctx->V + int64_t(slot) * k;
  sa.row_v16 = ctx->V16 ? ctx->V16 + int64_t(slot) * k : nullptr;
  sa.slab_ctr = ctx->slab_ctr; sa.vmax = ctx->vmax;
  sa.bar = ctx->bar;
  sa.phase_begin = pb; sa.phase_end = pe;
  void* args[] = {&sa};
  EFCP_CUDA(cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(k_select_insert),
                                        dim3(ctx->sel_grid), dim3(kSelThreads), args,
                                        kSelSmemBytes, st));
  EFCP_LAUNCHED();
  return EFCP_OK;
}

// Scalar products of every window row with the new row (one partial per slab and row).
int launch_sp(efcp_ctx* ctx, int slot, cudaStream_t st) {
  const int64_t k = ctx->k, d = ctx->d;
  const int m = ctx->m;
  const bool acc_mode = (ctx->flags & EFCP_RHS_ACCUMULATOR) != 0;
  const size_t smem = slab_smem_bytes(ctx->W, m);
#define EFCP_SP_LAUNCH1(ACC, VT, SHORT, VPTR)                                                  \
  k_sp_rows<ACC, VT, SHORT><<<ctx->grid_slab, kSlabThreads, smem, st>>>(                       \
      ctx->R, VPTR, ctx->V, ctx->offs, k, m, ctx->W, ctx->n_slabs, slot, ctx->slab_part,       \
      ctx->slab_ctr, ctx->order, ctx->e, d)
#define EFCP_SP_LAUNCH(ACC, VT, VPTR)                                                          \
  do {                                                                                         \
    if (ctx->short_rows) EFCP_SP_LAUNCH1(ACC, VT, true, VPTR);                                 \
    else EFCP_SP_LAUNCH1(ACC, VT, false, VPTR);                                                \
  } while (0)
  if (ctx->V16) EFCP_SP_LAUNCH(false, bf16raw, ctx->V16);
  else if (acc_mode) EFCP_SP_LAUNCH(true, float, ctx->V);
  else EFCP_SP_LAUNCH(false, float, ctx->V);
#undef EFCP_SP_LAUNCH1
#undef EFCP_SP_LAUNCH
  EFCP_LAUNCHED();
  return EFCP_OK;
}

// Phases [pb, pe) of the m x m kernel.
int launch_mxm(efcp_ctx* ctx, int slot, int pb, int pe, cudaStream_t st) {
  const int m = ctx->m;
  const Vecs v = vecs_of(ctx);
  MxmArgs ma{};
  ma.slab_part = ctx->slab_part; ma.partial = ctx->partial;
  ma.n_slabs = ctx->n_slabs;
  ma.parts = ctx->n_slabs < kSpParts ? ctx->n_slabs : kSpParts;
  ma.m = m; ma.slot = slot; ma.acc = (ctx->flags & EFCP_RHS_ACCUMULATOR) ? 1 : 0;
  ma.mlambda = double(m) * double(ctx->lambda); ma.lambda = double(ctx->lambda);
  ma.S = ctx->S; ma.B = ctx->B;
  ma.delta = v.delta; ma.aprime = v.aprime; ma.y = v.y; ma.bold = v.bold; ma.w = v.w;
  ma.res = v.res; ma.dw = v.dw; ma.rhs = v.rhs;
  ma.sc = ctx->sc; ma.bar = ctx->bar + 2;
  ma.phase_begin = pb; ma.phase_end = pe;
  ma.fuse12 = (pb <= 1 && pe > 2) ? 1 : 0;  // both in this launch: nothing to exchange between
  void* args[] = {&ma};
  EFCP_CUDA(cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(k_mxm),
                                        dim3(ctx->mxm_grid), dim3(kMxmThreads), args,
                                        mxm_smem_bytes(m), st));
  EFCP_LAUNCHED();
  return EFCP_OK;
}

// Sparse GGT: eigendecomposition of S and the weights of u over the window rows.
int launch_ggt(efcp_ctx* ctx, int slot, cudaStream_t st) {
  const int m = ctx->m;
  const Vecs v = vecs_of(ctx);
  if (ggt_slots(m) <= 2)
    k_ggt_weights<2><<<1, kGgtThreads, ggt_smem_bytes(m), st>>>(
        ctx->S, m, slot, double(ctx->lambda), v.w, ctx->wf, ctx->sc, ctx->ggt_rot);
  else
    k_ggt_weights<4><<<1, kGgtThreads, ggt_smem_bytes(m), st>>>(
        ctx->S, m, slot, double(ctx->lambda), v.w, ctx->wf, ctx->sc, ctx->ggt_rot);
  EFCP_LAUNCHED();
  return EFCP_OK;
}

// Linear combination of the window rows into `update` (or straight into the parameters).
// count < 0: all slabs, heavy first.  Otherwise the slabs slab0 .. slab0 + count - 1 in
// their natural order, with work counter number `ctr` (1..15).
int launch_lcg(efcp_ctx* ctx, float* update, LcgApply ap, cudaStream_t st, int slab0 = 0,
               int count = -1, int ctr = 1) {
  const int64_t k = ctx->k, d = ctx->d;
  const int m = ctx->m;
  const Vecs v = vecs_of(ctx);
  const bool acc_mode = (ctx->flags & EFCP_RHS_ACCUMULATOR) != 0;
  const bool ggt = (ctx->flags & EFCP_PRECOND_GGT) != 0;
  const size_t smem = slab_smem_bytes(ctx->W, m);
  const bool uvec = (reinterpret_cast<uintptr_t>(update) & 15) == 0;
  const float inv_lambda = 1.0f / ctx->lambda;
  const double* dw = ggt ? nullptr : v.dw;
  const int n_launch = count < 0 ? ctx->n_slabs : count;
  const int grid = std::min(ctx->grid_slab, n_launch);
  const int32_t* order = count < 0 ? ctx->order : nullptr;
#define EFCP_LCG_LAUNCH1(VEC, ACC, VT, SHORT, VPTR)                                            \
  k_lcg<VEC, ACC, VT, false, SHORT><<<grid, kSlabThreads, smem, st>>>(                         \
      ctx->R, VPTR, ctx->offs, k, m, ctx->W, n_launch, v.w, dw, v.wfin, update, d,             \
      ctx->slab_ctr + ctr, order, slab0, ctx->e, inv_lambda, ap)
#define EFCP_LCG_FIXED_LAUNCH1(VEC, VT, SHORT, VPTR)                                            \
  k_lcg<VEC, false, VT, true, SHORT><<<grid, kSlabThreads, smem, st>>>(                        \
      ctx->R, VPTR, ctx->offs, k, m, ctx->W, n_launch, v.w, dw, v.wfin, update, d,             \
      ctx->slab_ctr + ctr, order, slab0, ctx->e, inv_lambda, ap, ctx->vmax, ctx->lcg_redo,     \
      ctx->lcg_tol2)
#define EFCP_LCG_LAUNCH(VEC, ACC, VT, VPTR)                                                    \
  do {                                                                                         \
    if (ctx->short_rows) EFCP_LCG_LAUNCH1(VEC, ACC, VT, true, VPTR);                           \
    else EFCP_LCG_LAUNCH1(VEC, ACC, VT, false, VPTR);                                          \
  } while (0)
#define EFCP_LCG_FIXED_LAUNCH(VEC, VT, VPTR)                                                    \
  do {                                                                                         \
    if (ctx->short_rows) EFCP_LCG_FIXED_LAUNCH1(VEC, VT, true, VPTR);                          \
    else EFCP_LCG_FIXED_LAUNCH1(VEC, VT, false, VPTR);                                         \
  } while (0)
  if (ctx->vmax) {
    if (ctx->V16) {
      if (uvec) EFCP_LCG_FIXED_LAUNCH(true, bf16raw, ctx->V16);
      else EFCP_LCG_FIXED_LAUNCH(false, bf16raw, ctx->V16);
    } else {
      if (uvec) EFCP_LCG_FIXED_LAUNCH(true, float, ctx->V);
      else EFCP_LCG_FIXED_LAUNCH(false, float, ctx->V);
    }
  } else if (ctx->V16) {
    if (uvec) EFCP_LCG_LAUNCH(true, false, bf16raw, ctx->V16);
    else EFCP_LCG_LAUNCH(false, false, bf16raw, ctx->V16);
  } else if (acc_mode) {
    if (uvec) EFCP_LCG_LAUNCH(true, true, float, ctx->V);
    else EFCP_LCG_LAUNCH(false, true, float, ctx->V);
  } else {
    if (uvec) EFCP_LCG_LAUNCH(true, false, float, ctx->V);
    else EFCP_LCG_LAUNCH(false, false, float, ctx->V);
  }
#undef EFCP_LCG_LAUNCH
#undef EFCP_LCG_FIXED_LAUNCH
#undef EFCP_LCG_LAUNCH1
#undef EFCP_LCG_FIXED_LAUNCH1
  EFCP_LAUNCHED();
  return EFCP_OK;
}

// EFCP_DEBUG_CHECKS: the new row's offsets, slab membership and 16-bit stream, and the slab
// weights; a violation becomes the sticky internal-error status.
int launch_debug_checks(efcp_ctx* ctx, int slot, cudaStream_t st) {
  k_validate_rows<<<dim3(ctx->n_slabs, 1), 128, 0, st>>>(
      ctx->I, ctx->R, ctx->offs, ctx->k, ctx->d, ctx->m, ctx->W, ctx->n_slabs, slot, slot + 1,
      ctx->shard_tot ? 0 : 1, ctx->dbg_bad);
  EFCP_LAUNCHED();
  k_validate_colsum<<<ctx->n_slabs + 1, 256, 0, st>>>(ctx->offs, ctx->colsum, ctx->m,
                                                      ctx->n_slabs, ctx->dbg_bad);
  EFCP_LAUNCHED();
  k_fold_bad<<<1, 1, 0, st>>>(ctx->dbg_bad, ctx->sc);
  EFCP_LAUNCHED();
  return EFCP_OK;
}

#define EFCP_TRY(call)             \
  do {                             \
    const int rc__ = (call);       \
    if (rc__ != EFCP_OK) return rc__; \
  } while (0)

// One step: five launches (six for Sparse GGT).  With ap.theta set the linear combination
// updates the parameters in place of writing u (update may then be NULL).
// host_update != nullptr (efcp_step_host): the linear combination runs in kHostRanges launches
// over consecutive ranges of slabs, and every finished range of `update` starts its copy to
// host_update on the handle's copy stream while the next range is being accumulated.
int step_impl(efcp_ctx* ctx, const float* grad, float* update, void* stream_, LcgApply ap,
              float* host_update = nullptr) {
  if (!ctx || !grad || (!update && !ap.theta) || grad == update) return EFCP_EINVAL;
  if (ctx->shard_tot) return EFCP_EINVAL;  // a shard steps through efcp_shard_phase
  cudaStream_t st = static_cast<cudaStream_t>(stream_);
  EFCP_CUDA(cudaSetDevice(ctx->device));  // the launches below go to the handle's device
  const int slot = int(ctx->t % ctx->m);
  const bool ggt = (ctx->flags & EFCP_PRECOND_GGT) != 0;
  ctx->launches = 0;
  prof_mark(ctx, 0, st);
  EFCP_TRY(launch_ef(ctx, grad, st));
  // global Top-k: exact selection, residual and ring insert; block-wise Top-k has selected
  // already, only the ring insert is left
  if (ctx->split_phases) {
    for (int ph = ctx->block ? 4 : 0; ph < kSelPhases; ++ph)
      EFCP_TRY(launch_select(ctx, slot, ph, ph + 1, st));
  } else {
    EFCP_TRY(launch_select(ctx, slot, ctx->block ? 4 : 0, kSelPhases, st));
  }
  prof_mark(ctx, 1, st);
  EFCP_TRY(launch_sp(ctx, slot, st));
  prof_mark(ctx, 2, st);
  // m x m: sums of the slab partials, S row/column, remove-and-border update of the inverse,
  // weights, residual and the refinement's correction (Sparse GGT: the sums and S, then its
  // eigendecomposition)
  if (ctx->split_phases) {
    for (int ph = 0; ph < (ggt ? 3 : kMxmPhases); ++ph)
      EFCP_TRY(launch_mxm(ctx, slot, ph, ph + 1, st));
  } else {
    EFCP_TRY(launch_mxm(ctx, slot, 0, ggt ? 3 : kMxmPhases, st));
  }
  if (ggt) EFCP_TRY(launch_ggt(ctx, slot, st));
  prof_mark(ctx, 3, st);
  if (host_update && ctx->n_slabs >= kHostRanges * ctx->num_sms) {
    for (int q = 0; q < kHostRanges; ++q) {
      const int s0 = int(int64_t(ctx->n_slabs) * q / kHostRanges);
      const int s1 = int(int64_t(ctx->n_slabs) * (q + 1) / kHostRanges);
      EFCP_TRY(launch_lcg(ctx, update, ap, st, s0, s1 - s0, 1 + q));
      EFCP_CUDA(cudaEventRecord(ctx->host_ev[q], st));
      EFCP_CUDA(cudaStreamWaitEvent(ctx->copy_stream, ctx->host_ev[q], 0));
      const int64_t lo = int64_t(s0) * ctx->W, hi = std::min<int64_t>(ctx->d, int64_t(s1) * ctx->W);
      EFCP_CUDA(cudaMemcpyAsync(host_update + lo, update + lo, size_t(hi - lo) * 4,
                                cudaMemcpyDeviceToHost, ctx->copy_stream));
    }
  } else {
    EFCP_TRY(launch_lcg(ctx, update, ap, st));
    if (host_update)
      EFCP_CUDA(cudaMemcpyAsync(host_update, update, size_t(ctx->d) * 4, cudaMemcpyDeviceToHost,
                                st));
  }
  prof_mark(ctx, 4, st);
  if (ctx->flags & EFCP_DEBUG_CHECKS) EFCP_TRY(launch_debug_checks(ctx, slot, st));
  if (ctx->prof_on && ctx->prof_n < ctx->prof_cap) ++ctx->prof_n;
  ctx->t += 1;
  return EFCP_OK;
}

}  // namespace

extern "C" {

/*
 * Coordinate-sharded state.  Phase p of a step (0..5) runs on every shard, then buffer p is
 * summed over the shards (an all-reduce), then phase p + 1 runs:
 *   0  a = xi + g on the shard's coordinates, digit-1 histogram      -> buffer 0: histogram 1
 *   1  threshold bin of digit 1 (from the summed histogram), digit 2 -> buffer 1: histogram 2
 *   2  threshold bin of digit 2, digit 3                             -> buffer 2: histogram 3
 *   3  exact threshold key, the shard's counts above and at the key  -> buffer 3: the counts
 *   4  selection (equal keys go to the shards of lower coordinates first), ring insert,
 *      the shard's part of the scalar products                       -> buffer 4: delta
 *   5  S, the m x m stage (replicated), the shard's part of the update
 */
int efcp_shard_phase(efcp_ctx* ctx, int32_t phase, const float* grad, float* update,
                     void* stream_) {
  if (!ctx || !ctx->shard_tot || phase < 0 || phase > 5) return EFCP_EINVAL;
  if ((phase == 0 && !grad) || (phase == 5 && !update) || phase != ctx->next_phase)
    return EFCP_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(stream_);
  EFCP_CUDA(cudaSetDevice(ctx->device));
  const int slot = int(ctx->t % ctx->m);
  switch (phase) {
    case 0:
      ctx->launches = 0;
      EFCP_CUDA(cudaMemsetAsync(ctx->shard_tot, 0, size_t(ctx->n_shards) * 8, st));
      EFCP_TRY(launch_ef(ctx, grad, st));
      break;
    case 1: EFCP_TRY(launch_select(ctx, slot, 0, 1, st)); break;
    case 2: EFCP_TRY(launch_select(ctx, slot, 1, 2, st)); break;
    case 3: EFCP_TRY(launch_select(ctx, slot, 2, 3, st)); break;
    case 4:
      EFCP_TRY(launch_select(ctx, slot, 3, kSelPhases, st));
      EFCP_TRY(launch_sp(ctx, slot, st));
      EFCP_TRY(launch_mxm(ctx, slot, 0, 2, st));
      break;
    default:
      EFCP_TRY(launch_mxm(ctx, slot, 2, kMxmPhases, st));
      EFCP_TRY(launch_lcg(ctx, update, LcgApply{nullptr, 0.f, 0.f}, st));
      if (ctx->flags & EFCP_DEBUG_CHECKS) EFCP_TRY(launch_debug_checks(ctx, slot, st));
      ctx->t += 1;
      break;
  }
  ctx->next_phase = (phase + 1) % 6;
  return EFCP_OK;
}

int efcp_shard_buffer(efcp_ctx* ctx, int32_t phase, void** dev_ptr, int64_t* count,
                      int32_t* is_f64) {
  if (!ctx || !ctx->shard_tot || !dev_ptr || !count || !is_f64 || phase < 0 || phase > 4)
    return EFCP_EINVAL;
  *is_f64 = phase == 4 ? 1 : 0;
  switch (phase) {
    case 0: *dev_ptr = ctx->hist; *count = kBins1; break;
    case 1: *dev_ptr = ctx->hist + kBins1; *count = kBins2; break;
    case 2: *dev_ptr = ctx->hist + kBins1 + kBins2; *count = kBins3; break;
    case 3: *dev_ptr = ctx->shard_tot; *count = 2 * int64_t(ctx->n_shards); break;
    default: *dev_ptr = ctx->vecs; *count = ctx->m; break;
  }
  return EFCP_OK;
}

int efcp_create_shard(efcp_ctx** out, int64_t d_global, int64_t d_lo, int64_t d_hi, int32_t m,
                      int64_t k_global, int64_t row_cap, float lambda, uint32_t flags,
                      int32_t shard, int32_t n_shards) {
  if (!out) return EFCP_EINVAL;
  *out = nullptr;
  if (n_shards < 1 || n_shards > 1024 || shard < 0 || shard >= n_shards || d_lo < 0 ||
      d_hi <= d_lo || d_hi > d_global || !valid_args(d_global, m, k_global))
    return EFCP_EINVAL;
  if (flags & (EFCP_RHS_ACCUMULATOR | EFCP_PRECOND_GGT)) return EFCP_EINVAL;
  const int64_t d_loc = d_hi - d_lo;
  if (row_cap <= 0) row_cap = std::min(k_global, d_loc);  // whatever the shard could be given
  if (row_cap > d_loc) return EFCP_EINVAL;
  ShardSpec sp{d_global, k_global, shard, n_shards};
  return create_impl(out, d_loc, m, row_cap, lambda, flags, 0, nullptr, 0, true, &sp);
}

int64_t efcp_row_count(efcp_ctx* ctx, int32_t slot) {
  if (!ctx || slot < 0 || slot >= ctx->m) return -1;
  if (!ctx->shard_tot) return ctx->k;
  int32_t n = 0;
  if (cudaSetDevice(ctx->device) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess ||
      cudaMemcpy(&n, ctx->offs + int64_t(ctx->n_slabs) * ctx->m + slot, 4,
                 cudaMemcpyDeviceToHost) != cudaSuccess)
    return -1;
  return n;
}

int efcp_step(efcp_ctx* ctx, const float* grad, float* update, void* stream) {
  if (!update) return EFCP_EINVAL;
  return step_impl(ctx, grad, update, stream, LcgApply{nullptr, 0.f, 0.f});
}

int efcp_update_norm(efcp_ctx* ctx, const float* update, double* host_out, void* stream_) {
  if (!ctx || !update) return EFCP_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(stream_);
  EFCP_CUDA(cudaSetDevice(ctx->device));
  const int64_t want = (ctx->d + 8 * kUpdThreads - 1) / (8 * kUpdThreads);
  const int nb = int(std::max<int64_t>(1, std::min<int64_t>({want, int64_t(ctx->num_sms) * 8,
                                                             int64_t(kUpdMaxBlocks)})));
  if ((reinterpret_cast<uintptr_t>(update) & 15) == 0)
    k_update_sumsq<true><<<nb, kUpdThreads, 0, st>>>(update, ctx->d, ctx->upd_norm + 1);
  else
    k_update_sumsq<false><<<nb, kUpdThreads, 0, st>>>(update, ctx->d, ctx->upd_norm + 1);
  EFCP_LAUNCHED();
  k_sum_parts<<<1, 256, 0, st>>>(ctx->upd_norm + 1, nb, ctx->upd_norm);
  EFCP_LAUNCHED();
  ctx->norm_t = ctx->t;
  if (host_out) {
    double s = 0.0;
    EFCP_CUDA(cudaMemcpyAsync(&s, ctx->upd_norm, 8, cudaMemcpyDeviceToHost, st));
    EFCP_CUDA(cudaStreamSynchronize(st));
    *host_out = std::sqrt(s);
  }
  return EFCP_OK;
}

int efcp_apply_update(efcp_ctx* ctx, float* theta, const float* update, int64_t n, float eta,
                      float gamma, float clip_norm, void* stream_) {
  if (!ctx || !theta || !update || theta == update || n < 1 || n > ctx->d) return EFCP_EINVAL;
  if (!(eta >= 0.f) || !(gamma >= 0.f) || !(clip_norm >= 0.f) || std::isinf(eta) ||
      std::isinf(gamma) || std::isinf(clip_norm))
    return EFCP_EINVAL;
  if (clip_norm > 0.f && ctx->norm_t != ctx->t) return EFCP_EINVAL;  // no norm of this step's u
  cudaStream_t st = static_cast<cudaStream_t>(stream_);
  EFCP_CUDA(cudaSetDevice(ctx->device));
  const float decay = float(1.0 - double(gamma) * double(eta));
  const int64_t want = (n + 4 * kUpdThreads - 1) / (4 * kUpdThreads);
  const int nb = int(std::max<int64_t>(1, std::min<int64_t>(want, int64_t(ctx->num_sms) * 16)));
  const bool vec = ((reinterpret_cast<uintptr_t>(theta) | reinterpret_cast<uintptr_t>(update)) & 15) == 0;
  if (vec)
    k_apply_update<true><<<nb, kUpdThreads, 0, st>>>(theta, update, n, decay, double(eta),
                                                     double(clip_norm), ctx->upd_norm);
  else
    k_apply_update<false><<<nb, kUpdThreads, 0, st>>>(theta, update, n, decay, double(eta),
                                                      double(clip_norm), ctx->upd_norm);
  EFCP_LAUNCHED();
  return EFCP_OK;
}

int efcp_step_apply(efcp_ctx* ctx, const float* grad, float* theta, float* update, float eta,
                    float gamma, float clip_norm, void* stream_) {
  if (!ctx || !theta || theta == grad) return EFCP_EINVAL;
  if (!(eta >= 0.f) || !(gamma >= 0.f) || !(clip_norm >= 0.f) || std::isinf(eta) ||
      std::isinf(gamma) || std::isinf(clip_norm))
    return EFCP_EINVAL;  // before the step: a rejected call leaves the state untouched
  if (!update) {
    // nobody wants u: the linear combination applies it to theta slab by slab
    if (clip_norm > 0.f) return EFCP_EINVAL;  // clipping needs |u| before any of it is applied
    const float decay = float(1.0 - double(gamma) * double(eta));
    return step_impl(ctx, grad, nullptr, stream_, LcgApply{theta, decay, -eta});
  }
  int rc = efcp_step(ctx, grad, update, stream_);
  if (rc != EFCP_OK) return rc;
  if (clip_norm > 0.f && (rc = efcp_update_norm(ctx, update, nullptr, stream_)) != EFCP_OK) return rc;
  rc = efcp_apply_update(ctx, theta, update, ctx->d, eta, gamma, clip_norm, stream_);
  return rc;
}

int efcp_step_host(efcp_ctx* ctx, const float* grad, float* update, void* stream_) {
  if (!ctx || !grad || !update) return EFCP_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(stream_);
  EFCP_CUDA(cudaSetDevice(ctx->device));
  if (!ctx->stage_g) {
    int rc;
    if ((rc = dev_alloc(ctx, &ctx->stage_g, ctx->d * 4))) return rc;
    if ((rc = dev_alloc(ctx, &ctx->stage_u, ctx->d * 4))) return rc;
  }
  if (!ctx->copy_stream) {
    EFCP_CUDA(cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking));
    for (cudaEvent_t& ev : ctx->host_ev) EFCP_CUDA(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
  }
  EFCP_CUDA(cudaMemcpyAsync(ctx->stage_g, grad, size_t(ctx->d) * 4, cudaMemcpyHostToDevice, st));
  const int rc = step_impl(ctx, ctx->stage_g, ctx->stage_u, stream_, LcgApply{nullptr, 0.f, 0.f},
                           update);
  if (rc != EFCP_OK) return rc;
  EFCP_CUDA(cudaStreamSynchronize(st));
  EFCP_CUDA(cudaStreamSynchronize(ctx->copy_stream));
  return EFCP_OK;
}

int efcp_get_error(efcp_ctx* ctx, float* host_e) {
  if (!ctx || !host_e) return EFCP_EINVAL;
  const int rc = sync_status(ctx);
  if (rc == EFCP_ECUDA) return rc;
  EFCP_CUDA(cudaMemcpy(host_e, ctx->e, size_t(ctx->d) * 4, cudaMemcpyDeviceToHost));
  return rc;
}

int efcp_get_row(efcp_ctx* ctx, int32_t slot, int32_t* host_idx, float* host_val) {
  if (!ctx || !host_idx || !host_val || slot < 0 || slot >= ctx->m) return EFCP_EINVAL;
  const int rc = sync_status(ctx);
  if (rc == EFCP_ECUDA) return rc;
  const size_t bytes = size_t(ctx->k) * 4;
  EFCP_CUDA(cudaMemcpy(host_idx, ctx->I + int64_t(slot) * ctx->k, bytes, cudaMemcpyDeviceToHost));
  EFCP_CUDA(cudaMemcpy(host_val, ctx->V + int64_t(slot) * ctx->k, bytes, cudaMemcpyDeviceToHost));
  int64_t n = ctx->k;  // a shard's row holds what the step gave it; the rest reads as (0, 0)
  if (ctx->shard_tot) {
    int32_t cnt = 0;
    EFCP_CUDA(cudaMemcpy(&cnt, ctx->offs + int64_t(ctx->n_slabs) * ctx->m + slot, 4,
                         cudaMemcpyDeviceToHost));
    n = std::max<int64_t>(0, std::min<int64_t>(cnt, ctx->k));
    for (int64_t j = n; j < ctx->k; ++j) {
      host_idx[j] = 0;
      host_val[j] = 0.f;
    }
  }
  // the device keeps every slab segment of a row in a bank-interleaved order; callers get
  // the row in ascending index order (indices within a row are distinct)
  try {
    std::vector<std::pair<int32_t, float>> tmp(static_cast<size_t>(n));
    for (int64_t j = 0; j < n; ++j) tmp[size_t(j)] = {host_idx[j], host_val[j]};
    std::sort(tmp.begin(), tmp.end(),
              [](const std::pair<int32_t, float>& a, const std::pair<int32_t, float>& b) {
                return a.first < b.first;
              });
    for (int64_t j = 0; j < n; ++j) {
      host_idx[j] = tmp[size_t(j)].first;
      host_val[j] = tmp[size_t(j)].second;
    }
  } catch (const std::bad_alloc&) {
    return EFCP_ENOMEM;
  }
  return rc;
}

int efcp_get_gram(efcp_ctx* ctx, double* host_S) {
  if (!ctx || !host_S) return EFCP_EINVAL;
  const int rc = sync_status(ctx);
  if (rc == EFCP_ECUDA) return rc;
  EFCP_CUDA(cudaMemcpy(host_S, ctx->S, size_t(ctx->m) * ctx->m * 8, cudaMemcpyDeviceToHost));
  return rc;
}

int efcp_get_weights(efcp_ctx* ctx, double* host_w) {
  if (!ctx || !host_w) return EFCP_EINVAL;
  const int rc = sync_status(ctx);
  if (rc == EFCP_ECUDA) return rc;
  EFCP_CUDA(cudaMemcpy(host_w, ctx->vecs + int64_t(9) * ctx->m, size_t(ctx->m) * 8,
                       cudaMemcpyDeviceToHost));
  return rc;
}

int efcp_get_window(efcp_ctx* ctx, const int32_t** dev_I, const float** dev_V) {
  if (!ctx || !dev_I || !dev_V) return EFCP_EINVAL;
  const int rc = sync_status(ctx);
  if (rc == EFCP_ECUDA) return rc;
  *dev_I = ctx->I;
  *dev_V = ctx->V;
  return rc;
}

namespace {

struct StateHeader {
  uint64_t magic;
  int64_t d, k, t;
  int32_t m, W, n_slabs;
  uint32_t flags;
  float lambda;
  uint32_t pad;  // block length of block-wise Top-k (0: global)
};
constexpr uint64_t kStateMagic = 0x3130505443464645ull;  // "EFCPTP01"

struct StatePart {
  void* dev;
  int64_t bytes;
};

// the device arrays a checkpoint holds, in file order
std::vector<StatePart> state_parts(efcp_ctx* ctx) {
  const int64_t mk = int64_t(ctx->m) * ctx->k, mm = int64_t(ctx->m) * ctx->m;
  std::vector<StatePart> p = {
      {ctx->e, ctx->d * 4},
      {ctx->I, mk * 4},
      {ctx->V, mk * 4},
      {ctx->R, mk * 2},
      {ctx->offs, int64_t(ctx->n_slabs + 1) * ctx->m * 4},
      {ctx->colsum, int64_t(ctx->n_slabs + 1) * 8},
      {ctx->S, mm * 8},
      {ctx->B, mm * 8},
  };
  if (ctx->V16) p.push_back({ctx->V16, mk * 2});
  return p;
}

// sum of squares of e in fp64: per-block partials, then one block
__global__ void __launch_bounds__(256) k_sumsq(const float* __restrict__ e, int64_t d,
                                                double* __restrict__ part) {
  __shared__ double sm[32];
  double acc = 0.0;
  for (int64_t j = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; j < d;
       j += int64_t(gridDim.x) * blockDim.x) {
    const double v = double(e[j]);
    acc += v * v;
  }
  acc = block_sum(acc, sm);
  if (threadIdx.x == 0) part[blockIdx.x] = acc;
}
}  // namespace


int efcp_validate(efcp_ctx* ctx, int64_t* bad_out) {
  if (!ctx) return EFCP_EINVAL;
  const int rc = sync_status(ctx);
  if (rc != EFCP_OK) return rc;
  // scratch: the SP partial buffer is idle between steps
  unsigned long long* bad = reinterpret_cast<unsigned long long*>(ctx->partial);
  EFCP_CUDA(cudaMemset(bad, 0, 8));
  const int rows = int(ctx->t < ctx->m ? ctx->t : ctx->m);
  if (rows > 0) {
    k_validate_rows<<<dim3(ctx->n_slabs, rows), 128>>>(ctx->I, ctx->R, ctx->offs, ctx->k, ctx->d,
                                                       ctx->m, ctx->W, ctx->n_slabs, 0, rows,
                                                       ctx->shard_tot ? 0 : 1, bad);
  }
  k_validate_colsum<<<ctx->n_slabs + 1, 256>>>(ctx->offs, ctx->colsum, ctx->m, ctx->n_slabs, bad);
  unsigned long long h = 0;
  EFCP_CUDA(cudaMemcpy(&h, bad, 8, cudaMemcpyDeviceToHost));
  if (bad_out) *bad_out = int64_t(h);
  return h ? EFCP_EINTERNAL : EFCP_OK;
}

int64_t efcp_state_size(efcp_ctx* ctx) {
  if (!ctx) return -1;
  int64_t b = int64_t(sizeof(StateHeader));
  for (const StatePart& p : state_parts(ctx)) b += p.bytes;
  return b;
}

int efcp_state_export(efcp_ctx* ctx, void* host_buf, int64_t bytes) {
  if (!ctx || !host_buf || bytes < efcp_state_size(ctx)) return EFCP_EINVAL;
  const int rc = sync_status(ctx);
  if (rc == EFCP_ECUDA) return rc;
  StateHeader h{};
  h.magic = kStateMagic; h.d = ctx->d; h.k = ctx->k; h.t = ctx->t; h.m = ctx->m; h.W = ctx->W;
  h.n_slabs = ctx->n_slabs; h.flags = ctx->flags; h.lambda = ctx->lambda;
  h.pad = uint32_t(ctx->block);
  unsigned char* out = static_cast<unsigned char*>(host_buf);
  std::memcpy(out, &h, sizeof(h));
  out += sizeof(h);
  for (const StatePart& p : state_parts(ctx)) {
    EFCP_CUDA(cudaMemcpy(out, p.dev, size_t(p.bytes), cudaMemcpyDeviceToHost));
    out += p.bytes;
  }
  return rc;
}

int efcp_state_import(efcp_ctx* ctx, const void* host_buf, int64_t bytes) {
  if (!ctx || !host_buf || bytes < efcp_state_size(ctx)) return EFCP_EINVAL;
  StateHeader h;
  std::memcpy(&h, host_buf, sizeof(h));
  if (h.magic != kStateMagic || h.d != ctx->d || h.k != ctx->k || h.m != ctx->m ||
      h.W != ctx->W || h.n_slabs != ctx->n_slabs || (h.flags & ~EFCP_LCG_FP32) != (ctx->flags & ~EFCP_LCG_FP32) ||
      h.pad != uint32_t(ctx->block) ||
      std::memcmp(&h.lambda, &ctx->lambda, 4) != 0 || h.t < 0)
    return EFCP_EINVAL;
  EFCP_CUDA(cudaSetDevice(ctx->device));
  EFCP_CUDA(cudaDeviceSynchronize());
  const unsigned char* in = static_cast<const unsigned char*>(host_buf) + sizeof(h);
  for (const StatePart& p : state_parts(ctx)) {
    EFCP_CUDA(cudaMemcpy(p.dev, in, size_t(p.bytes), cudaMemcpyHostToDevice));
    in += p.bytes;
  }
  // scalars: clear the sticky status and the previous threshold (the next step takes the
  // two-pass route once; the selection does not depend on the route)
  EFCP_CUDA(cudaMemset(ctx->sc, 0, sizeof(Scalars)));
  EFCP_CUDA(cudaMemset(ctx->hist, 0, (kBins1 + kBins2 + kBins3) * 4));
  if (ctx->vmax) {  // derived from the window: rebuilt rather than stored
    k_vmax_all<<<ctx->n_slabs, 256>>>(ctx->V, ctx->offs, ctx->k, ctx->m, ctx->vmax);
    EFCP_CUDA(cudaGetLastError());
    EFCP_CUDA(cudaDeviceSynchronize());
  }
  ctx->t = h.t;
  return EFCP_OK;
}

int64_t efcp_fixed_point_fallbacks(efcp_ctx* ctx) {
  if (!ctx) return -1;
  if (!ctx->lcg_redo) return 0;
  unsigned long long v = 0;
  if (cudaSetDevice(ctx->device) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess ||
      cudaMemcpy(&v, ctx->lcg_redo, 8, cudaMemcpyDeviceToHost) != cudaSuccess)
    return -1;
  return int64_t(v);
}

int efcp_error_norm(efcp_ctx* ctx, double* out) {
  if (!ctx || !out) return EFCP_EINVAL;
  const int rc = sync_status(ctx);
  if (rc == EFCP_ECUDA) return rc;
  // scratch: the SP partial buffers are idle between steps (m >= 1 doubles each; use slab_part)
  const int blocks = int(std::min<int64_t>(ctx->num_sms * 4, int64_t(ctx->n_slabs) * ctx->m - 1));
  const int nb = blocks < 1 ? 1 : blocks;
  if (int64_t(ctx->n_slabs) * ctx->m < 2) {  // degenerate sizes: do it on the host
    std::vector<float> h(static_cast<size_t>(ctx->d));
    EFCP_CUDA(cudaMemcpy(h.data(), ctx->e, size_t(ctx->d) * 4, cudaMemcpyDeviceToHost));
    double s = 0.0;
    for (float v : h) s += double(v) * double(v);
    *out = std::sqrt(s);
    return rc;
  }
  k_sumsq<<<nb, 256>>>(ctx->e, ctx->d, ctx->slab_part + 1);
  k_sum_parts<<<1, 256>>>(ctx->slab_part + 1, nb, ctx->slab_part);
  double s = 0.0;
  EFCP_CUDA(cudaMemcpy(&s, ctx->slab_part, 8, cudaMemcpyDeviceToHost));
  *out = std::sqrt(s);
  return rc;
}

int64_t efcp_step_count(efcp_ctx* ctx) { return ctx ? ctx->t : -1; }

int efcp_test_hook(efcp_ctx* ctx, int32_t hook, int32_t value) {
  if (!ctx || hook != EFCP_HOOK_DROP_BLOCK_LOADS) return EFCP_EINVAL;
  ctx->hook_drop_loads = value ? 1 : 0;
  return EFCP_OK;
}

int efcp_status(efcp_ctx* ctx) {
  if (!ctx) return EFCP_EINVAL;
  return sync_status(ctx);
}

int efcp_last_cuda_error(efcp_ctx* ctx) { return ctx ? ctx->last_cuda : 0; }

double efcp_last_residual(efcp_ctx* ctx) {
  if (!ctx) return -1.0;
  if (cudaSetDevice(ctx->device) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess)
    return -1.0;
  Scalars h;
  if (cudaMemcpy(&h, ctx->sc, sizeof(h), cudaMemcpyDeviceToHost) != cudaSuccess) return -1.0;
  return h.resid;
}

int32_t efcp_launches_per_step(efcp_ctx* ctx) { return ctx ? ctx->launches : -1; }

int efcp_profile_begin(efcp_ctx* ctx, int32_t max_steps) {
  if (!ctx || max_steps < 1 || max_steps > 4096) return EFCP_EINVAL;
  EFCP_CUDA(cudaSetDevice(ctx->device));
  while (int(ctx->prof_ev.size()) < max_steps * 5) {
    cudaEvent_t ev;
    EFCP_CUDA(cudaEventCreate(&ev));
    ctx->prof_ev.push_back(ev);
  }
  ctx->prof_cap = max_steps;
  ctx->prof_n = 0;
  ctx->prof_on = true;
  return EFCP_OK;
}

int efcp_profile_end(efcp_ctx* ctx, double* ms_out, int32_t* steps_out) {
  if (!ctx || !ms_out || !steps_out) return EFCP_EINVAL;
  ctx->prof_on = false;
  EFCP_CUDA(cudaSetDevice(ctx->device));
  EFCP_CUDA(cudaDeviceSynchronize());
  for (int q = 0; q < 4; ++q) ms_out[q] = 0.0;
  for (int i = 0; i < ctx->prof_n; ++i) {
    for (int q = 0; q < 4; ++q) {
      float ms = 0.f;
      EFCP_CUDA(cudaEventElapsedTime(&ms, ctx->prof_ev[size_t(i) * 5 + q],
                                     ctx->prof_ev[size_t(i) * 5 + q + 1]));
      ms_out[q] += double(ms);
    }
  }
  *steps_out = ctx->prof_n;
  ctx->prof_n = 0;
  return EFCP_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------
// efcp_topk_static: the Top-k selection with its scratch memory in a fixed array of the
// library image, for callers that cannot allocate (see include/efcp.h).
namespace {

constexpr int64_t kStaticMaxD = EFCP_TOPK_STATIC_MAX_D;
constexpr int64_t kStaticMaxChunks = (kStaticMaxD + kChunk - 1) / kChunk;
// layout of the array (every part 256-byte aligned)
constexpr int64_t kOffHist = 0;                                            // 3 histograms
constexpr int64_t kOffScalars = kOffHist + align256c((kBins1 + kBins2 + kBins3) * 4);
constexpr int64_t kOffChunk = kOffScalars + align256c(int64_t(sizeof(Scalars)));
constexpr int64_t kOffSelGt = kOffChunk + align256c((kStaticMaxChunks + 1) * 4);
constexpr int64_t kOffSelEq = kOffSelGt + align256c((kStaticMaxChunks + 1) * 4);
constexpr int64_t kOffCandIdx = kOffSelEq + align256c((kStaticMaxChunks + 1) * 4);
constexpr int64_t kOffCandVal = kOffCandIdx + align256c(kStaticMaxD * 4);
constexpr int64_t kStaticBytes = kOffCandVal + align256c(kStaticMaxD * 4);

// In host code this name is only a handle for cudaGetSymbolAddress, never an address.
static __device__ __align__(256) unsigned char g_topk_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
unsigned char* g_static_ptr[kMaxDevices] = {};  // device address of the array, per device
int g_static_sms[kMaxDevices] = {};

// Digit-1 histogram of the magnitude keys of a (the part of k_ef_spec that does not
// touch an error buffer).
__global__ void __launch_bounds__(512) k_hist1_only(const float* __restrict__ a, int64_t d,
                                                    uint32_t* __restrict__ hist1) {
  __shared__ uint32_t h[kBins1];
  for (int i = threadIdx.x; i < kBins1; i += blockDim.x) h[i] = 0u;
  __syncthreads();
  for (int64_t j = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; j < d;
       j += int64_t(gridDim.x) * blockDim.x)
    atomicAdd(&h[mag_key(a[j]) >> kShift1], 1u);
  __syncthreads();
  for (int i = threadIdx.x; i < kBins1; i += blockDim.x) {
    const uint32_t c = h[i];
    if (c) atomicAdd(&hist1[i], c);
  }
}

// Final ordered compaction of the stand-alone selection: the kept
// (index, value) pairs in ascending index order.
__global__ void __launch_bounds__(kChunkThreads) k_write_sel_only(
    const int32_t* __restrict__ cand_idx, const float* __restrict__ cand_val, const Scalars* sc,
    const int32_t* __restrict__ off_gt, const int32_t* __restrict__ pre_eq,
    int32_t* __restrict__ out_idx, float* __restrict__ out_val, int64_t k_total) {
  __shared__ int sm[33];
  const int n = sc->n_cand;
  const uint32_t T = sc->T;
  const int n_eq = int(sc->n_eq);
  const int n_cc = (n + kChunk - 1) / kChunk;
  for (int c = blockIdx.x; c < n_cc; c += gridDim.x) {
    const int64_t base = int64_t(c) * kChunk + threadIdx.x * kPerThread;
    float v[kPerThread];
    bool ok[kPerThread];
    load_chunk8(cand_val, base, n, v, ok);
    bool is_eq[kPerThread];
    int my_eq = 0;
#pragma unroll
    for (int q = 0; q < kPerThread; ++q) {
      const uint32_t key = mag_key(v[q]);
      is_eq[q] = ok[q] && key == T;
      ok[q] = ok[q] && key > T;
      my_eq += is_eq[q] ? 1 : 0;
    }
    int tot;
    const int eq_before_chunk = pre_eq[c];
    int eq_rank = eq_before_chunk + block_excl_scan<int>(my_eq, &tot, sm);
    int my_sel = 0;
#pragma unroll
    for (int q = 0; q < kPerThread; ++q) {
      if (is_eq[q]) {
        ok[q] = eq_rank < n_eq;
        ++eq_rank;
      }
      my_sel += ok[q] ? 1 : 0;
    }
    int64_t pos = int64_t(off_gt[c]) + min(eq_before_chunk, n_eq) +
                  block_excl_scan<int>(my_sel, &tot, sm);
#pragma unroll
    for (int q = 0; q < kPerThread; ++q) {
      if (ok[q] && pos < k_total) {
        out_idx[pos] = cand_idx[base + q];
        out_val[pos] = v[q];
        ++pos;
      }
    }
  }
}

}  // namespace

extern "C" int efcp_topk_static(const float* a, int64_t d, int64_t k, int32_t* idx, float* val,
                                void* stream_) {
  if (!a || !idx || !val || d < 1 || k < 1 || k > d) return EFCP_EINVAL;
  // the selection kernels read `a` with 16-byte vector loads
  if (reinterpret_cast<uintptr_t>(a) & 15) return EFCP_EINVAL;
  if (d > kStaticMaxD) return EFCP_ETOOBIG;
  cudaStream_t st = static_cast<cudaStream_t>(stream_);
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    (void)cudaGetLastError();
    return EFCP_ECUDA;
  }
  unsigned char* base = nullptr;
  int sms = 0;
  {
    // set-up, once per device, with that device current: the device address of the array
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_ptr[dev]) {
      unsigned char* p = nullptr;
      int n = 0;
      if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_topk_scratch) != cudaSuccess ||
          cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
          !p || n < 1) {
        (void)cudaGetLastError();
        return EFCP_ECUDA;
      }
      g_static_ptr[dev] = p;
      g_static_sms[dev] = n;
    }
    base = g_static_ptr[dev];
    sms = g_static_sms[dev];
  }
  uint32_t* hist1 = reinterpret_cast<uint32_t*>(base + kOffHist);
  uint32_t* hist2 = hist1 + kBins1;
  uint32_t* hist3 = hist2 + kBins2;
  Scalars* sc = reinterpret_cast<Scalars*>(base + kOffScalars);
  int32_t* chunk_off = reinterpret_cast<int32_t*>(base + kOffChunk);
  int32_t* sel_gt = reinterpret_cast<int32_t*>(base + kOffSelGt);
  int32_t* sel_eq = reinterpret_cast<int32_t*>(base + kOffSelEq);
  int32_t* cand_idx = reinterpret_cast<int32_t*>(base + kOffCandIdx);
  float* cand_val = reinterpret_cast<float*>(base + kOffCandVal);
  const int n_chunks = int((d + kChunk - 1) / kChunk);
  // the array keeps the last call's contents: histograms and scalars must start at zero
  if (cudaMemsetAsync(base + kOffHist, 0, size_t(kOffChunk - kOffHist), st) != cudaSuccess) {
    (void)cudaGetLastError();
    return EFCP_ECUDA;
  }
  const int cand_grid = sms * 4;
  k_hist1_only<<<sms * 2, 512, 0, st>>>(a, d, hist1);
  k_pick<kBins1, 1><<<1, 1024, 0, st>>>(hist1, sc, uint32_t(k));
  k_count_chunks<<<n_chunks, kChunkThreads, 0, st>>>(a, d, sc, chunk_off, n_chunks);
  k_scan_counts<<<1, 1024, 0, st>>>(chunk_off, n_chunks, &sc->n_cand);
  k_compact_cand<<<n_chunks, kChunkThreads, 0, st>>>(a, d, sc, chunk_off, cand_idx, cand_val,
                                                     hist2, n_chunks);
  k_pick<kBins2, 2><<<1, 1024, 0, st>>>(hist2, sc, uint32_t(k));
  k_hist3<<<cand_grid, 256, 0, st>>>(cand_val, sc, hist3);
  k_pick<kBins3, 3><<<1, 1024, 0, st>>>(hist3, sc, uint32_t(k));
  k_count_sel<<<cand_grid, kChunkThreads, 0, st>>>(cand_val, sc, sel_gt, sel_eq);
  k_scan_sel<<<1, 1024, 0, st>>>(sel_gt, sel_eq, sc, uint32_t(k));
  k_write_sel_only<<<cand_grid, kChunkThreads, 0, st>>>(cand_idx, cand_val, sc, sel_gt, sel_eq,
                                                        idx, val, k);
  if (cudaGetLastError() != cudaSuccess) return EFCP_ECUDA;
  return EFCP_OK;
}
