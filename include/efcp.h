/*
 * efcp.h - C ABI of the B200 (sm_100a) EFCP / Sparse M-FAC step library.
 *
 * One handle owns the whole optimizer state of one parameter vector of
 * dimension d on one GPU: the error-feedback buffer xi (Algorithm 1),
 * the sparse ring buffer G = (I, V) of the last m compressed accumulators
 * (Section 3.1, "Sparsity format for G"), the m x m scalar-product matrix
 * S = G G^T (Section 2.1, "Scalar Products (SP)") and the inverse of
 * m*lambda*I + S from which the coefficients of Eq. (2) are read.
 *
 * Conventions for every call
 *   - returns EFCP_OK (0) or a negative EFCP_E* code; never throws, never aborts;
 *   - "device" pointers are CUDA device pointers valid on the handle's device,
 *     "host" pointers are ordinary host memory; nothing is retained after return
 *     except by the asynchronous work that efcp_step enqueues on the stream;
 *   - the caller owns grad, update and the stream; the handle owns all state and
 *     scratch, allocated once in efcp_create* on the device current at that time.
 *   - a handle is not thread-safe; steps on one handle are ordered by the stream.
 */
#ifndef EFCP_H_
#define EFCP_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct efcp_ctx efcp_ctx;

#define EFCP_OK        0
#define EFCP_EINVAL   -1  /* bad argument (null pointer, size out of range, bad lambda)   */
#define EFCP_ENOMEM   -2  /* device or host allocation failed                              */
#define EFCP_ECUDA    -3  /* a CUDA runtime call or launch failed (efcp_last_cuda_error)  */
#define EFCP_ENUMERIC -4  /* non-finite gradient entry, or a non-positive pivot in the
                             m x m update (window numerically singular for this lambda)  */
#define EFCP_ETIMEOUT -5  /* a bounded device-side wait gave up                            */
#define EFCP_EINTERNAL -6 /* an internal consistency check failed (selection count != k)  */
#define EFCP_ETOOBIG  -7  /* size beyond the fixed capacity of an allocation-free entry point */

/*
 * Environment variables read by efcp_create* (testing and tuning aids; none changes what a
 * step computes beyond the rounding of the update):
 *   EFCP_NO_SPEC=1        Top-k always takes the exact two-pass candidate route instead of the
 *                         candidates set aside while a = xi + g is formed.  Same selection.
 *   EFCP_LCG=fp32|fixed   overrides the EFCP_LCG_FP32 flag (accumulator of the linear combination).
 *   EFCP_LCG_FIXED_TOL=x  0 <= x <= 1e-4: relative error a slab of the fixed-point accumulator
 *                         may have before it is accumulated again in fp32 (default 1e-5; 0
 *                         sends every slab through the fp32 route).
 *   EFCP_SPLIT_PHASES=1   the two cooperative kernels of a step are launched once per phase
 *                         instead of once per step, so that a profiler's launch list shows
 *                         what each phase costs.  Same results, more launches.
 *   EFCP_SLAB_W=n         slab width in coordinates (multiple of 32, 256..49152) instead of the
 *                         width chosen from d, m and the SM count.  The width is part of a
 *                         checkpoint's header: a state imports only into a handle created with
 *                         the same width.
 */

/* flags for efcp_create_ex */
#define EFCP_RHS_COMPRESSED  0u /* u_t = A(c_t): precondition the compressed accumulator
                                   (Algorithm 1) - the default                             */
#define EFCP_RHS_ACCUMULATOR 1u /* precondition the full accumulator a_t = xi_t + c_t
                                   (u = F^-1 a_t; costs one more read of xi in SP and LCG)  */

#define EFCP_VALUES_BF16     2u /* window values in bfloat16 (Section 3.1, "Format for V"):
                                   the kept values are rounded to bfloat16 (nearest even),
                                   c holds the rounded values and xi = a - c keeps the
                                   rounding residue, so a = xi + c stays exact.  SP and LCG
                                   then read 4 bytes per window entry instead of 6.  Cannot
                                   be combined with EFCP_RHS_ACCUMULATOR.                   */

#define EFCP_PRECOND_GGT     4u /* Sparse GGT instead of Sparse M-FAC (appendix "Sparse GGT"):
                                   u_t = ((sum_i c_i c_i^T)^(1/2) + eps I)^-1 c_t over the
                                   window rows c_i, with eps passed in the `lambda` argument.
                                   Error feedback, Top-k, the window and the scalar products
                                   are unchanged; the m x m stage becomes a symmetric
                                   eigendecomposition, held in one SM's shared memory, which
                                   limits m to 160.  Not with EFCP_RHS_ACCUMULATOR (GGT
                                   preconditions the compressed accumulator).  For this mode
                                   efcp_get_weights returns the coefficients of u over the
                                   window rows and efcp_last_residual the relative
                                   off-diagonal norm the eigendecomposition stopped at;
                                   EFCP_ENUMERIC means it did not converge.                  */

#define EFCP_LCG_FP32        8u /* The linear combination (Section 2.1 "LCG", Section 3.1 "Sparse
                                   LCG") accumulates a slab of u in shared memory.  By default
                                   the accumulator is int32 fixed point: the shared-memory adds
                                   cost less than half of fp32 ones, and a slab's result does
                                   not depend on the order of the adds.  The scale of a slab
                                   comes from a bound that excludes overflow; a slab whose
                                   rounding error (estimated from the number of entries and
                                   the step of the grid) could exceed 1e-5 of its norm is
                                   accumulated again in fp32, so the update stays within the
                                   same 1e-4 of the exact one (efcp_fixed_point_fallbacks
                                   counts those slabs).  This flag selects fp32 atomic adds
                                   for every slab instead.  EFCP_RHS_ACCUMULATOR always uses
                                   fp32 adds.  The choice is not part of the state: a state
                                   exported with one setting imports into the other.          */

#define EFCP_DEBUG_CHECKS   16u /* After every step the library checks, on the device and on the
                                   step's stream, what it derived from the new row (offset
                                   table, slab membership of every entry, the 16-bit index
                                   stream, the slab weights); a violation turns into the sticky
                                   status EFCP_EINTERNAL.  Three more small launches per step.   */

/*
 * efcp_create / efcp_create_ex - the initialisation of Algorithm 1: set up an empty window and
 * xi_0 = 0 for dimension d, window length m, k kept entries per step (Top-k of
 * Section 3.1, k given as a count) and damping lambda (F_0 = lambda I, Section 2.1).
 * Requires 1 <= k <= d < 2^31, 1 <= m <= 4096, lambda finite and > 0.
 * Rows not written yet count as zero gradients; the 1/m of the empirical Fisher
 * always uses the capacity m.  *out receives the handle (NULL on failure).
 */
int efcp_create(efcp_ctx** out, int64_t d, int32_t m, int64_t k, float lambda);
int efcp_create_ex(efcp_ctx** out, int64_t d, int32_t m, int64_t k, float lambda,
                   uint32_t flags);

/*
 * efcp_create_blockwise - the same optimizer with Top-k applied in blocks (Section 3.1,
 * "Sparsity Pattern"): the coordinates are cut into blocks of `block` coordinates and every
 * block keeps exactly ceil(len * k / d) entries of largest magnitude, len being the block's
 * length (the last block may be shorter), ties to the lower index; at 1 % density that is
 * the paper's ceil(B / 100) per block.  A row of the window then holds efcp_row_length(ctx)
 * entries (the sum over the blocks, a little above k), and every efcp_get_* call that speaks
 * of k entries means that many.  Everything after the selection is as in efcp_create_ex.
 *   block: a multiple of 32 in [32, 16384].
 */
int efcp_create_blockwise(efcp_ctx** out, int64_t d, int32_t m, int64_t k, float lambda,
                          uint32_t flags, int32_t block);

/*
 * Caller-supplied memory (the ownership rule of the problem statement's create call: the
 * handle owns its state, the caller may own the memory it lives in).
 *   efcp_workspace_bytes : device bytes a handle for these arguments needs in total (state and
 *                          scratch; the same list of buffers efcp_create_blockwise allocates,
 *                          for the SM count of the current device, or of a B200 when there is
 *                          no device); -1 for invalid arguments.  efcp_step_host needs
 *                          8 d + 512 bytes more for its staging copies of grad and update.
 *   efcp_create_in       : efcp_create_blockwise (block = 0: global Top-k) that takes every
 *                          buffer from `workspace` (device, 256-byte aligned, workspace_bytes
 *                          long) and never calls cudaMalloc; EFCP_ENOMEM when it is too
 *                          small.  The workspace stays the caller's: efcp_destroy does not
 *                          free it, and it must outlive the handle.
 */
int64_t efcp_workspace_bytes(int64_t d, int32_t m, int64_t k, uint32_t flags, int32_t block);
int efcp_create_in(efcp_ctx** out, int64_t d, int32_t m, int64_t k, float lambda, uint32_t flags,
                   int32_t block, void* workspace, int64_t workspace_bytes);

/* Entries per window row: k, or the block-wise total (-1 for a NULL handle). */
int64_t efcp_row_length(efcp_ctx* ctx);

/*
 * efcp_step - the body of Algorithm 1's loop for one gradient, without the parameter update:
 *     a = xi + g                      (fp32, one rounding per coordinate)
 *     c = TopK_k(a)                   (global over d, exact, ties to the lower index)
 *     xi = a - c                      (kept coordinates become +0)
 *     row (t-1) mod m of G = c        (indices ascending)
 *     u = (lambda I + (1/m) G^T G)^-1 x,  x = c (default) or a (EFCP_RHS_ACCUMULATOR),
 * the last line evaluated as Eq. (2), a linear combination of the window rows with
 * coefficients obtained from S (Section 2.1).
 *   grad   device, d floats, read only.
 *   update device, d floats, every element overwritten; must not alias grad.
 *   stream a cudaStream_t (NULL = default stream).  All work is enqueued on it and
 *          the call returns without waiting.  Learning rate, weight decay and the
 *          parameter update are left to the caller (or to efcp_apply_update).
 * Errors detected on the device (EFCP_ENUMERIC, ...) are sticky and reported by
 * efcp_status or the next efcp_get_* call.
 */
int efcp_step(efcp_ctx* ctx, const float* grad, float* update, void* stream);

/*
 * efcp_step_host - the same step for callers whose gradient and update live in host
 * memory (pinned memory gives the best copy rate): copies grad to the device, runs
 * the step, copies the update back and waits.  For large d the linear combination runs
 * over four consecutive ranges of coordinates, and every finished range of the update
 * starts its way to the host (on a stream of the handle's own) while the next range is
 * still being accumulated.
 *   grad, update: host, d floats each.
 */
int efcp_step_host(efcp_ctx* ctx, const float* grad, float* update, void* stream);

/* Frees all device and host memory of the handle (waits for the device first). */
int efcp_destroy(efcp_ctx* ctx);

/*
 * State inspection (parity tests, checkpointing).  Each call waits for all work
 * queued on the handle's device, then copies to host memory:
 *   efcp_get_error : xi, d floats.
 *   efcp_get_row   : ring slot `slot` (0 <= slot < m): k ascending indices and the k
 *                    values.  A slot never written reads as indices 0..k-1, values 0.
 *   efcp_get_gram  : S = G G^T, m*m doubles, row-major, exactly symmetric
 *                    (Section 2.1: row and column i are replaced together).
 *   efcp_get_weights: the m fp64 weights w of the last step's linear combination:
 *                    update = sum_r w_r row_r in the default mode,
 *                    update = xi/lambda + sum_r w_r row_r with EFCP_RHS_ACCUMULATOR.
 * Returns the sticky device status if it is an error, else EFCP_OK.
 */
int efcp_get_error(efcp_ctx* ctx, float* host_e);
int efcp_get_row(efcp_ctx* ctx, int32_t slot, int32_t* host_idx, float* host_val);
int efcp_get_gram(efcp_ctx* ctx, double* host_S);
int efcp_get_weights(efcp_ctx* ctx, double* host_w);

/*
 * efcp_get_window - device pointers to the ring buffer G = (I, V) for read-only
 * inspection by code running on the same device (tests compute residuals of the defining
 * linear system at sizes where copying the window to the host is too slow).  Waits for the
 * device first.  *dev_I and *dev_V point to m rows of k entries each (row = ring slot);
 * inside a row the entries of each slab of coordinates are contiguous but not sorted
 * (Section 3.1 leaves the order inside a row open; efcp_get_row returns ascending order).
 * The pointers stay valid until efcp_destroy; writing through them is undefined.
 */
int efcp_get_window(efcp_ctx* ctx, const int32_t** dev_I, const float** dev_V);

/*
 * Checkpoint / resume.  The optimizer state of Algorithm 1 is xi and the window G (plus what
 * the library derives from them: S, the inverse, the offset table, the index and value
 * streams); efcp_state_export copies all of it into host memory, efcp_state_import puts it
 * back into a handle created with the same d, m, k, lambda and flags on the same kind of
 * GPU (the slab width, which depends on d, m and the SM count, must agree).  A run resumed
 * from an imported state continues like the run that exported it: the state bit for bit,
 * the updates up to the fp32 rounding of their accumulation order.
 *   efcp_state_size   : bytes efcp_state_export writes (-1 for a NULL handle).
 *   efcp_state_export : waits for the device; host_buf needs efcp_state_size bytes.
 *   efcp_state_import : waits for the device; EFCP_EINVAL when the header does not match
 *                       the handle or `bytes` is too small.
 */
int64_t efcp_state_size(efcp_ctx* ctx);
int efcp_state_export(efcp_ctx* ctx, void* host_buf, int64_t bytes);
int efcp_state_import(efcp_ctx* ctx, const void* host_buf, int64_t bytes);

/*
 * efcp_error_norm - the Euclidean norm of the error buffer xi (fp64 accumulation), the
 * numerator of the error-feedback evolution metric |xi_t| / (|g_1| + ... + |g_t|) of
 * Section 4 ("Error Feedback Evolution During Training"); the gradient norms are the
 * caller's.  Waits for the device.  *out (host) receives the norm.
 */
int efcp_error_norm(efcp_ctx* ctx, double* out);

/*
 * The parameter update (last line of the loop of Algorithm 1) with the decoupled weight
 * decay of Section 2 (the paragraph on the interaction with regularisation):
 *     theta <- (1 - gamma eta) theta - eta s u,
 * where s = 1, or, with clipping of the preconditioned gradient's norm as in the
 * hyper-parameter appendix (clip_norm > 0), s = min(1, clip_norm / |u|_2).
 *
 *   efcp_update_norm  : |u|_2 over the d entries of `update` (device; fp64 accumulation in a
 *                       fixed order), kept on the device for the efcp_apply_update calls
 *                       that follow.  Asynchronous on `stream` when host_out is NULL;
 *                       otherwise waits for the stream and stores the norm in *host_out.
 *   efcp_apply_update : the formula above on n coordinates, theta and update (device, n
 *                       floats each, any alignment) being the same sub-range of the
 *                       parameter vector and of u; groups of parameters with their own eta
 *                       and gamma are separate calls.  With clip_norm > 0, s uses the norm of
 *                       the last efcp_update_norm call, which has to have been made since the
 *                       last efcp_step (EFCP_EINVAL otherwise).  fp32 arithmetic: (1 - gamma
 *                       eta) and eta s are formed in fp64 and rounded once, the update is one
 *                       multiply and one fused multiply-add per coordinate.  Asynchronous.
 *   efcp_step_apply   : efcp_step, then efcp_update_norm (if clip_norm > 0) and
 *                       efcp_apply_update over all d coordinates, on the same stream;
 *                       `update` receives u.  With update == NULL (and clip_norm == 0,
 *                       EFCP_EINVAL otherwise: clipping needs |u| before any of it is applied)
 *                       u is never written: the linear combination updates theta slab by
 *                       slab from shared memory, which saves the write and one read of u.
 *                       The arithmetic per coordinate is the same.
 * eta >= 0, gamma >= 0, clip_norm >= 0 and finite, 1 <= n <= d; EFCP_EINVAL otherwise.
 */
int efcp_update_norm(efcp_ctx* ctx, const float* update, double* host_out, void* stream);
int efcp_apply_update(efcp_ctx* ctx, float* theta, const float* update, int64_t n, float eta,
                      float gamma, float clip_norm, void* stream);
int efcp_step_apply(efcp_ctx* ctx, const float* grad, float* theta, float* update, float eta,
                    float gamma, float clip_norm, void* stream);

/*
 * efcp_validate - consistency check of the window's derived structures (a debugging aid; the
 * memory checker of the CUDA toolkit is not always available).  For every written row it
 * verifies on the device that the offset table is monotone and ends at the row length, that
 * every entry lies in the slab its segment belongs to, that the 16-bit stream agrees with
 * the indices, and that the slab weights equal the column sums of the offset table.  Waits
 * for the device.  Returns EFCP_OK, EFCP_EINTERNAL when a check fails (*bad, if not NULL,
 * receives the number of violations), or the sticky status if that is an error.
 */
int efcp_validate(efcp_ctx* ctx, int64_t* bad);

/*
 * Coordinate-sharded state: one optimizer state spread over several GPUs by ranges of
 * coordinates.  The paper runs on one GPU and has no counterpart of this; the split follows
 * from the method: error feedback, the window rows and the update are separable by
 * coordinate, the Top-k threshold and the scalar products are sums over the shards.  Shard r of
 * n holds the coordinates [d_lo, d_hi) (ranges ascending with r, disjoint, covering
 * [0, d_global)): its part of xi, of every window row and of u; S and the m x m stage are
 * replicated.  k_global is the number of entries kept over all shards; a row of a shard holds
 * as many of them as fall into its range, at most row_cap (<= 0: min(k_global, d_hi - d_lo),
 * the worst case; a step that would need more raises EFCP_EINTERNAL).  Indices inside a shard
 * are relative to d_lo.  Flags: EFCP_VALUES_BF16, EFCP_LCG_FP32, EFCP_DEBUG_CHECKS.
 *
 * A step is six phases.  Every shard runs efcp_shard_phase(p), then buffer p of all shards
 * (efcp_shard_buffer) is summed element-wise over the shards and the sum stored back in every
 * shard's buffer - an all-reduce, e.g. NCCL's on the step's stream - then phase p + 1 runs:
 *   p = 0  a = xi + g (needs grad: device, d_hi - d_lo floats)    buffer: 4096 uint32
 *   p = 1  first digit of the threshold key                         buffer: 1024 uint32
 *   p = 2  second digit                                             buffer: 512 uint32
 *   p = 3  the key; entries above / equal to it on this shard       buffer: 2 n uint32
 *   p = 4  selection (ties at the key go to lower coordinates first), residual, ring insert,
 *          this shard's part of the scalar products                 buffer: m doubles
 *   p = 5  S, coefficients, this shard's part of u (needs update: device, d_hi - d_lo floats)
 * Unsigned sums may be formed as signed 32-bit sums (the bits are the same).  Nothing in the
 * library reads another GPU's memory; the exchanges are the caller's.  Phases must be called
 * in order (EFCP_EINVAL otherwise).  The state (xi, rows) equals that of an unsharded handle
 * bit for bit; u agrees up to the rounding of the summed scalar products.
 *   efcp_row_count : entries ring slot `slot` holds (k for an unsharded handle); efcp_get_row
 *                    returns that many, then (0, 0) up to the row capacity.  Waits for the device.
 */
int efcp_create_shard(efcp_ctx** out, int64_t d_global, int64_t d_lo, int64_t d_hi, int32_t m,
                      int64_t k_global, int64_t row_cap, float lambda, uint32_t flags,
                      int32_t shard, int32_t n_shards);
int efcp_shard_phase(efcp_ctx* ctx, int32_t phase, const float* grad, float* update,
                     void* stream);
int efcp_shard_buffer(efcp_ctx* ctx, int32_t phase, void** dev_ptr, int64_t* count,
                      int32_t* is_f64);
int64_t efcp_row_count(efcp_ctx* ctx, int32_t slot);

/*
 * efcp_test_hook - switches for failure-detection tests; never needed in production.
 *   EFCP_HOOK_DROP_BLOCK_LOADS (value 0/1): the block-wise Top-k kernel arms the barrier it
 *       waits on for its bulk copies of xi and g but does not issue the copies, so nothing is
 *       in flight and the kernel's bounded wait (about a second) runs out: the step ends with
 *       the sticky status EFCP_ETIMEOUT and an undefined result, the context stays usable,
 *       the handle can be destroyed.  Only handles from efcp_create_blockwise are affected.
 * Returns EFCP_EINVAL for an unknown hook.
 */
#define EFCP_HOOK_DROP_BLOCK_LOADS 1
int efcp_test_hook(efcp_ctx* ctx, int32_t hook, int32_t value);

/* Number of completed efcp_step calls on this handle (-1 for a NULL handle). */
int64_t efcp_step_count(efcp_ctx* ctx);

/* Waits for the device and returns the sticky status (EFCP_OK or an error code). */
int efcp_status(efcp_ctx* ctx);

/* The cudaError_t recorded with the last EFCP_ECUDA on this handle (0 if none). */
int efcp_last_cuda_error(efcp_ctx* ctx);

/*
 * Relative residual |m e_i - (m lambda I + S) w| / m of the last step's m x m solve
 * (fp64), a drift monitor for the incrementally updated inverse.  Waits for the device.
 */
double efcp_last_residual(efcp_ctx* ctx);

/* efcp_workspace_bytes for the default mode (no flags, global Top-k). */
int64_t efcp_state_bytes(int64_t d, int32_t m, int64_t k);

/* Slabs of the update that the fixed-point accumulator handed to fp32 since the handle was
 * created (0 with EFCP_LCG_FP32, -1 for a NULL handle or a CUDA error).  Waits for the device. */
int64_t efcp_fixed_point_fallbacks(efcp_ctx* ctx);

/* Number of kernels one efcp_step launches for this handle. */
int32_t efcp_launches_per_step(efcp_ctx* ctx);

/*
 * Stage timing with CUDA events recorded on the step's own stream.
 *   efcp_profile_begin : from the next efcp_step on, record events around the four
 *                        stages of a step, for at most max_steps steps (1..4096).
 *   efcp_profile_end   : waits for the device, adds up the elapsed times of the steps
 *                        recorded since efcp_profile_begin and stops recording.
 *                        ms_out (host, 4 doubles) receives the totals in milliseconds:
 *                        [0] error feedback + Top-k + ring insert (Algorithm 1),
 *                        [1] the scalar-product (SP) kernel alone,
 *                        [2] the m x m stage,
 *                        [3] the linear-combination (LCG) kernel alone;
 *                        *steps_out (host) receives the number of steps recorded.
 */
int efcp_profile_begin(efcp_ctx* ctx, int32_t max_steps);
int efcp_profile_end(efcp_ctx* ctx, double* ms_out, int32_t* steps_out);

/*
 * efcp_topk_static - the exact Top-k selection of efcp_step (k largest magnitudes, ties to
 * the lower index, pairs in ascending index order) as a stand-alone call that allocates
 * nothing.  The paper has no counterpart of this call; it exists for callers that must
 * not allocate device memory: code running while a memory pool or another framework owns
 * all free device memory, code inside a region where cudaMalloc's implicit device-wide
 * synchronisation is not acceptable, and start-up paths that must not fail with
 * out-of-memory.  efcp_create, by contrast, calls cudaMalloc.
 *
 * The scratch memory of the selection (histograms, chunk counters and the candidate list,
 * 8 bytes per element of `a`) lives in one fixed array inside the library image,
 * EFCP_TOPK_STATIC_MAX_D elements long: about 8.1 MiB that every GPU which loads the
 * library holds until the process exits.
 *   a      device, d floats, read only, 16-byte aligned (the kernels read it with vector
 *          loads; a view that starts at an odd element of a larger buffer is refused
 *          with EFCP_EINVAL rather than read).
 *   idx    device, k int32: receives the kept indices, ascending.
 *   val    device, k floats: receives a[idx[j]].
 *   stream a cudaStream_t (NULL = default stream); the work is enqueued, not awaited.
 * Non-finite entries are ranked, not reported: magnitudes are ordered by their IEEE bit
 * pattern, so Inf ranks above every finite value and NaN above Inf, and unlike efcp_step
 * this call has no handle whose status could record them.
 * Returns EFCP_EINVAL for null pointers, a misaligned `a` or k outside 1..d, EFCP_ETOOBIG when
 * d > EFCP_TOPK_STATIC_MAX_D (nothing is enqueued), EFCP_ECUDA when a runtime call fails.
 * The first call on each device looks up the array's device address and the SM count;
 * make that first call outside any stream capture.  All calls on a device share the one
 * array: the call clears the parts that must start at zero, and two calls whose GPU work
 * overlaps (different streams, different host threads) race on it - serialise them.
 */
#define EFCP_TOPK_STATIC_MAX_D (1 << 20)
int efcp_topk_static(const float* a, int64_t d, int64_t k, int32_t* idx, float* val, void* stream);

/* Static description of an EFCP_* code. */
const char* efcp_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* EFCP_H_ */
