/*
 * prm.h - C ABI of the Periodic Row-wise Muon optimizer step for NVIDIA B200.
 *
 * The library performs, for a list of 2-D weight matrices, the matrix branch
 * of the paper's Algorithm 1 ("Periodic Row-wise Muon"): momentum update,
 * orientation, then either the NS5 spectral refresh (Eq. periodic-direction,
 * rho_t = 1; recurrence of Appendix Eq. app-ns-recurrence) or the row-wise
 * normalised direction gamma * RowNorm_eps (Eq. rownorm, rho_t = 0), and the
 * decoupled-weight-decay parameter update of Eq. periodic-direction.
 *
 * Conventions
 *   - Matrices are stored row-major, contiguous, rows x cols; "wide" means
 *     rows <= cols, "tall" means rows > cols.  The orientation map of
 *     Section 3.1 transposes tall matrices, so RowNorm normalises stored
 *     rows of wide matrices and stored COLUMNS of tall ones.
 *   - All matrix pointers are DEVICE pointers, 16-byte aligned.  The arrays
 *     of pointers handed to prm_step are HOST arrays of length n_mats.
 *   - The caller owns parameters, gradients, momentum, the workspace and the
 *     stream.  prm_step enqueues work on the stream and returns; it never
 *     synchronises and never allocates device memory.
 *   - Every function returns PRM_OK (0) or a negative error code; nothing
 *     aborts the process.  prm_last_error() gives a text for the last error
 *     on that handle.
 *   - There is no CPU fallback: without a CUDA device the compute entry
 *     points return PRM_ERR_CUDA.
 */
#ifndef PRM_H_
#define PRM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define PRM_API __attribute__((visibility("default")))
#else
#define PRM_API
#endif

#define PRM_OK                  0
#define PRM_ERR_ARG            -1   /* null pointer, K < 1, bad option key or value */
#define PRM_ERR_SHAPE          -2   /* non-positive or unsupported dimension */
#define PRM_ERR_ALIGN          -3   /* device pointer not 16-byte aligned */
#define PRM_ERR_WORKSPACE      -4   /* workspace missing or too small */
#define PRM_ERR_CUDA           -5   /* a CUDA runtime/driver call failed */
#define PRM_ERR_DEVICE_TIMEOUT -6   /* a bounded device-side wait expired */
#define PRM_ERR_STATE          -7   /* call not allowed in this state */

/* Option keys for prm_set_option. */
#define PRM_OPT_GAMMA        1  /* RowNorm multiplier gamma (Section 3.2), default 0.15 */
#define PRM_OPT_EPS_ROW      2  /* epsilon of Eq. rownorm, default 1e-8 */
#define PRM_OPT_EPS_NS       3  /* epsilon added to ||X||_F before NS5, default 1e-7 */
#define PRM_OPT_SCALE_MODE   4  /* s(W): 0 -> 1; 1 (default) -> sqrt(max(1, rows/cols));
                                   2 -> 0.2*sqrt(max(rows, cols)) */
#define PRM_OPT_IO_DTYPE     5  /* 0 (default): bf16 params and grads; 1: fp32 params and
                                   grads.  Momentum is fp32 in both.  Before set_workspace. */
#define PRM_OPT_CHECK_MODE   6  /* 0 (default): NS5 on tensor cores, bf16 operands, fp32
                                   accumulate; 1: NS5 in fp32 on CUDA cores (slow, for
                                   verification).  Before set_workspace. */
#define PRM_OPT_LR           7  /* eta_t; may be changed between any two steps */
#define PRM_OPT_WD           8  /* lambda; may be changed between any two steps */
#define PRM_OPT_NS_WORKSPACE_BYTES 9 /* soft cap on the NS5 part of the workspace, default
                                   8 GiB; matrices of one shape group are refreshed in
                                   sub-batches that fit.  Before set_workspace. */
/* Variants of the ablation table (Table 3a of the paper); may be changed between steps. */
#define PRM_OPT_GAMMA_NS    10  /* multiplier on the NS5 branch, default 1 (the paper's method);
                                   "scalar-controlled" sets it to gamma */
#define PRM_OPT_NO_REFRESH  11  /* 1: RowNorm at every step, no NS5 schedule; default 0 */
/* How the tensor-core path evaluates the five NS5 iterations (Appendix "Cost of
 * NS5").  The iteration X <- aX + BX with A = X X^T, B = bA + cA^2 keeps every A_k
 * a polynomial in A_0, and A_{k+1} = (aI + B_k) A_k (aI + B_k).
 *   0: all five iterations as printed, 15 r^2 c + 5 r^3 flop per matrix (with
 *      triangle-only symmetric products).
 *   1: for matrices with at least 1024 oriented rows r and c >= 1.5 r columns
 *      the first three iterations work on r x r matrices only (A_1, A_2 and the
 *      product of the three factors aI + B_k from r x r products), then X_3
 *      comes from one r x c product and the last two iterations run as
 *      printed: 9 r^2 c + 11 r^3 flop, the same result in exact arithmetic and
 *      the same measured error as 0.
 *   2 (default): as 1, and beyond c = 2 r the Gram matrix of the fifth iteration
 *      is taken from the fourth's (A_4 = (aI + B_3) A_3 (aI + B_3), two r x r
 *      products instead of X_4 X_4^T): 8 r^2 c + 13 r^3 flop.  Measured error
 *      against the fp64 recurrence 5-50 % above that of 0 and 1 on the
 *      benchmark's inputs (at most 1.1e-2 relative Frobenius error).
 * The check mode always runs the iterations as printed.  Before set_workspace
 * (the workspace holds two more r x r matrices per refreshed matrix with 1 or 2). */
#define PRM_OPT_NS_GRAM_SPAN 12
/* Which kernels take the row step (rho_t = 0) of TALL matrices, where RowNorm
 * (Eq. rownorm, on the transposed matrix of Section 3.1) normalises stored columns:
 *   0 (default), 1: two passes over gradient and momentum (20 bytes per element);
 *   2: one pass over HBM (14 bytes per element: the data waits in shared memory
 *      for the column norms) for bf16 matrices with cols % 8 == 0 and at most
 *      ~25000 rows, two passes for the rest.  Fewer bytes, but bound by the SMs'
 *      instruction issue: faster than the two passes at full SM clock, slower at
 *      the reduced clock that follows a power-capped refresh.
 * Both give the same result up to the order of the fp32 sums.  Before set_workspace. */
#define PRM_OPT_TALL_KERNEL 13
/* Accuracy option of the tensor-core NS5 (the paper fixes no arithmetic format for
 * Eq. app-ns-recurrence; the default stores every operand in bf16).  For inputs whose
 * spectrum has a few singular values far above the rest, the bf16 rounding of the
 * NS5 input X_0 alone, whose noise is then of the order of the small singular values,
 * puts the result 5-6e-2 (relative Frobenius) from the fp64 recurrence.
 *   0 (default): X_0 stored as one bf16 matrix.
 *   1: X_0 stored as two bf16 matrices H = bf16(X_0), L = bf16(X_0 - H).  Matrices
 *      with more than 768 oriented rows take the Gram-space order of
 *      PRM_OPT_NS_GRAM_SPAN whatever their aspect ratio; in it X_0 enters two
 *      products only, X_0 X_0^T (computed as H H^T + H L^T + L H^T) and Q X_0
 *      (Q H + Q L): 4 r^2 c more flop per matrix (+ 25-35 % on the benchmark's
 *      shapes), one more r x c matrix of workspace per refreshed matrix.  Smaller
 *      matrices are refreshed in fp32 on CUDA cores, like those with fewer than 64
 *      rows (the Gram-space order costs them more accuracy on ordinary inputs than
 *      the second plane returns).  Brings the inputs described above inside the
 *      2e-2 of all others.  prm_refresh_segments keeps one plane: its input is
 *      the bf16 payload of the exchange, which has no second plane to offer.
 * Before set_workspace. */
#define PRM_OPT_NS_SPLIT_INPUT 14
/* Which kernels take the row step (rho_t = 0) of WIDE matrices (Eq. rownorm on stored rows)
 * and their NS5 pre-pass (momentum update, direction input, Frobenius sum):
 *   0 (default): for bf16 matrices with cols % 8 == 0 (row step: at most 24576 columns)
 *      persistent kernels, one CTA per SM, whose producer warp streams the rows in with bulk
 *      asynchronous copies ahead of the warps that work on them; the kernels of 1 for the rest.
 *   1: row step with one stored row per CTA (per cluster beyond 32768 columns), pre-pass with
 *      4 rows x 2048 columns per CTA; loads held in registers.
 * Same arithmetic and bytes per element either way; sums are added in another order, so the
 * two agree to rounding, not bit for bit.  May be changed between steps. */
#define PRM_OPT_WIDE_KERNEL 15


typedef struct prm_ctx prm_ctx;

/*
 * Create a handle for n_mats matrices (Algorithm 1's Muon set W_M).
 *   shapes   host array of 2*n_mats int64: (rows, cols) of matrix i at [2i], [2i+1]
 *   K        refresh period, K >= 1; step t refreshes iff t mod K == 0 (Section 3.2)
 *   beta     momentum coefficient of M_t = beta*M_{t-1} + (1-beta)*G_t
 *   nesterov 0: direction from M_t; 1: from beta*M_t + (1-beta)*G_t
 *   lr, wd   eta_t and lambda of Eq. periodic-direction
 * Uses the CUDA device current at the time of the call.  Allocates only host
 * memory.  On failure *out is NULL.
 */
PRM_API int prm_create(prm_ctx** out, const int64_t* shapes, int n_mats,
               int K, float beta, int nesterov, float lr, float wd);

/* Set an option (keys above).  Returns PRM_ERR_STATE for options that must be
 * set before prm_set_workspace once a workspace is attached. */
PRM_API int prm_set_option(prm_ctx* ctx, int key, double value);

/* Bytes of device workspace needed with the current options (pointer tables,
 * column-norm scratch of tall row-steps, NS5 operands).  0 on a NULL handle. */
PRM_API size_t prm_workspace_bytes(const prm_ctx* ctx);

/* Attach caller-allocated device workspace (256-byte aligned, at least
 * prm_workspace_bytes).  The library keeps the pointer until prm_destroy or
 * the next prm_set_workspace; the caller frees it afterwards. */
PRM_API int prm_set_workspace(prm_ctx* ctx, void* dev_ptr, size_t bytes);

/*
 * One optimizer step for all matrices (Algorithm 1 lines 2-9 for step t =
 * step_idx, zero-based): updates momentum[i] and params[i] in place, reads
 * grads[i].  params/grads: bf16 or fp32 per PRM_OPT_IO_DTYPE; momentum: fp32.
 * The branch depends only on step_idx mod K; steps need not be consecutive.
 * cuda_stream is a cudaStream_t (NULL = default stream).  Calls on one handle
 * must be ordered on one stream, or separated by synchronisation.
 * The first step on a handle, and any step that is given a pointer it has not
 * seen at that position before, also uploads the pointer tables (and the tensor
 * maps over the matrices) with host-to-device copies from pageable host memory:
 * such a step blocks the host until the bytes are staged and cannot run inside
 * a stream capture.  Steps with unchanged pointers only launch kernels.
 */
PRM_API int prm_step(prm_ctx* ctx, void* const* params, const void* const* grads,
             float* const* momentum, int64_t step_idx, void* cuda_stream);

/*
 * Same step, but this step's gradients come from HOST memory:
 * grads_host[i] (rows*cols elements of the I/O dtype, ideally pinned) is
 * copied to grads_dev[i] with one asynchronous copy per matrix, then the step
 * runs as in prm_step.  The copies run on a stream owned by the handle,
 * ordered after everything already queued on cuda_stream; the kernels of a
 * shape group wait only for that group's gradients, so the copy of the next
 * group overlaps the work of the current one.  Everything the call enqueues is
 * complete when cuda_stream is.
 */
PRM_API int prm_step_h2d(prm_ctx* ctx, void* const* params, void* const* grads_dev,
                 const void* const* grads_host, float* const* momentum,
                 int64_t step_idx, void* cuda_stream);

/*
 * The schedule and the shape grouping, without touching the device.
 *   is_refresh      1 iff step_idx mod K == 0 (and PRM_OPT_NO_REFRESH is off)
 *   n_groups        number of distinct (rows, cols) pairs
 *   group_of_mat    [n_mats] group id, ids numbered by first appearance
 *   order_in_group  [n_mats] position inside the group, caller order kept
 * Any output pointer may be NULL.
 */
PRM_API int prm_plan(const prm_ctx* ctx, int64_t step_idx, int* is_refresh,
             int* n_groups, int* group_of_mat, int* order_in_group);

/*
 * One shape group of the plan (0 <= group < n_groups): its stored shape, the
 * number of matrices, how many of them one refresh sub-batch holds with the
 * current workspace cap, how many leading NS5 iterations the refresh runs in
 * Gram space (0 or 3, see PRM_OPT_NS_GRAM_SPAN), and the flop one refresh of
 * one such matrix executes in its NS5 products (X X^T products counted r^2 c,
 * r x c products 2 r^2 c, symmetric r x r products r^3, r <= c the oriented
 * shape).  Host only.  Any output pointer may be NULL.  PRM_ERR_ARG for a
 * group out of range.
 */
PRM_API int prm_group_info(const prm_ctx* ctx, int group, int64_t* rows, int64_t* cols,
                   int* count, int* ns_batch, int* gram_iters, double* ns5_flop);

/* Reads the device status word (synchronises the device first): PRM_OK, or
 * PRM_ERR_DEVICE_TIMEOUT if a kernel gave up on a bounded wait since the last
 * call; the word is cleared. */
PRM_API int prm_status(prm_ctx* ctx);

/*
 * Self-test of the device-side failure path.  Every wait inside the kernels
 * (on TMA, tensor-core and epilogue barriers) is bounded; a wait that runs out
 * raises the status word and the kernel drains and returns, so the context
 * stays usable.  This call launches a one-thread kernel that waits limit_ms
 * (at most 1000) on a barrier nothing completes and then does exactly that:
 * after it, prm_status returns PRM_ERR_DEVICE_TIMEOUT once and PRM_OK again
 * afterwards.  Nothing faults, traps or hangs.
 */
PRM_API int prm_selftest_timeout(prm_ctx* ctx, double limit_ms, void* cuda_stream);

/* Text of the last error on this handle ("" if none).  Valid until the next
 * call on the handle.  With ctx == NULL: the last prm_create error. */
PRM_API const char* prm_last_error(const prm_ctx* ctx);

/* Number of kernels the library has launched through this handle so far. */
PRM_API int64_t prm_launch_count(const prm_ctx* ctx);

/*
 * Optional per-kernel-class device timing.  prm_profile(ctx, 1) makes every
 * following prm_step bracket each kernel class with CUDA events on the step's
 * stream (no device memory is allocated); prm_profile(ctx, 0) stops it.
 * prm_profile_read waits for the recorded events and adds up, per class, the
 * elapsed milliseconds and the number of kernel launches since the last read.
 * ms and launches are host arrays of n_classes entries (PRM_PROF_COUNT).
 */
#define PRM_PROF_ROW_WIDE      0  /* fused row step, wide matrices */
#define PRM_PROF_ROW_TALL      1  /* row step, tall matrices (3 kernels) */
#define PRM_PROF_PREPASS       2  /* NS5 pre-pass and norm (2 kernels) */
#define PRM_PROF_GRAM          3  /* A = X X^T */
#define PRM_PROF_POLY          4  /* B = b A + c A^2 */
#define PRM_PROF_UPDATE        5  /* X <- a X + B X */
#define PRM_PROF_UPDATE_FINAL  6  /* last X update fused with the parameter update */
#define PRM_PROF_GRAMSPACE     7  /* r x r products of the Gram-space iterations (PRM_OPT_NS_GRAM_SPAN) */
#define PRM_PROF_COUNT         8
PRM_API int prm_profile(prm_ctx* ctx, int enable);
PRM_API int prm_profile_read(prm_ctx* ctx, double* ms, int64_t* launches, int n_classes);

/*
 * Row step of ONE tall matrix (rows > cols) that allocates nothing.  (The
 * paper has no counterpart: this entry point exists for the library's users,
 * not for the method.)
 *
 * It is meant for callers that cannot allocate device memory and so cannot
 * give prm_step a workspace: code running inside a process whose memory pool
 * already owns the GPU's memory, or a loop that must stay clear of the
 * device-wide synchronisation inside cudaMalloc/cudaFree.  The column
 * partial sums and column norms that the tall row step needs live in a fixed
 * 4 MiB array inside the library image (held by every GPU that uses the
 * library, from the moment the driver loads the module until the process
 * exits).  The call itself performs no cudaMalloc,
 * cudaFree or other allocating call.
 *
 *   param, grad   device pointers, rows x cols row-major, bf16 (io_fp32 = 0)
 *                 or fp32 (io_fp32 = 1); param is updated in place
 *   momentum      device pointer, fp32, updated in place
 *   scale         the shape factor s(W) to apply (e.g. sqrt(rows/cols))
 *   other scalars as in prm_create / prm_set_option
 *   errbuf        optional host buffer for an error text (may be NULL)
 * Computes exactly what prm_step computes for a tall matrix on a non-refresh
 * step.  Limits: cols a multiple of 8, and (ceil(rows/128) + 1) * cols <=
 * 1048576 floats; larger matrices are refused with PRM_ERR_WORKSPACE and a
 * message, before anything is launched.  Wide matrices are refused with
 * PRM_ERR_SHAPE (their row step needs no scratch).
 *
 * The first call on each device looks up the array's device address (with that
 * device current); make that first call outside any stream capture.  All
 * calls share the one array: it keeps the previous call's contents, none of
 * which is read before being overwritten, and calls that overlap on the GPU
 * (different streams without ordering) race on it.
 */
PRM_API int prm_rowstep_tall_noalloc(void* param, const void* grad, float* momentum,
                                     int64_t rows, int64_t cols, int io_fp32, float beta,
                                     int nesterov, float lr, float wd, float gamma, float eps_row,
                                     float scale, void* cuda_stream, char* errbuf,
                                     size_t errbuf_len);

/*
 * AdamW for the parameters outside the Muon set (Algorithm 1 line 11: biases,
 * normalisation parameters and everything outside the transformer blocks are
 * still updated by the baseline's AdamW; hyper-parameter table: lr 1e-4,
 * betas (0.9, 0.95), eps 1e-8, weight decay 0.01).  Decoupled form with bias
 * correction, step >= 1 is the 1-based step count:
 *   p <- p*(1 - lr*wd);  m <- beta1*m + (1-beta1)*g;  v <- beta2*v + (1-beta2)*g^2
 *   p <- p - lr * (m/(1-beta1^step)) / (sqrt(v/(1-beta2^step)) + eps)
 * params/grads/exp_avg/exp_avg_sq: HOST arrays of n_tensors DEVICE pointers
 * (16-byte aligned); tensor i holds numel[i] contiguous elements of any shape;
 * params and grads are bf16 (io_fp32 = 0) or fp32, the moments fp32, all
 * updated in place.  Needs no handle and no workspace; enqueues on cuda_stream.
 */
PRM_API int prm_adamw_step(int n_tensors, void* const* params, const void* const* grads,
                           float* const* exp_avg, float* const* exp_avg_sq, const int64_t* numel,
                           int io_fp32, float lr, float beta1, float beta2, float eps, float wd,
                           int64_t step, void* cuda_stream);

/*
 * Sharded tall RowNorm (Section 3.3, Eq. sharded-tall-rownorm; Algorithm 2
 * lines 9-13): the row step of a tall matrix (global rows > cols) whose rows
 * are split over ranks.  Each rank holds rows_local consecutive rows.
 *
 * prm_tall_shard_stats   updates the local momentum rows in place and writes
 *   the local column sums of squares of the direction input, colsumsq_out[j] =
 *   sum over local rows of U_ij^2 (cols floats, device; no square root).
 *   scratch: device, prm_tall_shard_scratch_bytes(rows_local, cols) bytes.
 * The caller then SUMS colsumsq over all ranks (one all-reduce of cols floats
 * per matrix; the buffers of all tall matrices may be packed into one).
 * prm_tall_shard_apply    finishes the local rows with the global sums:
 *   nu_j = max(sqrt(colsumsq[j]), eps_row) (square root first, then the clamp),
 *   W_ij <- (1 - lr*wd) W_ij - lr*scale*gamma*U_ij/nu_j, where scale is s(W) of
 *   the GLOBAL shape, e.g. sqrt(global_rows/cols).
 * Both need cols % 8 == 0 and 16-byte aligned pointers; params/grads bf16
 * (io_fp32 = 0) or fp32, momentum fp32.  With one shard holding all rows the
 * pair computes exactly prm_step's tall row step.
 */
PRM_API size_t prm_tall_shard_scratch_bytes(int64_t rows_local, int64_t cols);
PRM_API int prm_tall_shard_stats(const void* grad_shard, float* momentum_shard, int64_t rows_local,
                                 int64_t cols, int io_fp32, float beta, int nesterov,
                                 float* colsumsq_out, float* scratch, size_t scratch_bytes,
                                 void* cuda_stream);
PRM_API int prm_tall_shard_apply(void* param_shard, const void* grad_shard, const float* momentum_shard,
                                 int64_t rows_local, int64_t cols, int io_fp32, float beta, int nesterov,
                                 float lr, float wd, float gamma, float eps_row, float scale,
                                 const float* colsumsq, void* cuda_stream);

/*
 * Refresh over row shards: the bucketed all-gather pipeline (Section 3.3,
 * "Distributed Execution"; Algorithm 2 lines 1-7; appendix "Idealized overlap
 * model").  Every stored matrix is split over `world` ranks by rows as
 * torch.chunk splits dim 0: chunk = ceil(rows / world), rank q owns rows
 * [q*chunk, min(rows, (q+1)*chunk)) (possibly none).  The Muon matrices are
 * partitioned into communication buckets; per bucket every rank fills one
 * SEGMENT of bf16 elements, the segments are all-gathered (by the caller:
 * NCCL or any other transport), and every rank then refreshes the bucket's
 * full matrices and updates its own rows.  While one bucket is refreshed the
 * next one is gathered.  The library does the device work on both sides of
 * the exchange and the planning; it contains no communication.
 *
 * prm_shard_rows     the row range of one rank (host).
 * prm_bucket_plan    host.  Walks the matrices shape group by shape group
 *   (groups in order of first appearance, caller order inside a group, so that
 *   a bucket holds matrices NS5 can batch); matrix i
 *   reserves ceil8(chunk_i * cols_i) elements in every rank's segment
 *   (offset_in_segment[i], a multiple of 8); a new bucket starts when the
 *   gathered payload world * 2 bytes * segment would exceed bucket_bytes (a
 *   bucket always holds at least one matrix).  Outputs: bucket_of_mat[n_mats],
 *   offset_in_segment[n_mats], *n_buckets, segment_elems[b] for b < *n_buckets
 *   (array of n_mats entries).
 * prm_shard_momentum_pack   device.  Algorithm 1 line 2 on this rank's rows of
 *   one matrix (momentum_shard updated in place) and the direction input U
 *   (M_t, or beta*M_t + (1-beta)*G_t with nesterov) rounded to bf16 into
 *   u_out, which points at the matrix's place in this rank's segment;
 *   reserved_elems >= rows_local*cols elements are written, the tail as
 *   zeros.  grad bf16 (io_fp32 = 0) or fp32; pointers 16-byte aligned.
 *   bf16 is what the single-GPU refresh feeds NS5 as well, so sharding does
 *   not change the NS5 input.
 * prm_refresh_gathered      device, on a handle created over the GLOBAL
 *   shapes with a workspace attached.  mats[k] (k < n): indices, in the
 *   handle's matrix order, of the bucket's matrices; gathered: the all-gather
 *   result, world segments of segment_elems bf16 elements, rank q's at
 *   q*segment_elems; offsets[k]: offset_in_segment of mats[k];
 *   param_shards[k]: this rank's rows of parameter mats[k] (bf16 or fp32 per
 *   PRM_OPT_IO_DTYPE; may be NULL when the rank owns no row).  Per shape
 *   group and sub-batch: the full oriented matrices are rebuilt from the
 *   segments straight into the NS5 workspace (with the Frobenius norm), NS5
 *   runs as in prm_step, and W_shard <- (1 - lr*wd) W_shard - lr*s(W)*X_5 is
 *   applied to rows [row_start, row_start + row_count) only; s(W) uses the
 *   global shape.  The gathered buffer may be reused as soon as the call's
 *   work on cuda_stream has passed the rebuild of its last sub-batch, i.e.
 *   after the call's work completes.  mats, offsets and param_shards are HOST
 *   arrays.  Errors as for prm_step; PRM_ERR_SHAPE if a matrix does not fit
 *   its segment.
 * prm_refresh_segments      the same, but the world segments are given by
 *   their own device pointers (HOST array of world pointers, 2-byte aligned,
 *   16-byte aligned for vector loads; at most 64 ranks).  A pointer may map
 *   ANOTHER GPU's memory (CUDA IPC, symmetric memory): the rebuild then reads
 *   the rows with plain loads over NVLink straight from the buffers the
 *   owners packed them into, and the all-gather and its receive buffer
 *   disappear into the pre-pass (no TMA and no multicast are involved in these
 *   loads).  The caller orders the reads after every owner's pack (a
 *   cross-rank barrier on the streams) and keeps a segment unchanged until all
 *   ranks have passed the call's rebuild.
 * prm_pipeline_model  host.  Ideal two-stage pipeline over n_buckets buckets
 *   with all-gather times a[l] and compute times c[l] (Eq. app-pipeline-time,
 *   Eq. app-exposed-communication):
 *     t_pipe = a[0] + sum_{l < n-1} max(c[l], a[l+1]) + c[n-1]
 *     t_comm_exposed = a[0] + sum_{l < n-1} max(0, a[l+1] - c[l])
 */
PRM_API int prm_shard_rows(int64_t rows, int world, int rank, int64_t* row_start, int64_t* row_count);
PRM_API int prm_bucket_plan(const int64_t* shapes, int n_mats, int world, int64_t bucket_bytes,
                            int* bucket_of_mat, int64_t* offset_in_segment, int* n_buckets,
                            int64_t* segment_elems);
PRM_API int prm_shard_momentum_pack(const void* grad_shard, float* momentum_shard, int64_t rows_local,
                                    int64_t cols, int64_t reserved_elems, int io_fp32, float beta,
                                    int nesterov, void* u_out, void* cuda_stream);
PRM_API int prm_refresh_gathered(prm_ctx* ctx, const int* mats, int n, const void* gathered,
                                 int64_t segment_elems, const int64_t* offsets, int world, int rank,
                                 void* const* param_shards, void* cuda_stream);
PRM_API int prm_refresh_segments(prm_ctx* ctx, const int* mats, int n, const void* const* segments,
                                 int64_t segment_elems, const int64_t* offsets, int world, int rank,
                                 void* const* param_shards, void* cuda_stream);
PRM_API int prm_pipeline_model(const double* a, const double* c, int n_buckets, double* t_pipe,
                               double* t_comm_exposed);

/*
 * The partition that needs no optimizer collective: whole matrices assigned
 * to ranks.  Every matrix's update is independent of every other's (Algorithm
 * 1 lines 4-10), so a rank that owns a matrix (parameter, gradient, momentum)
 * runs prm_step on its own list and nothing is exchanged; Section 3.3's
 * collectives exist only because dim-0 sharding splits each matrix.  Host
 * only: longest-processing-time greedy on the NS5 flop the default schedule
 * executes for each matrix (PRM_OPT_NS_GRAM_SPAN = 2: 8 r^2 c + 13 r^3 where the
 * Gram-space iterations apply, else 15 r^2 c + 5 r^3; decreasing cost, ties
 * by index; least-loaded rank, ties by
 * rank).  owner_of_mat[n_mats] receives the rank of each matrix, cost_out[world]
 * (may be NULL) the flop assigned to each rank.  The paper does not describe
 * this layout; it is offered beside the paper's.
 */
PRM_API int prm_partition_matrices(const int64_t* shapes, int n_mats, int world, int* owner_of_mat,
                                   double* cost_out);

/*
 * The shape-dependent update scale s(W) of Eq. finite_ns5 for a stored
 * rows x cols matrix under PRM_OPT_SCALE_MODE `mode` (the paper names s(W) and
 * does not define it; the modes are listed at the option).  Host only.  A
 * caller that applies the row step to a row SHARD (prm_tall_shard_apply) passes
 * the scale of the whole matrix, which this returns; 0 on a bad argument.
 */
PRM_API double prm_shape_scale(int mode, int64_t rows, int64_t cols);

/* Frees host resources.  Device memory belongs to the caller. */
PRM_API int prm_destroy(prm_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* PRM_H_ */
