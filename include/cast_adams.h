/*
 * cast_adams.h -- C ABI of the fused AdamS N:M optimizer step for NVIDIA B200 (sm_100a).
 *
 * One call performs, for every parameter of a row-major weight matrix W (rows x cols,
 * cols = input dimension), one iteration of the AdamS optimizer of CAST (arxiv 2509.25996):
 *
 *   - N:M magnitude selection per group of M consecutive columns            (Eq. 3, 4, 6)
 *   - first moment           mu   = beta1 m + (1 - beta1) g                  (Alg. 1 / Eq. 8)
 *   - proportional L1 decay  mu~  = (1 - a) mu + a lambda Sign(w), a = t/T,
 *                            on entries outside the kept set, mu~ = mu inside (Eq. 7, Alg. 1)
 *   - second moment          v    = beta2 v + (1 - beta2) mu~^2               (Eq. 8)
 *   - bias-corrected update  w    = w - lr (mu~/(1-beta1^t)) / (sqrt(v/(1-beta2^t)) + eps)
 *   - forward weight         Diag(A~) W~ (Eq. 12), pruned by the mask (Alg. 2, final loop), as bf16
 *   - mask metadata, one bit per parameter (Remark of Sec. 4.1), optional flip count (App. C)
 *
 * Conventions shared by every entry point
 *   - Returns CAST_OK (0) or a negative status.  Nothing throws, aborts or synchronises the
 *     device; all argument checks run on the host before any launch.  After CAST_ERR_CUDA,
 *     cast_last_cuda_error() gives the cudaError_t that was seen on this thread.
 *   - "device pointer" = memory reachable from the current CUDA device; "host pointer" = ordinary
 *     host memory.  The caller owns every buffer and keeps it alive until `stream` has passed the
 *     work.  Buffers of one matrix must not overlap each other.
 *   - w, m, v are updated IN PLACE.  Non-finite inputs are not checked; results are then
 *     unspecified (the paper is silent).
 *   - Shapes: cols % 32 == 0 (a metadata word describes 32 consecutive columns of one row),
 *     cols % M == 0, M in {2, 4, 8, 16, 32}, 1 <= N <= M, rows*cols < 2^31 per matrix.
 *     Every device pointer is 16-byte aligned.
 *   - bf16 values are passed as raw 16-bit patterns (cast_bf16).
 *
 * Metadata layout (the paper fixes only its size; the layout is defined here):
 *   uint32 words, row-major, cols/32 words per row.  Group i of row r owns the M-bit field at
 *   bit offset (i*M) mod 32 of word r*(cols/32) + (i*M)/32.
 *     bitmask form (CAST_F_META_BITMASK, any N:M): bit j of the field is set iff column i*M+j is kept.
 *     index form   (default, 2:4 only):            field = lo | hi << 2 with lo < hi the positions
 *                                                   (0..3) of the two kept columns.
 */
#ifndef CAST_ADAMS_H
#define CAST_ADAMS_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define CAST_API __attribute__((visibility("default")))
#else
#define CAST_API
#endif

typedef uint16_t cast_bf16;      /* raw bfloat16 bits                        */
typedef void*    cast_stream_t;  /* a cudaStream_t (NULL = the default stream) */

enum cast_status {
    CAST_OK         =  0,
    CAST_ERR_NULL   = -1,   /* a required pointer is NULL                                   */
    CAST_ERR_SHAPE  = -2,   /* rows/cols/segment sizes violate the shape rules              */
    CAST_ERR_ALIGN  = -3,   /* a device pointer is not 16-byte aligned                      */
    CAST_ERR_NM     = -4,   /* unsupported N:M, or index-form metadata asked for N:M != 2:4 */
    CAST_ERR_HYPER  = -5,   /* hyper-parameter out of range (see cast_adams_step)           */
    CAST_ERR_CUDA   = -6,   /* a CUDA runtime call failed; see cast_last_cuda_error()       */
    CAST_ERR_PLAN   = -7,   /* invalid plan / context handle, or it is too small            */
    CAST_ERR_ALIAS  = -8,   /* two buffers of one matrix overlap                            */
    CAST_ERR_MEMORY = -9,   /* a pointer is not of the required kind (device / host)        */
    CAST_ERR_STAGING = -10  /* an earlier step of this plan gave up waiting for one of its bulk
                               copies (see CAST_F_BULK_STAGING): a tile of the state was left as it
                               was; the plan refuses further steps                            */
};

enum cast_flags {
    CAST_F_RESELECT      = 1u << 0, /* choose the kept set from |w_{t-1}| now (Eq. 6).  Without it the
                                       kept set is decoded from `meta` (mask reuse between the refreshes
                                       the paper makes every T1 = 10 iterations, Sec. 4.1)             */
    CAST_F_COUNT_FLIPS   = 1u << 1, /* add ||mask_t - mask_{t-1}||_0 (numerator of the flip rate r_t,
                                       App. C) to *flip_count; mask_{t-1} is read from `meta`          */
    CAST_F_META_BITMASK  = 1u << 2, /* bitmask-form metadata (required unless N:M == 2:4)              */
    CAST_F_V_KEPT_FROM_G = 1u << 3, /* alternate reading of Eq. 8: kept entries feed g^2 (textbook Adam)
                                       into v; entries outside the kept set still feed mu~^2           */
    CAST_F_EMIT_DENSE    = 1u << 4, /* emit Diag(A~) W~ for all entries (the dense training-time forward
                                       weight of Alg. 2) instead of the pruned product                  */
    CAST_F_GRAD_OF_SCALED = 1u << 6, /* `g` is the gradient with respect to the scaled weight Diag(A~) W~ that the
                                       forward pass used (Eq. 12) instead of the gradient with respect to W: the
                                       step applies the chain rule dL/dW = A (.) g itself and, where a scale_grad
                                       buffer is given, adds dL/dA[r, s] = sum_{c in segment s} g[r, c] W_{t-1}[r, c]
                                       to it.  Which A: the forward pass that produced g used the scale of the
                                       PREVIOUS emission; once the scale is trained (cast_scale_adam_step between
                                       the steps) that is no longer the `scale` buffer, which holds the updated
                                       A_t for this step's emission.  Give the previous one as `scale_chain` of the
                                       matrix (cast_plan_scale_adam_step maintains it); without it the factor is
                                       `scale` as it stands, i.e. exact while the scale is fixed and one scale
                                       update (relative size lr_A) off while it is trained                  */
    CAST_F_EMIT_COMPRESSED = 1u << 5, /* emit only the kept entries of the pruned product (Alg. 2, final loop):
                                       w_fwd_bf16 is then [rows][cols*N/M], the N kept values of each group in
                                       column order; with the metadata it is the whole pruned matrix, and a
                                       step writes 2 N/M instead of 2 bytes per parameter.  M <= 8 only; not
                                       together with CAST_F_EMIT_DENSE                                   */
    CAST_F_MASK_STATS    = 1u << 7, /* the step also adds the mask statistics the paper monitors (App. C) to a
                                       cast_mask_stats_t, from the registers it holds anyway: ||W_t (.) M_t||_1 and
                                       ||W_t||_1 on the UPDATED weights with this step's kept set M_t, and
                                       ||M_t - M_ref||_0 against the reference mask `meta_ref` of the matrix (the
                                       initial mask for the initial flip rate i_t; 0 is added where meta_ref is
                                       NULL).  Only cast_plan_step_stats takes this flag, on a plan created
                                       with it (other entry points answer CAST_ERR_PLAN)                  */
    CAST_F_BULK_STAGING  = 1u << 8, /* Two switches that choose how a step moves its data, not what it computes
                                       (results are identical bit for bit).  The plain access path is one thread =
                                       8 consecutive columns by 128-bit loads and stores.  The staged path moves
                                       each 1024-parameter tile with bulk asynchronous copies through shared
                                       memory; it is built for: 2:4 with any of CAST_F_RESELECT,
                                       CAST_F_COUNT_FLIPS, CAST_F_META_BITMASK, CAST_F_EMIT_DENSE (not dense and
                                       bitmask together) and with CAST_F_RESELECT | CAST_F_EMIT_COMPRESSED; groups
                                       of 4 or 8 under general N:M with CAST_F_RESELECT |
                                       CAST_F_META_BITMASK, with or without CAST_F_COUNT_FLIPS; 2:4 with
                                       CAST_F_EMIT_DENSE | CAST_F_MASK_STATS (plans).  On B200 it is as fast as
                                       the plain path in short runs and 0-3 % faster in sustained ones.
                                       Without either switch: a plan step (cast_plan_step) over at least
                                       16.8 M parameters takes the staged path where it is built, everything
                                       else the plain one.
                                       CAST_F_BULK_STAGING asks for the staged path (CAST_ERR_NM where it is not
                                       built), CAST_F_PLAIN_ACCESS for the plain one.  The staged path's one
                                       failure mode: its wait for a copy is bounded; a tile whose data has not
                                       arrived by then is left as it was, counted (cast_bulk_timeout_count), and a
                                       plan refuses its next step with CAST_ERR_STAGING                        */
    CAST_F_PLAIN_ACCESS  = 1u << 9
};

/*
 * Accumulator of the mask statistics of App. C (cast_mask_stats, cast_plan_mask_stats and the steps that carry
 * CAST_F_MASK_STATS add to it; the caller zeroes it):
 *
 *   mask_diff      += ||M - M_ref||_0   numerator of the flip rate r_t when M_ref is the previous mask, of the
 *                                       initial flip rate i_t when it is the initial mask (0 without a reference)
 *   kept_abs_sum   += ||W (.) M||_1     numerator of the sparse weight ratio S_t
 *   total_abs_sum  += ||W||_1           its denominator
 *
 * The denominators of r_t and i_t are the parameter counts, which the caller knows.  Sums are formed in fp64
 * (their last bits depend on the order in which CTAs add their parts).
 */
typedef struct cast_mask_stats {
    unsigned long long mask_diff;
    unsigned long long reserved_;     /* keeps the doubles 16-byte aligned; never written */
    double kept_abs_sum;
    double total_abs_sum;
} cast_mask_stats_t;

/*
 * cast_adams_step -- one AdamS iteration (Alg. 1 loop body, Eq. 6-8; Eq. 12 for the emitted weight)
 * over one matrix, asynchronous on `stream`.
 *
 *   w, m, v      device, fp32 [rows*cols], in/out: master weight, first moment (stored undecayed),
 *                second moment.
 *   g            device, bf16 [rows*cols], in: gradient of this iteration.
 *   w_fwd_bf16   device, bf16 [rows*cols] ([rows*cols*N/M] with CAST_F_EMIT_COMPRESSED), out: bf16(A[r, c / (cols/scale_groups)] * w_new[r, c]) where
 *                kept, +0.0 (0x0000) elsewhere (all entries with CAST_F_EMIT_DENSE).  Rounding is to
 *                nearest even of the fp32 product.
 *   meta         device, uint32 [rows*cols/32], in/out (layout above).  Read when CAST_F_RESELECT is
 *                absent or CAST_F_COUNT_FLIPS is set; written when CAST_F_RESELECT is set (a reused mask
 *                is left as it is).
 *   scale        device, fp32 [rows][scale_groups] (the matrix A of Eq. 12, n = scale_groups), or NULL
 *                for A = 1.  Requires scale_groups >= 1, cols % scale_groups == 0 and
 *                (cols/scale_groups) % max(M, 8) == 0.
 *   N, M         keep N of every M consecutive columns; the kept set is chosen on the weights before
 *                this update, larger magnitude first, lower column first among equal magnitudes.
 *   lr           finite.  beta1, beta2 in [0, 1).  eps > 0.  l1_coeff (lambda of Eq. 7) finite.
 *                Accuracy domain: the step is evaluated in fp32 (first-moment sums in fp64, approximate
 *                square root and reciprocal with a relative error below ~5e-7 on the update term).  Its
 *                results are within max(1e-6 relative, 1e-9 absolute) of an fp64 evaluation of Alg. 1 as
 *                long as the per-step update |lr mu^ / (sqrt(v^) + eps)| stays below ~1e-3 (with
 *                beta = 0.9/0.95 that is lr up to ~2e-4); for larger updates the error stays ~5e-7
 *                RELATIVE TO THE UPDATE, which then exceeds the 1e-9 absolute floor for weights near
 *                zero -- as it does for any fp32 evaluation, IEEE square root and division included.
 *   step         t >= 1;  total_steps  T >= t;  the decay weight is alpha_t = t/T.
 *   flags        OR of cast_flags.
 *   flip_count   device, one unsigned 64-bit counter the step ADDS to (the caller zeroes it); may be
 *                NULL unless CAST_F_COUNT_FLIPS is set.
 *
 * Errors: any violated rule above returns its status and launches nothing.
 */
CAST_API int cast_adams_step(float* w, float* m, float* v, const cast_bf16* g,
                    cast_bf16* w_fwd_bf16, uint32_t* meta,
                    const float* scale, int scale_groups,
                    int64_t rows, int64_t cols, int N, int M,
                    float lr, float beta1, float beta2, float eps, float l1_coeff,
                    int64_t step, int64_t total_steps,
                    uint32_t flags, unsigned long long* flip_count,
                    cast_stream_t stream);

/* One matrix of a multi-tensor plan (or of cast_adams_step_ex); fields as the arguments of cast_adams_step. */
typedef struct cast_tensor {
    float* w; float* m; float* v;
    const cast_bf16* g;
    cast_bf16* w_fwd;
    uint32_t* meta;
    const float* scale;      /* may be NULL */
    int32_t scale_groups;    /* ignored when scale is NULL */
    int64_t rows, cols;
    float* scale_grad;       /* device, fp32 [rows][scale_groups], ADDED to by steps that carry
                                CAST_F_GRAD_OF_SCALED (zero it before the step); may be NULL; needs `scale` */
    const uint32_t* meta_ref;/* device, uint32 [rows*cols/32], same form as `meta`: the reference mask of
                                CAST_F_MASK_STATS (never written); may be NULL                              */
    const float* scale_chain;/* device, fp32 [rows][scale_groups]: the scale the forward pass that produced `g` was
                                emitted with, where that is not `scale` any more (the scale is being trained and
                                has been updated since).  Read only by steps with CAST_F_GRAD_OF_SCALED, as the
                                factor of the chain rule dL/dW = A (.) g; `scale` still scales the emission.
                                NULL = use `scale`.  cast_plan_scale_adam_step keeps it up to date itself (it
                                stores each scale's value before the update there); needs `scale`              */
} cast_tensor_t;

/* Hyper-parameters of one iteration (Alg. 1 inputs); ranges as in cast_adams_step. */
typedef struct cast_hyper {
    float lr, beta1, beta2, eps, l1_coeff;
    int64_t step, total_steps;
    uint32_t flags;
} cast_hyper_t;

/*
 * cast_adams_step_ex -- cast_adams_step with the matrix and the hyper-parameters passed as structures, which
 * also carries the optional scale-gradient buffer of CAST_F_GRAD_OF_SCALED.  Same checks, same kernel.
 */
CAST_API int cast_adams_step_ex(const cast_tensor_t* tensor, int N, int M, const cast_hyper_t* hyper,
                       unsigned long long* flip_count, cast_stream_t stream);

/*
 * cast_scale_adam_step -- the optimizer step of the scale matrix A of Eq. 12, which the paper learns jointly
 * with the weights (Sec. 4.2) without naming its optimizer: plain Adam with bias correction (Alg. 1 without
 * its mask and decay lines), element-wise over `n` = rows * scale_groups entries, in fp64 internally.
 *
 *   a, m_a, v_a   device, fp32 [n], in/out: the scale entries and their two moments.
 *   grad          device, fp32 [n]: dL/dA as accumulated by steps with CAST_F_GRAD_OF_SCALED; set to zero
 *                 after use when clear_grad != 0 (ready for the next iteration's accumulation).
 *   lr finite; beta1, beta2 in [0, 1); eps > 0; step >= 1.
 * Asynchronous on `stream`; queue it after the AdamS steps of the iteration on the same stream.
 */
CAST_API int cast_scale_adam_step(float* a, float* m_a, float* v_a, float* grad, int64_t n,
                         float lr, float beta1, float beta2, float eps, int64_t step,
                         int clear_grad, cast_stream_t stream);

/*
 * cast_plan_scale_adam_step -- cast_scale_adam_step for the scale matrix of every matrix of a plan in one launch.
 * The scales and their gradients are the `scale` and `scale_grad` buffers the plan's descriptors name (every matrix
 * must have both; the scale buffers are UPDATED by this call although the descriptor declares them const for the
 * step); `m_a` and `v_a` are HOST arrays of n_tensors device pointers to the two moments of each scale matrix
 * (fp32 [rows * scale_groups]).  Where a matrix has a `scale_chain` buffer, the scale's value BEFORE this update is
 * stored there (the forward pass of the coming iteration was emitted with it, so it is the chain-rule factor of the
 * next step).  Other arguments as cast_scale_adam_step.
 */
CAST_API int cast_plan_scale_adam_step(void* plan, float* const* m_a, float* const* v_a,
                              float lr, float beta1, float beta2, float eps, int64_t step,
                              int clear_grad, cast_stream_t stream);

/*
 * Multi-tensor plan: the AdamS iteration of Alg. 1 over "each parameter theta in Theta", i.e. over
 * every prunable matrix of the model, in ONE kernel launch per 320 matrices.
 *
 * cast_plan_create  validates `n_tensors` descriptors (host array, copied) and returns an opaque handle
 *                   in *plan_out.  The plan is host memory only: it holds the launch tables, which travel
 *                   to the device as kernel parameters at every step, and allocates nothing on the
 *                   device (but see CAST_F_MASK_STATS under cast_plan_create_ex); it also holds one word of
 *                   page-locked host memory in which staged steps report a copy they gave up on.  All matrices share N:M.  The buffers named by the descriptors stay owned by
 *                   the caller and must outlive the plan's use.
 * cast_plan_step    launches one grid over all matrices on `stream` (ceil(n_tensors / 320) grids for
 *                   larger lists); arguments as cast_adams_step.  The plan may be stepped any number of
 *                   times, on any stream of its device; two steps of one plan must not overlap in time
 *                   (they update the same state).
 * cast_plan_destroy frees the handle (no device work).
 */
CAST_API int cast_plan_create(const cast_tensor_t* tensors, int n_tensors, int N, int M, void** plan_out);
/* As cast_plan_create, with plan_flags = OR of
 *   CAST_F_EMIT_COMPRESSED  the w_fwd buffers have the compressed size.  Every step of such a plan must carry that
 *                           flag, and a step of an ordinary plan must not (CAST_ERR_PLAN otherwise): the buffer
 *                           sizes are fixed when the plan is made;
 *   CAST_F_MASK_STATS       the plan may take steps with the statistics epilogue (cast_plan_step_stats); this is
 *                           the one case in which a plan allocates device memory (32 KB).
 * 0 = cast_plan_create. */
CAST_API int cast_plan_create_ex(const cast_tensor_t* tensors, int n_tensors, int N, int M, uint32_t plan_flags,
                        void** plan_out);
CAST_API int cast_plan_step(void* plan, const cast_hyper_t* hyper, unsigned long long* flip_count,
                   cast_stream_t stream);
/*
 * cast_plan_step_stats -- cast_plan_step that may carry CAST_F_MASK_STATS: the i_t and S_t sums of App. C come out
 * of the step itself (it holds |w_t|, the kept set and the stored metadata in registers), next to the flip count,
 * instead of a second pass over the weights (cast_plan_mask_stats, 4.25 B per parameter).
 *   stats   device, 8-byte aligned, ADDED to (the caller zeroes it); required with the flag, ignored without it.
 *           Values: see cast_mask_stats_t; W is the weight after this update, M the kept set of this step
 *           (selected now or reused), M_ref the `meta_ref` of each matrix as given when the plan was created.
 * The plan must have been created with CAST_F_MASK_STATS among its plan_flags (CAST_ERR_PLAN otherwise): such a
 * plan owns 32 KB of device memory (1024 partial accumulators that the step's CTAs add to, so that their atomics
 * do not queue on one address), allocated by cast_plan_create_ex and freed by cast_plan_destroy.  A step with the
 * flag launches one more, one-CTA kernel that folds the partial sums into `stats` and clears them.
 */
CAST_API int cast_plan_step_stats(void* plan, const cast_hyper_t* hyper, unsigned long long* flip_count,
                         cast_mask_stats_t* stats, cast_stream_t stream);
CAST_API int cast_plan_destroy(void* plan);
/* Fault injection on the host, for tests of a caller's error handling: marks the plan exactly as a staged kernel does
 * when it gives up waiting for a bulk copy (see CAST_F_BULK_STAGING).  Every later step of the plan answers
 * CAST_ERR_STAGING; the plan can still be destroyed.  Touches no device. */
CAST_API int cast_plan_report_staging_failure(void* plan);

/*
 * Host-resident optimizer state (the same iteration of Alg. 1, with w, m, v, g, w_fwd, meta and scale
 * in HOST memory): the matrix is cut into blocks of whole rows that are copied to device staging
 * buffers, updated by the same kernel and copied back, with copies and kernels of consecutive blocks
 * overlapped on the context's own streams.
 *
 * cast_host_ctx_create  allocates the staging buffers for blocks of up to `max_block_params`
 *                       parameters (a multiple of 32, >= 1024) in `n_slots` (2..8) slots on the current
 *                       device.  Device memory used: about 28.2 bytes * max_block_params * n_slots.
 * cast_host_step        arguments as cast_adams_step but every pointer is a HOST pointer (page-locked
 *                       memory makes the copies asynchronous; pageable memory works and is slower).
 *                       flip_count is a host counter that is added to.  The call returns when all work
 *                       is queued; results are valid after cast_host_ctx_sync.  A matrix whose rows are
 *                       longer than max_block_params is rejected with CAST_ERR_PLAN.  If a CUDA call fails
 *                       part-way (CAST_ERR_CUDA), the call first waits for every copy it has already queued
 *                       and then returns: nothing touches the host buffers afterwards, but they may hold a
 *                       partly updated state.
 * cast_host_ctx_sync    waits for everything queued through the context and folds the flip counts.
 * cast_host_ctx_destroy waits, then frees streams and buffers.
 */
CAST_API int cast_host_ctx_create(int64_t max_block_params, int n_slots, void** ctx_out);
CAST_API int cast_host_step(void* ctx,
                   float* w, float* m, float* v, const cast_bf16* g,
                   cast_bf16* w_fwd_bf16, uint32_t* meta,
                   const float* scale, int scale_groups,
                   int64_t rows, int64_t cols, int N, int M,
                   float lr, float beta1, float beta2, float eps, float l1_coeff,
                   int64_t step, int64_t total_steps,
                   uint32_t flags, unsigned long long* flip_count);
CAST_API int cast_host_ctx_sync(void* ctx);
CAST_API int cast_host_ctx_destroy(void* ctx);

/*
 * cast_kd_loss -- the training loss of Sec. 4.3 (Eq. 13) for every token, and its gradient:
 *
 *     loss[i] = eta * D_KL(P_t || P_s) + (1 - eta) * L_ce,   P_s = softmax(student row i), P_t = softmax(teacher row i),
 *               L_ce = -log P_s(labels[i])
 *     grad    = grad_scale * (P_s - eta P_t - (1 - eta) onehot(labels[i]))      (d loss[i] / d student row i)
 *
 *   student_logits, teacher_logits   device, bf16 [tokens][vocab].
 *   labels        device, int32 [tokens]; a negative label (or one >= vocab) means the token has no target: its
 *                 cross-entropy term and that term's gradient are left out (the paper does not treat padding).
 *   loss          device, fp32 [tokens], out.  The paper does not say how tokens are reduced; sum or average them.
 *   grad_logits   device, bf16 [tokens][vocab], out, or NULL for the loss alone.  grad_scale carries the
 *                 reduction (1/tokens for a mean) and any loss scaling.
 *   eta in [0, 1]; grad_scale finite.  Logits are expected to be finite.
 * Rows with vocab % 8 == 0 and 16-byte aligned buffers take the vector path; anything else a slower scalar path
 * with the same results.  Asynchronous on `stream`.
 */
CAST_API int cast_kd_loss(const cast_bf16* student_logits, const cast_bf16* teacher_logits, const int32_t* labels,
                 float* loss, cast_bf16* grad_logits, int64_t tokens, int64_t vocab,
                 float eta, float grad_scale, cast_stream_t stream);

/*
 * cast_prune_fold -- the final pruning of Alg. 2 (its last loop; the last lines of Alg. 1): W^ = W (.) M with the
 * scale of Eq. 12 folded into the weights, as bf16.  No optimizer state is read or written.
 *
 *   w        device, fp32 [rows*cols]: the trained weights.
 *   scale    device, fp32 [rows][scale_groups] or NULL (A = 1); shape rules as cast_adams_step.
 *   meta     device, uint32 [rows*cols/32], in/out: with CAST_F_RESELECT the mask is chosen now from |w| (Eq. 6,
 *            exactly N per group, ties to the lower column) and written; without it the stored mask is used
 *            (and rewritten unchanged).
 *   out      device, bf16 [rows*cols] (pruned slots +0.0), or with CAST_F_EMIT_COMPRESSED [rows*cols*N/M], the N
 *            kept values of each group in column order (M <= 8).  Values are bf16(A * w), round to nearest even.
 *   flags    OR of CAST_F_RESELECT, CAST_F_META_BITMASK (required unless N:M == 2:4), CAST_F_EMIT_COMPRESSED.
 * Asynchronous on `stream`.  Errors as cast_adams_step; nothing is launched on an error.
 */
CAST_API int cast_prune_fold(const float* w, const float* scale, int scale_groups, uint32_t* meta, cast_bf16* out,
                    int64_t rows, int64_t cols, int N, int M, uint32_t flags, cast_stream_t stream);

/*
 * cast_plan_prune_fold -- cast_prune_fold over every matrix of a plan in one launch (per 320 matrices): weights,
 * scales and metadata are the ones the plan's descriptors name; `out` is a HOST array of n_tensors device pointers,
 * one output buffer per matrix (sizes as in cast_prune_fold).  flags as cast_prune_fold.
 */
CAST_API int cast_plan_prune_fold(void* plan, cast_bf16* const* out, uint32_t flags, cast_stream_t stream);

/*
 * cast_mask_stats -- the mask statistics the paper monitors during training (App. C), for one matrix, as a pass of
 * its own over whatever (W, M, M_ref) the caller names (cast_mask_stats_t above says what is added).
 *
 *   w          device, fp32 [rows*cols]: the weights W.
 *   meta       device, uint32 [rows*cols/32]: the mask M in the metadata layout described at the top.
 *   meta_ref   device, same shape and form as meta, or NULL.
 *   M          group size (2, 4, 8, 16, 32); flags: CAST_F_META_BITMASK or 0 (index form, M == 4 only).
 *   stats      device, 8-byte aligned; the call ADDS to it (zero it before the first matrix of a model, then
 *              call once per matrix to get the model-wide sums of App. C).
 * Asynchronous on `stream`.  Errors as cast_adams_step; nothing is launched on an error.
 */
CAST_API int cast_mask_stats(const float* w, const uint32_t* meta, const uint32_t* meta_ref,
                    int64_t rows, int64_t cols, int M, uint32_t flags,
                    cast_mask_stats_t* stats, cast_stream_t stream);

/*
 * cast_plan_mask_stats -- cast_mask_stats over every matrix of a plan in one launch (per 320 matrices), with
 * the weights and masks the plan's descriptors name.  `meta_ref` is a HOST array of n_tensors device pointers
 * (the reference mask of each matrix, same shape and form as its mask), or NULL for no reference.  `flags`
 * is CAST_F_META_BITMASK or 0 and must name the form the plan's steps write.  `stats` as in cast_mask_stats.
 */
CAST_API int cast_plan_mask_stats(void* plan, const uint32_t* const* meta_ref, uint32_t flags,
                         cast_mask_stats_t* stats, cast_stream_t stream);

/*
 * cast_host_step_static -- cast_host_step for callers that must not allocate device memory.
 * (The paper has no counterpart to this entry point: it is a packaging variant of the call above.)
 *
 * cast_host_ctx_create reserves its staging slots with cudaMalloc.  A caller whose framework allocator
 * already owns all device memory, that cannot afford the device-wide synchronisation an allocation or a
 * free implies, or that may not grow its device footprint after start-up, uses this call instead: the
 * staging area is a fixed array inside the library image (about 16.6 MiB, held by every GPU on which the
 * process uses the library, until the process exits), and the call allocates and frees nothing, on the
 * device or through any other library.
 *
 *   When the memory is taken: the CUDA runtime loads device code lazily by default, so the image that holds the
 *   staging area is placed in device memory by the FIRST call on each device, not when the library is opened.
 *   That first call needs about 16.6 MiB of free device memory (it fails with CAST_ERR_CUDA otherwise) and may
 *   synchronise the device.  Make it once per device at start-up -- any small matrix will do -- before the
 *   framework's allocator takes the memory and outside any stream capture; or run the process with
 *   CUDA_MODULE_LOADING=EAGER, which moves the loading to context creation.  Later calls leave the amount of
 *   free device memory exactly as they find it.
 *
 *   Arguments as cast_host_step (every data pointer is a HOST pointer; flip_count is a host counter that
 *   is added to), plus `stream`, on which the copies and the kernel are queued.
 *   Limit: rows * cols <= CAST_STATIC_MAX_PARAMS; a larger matrix is refused with CAST_ERR_PLAN (the
 *   staging area is too small) and nothing is queued.  Cut larger matrices into blocks of whole rows.
 *   The call is synchronous: it returns after `stream` has finished the step, with the results in the
 *   host buffers.  This also holds when a CUDA call fails part-way (CAST_ERR_CUDA): the stream is drained
 *   before the error is returned, and the host buffers may then hold a partly updated state.
 *   The first call on each device looks up the device address of the staging area (with that device
 *   current); make that first call outside any stream capture.
 *   All calls of a process on one device share the one staging area, which keeps the contents the
 *   previous call left (the call clears the only part that must start at zero, its flip counter).
 *   Two calls that overlap in time on the same device -- from two host threads, on the same or different
 *   streams -- race on it and corrupt each other's results: serialise them.
 */
#define CAST_STATIC_MAX_PARAMS 1048576
CAST_API int cast_host_step_static(float* w, float* m, float* v, const cast_bf16* g,
                   cast_bf16* w_fwd_bf16, uint32_t* meta,
                   const float* scale, int scale_groups,
                   int64_t rows, int64_t cols, int N, int M,
                   float lr, float beta1, float beta2, float eps, float l1_coeff,
                   int64_t step, int64_t total_steps,
                   uint32_t flags, unsigned long long* flip_count,
                   cast_stream_t stream);

/*
 * Measurement aids.  Neither computes anything of the method (the paper has no counterpart); a benchmark puts their
 * times beside a measured step.
 *
 * cast_probe_launch   launches an empty grid of n_ctas CTAs of 128 threads on `stream`: the cost of launching and
 *                     draining as many CTAs as a step over 1024 * n_ctas parameters has.
 * cast_probe_stream   performs the loads and stores of one AdamS step over n_params parameters (device buffers
 *                     sized as in cast_adams_step, n_params % 32 == 0, < 2^31) in the step's own launch shape and
 *                     access pattern, with no arithmetic between them: w, m, v come back with their signs flipped,
 *                     w_fwd receives the gradient's bits, meta is overwritten.  Its rate is the ceiling of a
 *                     28.125-byte-per-parameter step of this shape on the device at hand.
 */
CAST_API int cast_probe_launch(int64_t n_ctas, cast_stream_t stream);
CAST_API int cast_probe_stream(float* w, float* m, float* v, const cast_bf16* g, cast_bf16* w_fwd, uint32_t* meta,
                      int64_t n_params, cast_stream_t stream);

/* Steps with CAST_F_BULK_STAGING wait for their bulk copies with a bounded number of polls; a tile whose data
 * has not arrived by then is not updated and is counted.  *count_out receives that count over the life of the
 * process on the current device (0 in every healthy run).  Synchronises the device. */
CAST_API int cast_bulk_timeout_count(unsigned long long* count_out);

/* Static description of a status code (never NULL). */
CAST_API const char* cast_strerror(int status);

/* The cudaError_t behind the last CAST_ERR_CUDA returned on the calling thread (0 if none). */
CAST_API int cast_last_cuda_error(void);

/* Number of kernels this library has launched in the calling process (for launch accounting). */
CAST_API unsigned long long cast_kernel_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* CAST_ADAMS_H */
