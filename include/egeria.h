/*
 * egeria.h -- C ABI of the B200 (sm_100a) plasticity-evaluation library.
 *
 * The library evaluates the "training plasticity" of every monitored layer
 * module of a network (Egeria, Sec. 4.2.1, Eq. 1) and turns each module's
 * plasticity history into the freezing decision of Sec. 4.2.2 / Algorithm 1.
 *
 * Notation (the paper's): b = mini-batch size; module l has training and
 * reference activations A_T^(l), A_R^(l), flattened per sample to b x d_l;
 * P_i^(l) = plasticity at evaluation i; W = window (moving-average span, fit
 * window and number of consecutive low-slope evaluations); T = slope tolerance.
 *
 * Conventions for every call
 *   - "device" pointers are CUDA device memory owned by the caller; "host"
 *     pointers are ordinary host memory.  The library allocates no device
 *     memory: all scratch lives in the caller's workspace (see
 *     egeria_workspace_bytes).  (A context also holds a few KB of pinned host
 *     memory unless EGERIA_FLAG_EQUAL_SPLIT is given.)
 *   - cuda_stream is a cudaStream_t passed as void* (NULL = default stream).
 *     Calls enqueue work on it and return without synchronising, unless the
 *     call's comment says otherwise.
 *   - Activations are bfloat16, row-major [b, d_l] (sample-major), contiguous.
 *   - Errors are returned as egeria_status; nothing throws or aborts.  There is
 *     no CPU fallback: without an sm_100 device the compute calls fail with
 *     EGERIA_ERR_UNSUPPORTED_DEVICE or EGERIA_ERR_CUDA.
 *   - One context per stream; a context is not thread-safe.
 *   - A call on a context passes the kernel state that belongs to that call (which of two sets of
 *     progress counters and of partial slots to use, the serial number of the rule evaluation),
 *     and may enqueue small copies (a new work plan, the launch log of the adaptive split):
 *     enqueue every evaluation of a context through the library; replaying one from a
 *     captured CUDA graph would reuse that state and give wrong results.  The evaluation calls
 *     (egeria_sp_loss_batch, egeria_plasticity_evaluate and their _subset and _host forms)
 *     therefore return EGERIA_ERR_INVALID_ARG on a stream that is being captured, and record
 *     nothing.
 */
#ifndef EGERIA_H_
#define EGERIA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct egeria_ctx egeria_ctx; /* opaque, library-owned host object */

typedef enum {
    EGERIA_OK = 0,
    EGERIA_ERR_INVALID_ARG = 1,        /* NULL pointer, M < 1, b out of range, W < 1, ... */
    EGERIA_ERR_UNSUPPORTED_SHAPE = 2,  /* d_l < 1, b > 256, ... */
    EGERIA_ERR_UNSUPPORTED_DEVICE = 3, /* current device is not compute capability 10.x */
    EGERIA_ERR_WORKSPACE = 4,          /* workspace NULL, misaligned or too small */
    EGERIA_ERR_CUDA = 5,               /* a CUDA runtime/driver call failed */
    EGERIA_ERR_TIMEOUT = 6,            /* a bounded device-side wait ran out (see egeria_device_status) */
    EGERIA_ERR_CHECK = 7               /* checked build only: an index check inside a kernel failed (egeria_debug_check_record) */
} egeria_status;

enum {
    /* Use the literal test of Algorithm 1, slope < T, instead of |slope| < T. */
    EGERIA_FLAG_SIGNED_SLOPE = 1u,
    /* Compute every Gram matrix with the CUDA-core kernel (plain loads, FMA)
     * instead of the TMA + tcgen05 kernel.  Same results up to summation order. */
    EGERIA_FLAG_FORCE_SIMT = 2u,
    /* Keep the two row-normalised similarity matrices of every module in the
     * workspace so that egeria_debug_dump_gram can return them. */
    EGERIA_FLAG_KEEP_GRAMS = 4u,
    /* Reserve device staging for egeria_sp_loss_batch_host in the workspace. */
    EGERIA_FLAG_HOST_STAGING = 8u,
    /* Record a CUDA event before and after the evaluation kernel(s) of every
     * egeria_sp_loss_batch / egeria_plasticity_evaluate call, for
     * egeria_gram_kernel_time. */
    EGERIA_FLAG_TIME_GRAM = 16u,
    /* Always cut the work into equal shares.  Without this flag the first
     * evaluations of a context that keep every SM busy report how fast each
     * thread block streamed, and the shares then follow those rates (the SMs of
     * a B200 do not all get the same share of HBM bandwidth, and the placement of
     * thread blocks on SMs repeats from launch to launch): three evaluations are
     * measured, the shares are set, and this is repeated twice under the new
     * shares; three more evaluations under the final shares then decide whether
     * they stay (only if the slowest thread block streams at least 1 % faster than
     * under equal shares; else the split goes back to equal ones).  After the
     * twelfth such evaluation nothing changes any more.  The shares decide
     * how the fp32 partial sums are grouped, so with the adaptive split the
     * low-order bits of a loss can differ between evaluations across a change of
     * shares and from run to run; with this flag every evaluation of the same
     * inputs gives the same bits. */
    EGERIA_FLAG_EQUAL_SPLIT = 32u,
    /* Per-module tolerance [Sec. 4.2.2, "Hyperparameters guideline"]: T of a
     * module is 20 % of the largest |slope| in its initial 3 readings (a slope
     * exists from the 2nd reading on, so these are evaluations 1 and 2).  The T
     * given at creation is ignored; evaluations 0..2 of a module only set its
     * tolerance and are never stale. */
    EGERIA_FLAG_AUTO_T = 64u,
    /* Frontmost-active policy [Sec. 4.2.2: only the frontmost module that is
     * still active is monitored, so that the frozen modules always form a prefix;
     * Algorithm 1: freeze, then l <- l + 1].  Modules are ordered front to back.  Only module l = (number
     * of frozen modules) is advanced by an evaluation; when its counter reaches
     * W it is frozen, and the NEXT evaluation starts module l + 1 from a cleared
     * state.  out_mask is then a prefix mask (1 for the frozen modules) and
     * out_slopes holds this evaluation's slope for the monitored module, the
     * final slope of every frozen one and +inf for those not monitored yet. */
    EGERIA_FLAG_FRONTMOST = 128u,
    /* With EGERIA_FLAG_FRONTMOST: egeria_plasticity_evaluate computes the loss of the monitored
     * module ONLY [Sec. 3: only the activation of the frontmost module that is not frozen is
     * collected; Algorithm 1 is called with that one module].  Which module that is, is decided
     * on the device when the kernel starts (it reads the front the previous evaluation left), so
     * the caller never reads anything back: the work split of every possible front is kept on
     * the device, each spreading its one module over the whole GPU, and an evaluation costs
     * about that module's share of a full one.  Only out_losses[front] is written; out_mask
     * and out_slopes are reported as under EGERIA_FLAG_FRONTMOST.  The pointers of ALL modules
     * must still be valid (any of them may be the front), and every module must qualify for
     * the TMA + tcgen05 kernel (d_l a multiple of 8, 16-byte aligned pointers), else
     * EGERIA_ERR_UNSUPPORTED_SHAPE.  Once every module is frozen an evaluation does no work
     * beyond reporting the mask.  egeria_sp_loss_batch and the subset calls are not affected
     * (the subset form of the evaluation is refused: EGERIA_ERR_INVALID_ARG). */
    EGERIA_FLAG_FRONT_ONLY = 256u,
    /* Let consecutive evaluations of this context overlap on the GPU.  Every evaluation kernel
     * is launched as a programmatic dependent of the kernel before it in the stream: its thread
     * blocks set themselves up while that kernel's last blocks are still running, and then WAIT
     * for that kernel to have ended before they read an activation or touch the workspace.
     * With this flag the wait before the first read of the activations is left out: a thread
     * block of the next evaluation starts streaming on an SM as soon as the previous
     * evaluation's block there has ended, while other blocks of the previous evaluation are
     * still finishing their modules; everything the evaluations share (workspace, outputs, the
     * rule's state) is still touched only after the previous evaluation has ended entirely, so
     * results are the same.  THE CALLER PROMISES, by setting this flag, that the activations
     * passed to an evaluation are not written by the KERNEL that precedes that evaluation in
     * the stream (they were complete before it; e.g. several mini-batches' activations
     * collected first and evaluated one after the other).  (Copies are not kernels: an
     * evaluation still waits for a copy enqueued before it.)  Has no effect under
     * EGERIA_FLAG_TIME_GRAM (the timing events keep the kernels apart). */
    EGERIA_FLAG_OVERLAP = 512u
};

#define EGERIA_MAX_B 256          /* largest supported mini-batch size */
#define EGERIA_WORKSPACE_ALIGN 1024

/* Bytes of device workspace a context with these parameters needs.  Pure host
 * arithmetic (no CUDA call).  Returns 0 for invalid arguments.
 *   M      number of monitored modules (>= 1)
 *   d      host array [M], flattened per-sample size of each module (>= 1)
 *   b_max  largest b any call will pass (2..EGERIA_MAX_B)
 *   W      window (>= 1)
 *   flags  EGERIA_FLAG_* (KEEP_GRAMS and HOST_STAGING enlarge the workspace) */
size_t egeria_workspace_bytes(int M, const int64_t *d, int b_max, int W, uint32_t flags);

/* Create a context for M modules [inputs of Algorithm 1: W, T; module shapes].
 *   out        receives the context
 *   T          host array [M] of per-module tolerances, or NULL to use T_all
 *   workspace  device memory, EGERIA_WORKSPACE_ALIGN-aligned, caller-owned, at
 *              least egeria_workspace_bytes(...) long; must outlive the context
 * Clears the plasticity state (as egeria_plasticity_reset) synchronously on the
 * current device.  W = 1 is accepted but can never converge (no line through
 * one point). */
egeria_status egeria_plasticity_create(egeria_ctx **out, int M, const int64_t *d, int b_max,
                                       int W, const float *T, float T_all, void *workspace,
                                       size_t workspace_bytes, uint32_t flags);

/* Free the host object.  The workspace stays the caller's. */
egeria_status egeria_plasticity_destroy(egeria_ctx *ctx);

/* Plasticity of every module for one mini-batch [Sec. 4.2.1, Eq. 1]:
 *   G = A A^T (b x b, fp32 accumulation of bf16 products) for A_T and A_R,
 *   every row of G scaled to unit L2 norm (norms below 1e-12 are clamped, so an
 *   all-zero sample gives a zero row), P = ||G~_T - G~_R||_F^2 / b^2.
 *   At, Ar      host arrays [M] of device pointers, bf16 [b, d_l] each
 *   b           2..b_max
 *   d           host array [M]; must equal the d given at creation
 *   out_losses  device float [M]
 * Modules whose d_l is a multiple of 8 and whose pointers are 16-byte aligned
 * take the TMA + tcgen05 kernel; others take the CUDA-core kernel.
 * NaN/Inf in the inputs propagate to the loss. */
egeria_status egeria_sp_loss_batch(egeria_ctx *ctx, void *cuda_stream, const void *const *At,
                                   const void *const *Ar, int b, const int64_t *d,
                                   float *out_losses);

/* Same evaluation from HOST activations: copies every A_T, A_R to the staging
 * area of the workspace (needs EGERIA_FLAG_HOST_STAGING), evaluates, copies the
 * M losses back to out_losses_host and synchronises the stream before returning.
 *   At_host, Ar_host  host arrays [M] of host pointers (pinned memory copies
 *                     fastest), bf16 [b, d_l]
 *   out_losses_host   host float [M] */
egeria_status egeria_sp_loss_batch_host(egeria_ctx *ctx, void *cuda_stream,
                                        const void *const *At_host, const void *const *Ar_host,
                                        int b, const int64_t *d, float *out_losses_host);

/* One evaluation of the freezing rule for every module [Sec. 4.2.2, Eq. 2,
 * Algorithm 1]: append the new reading, smooth (mean of the last min(i+1, W)
 * readings), append to the module's list, fit a least-squares line to the last
 * min(len, W) smoothed values against 0,1,2,..., compare the slope with T
 * (|s| < T, strict; fewer than two points or NaN is "not stale"), update the
 * consecutive-stale counter; a module is converged once its counter reaches W
 * and its state then stops advancing.  All arithmetic is float64.
 *   losses      device float [M], e.g. the out_losses of egeria_sp_loss_batch
 *   out_slopes  device double [M] (slope of this evaluation; the last one for a
 *               module that had already converged), may be NULL
 *   out_mask    device uint8 [M], 1 = converged (freeze), may be NULL */
egeria_status egeria_plasticity_step(egeria_ctx *ctx, void *cuda_stream, const float *losses,
                                     double *out_slopes, uint8_t *out_mask);

/* One whole evaluation in one call: egeria_sp_loss_batch followed by
 * egeria_plasticity_step on the losses just computed [Algorithm 1,
 * checkPlasticity: calculateSPLoss, smoothPlasticity, windowLinearFit, counter].
 * The freezing rule of a module is advanced by the thread block that finishes
 * the module's loss, so no extra kernel is launched.  Arguments as in the two
 * calls; out_slopes and out_mask may be NULL.  Results are identical to the two
 * separate calls. */
egeria_status egeria_plasticity_evaluate(egeria_ctx *ctx, void *cuda_stream, const void *const *At,
                                         const void *const *Ar, int b, const int64_t *d,
                                         float *out_losses, double *out_slopes, uint8_t *out_mask);

/* The two calls above for a SUBSET of the modules: active is a host uint8 [M];
 * modules with active[m] == 0 are left out -- their pointers are not read (may be
 * NULL), no work is done for them, their entries of out_losses, out_slopes and
 * out_mask are not written and their freezing rule does not advance.  The work of
 * the active modules is spread over the whole GPU, so evaluating one module of
 * many costs about its share.  This is how the frontmost-active policy is meant
 * to be used [Sec. 3: only the activation of the frontmost module that is not
 * frozen is collected]: read out_mask back now and then and pass only the frontmost
 * module that is not frozen (under EGERIA_FLAG_FRONTMOST that module reports the
 * prefix mask and the slopes of all modules; if it is left out, or all modules
 * are frozen, nothing is reported).  At least one module must be active. */
egeria_status egeria_sp_loss_subset(egeria_ctx *ctx, void *cuda_stream, const void *const *At,
                                    const void *const *Ar, int b, const int64_t *d,
                                    const uint8_t *active, float *out_losses);
egeria_status egeria_plasticity_evaluate_subset(egeria_ctx *ctx, void *cuda_stream,
                                                const void *const *At, const void *const *Ar, int b,
                                                const int64_t *d, const uint8_t *active,
                                                float *out_losses, double *out_slopes,
                                                uint8_t *out_mask);

/* The same rule over whole histories, from a cleared state that is private to
 * the call (the context's step state is not touched; the window is the one in force).
 *   hist             device float [M, H] row-major raw readings
 *   out_slopes       device double [M, H]; NaN after a module converged; may be NULL
 *   out_mask         device uint8 [M]
 *   out_freeze_eval  device int32 [M]: evaluation index at which the counter
 *                    reached W, -1 if never; may be NULL */
egeria_status egeria_plasticity_replay(egeria_ctx *ctx, void *cuda_stream, const float *hist,
                                       int H, double *out_slopes, uint8_t *out_mask,
                                       int32_t *out_freeze_eval);

/* Clear the step state (histories, counters, masks, the front, the reference
 * learning rate) by hand, e.g. for an unfreezing criterion of the caller's own
 * [Sec. 4.2.2 "Unfreezing": cyclical schedules are left to the user; Algorithm 1
 * customizedUnfreeze].  If halve_W is non-zero the window in force is halved,
 * W <- max(2, floor(W / 2)), as the paper does for refreezing. */
egeria_status egeria_plasticity_reset(egeria_ctx *ctx, void *cuda_stream, int halve_W);

/* Unfreezing on learning-rate annealing [Sec. 4.2.2 "Unfreezing"; Algorithm 1, the
 * branch after the freeze step: unfreezeAllLayers, l <- l_0].  Tell the context the
 * learning rate in force for the evaluations that follow (host value; no CUDA work).
 * From then on every evaluation of the rule (egeria_plasticity_step,
 * egeria_plasticity_evaluate and their subset forms) is followed by the paper's
 * test, all of it on the device:
 *   - the rate in force at the first freeze after the start or the last restart is
 *     remembered (with EGERIA_FLAG_FRONTMOST that is the first module's freeze);
 *   - once lr <= that rate / 10 * (1 + 1e-6) -- a drop by a factor of ten or more;
 *     the slack lets a step decay by exactly 10x count when it was computed in
 *     single precision -- every module starts afresh (histories, counters, automatic
 *     tolerances), the front goes back to module 0, the window in force is halved,
 *     W <- max(2, floor(W / 2)), the remembered rate is forgotten, and the out_mask
 *     of that evaluation is cleared.  The reading of that evaluation has been
 *     consumed by the old state; the next evaluation is the first of the new run.
 * A rate that is not positive (or NaN, the state after creation) switches the rule
 * off: it is neither remembered nor tested.  The test costs one extra small kernel
 * launch, and only after the first evaluation under a changed rate. */
egeria_status egeria_plasticity_set_lr(egeria_ctx *ctx, double lr);

/* How often the unfreezing rule has restarted the modules of this context.
 * Waits for the stream of the last call and reads the count from the device;
 * -1 if that fails, 0 for a NULL context. */
int egeria_plasticity_restarts(const egeria_ctx *ctx);

/* Algorithm 1 WITH its learning-rate-based unfreezing over whole histories, from a
 * cleared state private to the call (starting with the context's window in force).
 *   hist            device float [M, H] row-major raw readings
 *   lr              device double [H]: learning rate at each evaluation; NULL = no
 *                   unfreezing (then this is egeria_plasticity_replay with more outputs)
 *   out_slopes      device double [M, H]; NaN where the module was not advanced; may be NULL
 *   out_frozen      device uint8 [H, M]: 1 where module m is frozen after evaluation i
 *                   (after the unfreezing test); may be NULL
 *   out_window      device int32 [H]: window in force during evaluation i; may be NULL
 *   out_restarted   device uint8 [H]: 1 if the unfreezing fired at the end of evaluation i; may be NULL
 *   out_mask        device uint8 [M]: frozen at the end of the history; may be NULL
 *   out_freeze_eval device int32 [M]: evaluation of the module's freeze in the last run, -1 if
 *                   it is not frozen at the end; may be NULL
 * One thread block runs all modules (a restart couples them).  More than 1280 modules
 * give EGERIA_ERR_UNSUPPORTED_SHAPE. */
egeria_status egeria_plasticity_replay_lr(egeria_ctx *ctx, void *cuda_stream, const float *hist,
                                          const double *lr, int H, double *out_slopes,
                                          uint8_t *out_frozen, int32_t *out_window,
                                          uint8_t *out_restarted, uint8_t *out_mask,
                                          int32_t *out_freeze_eval);

/* End of the bootstrapping stage [Sec. 3 "Bootstrapping stage": the changing rate
 * of the training loss is monitored in line with the plasticity; Sec. 4.2.2: the
 * changing rate that ends the stage is 10 %].  The training-loss readings are
 * smoothed (Eq. 2) and fitted like a plasticity series, with the window W given
 * at creation (>= 2); with a full window of W smoothed values, slope s and window
 * mean ybar, the changing rate is |s| (W - 1) / |ybar| -- the relative change of
 * the fitted line across the window -- and the stage ends at the first evaluation
 * whose rate is below rate_tol (the paper's value: 0.1).  The state is separate
 * from the modules' and is not touched by egeria_plasticity_reset.
 *   train_loss  device float [1]: the new reading
 *   out_rate    device double [1]: rate of this evaluation, NaN while the window
 *               is not full and once the stage has ended; may be NULL
 *   out_done    device uint8 [1]: 1 once the stage has ended; may be NULL */
egeria_status egeria_bootstrap_step(egeria_ctx *ctx, void *cuda_stream, const float *train_loss,
                                    float rate_tol, double *out_rate, uint8_t *out_done);

/* The same over a whole history, from a cleared state private to the call.
 *   loss_hist  device float [H]     out_rates  device double [H], may be NULL
 *   out_end    device int32 [1]: evaluation at which the stage ended, -1 if not */
egeria_status egeria_bootstrap_replay(egeria_ctx *ctx, void *cuda_stream, const float *loss_hist,
                                      int H, float rate_tol, double *out_rates, int32_t *out_end);

/* Start the bootstrapping detector of the context afresh. */
egeria_status egeria_bootstrap_reset(egeria_ctx *ctx, void *cuda_stream);

/* Checkpointing of the freezing-rule state (windows, counters, tolerances, the
 * front, the bootstrapping detector; not the work split).  export copies it,
 * with a small header, to a HOST buffer of at least
 * egeria_plasticity_state_bytes() bytes and synchronises the stream; import
 * restores it into a context created with the same M, W and rule flags (else
 * EGERIA_ERR_INVALID_ARG) and synchronises the stream.  A too small buffer gives
 * EGERIA_ERR_WORKSPACE.  The paper has no counterpart: it is what a training job
 * that checkpoints needs to resume with the same freezing decisions. */
size_t egeria_plasticity_state_bytes(const egeria_ctx *ctx);
egeria_status egeria_plasticity_export(egeria_ctx *ctx, void *cuda_stream, void *host_buffer,
                                       size_t buffer_bytes);
egeria_status egeria_plasticity_import(egeria_ctx *ctx, void *cuda_stream, const void *host_buffer,
                                       size_t buffer_bytes);

/* Window in force (halved by egeria_plasticity_reset and by the unfreezing rule).
 * It lives on the device: waits for the stream of the last call and reads it;
 * -1 if that fails, 0 for a NULL context. */
int egeria_plasticity_window(const egeria_ctx *ctx);

/* The per-thread-block shares of the adaptive split (see EGERIA_FLAG_EQUAL_SPLIT).
 * Copies up to max_weights of them to out_weights (host, may be NULL; 1.0 = the
 * equal share) and returns how many thread blocks the split is over once rates have
 * been measured (the shares are all 1.0 again if the measurement found them no better
 * than equal ones), 0 while nothing has been measured (or with EGERIA_FLAG_EQUAL_SPLIT),
 * -1 for a NULL context.  Never waits for the device. */
int egeria_split_weights(egeria_ctx *ctx, float *out_weights, int max_weights);

/* Test hook: copy the row-normalised similarity matrices of one module, as
 * left by the last egeria_sp_loss_batch, to device float [b, b] buffers.
 * Needs EGERIA_FLAG_KEEP_GRAMS. */
egeria_status egeria_debug_dump_gram(egeria_ctx *ctx, void *cuda_stream, int module,
                                     float *Gt_norm, float *Gr_norm);

/* Test hook: the static work split of one evaluation, pure host arithmetic.
 * Writes up to max_units rows {module, side (0 = T, 1 = R, 2 = both), first
 * 64-element block, number of blocks, CTA} to out_units and the unit count to
 * n_units.  n_ctas is the number of persistent CTAs to split over. */
egeria_status egeria_debug_plan(int M, const int64_t *d, int b, int n_ctas, int32_t *out_units,
                                int max_units, int *n_units);

/* Test hook: the same with one weight per CTA (host float [n_ctas], positive;
 * NULL = equal shares): CTA c's share of the blocks is weights[c] / sum. */
egeria_status egeria_debug_plan_weighted(int M, const int64_t *d, int b, int n_ctas,
                                         const float *weights, int32_t *out_units, int max_units,
                                         int *n_units);

/* 1 if this library was compiled with -DEGERIA_CHECKED (the build script makes such a second
 * library, libegeria_checked.so), else 0.  In a checked build the kernels compare every index
 * they take from a table in memory (unit table, slot ranges, first tasks, cursors) and every
 * offset into a partial slot, a warp's staging area, the chunk-sum scratch or tensor memory
 * with its bound before using it; a failed check records what it saw (the first failure
 * wins), makes the kernel skip that access -- nothing traps -- and egeria_device_status then
 * returns EGERIA_ERR_CHECK once.  It stands in for the memory-checking tools where those cannot
 * be run, and costs a few per cent.  The paper has no counterpart. */
int egeria_build_is_checked(void);

/* Test hook: the record of the first failed check since the last egeria_device_status that
 * reported one (host int32 [5]: which check -- 1 unit range, 2 unit, 3 tensor-memory columns,
 * 4 slot store, 5 first task, 6 task, 7 fetch, 8 chunk sum, 9 stage, 10 emptied range --, the
 * offending value's low and high words, thread block, thread); all zero if none.  Waits for
 * the stream of the last call and clears the record. */
egeria_status egeria_debug_check_record(egeria_ctx *ctx, int32_t *out_record);

/* Test hook: the help planned for the end of a launch, pure host arithmetic.  The rows of a
 * module are finished by the warps of the thread blocks that worked on it, so a module that got
 * few blocks has many rows per warp; some warps of the blocks of the well-off modules are told to
 * start with such a module's rows instead.  Writes, for every CTA c < n_ctas, out_help[2 c] = the
 * module it lends warps to (-1: none) and out_help[2 c + 1] = how many of its twelve epilogue
 * warps. */
egeria_status egeria_debug_plan_help(int M, const int64_t *d, int b, int n_ctas, int32_t *out_help);

/* Test hook: how the end of a launch is cut into tasks and who starts with which, pure host
 * arithmetic for the split egeria_debug_plan returns (only_module >= 0: that module evaluated
 * alone, as in a front-only evaluation).  A task is a row of G, or, for a module evaluated alone
 * at b <= 64 and cut into more partials than one pass of a warp's staging area holds, a (row,
 * chunk) pair.  Writes
 *   out_first[c * 12 + w]  the task epilogue warp w of CTA c starts with, (module << 16) | task,
 *                          or -1 (host int32 [n_ctas * 12]);
 *   out_tasks[2 m], out_tasks[2 m + 1]  module m's tasks and how many of them have a warp of their
 *                          own from the start; the module's cursor hands out the rest (host int32 [2 M]);
 *   *out_validate          1 if the kernel would tell an arrived partial row by its contents (every
 *                          task has its own warp and fits one pass), 0 if by the unit counters. */
egeria_status egeria_debug_plan_tasks(int M, const int64_t *d, int b, int n_ctas, int only_module,
                                      int32_t *out_first, int32_t *out_tasks, int *out_validate);

/* Test hook for the bounded waits: the NEXT evaluation kernel of this context (tensor-core
 * modules) runs with every wait limited to one millisecond instead of two seconds, and with one
 * hand-shake of its first thread block left out on purpose, so that the waits that depend on it
 * run out: kind 1 = that block's loader issues no load; kind 2 = its MMA issuer stops after its
 * first pipeline stage; 0 = cancel.  The block then leaves through the give-up path (waits for
 * its loads in flight, frees its tensor memory), the kernel returns, the losses of that
 * evaluation are not written and egeria_device_status reports EGERIA_ERR_TIMEOUT once; the
 * evaluation after that is an ordinary one.  Nothing traps or spins without bound.  Not for
 * production use. */
egeria_status egeria_debug_stall_next(egeria_ctx *ctx, int kind);

/* Synchronise the stream of the last call and report the device status word:
 * EGERIA_OK, or EGERIA_ERR_TIMEOUT if a bounded wait inside a kernel ran out
 * (the kernel then skipped its remaining work; results are invalid). */
egeria_status egeria_device_status(egeria_ctx *ctx);

/* Plasticity of ONE module with no workspace and no allocation of any kind.
 * The paper has no counterpart to this call; it exists for callers that cannot
 * obtain device memory at the moment they need an evaluation: code that runs
 * where cudaMalloc is forbidden or fails (a framework whose caching allocator
 * owns all of HBM so that a raw allocation fails, a plugin that is handed a
 * stream but no allocator, code that must not take the device-wide
 * synchronisation an allocation or free implies).  Such callers cannot size and
 * allocate the workspace a context needs either.
 *
 * The scratch of this call (partial Gram matrices, work split, tensor maps) is
 * a fixed 6 MiB array inside the library image; every GPU that loads the
 * library holds it until the process exits.  The price is a size limit:
 *   b  2..128 (larger b returns EGERIA_ERR_UNSUPPORTED_SHAPE), any d >= 1,
 * and the feature axis is split over 32 CTAs only, so it is slower than a
 * context on large d; each call also builds its work split and tensor maps on
 * the host and sends them with one small copy (a context keeps them on the
 * device).  Same arithmetic as egeria_sp_loss_batch.
 *   At, Ar    device bf16 [b, d] (caller-owned)     out_loss  device float [1]
 * The first call on each device looks up the array's device address and sets
 * kernel attributes (with that device current).  No call of this entry point
 * may be recorded into a CUDA graph: every call copies from host memory that
 * is gone when it returns, so a call on a capturing stream is refused with
 * EGERIA_ERR_INVALID_ARG (that goes for the first call and for all later ones).
 * All calls share the one array, which keeps the previous call's contents (the
 * call clears the words that must start at zero): two calls that overlap on
 * the GPU, from different streams or threads, race.  Calls on one stream are
 * safe back to back.  Not thread-safe.
 * If a bounded wait inside the kernel runs out, the kernel gives up and
 * out_loss is left NaN; egeria_sp_loss_static_status tells that case from a
 * NaN that came from the inputs. */
egeria_status egeria_sp_loss_static(void *cuda_stream, const void *At, const void *Ar, int b,
                                    int64_t d, float *out_loss);

/* Status word of the last egeria_sp_loss_static call on the current device:
 * EGERIA_OK, or EGERIA_ERR_TIMEOUT if a bounded wait inside its kernel ran out.
 * Call it after synchronising the stream of that call and before the next one
 * (which clears the word); it copies four bytes from the device and allocates
 * nothing. */
egeria_status egeria_sp_loss_static_status(void);

/* Measurement hook (needs EGERIA_FLAG_TIME_GRAM): device time, in milliseconds,
 * spent in the evaluation kernels of the egeria_sp_loss_batch /
 * egeria_plasticity_evaluate calls made since the last query (for tensor-core
 * modules that is the whole evaluation; the separate finalisation kernel of
 * CUDA-core modules is not included), and the number of those calls; at most
 * 4096 calls between two queries are timed.  Waits for the last recorded event.
 * Resets the tally. */
egeria_status egeria_gram_kernel_time(egeria_ctx *ctx, double *total_ms, int64_t *n_calls);

/* Number of kernels the library has launched through this context so far. */
int64_t egeria_launch_count(const egeria_ctx *ctx);

const char *egeria_status_string(egeria_status s);

#ifdef __cplusplus
}
#endif
#endif /* EGERIA_H_ */
