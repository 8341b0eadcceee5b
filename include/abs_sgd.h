/*
 * abs_sgd.h -- C ABI of the delayed synchronous step of ABS-SGD on one NVIDIA B200.
 *
 * Method: "A Delayed Synchronous SGD Algorithm with Adaptive Batch Size for Heterogeneous
 * GPU Clusters", arXiv 2308.15164, Algorithm 1.  Paper <-> library notation:
 *     N workers            = W          n parameters        = P
 *     G_t^i (accumulated)  = acc[set][i] (fp32, length P)
 *     M_t^i (batch size)   = b_i * M_r, b_i = number of abs_accumulate* calls of worker i
 *     learning rate gamma  = lr         compensation lambda = lambda_dc
 * The W workers of the paper are W gradient buffers in this GPU's memory, so the "global
 * synchronization" of Step 1 is an in-device weighted reduction; no collective is involved.
 * (Workers spread over several GPUs: the abs_global_* calls further down.)
 *
 * One iteration t (Algorithm 1, body of the while loop):
 *     abs_accumulate*(worker i, ...)   any number of times per worker, in any order
 *                                      (Step 2: G_t^i += g, M_t^i += M_r; the count is not
 *                                       preset -- the library counts calls)
 *     abs_sync_step()                  ends the iteration: the weighted average of the
 *                                      DELAYED gradients  Gbar_{t-1} = sum_i G_{t-1}^i / sum_i b_i
 *                                      (Step 1) is applied to x_t, giving x_{t+1}
 *                                      ("Update parameters"); the consumed set is cleared
 *                                      and becomes the target of iteration t+1.
 * Update rule (momentum and weight decay extend the paper's plain SGD; with momentum =
 * weight_decay = 0 it is exactly x_{t+1} = x_t - lr * Gtilde_t):
 *     Gtilde = Gbar + lambda_dc * Gbar*Gbar*(x_t - x_{t-1})         (Eq. 6; lambda_dc = 0: off)
 *     g = Gtilde + weight_decay * x ;  v = momentum * v + g ;  x = x - lr * v
 * If sum_i b_i = 0 for the delayed set (always at t = 0, where G_{-1} = 0) the step leaves
 * x and v untouched; buffers and counters still swap and t still advances.
 *
 * Conventions
 *   - All functions return an int status (ABS_OK or a negative ABS_E* code); none aborts,
 *     throws or blocks the host unless stated.  Argument errors are detected before any
 *     GPU work is enqueued.
 *   - "dev" pointers are device memory of the current CUDA device, "host" pointers host
 *     memory.  The caller owns every buffer it passes in (workspace, gradients, x/y,
 *     params0) and both streams; the context owns only host state and CUDA events.
 *   - Work is enqueued on the streams given in abs_config and follows CUDA stream order:
 *     an input buffer must stay valid and unchanged until the work enqueued by the call
 *     that received it has completed.
 *   - A context is not thread-safe; use one host thread per context.
 */
#ifndef ABS_SGD_H_
#define ABS_SGD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ABS_OK        0
#define ABS_EINVAL   (-1)  /* null / misaligned pointer, worker >= W, P = 0, W = 0 or > 64, bad dtype or flags */
#define ABS_ESTATE   (-2)  /* context destroyed or never initialised                                          */
#define ABS_ECUDA    (-3)  /* a CUDA runtime call failed; abs_last_error() gives the text                     */
#define ABS_ENOMEM   (-4)  /* workspace smaller than abs_workspace_bytes()                                    */
#define ABS_ETIMEOUT (-5)  /* a bounded device-side wait ran out                                              */
#define ABS_ELIMIT   (-6)  /* a size exceeds a fixed built-in capacity (abs_sync_step_noalloc: W > 64)        */

#define ABS_GRAD_F32   0u  /* abs_accumulate takes fp32 gradients */
#define ABS_GRAD_BF16  1u  /* abs_accumulate takes bf16 gradients (widened exactly to fp32) */

#define ABS_FLAG_PIPELINED  1u  /* Step 1 of iteration t runs on stream_sync, concurrently with Step 2 of t+1 */
#define ABS_FLAG_MLP        2u  /* the flat vector is a 2-layer MLP; enables abs_accumulate_mlp               */
#define ABS_FLAG_HOST_INPUT 4u  /* reserve staging so abs_accumulate_host may be used                         */
#define ABS_FLAG_OVERWRITE_FIRST 8u /* byte-saving variant: the fused step does not write zeros over the set it
                                       consumed; instead a worker's first micro-batch of an iteration stores
                                       (acc = g) rather than adds.  Same results; the fused step moves
                                       4*W_act + 16 instead of 8*W_act + 16 bytes per parameter and those first
                                       accumulates 8 (6 for bf16) instead of 12 (10).  Rows of workers that were
                                       idle keep stale values (never read).  abs_accumulate_mlp* store a worker's
                                       first gradient of an iteration in either mode (the row is then known
                                       to be empty), which saves the read of the W1 slice.                    */

#define ABS_FLAG_MLP_COALESCE 16u /* with ABS_FLAG_MLP: single abs_accumulate_mlp calls of a worker are gathered, up to
                                       four, and run as ONE batch (exactly what abs_accumulate_mlp_batch does with
                                       the same micro-batches: one forward GEMM over the stacked samples, one dW1
                                       GEMM with K = 64 n whose epilogue touches the accumulator slice once).  The
                                       call still reads x_dev / y_dev right away (its cast kernel is enqueued on
                                       stream_acc before it returns) and counts b_i right away; the rest of the
                                       gradient is enqueued when the group is full or when anything needs it:
                                       abs_sync_step / abs_global_begin (every micro-batch of iteration t is
                                       evaluated at x_t and lands in iteration t's accumulator), another kind of
                                       accumulate call for that worker, abs_wait, abs_check, abs_accumulator,
                                       abs_set_launch.  Results equal those of explicit batch calls over the same
                                       groups bit for bit, and those of ungrouped single calls to fp32 rounding.
                                       At most four groups wait at a time (the oldest is started when a fifth
                                       worker opens one).                                                       */

#define ABS_FLAG_GRAD_NORM 32u   /* the fused step also forms |Gbar|^2, the squared norm of the weighted average it
                                     applies (before Eq. 6 and weight decay): per-thread fp32 squares, summed in fp64
                                     by warp shuffles, one partial per CTA, added in a fixed order by the last CTA
                                     (reproducible run to run).  No extra memory traffic beyond 8 bytes per CTA.
                                     Read it with abs_grad_norm2.  Not with abs_global_*.                        */

#define ABS_FLAG_MLP_X_BF16 64u   /* with ABS_FLAG_MLP: abs_accumulate_mlp* take x_dev as bf16 values ([mlp_mb, mlp_in] row-major,
                                     2 bytes each) instead of fp32; they enter the GEMMs as they are (no rounding step) */

#define ABS_FLAG_MLP_DEFER 128u   /* with ABS_FLAG_MLP: a gradient call no longer touches its worker's accumulator row.
                                     Within an iteration every gradient is evaluated at the same x_t (Algorithm 1,
                                     Step 2), so a worker's sum of micro-batch gradients is ONE contraction over its
                                     stacked micro-batches, sum_j X_j^T dZ_j with K = 64 b_i, and may be formed late.
                                     A call runs forward, loss and layer-2 backward, bumps b_i, and leaves in the
                                     accumulator set's operand pool (about (3 mlp_in + 2 mlp_hidden) * 128 bytes per
                                     micro-batch) its dW1 operands bf16(X)^T, bf16(dZ)^T and its own db1 | dW2 | db2.
                                     Calls therefore need no order among themselves, not even those of one worker:
                                     they are spread over the library's internal streams call by call (results do not
                                     depend on that: every later sum runs in call order).  The rows are written when
                                     somebody needs them: when a row is read or added to (abs_accumulator,
                                     abs_accumulate*, abs_wait, abs_check, abs_state_export, abs_set_launch,
                                     abs_global_begin) or the pool (max(32, 16 W) micro-batches, at most 128) is full.
                                     At the end of an iteration (abs_sync_step) they are usually not written at all:
                                     when no row of the set was written during the iteration (gradient calls only;
                                     single-GPU step without ABS_FLAG_GRAD_NORM, mlp_hidden a multiple of 128) the step
                                     forms the weighted average of the W1 slice as one contraction over ALL micro-batches
                                     of all workers, (sum_j X_j^T dZ_j) / B, inside the kernel that applies the update,
                                     and the bias / W2 part from the pooled per-micro-batch partials (the rows then
                                     stay as they are: zero, or stale with ABS_FLAG_OVERWRITE_FIRST).  Otherwise the rows are completed first and the
                                     row-based step runs.  Either way the result equals that of the per-call path to
                                     fp32 rounding (one fp32 accumulation over K instead of rounded additions into the
                                     row).  Combines with every other flag; with ABS_FLAG_MLP_COALESCE single calls are
                                     gathered four at a time whoever their workers are.                             */

#define ABS_MAX_WORKERS 64u
#define ABS_MAX_RANKS   16u   /* GPUs taking part in abs_global_* (n_ranks * W <= ABS_MAX_WORKERS)        */
#define ABS_IPC_HANDLE_BYTES 64

/* Kernel classes, for abs_kernel_stats() and abs_set_launch(). */
#define ABS_K_ACCUMULATE 0   /* Step 2: acc += g                                        */
#define ABS_K_SYNC       1   /* Step 1 + update: weighted reduce, momentum SGD, clear   */
#define ABS_K_MLP_FWD    2   /* MLP: operand cast, forward GEMM, loss gradient          */
#define ABS_K_MLP_BWD    3   /* MLP: layer-2 backward, dZ, bias gradients               */
#define ABS_K_MLP_DW1    4   /* MLP: dW1 = X^T dZ on tcgen05, accumulated into acc      */
#define ABS_K_CHAIN      5   /* not a kernel: how consecutive kernels of a stream follow one another  */
#define ABS_K_COUNT      6

typedef struct abs_ctx abs_ctx;   /* opaque; host memory owned by the library */

typedef struct abs_config {
    uint64_t P;               /* number of parameters n (> 0)                                         */
    uint32_t W;               /* number of logical workers N (1..ABS_MAX_WORKERS)                     */
    float lr;                 /* gamma                                                                */
    float momentum;           /* mu; 0 = the paper's plain SGD                                        */
    float weight_decay;       /* coupled L2; 0 = the paper's plain SGD                                */
    float lambda_dc;          /* lambda of Eq. 6; 0 disables compensation                             */
    uint32_t grad_dtype;      /* ABS_GRAD_F32 or ABS_GRAD_BF16: element type of abs_accumulate inputs */
    uint32_t flags;           /* ABS_FLAG_*                                                           */
    uint32_t mlp_in, mlp_hidden, mlp_out, mlp_mb;  /* with ABS_FLAG_MLP: layer sizes and samples per
                                 micro-batch.  Flat layout: W1 [in,hidden] row-major, b1 [hidden],
                                 W2 [hidden,out] row-major, b2 [out]; P must equal their total.
                                 Limits: in % 128 == 0, hidden % 128 == 0, out <= 16, mb == 64.      */
    void *stream_acc;         /* cudaStream_t for Step 2 work (accumulation); NULL = default stream.  With
                                 ABS_FLAG_MLP a high-priority stream is worth having: the first kernel of
                                 every gradient call runs there and should not queue behind earlier calls'
                                 dW1 GEMMs (which the library runs at the lowest priority)              */
    void *stream_sync;        /* cudaStream_t for Step 1 work when ABS_FLAG_PIPELINED; must then
                                 differ from stream_acc                                               */
} abs_config;

/* Bytes of device workspace abs_init needs for this configuration (0 if cfg is invalid).
 * Holds: parameters x (two copies when pipelined), momentum v, the double-buffered per-worker
 * accumulators acc[2][W][P_pad] (P_pad = P rounded up to 256 elements), device counters,
 * and the MLP / host-input scratch when those flags are set. */
size_t abs_workspace_bytes(const abs_config *cfg);

/* Algorithm 1, "Initialization": t = 0, G_{-1}^i = 0, x_0 = params0.
 * workspace_dev: device memory, 256-byte aligned, >= abs_workspace_bytes(cfg); used until
 * abs_destroy.  params0_dev: P fp32 values, copied in (stream-ordered on stream_acc).
 * Errors: ABS_EINVAL (bad cfg/pointers), ABS_ENOMEM (workspace too small), ABS_ECUDA. */
int abs_init(abs_ctx **out, const abs_config *cfg, void *workspace_dev, size_t workspace_bytes,
             const float *params0_dev);

/* Algorithm 1, Step 2 (one reference batch of worker `worker`): G_t^i += grad, b_i += 1.
 * grad_dev: P contiguous elements of cfg.grad_dtype, 16-byte aligned, device memory; the
 * gradient of a micro-batch is the MEAN over its M_r samples.  Enqueued on stream_acc. */
int abs_accumulate(abs_ctx *ctx, uint32_t worker, const void *grad_dev);

/* Algorithm 1, Step 2 for n (1..8) reference batches of one worker whose gradients are all at hand:
 * G_t^i += g_0, += g_1, ... (added one after the other in list order, so the result equals n calls of
 * abs_accumulate bit for bit); b_i += n.  One pass over the accumulator row: (4 n + 8) bytes per parameter
 * for fp32 gradients (2 n + 8 for bf16) instead of 12 n (10 n).  grads_dev: HOST array of n device
 * pointers, each as for abs_accumulate; the array itself is read before the call returns.
 * Enqueued on stream_acc. */
int abs_accumulate_batch(abs_ctx *ctx, uint32_t worker, uint32_t n, const void *const *grads_dev);

/* Same as abs_accumulate for a gradient in (preferably pinned) HOST memory: copies it to
 * the device through an internal double-buffered staging area, then accumulates.  Needs
 * ABS_FLAG_HOST_INPUT.  grad_host must stay valid until the copy has completed (the call
 * may return earlier when the memory is pinned). */
int abs_accumulate_host(abs_ctx *ctx, uint32_t worker, const void *grad_host);

/* Algorithm 1, Step 2 with the gradient computed here: forward and backward pass of the
 * 2-layer ReLU MLP with mean softmax cross-entropy on one micro-batch, evaluated at the
 * current parameters x_t, and accumulated into worker `worker`'s buffer; b_i += 1.
 * x_dev: [mlp_mb, mlp_in] row-major, fp32 (bf16 with ABS_FLAG_MLP_X_BF16), 16-byte aligned; y_dev: [mlp_mb]
 * int32 class indices in [0, mlp_out).  GEMM operands are rounded to bf16 (nearest even) with fp32 accumulation;
 * dW1 = X^T dZ runs on the tcgen05 tensor cores and its epilogue adds into the accumulator.
 * Needs ABS_FLAG_MLP.  x_dev and y_dev are read by the first kernel only, which is enqueued on stream_acc
 * (they may be reused by later work on that stream).  The remaining kernels run on internal streams of
 * the worker (workers compute concurrently, as in the paper; what a worker's calls add to its row is added in call
 * order; the dW1 GEMM of a call runs on a second, lowest-priority stream of the worker, so that the worker's next
 * call can start beside it), which start after everything enqueued on stream_acc so far; abs_sync_step, abs_wait, abs_check,
 * abs_accumulate, abs_accumulate_host and abs_accumulator make stream_acc wait for all of them.  With
 * ABS_FLAG_MLP_DEFER a call adds nothing to the row and launches no dW1 kernel (see the flag): calls are then spread
 * over the internal streams whoever their workers are. */
int abs_accumulate_mlp(abs_ctx *ctx, uint32_t worker, const void *x_dev, const int32_t *y_dev);

/* n (1..8) consecutive reference batches of one worker in one call: the same computation as n calls of
 * abs_accumulate_mlp (forward, loss and backward of every micro-batch at x_t; b_i += n), but the n dW1
 * products are contracted by ONE tcgen05 GEMM with K = 64 n, so the worker's fp32 accumulator slice is
 * read and written once instead of n times -- that traffic, not the MMAs, bounds the kernel.  The sum
 * over the n micro-batches is formed in the fp32 TMEM accumulator, so results agree with n single
 * calls to fp32 rounding, not bit for bit.  x_dev: [n][mlp_mb][mlp_in] fp32 (bf16 with ABS_FLAG_MLP_X_BF16);
 * y_dev: [n][mlp_mb] int32. */
int abs_accumulate_mlp_batch(abs_ctx *ctx, uint32_t worker, uint32_t n, const void *x_dev, const int32_t *y_dev);

/* The same call for n (1..8) reference batches that are NOT adjacent in memory: x_devs[j] / y_devs[j] point to
 * micro-batch j ([mlp_mb, mlp_in] and [mlp_mb], aligned as for abs_accumulate_mlp); the two pointer arrays are host
 * memory and are read before the call returns.  One cast launch reads all n buffers (on stream_acc, like every
 * gradient call's first kernel); from there on the call is abs_accumulate_mlp_batch over the same micro-batches
 * in list order, bit for bit. */
int abs_accumulate_mlp_list(abs_ctx *ctx, uint32_t worker, uint32_t n, const void *const *x_devs,
                            const int32_t *const *y_devs);

/* Algorithm 1, Step 1 + compensation + "Update parameters" + t = t + 1 (see the file header).
 * Without ABS_FLAG_PIPELINED the fused kernel runs on stream_acc.  With it, the call makes
 * x_{t+1} (computed by the kernel launched one call earlier on stream_sync) visible to
 * stream_acc, and launches the kernel for the set just filled on stream_sync, so that it
 * overlaps the accumulation of iteration t+1.  Both modes publish the same x_1, x_2, ...
 * Never blocks the host. */
int abs_sync_step(abs_ctx *ctx);

/* Device pointer to the published parameters x_t (P fp32).  Work enqueued on stream_acc after
 * this call sees x_t; the pointer is valid until the next abs_sync_step.  Does not block. */
int abs_params(abs_ctx *ctx, const float **x_dev_out);

/* Copy the published parameters x_t to host memory (P fp32); blocks until the copy is done. */
int abs_params_host(abs_ctx *ctx, float *dst_host);

/* Device pointer to the momentum buffer v (P fp32) as of the published parameters.  In
 * pipelined mode v is being rewritten by the in-flight kernel; call abs_wait first. */
int abs_momentum(abs_ctx *ctx, const float **v_dev_out);

/* Device pointer to accumulator G^worker of set `set` (0 or 1), P fp32 (inspection / parity). */
int abs_accumulator(abs_ctx *ctx, uint32_t set, uint32_t worker, const float **acc_dev_out);

/* Logical state after the calls made so far (what Algorithm 1 holds at this point):
 * cnt_host[2][W] = b_i of both sets, *cur = index of the set the current iteration fills,
 * *t = iteration counter.  Host-side, never blocks.  Any output pointer may be NULL. */
int abs_counters(abs_ctx *ctx, int32_t *cnt_host, uint32_t *cur, uint64_t *t);

/* The b_i that sync step number `step` (0-based, < t, at most 63 steps back) consumed, as
 * counted ON THE DEVICE by the accumulate kernels and logged by the fused kernel before it
 * cleared them.  b_host[W].  Blocks until the logging kernel has finished. */
int abs_consumed(abs_ctx *ctx, uint64_t step, int32_t *b_host);

/* |Gbar|^2 of the weighted average that sync step `step` applied (0 if it applied nothing); same window
 * and blocking behaviour as abs_consumed.  Needs ABS_FLAG_GRAD_NORM.  (A run-time metric; the paper's
 * experiments log accuracy over time only.) */
int abs_grad_norm2(abs_ctx *ctx, uint64_t step, double *out);

/* Algorithm 1, Step 2 loop condition "while Step 1 not finished": *done = 0 while the fused kernel
 * launched by the last abs_sync_step (pipelined mode) is still running, 1 once it has completed
 * (always 1 in eager mode or when nothing is in flight).  Never blocks.  A driver that keeps
 * calling abs_accumulate* until *done becomes 1 gets the paper's adaptive batch size: b_i is
 * whatever the workers managed to compute while the synchronisation ran. */
int abs_step1_finished(abs_ctx *ctx, int *done);

/* gamma may change between iterations (Theorem 1 allows gamma_t).  The rate travels with the
 * gradients: the value in effect when abs_sync_step ends iteration t is the one used to apply
 * that iteration's gradients, i.e. it is the paper's gamma_{t+1} (x_{t+2} = x_{t+1} - gamma_{t+1} *
 * Gtilde_{t+1}).  Supplying it one iteration ahead is what lets Step 1 start the moment the
 * iteration ends; eager and pipelined mode follow the same rule. */
int abs_set_lr(abs_ctx *ctx, float lr);

/* Make stream_acc wait (on the device, not the host) for every kernel launched on
 * stream_sync so far.  Does not publish anything new. */
int abs_wait(abs_ctx *ctx);

/* Blocks until everything enqueued so far has finished and reports the device-side status:
 * ABS_OK, ABS_ECUDA (a stream reported an error) or ABS_ETIMEOUT (a kernel gave up a bounded
 * wait on an mbarrier; its output tile was not written). */
int abs_check(abs_ctx *ctx);

/* Failure-reporting self-test: enqueues (on stream_acc) one tiny kernel that waits, with the library's bounded
 * polling loop, for a barrier that nothing completes; it gives up within a fraction of a millisecond and records
 * the time-out exactly as a stuck copy pipeline of the fused step would.  The next abs_check then returns
 * ABS_ETIMEOUT once (and clears the record); the context and the GPU stay fully usable.  Nothing faults or hangs. */
int abs_selftest_timeout(abs_ctx *ctx);

/* Launch shape of a kernel class: CTAs per SM for the persistent grid (0 = default, -1 = one
 * tile per CTA) for ABS_K_ACCUMULATE and ABS_K_SYNC.  ABS_K_SYNC also takes -2: the fused step with its rows
 * staged through shared memory by the bulk-copy engine (cp.async.bulk loads and stores, mbarrier pipeline;
 * W <= 24 and no ABS_FLAG_GRAD_NORM, else the default kernel runs); same results bit for bit.  For the MLP classes the value selects
 * kernel variants instead (results agree within rounding):
 *   ABS_K_MLP_DW1  bit mask.  dW1 kernel: 0 = chosen per call (the persistent ring kernel when the tile is
 *                  stored or the call is K-batched, the register-prefetch kernel for single adds);
 *                  4 = persistent warp-specialised ring kernel (TMA store / reduce-add);
 *                  8 = one tile per CTA, accumulator tile prefetched into registers.
 *                  32 = the ring kernel keeps 128 x 64 tiles for K-batched calls (default there: 128 x 128).
 *                  128 = forward GEMM and ring dW1 kernel always with their deep pipelines, which take a whole
 *                  SM's shared memory (default: with W > 1, outside serial mode, their light forms of about
 *                  100 KB, so that CTAs of different workers' calls share an SM; same results bit for bit).
 *   ABS_K_MLP_BWD  1 = with ABS_FLAG_MLP_DEFER: the step never works from the pooled operands; every iteration's
 *                  rows are completed first (see the flag).  2 = the pooled step keeps 128 x 128 tiles (default:
 *                  128 x 256 where mlp_hidden is a multiple of 256).
 *   ABS_K_MLP_FWD  1 = serial mode: every kernel of a gradient call runs on stream_acc instead of the
 *                  worker's internal stream (for per-kernel timing).
 *   ABS_K_CHAIN    0 = consecutive kernels of a stream are chained by programmatic dependent launch: the next
 *                  kernel is made resident and does its set-up while the one ahead drains, and waits on the
 *                  device for that one's completion before it reads anything it wrote (default; same results);
 *                  1 = plain stream order. */
int abs_set_launch(abs_ctx *ctx, int kernel_class, int ctas_per_sm);

/* Per-kernel timing with CUDA events on the launching stream.  abs_profile(ctx, 1) starts
 * recording an event pair around every launch; abs_kernel_stats() blocks until recorded
 * work has finished and returns the number of launches and their summed duration since
 * profiling was switched on (or last reset by abs_profile(ctx, 1)). */
int abs_profile(abs_ctx *ctx, int enable);
int abs_kernel_stats(abs_ctx *ctx, int kernel_class, uint64_t *launches, double *total_ms);

/* Timeline of the timed launches.  abs_profile(ctx, 2) records, besides the totals, when each timed kernel (or
 * kernel group of a gradient call) started and stopped, in microseconds since the moment stream_acc reached the
 * abs_profile call.  stream: 0 = stream_acc, 1 = stream_sync, 2 + k = internal worker stream k.  A span starts
 * when its stream reaches the kernel (the kernel may still queue for SM resources behind other streams' kernels)
 * and ends when the kernel has finished, so overlapping spans of different streams show which kernels really ran
 * side by side.  abs_profile_timeline blocks until the recorded work has finished, writes up to `capacity` spans
 * to `out` (may be NULL) in launch order and the number recorded so far to *n. */
typedef struct abs_span {
    int32_t kernel_class;   /* ABS_K_* */
    int32_t stream;
    int32_t part;           /* ordinal of the kernel within its class for one gradient call (ABS_K_MLP_FWD: 0 = operand
                               cast, 1 = forward GEMM, 2 = bias / ReLU / partial logits); 0 otherwise */
    float start_us, stop_us;
} abs_span;
int abs_profile_timeline(abs_ctx *ctx, abs_span *out, size_t capacity, size_t *n);

/* Number of kernels this context has launched since abs_init. */
uint64_t abs_launch_count(abs_ctx *ctx);

/* Text of the last error on this context (never NULL; "" if none).  ctx may be NULL: then
 * the text of the last failed abs_init on this thread. */
const char *abs_last_error(abs_ctx *ctx);

/* Waits for the context's enqueued work, releases events and host state.  The workspace
 * is the caller's to free afterwards.  Using ctx after this returns ABS_ESTATE. */
int abs_destroy(abs_ctx *ctx);

/* ---------------------------------------------------------------------------------------------------
 * Step 1 across GPUs: the paper's own setting (Section 5.1-5.2: the workers are different GPUs and Step 1 is
 * the "global synchronization" of G_{t-1}^i and of the batch sizes M_{t-1}^i between them).
 *
 * One process and one context per GPU ("rank"); a context's W workers are that GPU's local workers, and the
 * global worker index of local worker i on rank q is q*W + i.  All ranks use the same abs_config (so their
 * workspaces have the same layout), ABS_FLAG_PIPELINED, and make the same sequence of abs_global_* calls.
 * abs_accumulate* are used as before; ONE iteration ends with, on every rank,
 *
 *     abs_global_begin(ctx, &counts, &n);     // x_{t+1} becomes visible to stream_acc; this rank's b_i go
 *                                             // into its slots of counts[0..n), zeros elsewhere
 *     <sum counts[0..n) (int32) over all ranks, in place, ordered on stream_sync>    -- exchange A
 *     abs_global_step(ctx);                   // the fused kernel, on stream_sync
 *     <any collective over all ranks ordered on stream_sync>                          -- exchange B
 *     abs_global_end(ctx);
 *
 * instead of abs_sync_step.  The two exchanges are the caller's (ncclAllReduce on stream_sync, or any
 * equivalent that is ordered with the work on that stream); they carry n <= 64 integers, not gradients.
 * Exchange A is the paper's batch-size synchronisation and also guarantees that every rank has finished
 * the iteration's accumulation before any kernel reads its rows; exchange B guarantees that every rank's
 * kernel has finished before anyone uses x_{t+1} or accumulates into the cleared set again.
 *
 * The gradients themselves are moved by the kernel of abs_global_step, not by a collective library: rank r
 * owns a contiguous slice of the flat vector (abs_global_slice); for its slice it reads every worker row
 * of every rank through the peer mappings given to abs_global_attach, forms
 * Gbar = sum_{q,i} G^{q,i} / sum_{q,i} b_{q,i} in global worker order, applies Eq. 6 / weight decay /
 * momentum exactly as abs_sync_step does, writes x_{t+1} into EVERY rank's parameter buffer (and bf16
 * copy), and writes zeros over what it read (not with ABS_FLAG_OVERWRITE_FIRST).  Per iteration a rank
 * receives (G-1)/G * W * 4 bytes per parameter and sends (G-1)/G * (W + 1) * 4: the volume of a
 * reduce-scatter plus an all-gather, in one pass.  Results equal a one-GPU context with G*W workers fed the
 * same gradients, bit for bit.  The momentum vector is sharded: a rank keeps only its slice of v current.
 * If all b are 0 the kernel copies x_t to x_{t+1} everywhere and leaves v alone.
 * --------------------------------------------------------------------------------------------------- */
typedef struct abs_peer_table {
    uint32_t n_ranks;                        /* G, 1..ABS_MAX_RANKS                                          */
    uint32_t rank;                           /* this context's rank                                          */
    void *workspace_dev[ABS_MAX_RANKS];      /* every rank's workspace (the pointer it gave abs_init) AS MAPPED
                                                IN THIS PROCESS: [rank] is the own workspace, the others come
                                                from abs_ipc_open (other processes) or are plain pointers
                                                (same process, peer access enabled)                          */
} abs_peer_table;

/* Once, after abs_init and before the first iteration ends; every rank's abs_init must have completed
 * (synchronise the streams and the processes first).  Errors: ABS_EINVAL (not pipelined, bad table,
 * n_ranks * W > 64, called twice).  After it, abs_sync_step returns ABS_EINVAL on this context. */
int abs_global_attach(abs_ctx *ctx, const abs_peer_table *peers);
/* See above.  *counts_dev: device pointer (inside the workspace) to n = n_ranks * W int32; valid until
 * abs_destroy.  Never block the host.  Calls out of order return ABS_EINVAL. */
int abs_global_begin(abs_ctx *ctx, int32_t **counts_dev, uint32_t *n_counts);
int abs_global_step(abs_ctx *ctx);
int abs_global_end(abs_ctx *ctx);
/* The slice of the flat vector this rank reduces and whose momentum it holds: elements [first, first+count). */
int abs_global_slice(abs_ctx *ctx, uint64_t *first, uint64_t *count);
/* The same partition without a context (host arithmetic only): the slices of ranks 0..n_ranks-1 are
 * consecutive, disjoint and cover [0, P); each starts on a multiple of 1024 elements; trailing ranks may
 * get an empty slice when P is small. */
int abs_global_partition(uint64_t P, uint32_t n_ranks, uint32_t rank, uint64_t *first, uint64_t *count);
/* abs_consumed for a context in multi-GPU mode: b_host[n_ranks * W], global worker order. */
int abs_global_consumed(abs_ctx *ctx, uint64_t step, int32_t *b_host);

/* CUDA IPC plumbing for ranks in separate processes.  abs_ipc_export: handle_out receives
 * ABS_IPC_HANDLE_BYTES bytes naming the device allocation that contains dev_ptr, *offset_out the offset of
 * dev_ptr inside it; send both to the peers.  abs_ipc_open (in a peer process, its GPU current): maps the
 * allocation and returns the address that corresponds to dev_ptr.  abs_ipc_close undoes abs_ipc_open.
 * The memory must come from cudaMalloc (not from a virtual-memory pool).  Status codes as everywhere. */
int abs_ipc_export(const void *dev_ptr, void *handle_out, uint64_t *offset_out);
int abs_ipc_open(const void *handle, uint64_t offset, void **dev_ptr_out);
int abs_ipc_close(void *dev_ptr, uint64_t offset);

/* Checkpoint and resume (the paper has no counterpart).  abs_state_export writes everything a later
 * abs_state_import needs to continue the run bit for bit: parameters (both buffers), momentum, both
 * accumulator sets, counters and logs, iteration counter, set index, rates in effect -- abs_state_bytes()
 * bytes of HOST memory, dominated by the accumulators (8 * W * P bytes).  Both calls block: they start any
 * waiting micro-batch groups and wait for everything enqueued on the context's streams.  Import needs a
 * context created with the same abs_config (streams and initial lr may differ; the saved rate wins) and, in
 * multi-GPU mode, attached with the same rank layout; it replaces the context's whole state.  Errors:
 * ABS_EINVAL (NULL / short buffer, foreign or mismatching state, called between abs_global_begin and
 * abs_global_end), ABS_ECUDA.  The log behind abs_grad_norm2 is not part of the state. */
size_t abs_state_bytes(abs_ctx *ctx);
int abs_state_export(abs_ctx *ctx, void *dst_host, size_t bytes);
int abs_state_import(abs_ctx *ctx, const void *src_host, size_t bytes);

/* One fused sync step on buffers the CALLER owns, for callers that cannot allocate device
 * memory.  (No counterpart in the paper: this is a packaging variant of the kernel behind
 * abs_sync_step, not another algorithm step.)
 *
 * Meant for code that runs inside someone else's memory budget -- an extension under a
 * framework that already reserved the GPU for its own pool, a job whose device memory was
 * carved up front, a loop that cannot afford the device-wide synchronisation of cudaMalloc /
 * cudaFree.  The call itself allocates nothing, on the host or on the device: the few words of
 * working memory the kernel needs (its CTA ticket and the log of consumed counts) live in a
 * 1 KiB array built into the library, which every GPU that loads the library holds until the
 * process exits.
 *
 * Computes, in place and on `stream`:  B = sum_i cnt[i];  if B > 0:
 *     Gbar = (sum_{i: cnt[i]>0} acc[i]) / B ;  g = Gbar + weight_decay*x ;  v = momentum*v + g ;
 *     x = x - lr*v ;  acc[i] = 0 for every i with cnt[i] > 0 ;
 * then cnt[i] = 0 for all i.  (No compensation term, no bf16 shadow.)
 *   x_dev, v_dev   P fp32 each, 16-byte aligned, updated in place
 *   acc_dev        W rows of fp32, row i at acc_dev + i*row_stride, 16-byte aligned
 *   row_stride, P  in elements; both multiples of 4, row_stride >= P
 *   cnt_dev        W int32 device counters b_i (input, cleared on output)
 *   stream         cudaStream_t (NULL = default stream)
 * All four buffers and the stream must belong to the CURRENT device (the built-in array used is the current
 * device's copy); buffers of another device, or host pointers, return ABS_EINVAL.
 * Limit: W <= 64 (what the built-in working memory can log); larger W returns ABS_ELIMIT and
 * nothing is launched.  Other bad arguments return ABS_EINVAL, CUDA failures ABS_ECUDA.
 * The step always runs the load/store form of the fused kernel (never the bulk-copy form abs_sync_step picks
 * for some worker counts): that form has no device-side wait that could run out, so a call that returned
 * ABS_OK either completes in full or shows up as a CUDA error on the stream.  Results equal abs_sync_step's
 * bit for bit (both forms compute the same bits).
 *
 * The first call on each device looks up the device address of the built-in array (one
 * cudaGetSymbolAddress, no allocation); make that first call outside any stream capture.
 * All calls on a device share the array and it keeps the previous call's contents (the call
 * clears the word that must start at zero), so two calls whose kernels may overlap on the GPU
 * -- different streams without an ordering between them -- race on it: order them. */
int abs_sync_step_noalloc(float *x_dev, float *v_dev, float *acc_dev, uint64_t row_stride, uint64_t P,
                          uint32_t W, int32_t *cnt_dev, float lr, float momentum, float weight_decay,
                          void *stream);

#ifdef __cplusplus
}
#endif
#endif /* ABS_SGD_H_ */
