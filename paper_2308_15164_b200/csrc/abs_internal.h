// Internal declarations shared by the host-side context and the kernel translation units.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "abs_sgd.h"

namespace abs_sgd {

constexpr int kMaxW = ABS_MAX_WORKERS;
constexpr int kLogDepth = 64;     // sync steps kept in the device-side consumed-count log
constexpr size_t kPadElems = 256; // accumulator row stride is P rounded up to this many elements

// ---- programmatic dependent launch ----------------------------------------------------------
// Consecutive kernels of a stream are chained so that kernel n+1 is made resident (CTAs scheduled, shared
// memory carved, barriers initialised, TMEM allocated) while kernel n is still draining.  Every kernel of this
// library executes pdl_wait() in every CTA before it touches anything an earlier kernel of its stream wrote --
// the wait returns once the predecessor grid has completed and its writes are visible -- and only THEN lets its
// own successor start (pdl_trigger()).  By induction, when a kernel starts, every kernel two or more places ahead
// of it in the stream has completed, so code in front of pdl_wait() may read what those wrote, but nothing
// the immediate predecessor writes.  Both instructions do nothing in a launch without the attribute.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#endif
// kernel<<<grid, block, smem, stream>>>(args...), with the programmatic-stream-serialization attribute when
// `chained` is set.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                 bool chained, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = chained ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<Args&&>(args)...);
}

// ---- Step 2: acc_row[j] += g[j], cnt[0] += 1 (Algorithm 1, Step 2) ------------------------
// grad_dtype: ABS_GRAD_F32 / ABS_GRAD_BF16.  P = number of valid elements in g.
// overwrite: acc_row[j] = g[j] instead (first micro-batch of a worker when the row is not kept zeroed).
// chained (here and below): launch with programmatic dependent launch on the kernel ahead on `stream`.
cudaError_t launch_accumulate(float* acc_row, const void* g, uint32_t grad_dtype, size_t P, int32_t* cnt, bool overwrite,
                              int ctas_per_sm, int num_sms, cudaStream_t stream, bool chained);

// ---- Step 1 + update (Algorithm 1, Step 1, Eq. 6, "Update parameters") --------------------
struct SyncArgs {
    const float* x_in;        // x_t            [P_pad]
    float* x_out;             // x_{t+1}        [P_pad] (may alias x_in)
    float* v;                 // momentum       [P_pad]
    float* acc;               // delayed set    [W][row_stride]
    unsigned long long row_stride;  // elements between worker rows (multiple of 4)
    unsigned long long n_vec;       // P_pad / 4
    int W;
    int32_t* cnt;             // [W]  device counters of the delayed set (b_i); cleared by the kernel
    int32_t* log_row;         // [W]  receives the consumed b_i
    unsigned int* ticket;     // last-CTA-done ticket, zero on entry and on exit
    float lr, mu, wd;
    float lambda_dc;          // Eq. 6 coefficient
    float disp_scale;         // x_t - x_{t-1} = -disp_scale * v   (0 when the previous step was a no-op)
    __nv_bfloat16* shadow;    // optional bf16 copy of x_{t+1} [P_pad], or nullptr
    int zero_acc;             // 1: overwrite the consumed rows with zeros; 0: leave them (overwrite-first mode)
    double* norm_part;        // optional: one slot per CTA for the partial sums of |Gbar|^2 ...
    double* norm_out;         // ... and where the last CTA puts the total (nullptr: the norm is not computed)
    unsigned int norm_slots;  // slots in norm_part
    int overlapped;           // the launch runs beside the next iteration's accumulate kernels (pipelined mode)
    int* status;              // optional device status word (ABS_ETIMEOUT if a bounded wait of the bulk-copy kernel ran out)
    int tma_one_cta;          // bulk-copy form: 0 = as many CTAs per SM as its budget holds; n > 0 = one CTA per SM with n stages
    int plain_only;           // 1: never the bulk-copy form (a caller without a status word to report its time-outs through)
};
// n (1..kMaxAccBatch) gradients of one worker added in one pass over its accumulator row, in list order.
constexpr int kMaxAccBatch = 8;
struct GradList {
    const void* p[kMaxAccBatch];
};
cudaError_t launch_accumulate_multi(float* acc_row, const GradList& gl, int n, uint32_t grad_dtype, size_t P, int32_t* cnt,
                                    bool overwrite, int ctas_per_sm, int num_sms, cudaStream_t stream, bool chained);
// ctas_per_sm: 0 = default shape, -1 = one tile per CTA, > 0 = persistent grid, -2 = the bulk-copy kernel below
// where it applies (else the default).
cudaError_t launch_sync(const SyncArgs& a, int ctas_per_sm, int num_sms, cudaStream_t stream, bool chained);
// Same step with the rows staged through shared memory by cp.async.bulk (sync_tma.cu).  cudaErrorNotSupported for
// W > kSyncTmaMaxW or when the gradient norm is wanted: the caller then uses launch_sync.
constexpr int kSyncTmaMaxW = 24;
cudaError_t launch_sync_tma(const SyncArgs& a, int num_sms, cudaStream_t stream, bool chained);
// One small launch whose only wait can never be satisfied: it gives up after a few thousand polls and writes
// ABS_ETIMEOUT to *status (the path a stuck pipeline takes), leaving the context usable.
cudaError_t launch_bounded_wait_selftest(int* status, cudaStream_t stream);

// ---- Step 1 across GPUs (Algorithm 1, Step 1 as the paper runs it: workers on different GPUs) -----
// Rank r reduces, updates and redistributes the vectors [vec_lo, vec_hi) of the flat parameter: it reads that
// slice of every worker row of every rank (its own rows and the peers' rows through peer mappings), applies the
// same update as k_sync, stores x_{t+1} into every rank's output buffer and clears the slice of every row it read.
constexpr int kMaxRanks = ABS_MAX_RANKS;
struct GlobalSyncArgs {
    const float* x_in;                    // this rank's x_t [P_pad]
    float* v;                             // this rank's momentum; only [vec_lo, vec_hi) is kept up to date
    float* acc[kMaxRanks];                // rank q's set being applied, [W_local][row_stride], as mapped here
    float* x_out[kMaxRanks];              // rank q's buffer for x_{t+1}
    __nv_bfloat16* shadow[kMaxRanks];     // rank q's bf16 copy of x_{t+1}, or nullptr
    unsigned long long row_stride;        // elements between worker rows
    unsigned long long vec_lo, vec_hi;    // this rank's slice, in float4 vectors
    int G, W_local;
    const int32_t* cnt_all;               // [G * W_local] b_i of every worker of every rank (exchanged beforehand)
    int32_t* log_row;                     // [G * W_local] receives the consumed b_i
    unsigned int* ticket;                 // last-CTA-done ticket, zero on entry and on exit
    int* applied;                         // in: 1 if the previous step changed x; out: whether this one did
    float lr, mu, wd, lambda_dc;
    float disp_scale;                     // rate of the previous step (x_t - x_{t-1} = -disp_scale * v if it applied)
    int zero_acc;
};
cudaError_t launch_sync_global(const GlobalSyncArgs& a, int ctas_per_sm, int num_sms, cudaStream_t stream, bool chained);
// gcnt[j] = (own_lo <= j < own_lo + W_local) ? cnt[j - own_lo] : 0 for j < n_total;  cnt[0..W_local) = 0.
cudaError_t launch_global_counts(int32_t* gcnt, int32_t* cnt, int own_lo, int W_local, int n_total, cudaStream_t stream);

// bf16 copy of an fp32 vector (n multiple of 4): used once at init for the MLP weight shadow.
cudaError_t launch_cast_bf16(const float* src, __nv_bfloat16* dst, size_t n, int num_sms, cudaStream_t stream);

// ---- MLP micro-batch gradient (Step 2 with the gradient computed on the device) ----------
constexpr int kMlpMaxBatch = 8;     // micro-batches one gradient call may carry
constexpr int kMlpGatherMax = 4;    // micro-batches ABS_FLAG_MLP_COALESCE gathers into one group
// Internal bit of the `variant` argument below (set by the context, never by abs_set_launch): forward GEMM and ring
// dW1 kernel in their light shared-memory configurations, so that CTAs of different workers' calls share an SM.
constexpr int kMlpLightBit = 256;
// Which kernels of a gradient call are launched chained to the kernel ahead (bits of the `chain` argument of
// launch_mlp_front; the cast and the dW1 kernel take a bool).
constexpr int kChainCast = 1, kChainFwd1 = 2, kChainFwd2 = 4, kChainBwd = 8, kChainDw1 = 16;
constexpr int kMlpStreams = 8;   // internal worker streams (worker i runs on stream i % kMlpStreams)
constexpr int kMlpSets = 8;      // scratch sets, one per call in flight, taken round-robin
struct MlpDims {
    int d_in, d_hidden, d_out, mb;
};
// Micro-batches one dW1 launch may contract (K = 64 per micro-batch) and the slots of the stacked operand
// tensors that hold them, in contraction order.
constexpr int kMlpMaxSlots = 128;
struct MlpSlots {
    uint16_t s[kMlpMaxSlots];
};
struct MlpWorkers {      // worker of each micro-batch of a pooled gradient call
    uint8_t w[8];
};
struct alignas(64) TmapBytes {   // storage for one CUtensorMap (encoded on the host, passed by value to kernels)
    unsigned char b[128];
};
struct MlpScratch {      // device pointers carved from the workspace (all hidden-major, see mlp.cu)
    __nv_bfloat16* xb;   // [mb][d_in]            bf16(X)
    __nv_bfloat16* xtb;  // [4][d_in][mb]         bf16(X)^T of up to 4 stacked micro-batches: K-major A operand of dW1
    float* zpart;        // [split][d_hidden][mb] split-K partial sums of the forward GEMM
    __nv_bfloat16* hbt;  // [d_hidden][mb]        bf16(relu(Z))^T
    __nv_bfloat16* dzt;  // [4][d_hidden][mb]     bf16(dZ)^T of up to 4 stacked micro-batches: K-major B operand of dW1
    float* lpart;        // [d_hidden/32][mb][16] partial logits per CTA of k_fwd2
    float* gpart;        // [groups][mb][16]      partial logits per group of 8 CTAs
    int32_t* ycopy;      // [4][mb]               labels of the call's micro-batches (copied by k_cast_x)
    float* bpart;        // [4][d_hidden/32][4][256] partial dW2 / db1 / db2 sums of k_bwd, per micro-batch of a call
    unsigned int* tickets_b;  // [d_hidden/32]     "last CTA done" tickets of k_bwd (zero between launches)
    unsigned int* tickets;  // [groups]           "last CTA done" tickets of the logit reduction (zero between launches)
    unsigned int* tickets2; // [4]                second level of that reduction, one per micro-batch of a call
    float* dlbuf;        // [4][2][mb][16]        dL of each micro-batch: unrounded, and rounded to bf16
    int* status;         // device status word: ABS_ETIMEOUT if a bounded wait ran out
    void* zero_from;     // region that must be zero before first use (tickets + status) ...
    size_t zero_bytes;   // ... and its size
    int num_sms;         // SM count of the device (grid of the persistent dW1 kernel)
    TmapBytes tmap_xt, tmap_dzt;   // dW1 operands
    TmapBytes tmap_xb, tmap_w1[2]; // forward GEMM operands (W1 of each bf16 shadow copy)
};
// ABS_FLAG_MLP_DEFER: the dW1 operands of an accumulator set's gradient calls are kept (bf16(X)^T and bf16(dZ)^T,
// (d_in + d_hidden) * 128 bytes per micro-batch) in `cap` slots instead of being contracted call by call.
// A slot also holds what else a call hands from one of its kernels to the next across streams -- bf16(X) for the
// forward GEMM, the labels -- and the micro-batch's db1 | dW2 | db2 (laid out like the row behind W1): in this
// mode a call adds nothing to the row, so calls of one worker need no order among themselves.
struct MlpPool {
    __nv_bfloat16* xtb;  // [cap][d_in][mb]
    __nv_bfloat16* dzt;  // [cap][d_hidden][mb]
    __nv_bfloat16* xb;   // [cap][mb][d_in]
    int32_t* ycopy;      // [cap][mb]
    float* part;         // [cap][part_stride]: db1 [d_hidden] | dW2 [d_hidden][d_out] | db2 [d_out]
    size_t part_stride;  // floats
    int cap;
    TmapBytes tmap_xt, tmap_dzt, tmap_xb;
    TmapBytes tmap_dzt128, tmap_dzt256;   // dZ^T in boxes of 128 / 256 rows (one TMA copy per operand slot of k_sync_w1)
};
size_t mlp_pool_bytes(const MlpDims& d, int cap);
cudaError_t mlp_pool_init(MlpPool* p, const MlpDims& d, int cap, void* base);
size_t mlp_scratch_bytes(const MlpDims& d);
// Lays the scratch out at `base` (1024-B aligned) and encodes the operand TMA descriptors (host call).
cudaError_t mlp_scratch_init(MlpScratch* s, const MlpDims& d, void* base, __nv_bfloat16* shadow0,
                             __nv_bfloat16* shadow1, const char** err);
// TMA descriptor of the W1 slice of one worker's accumulator row (fp32 [d_in][d_hidden]).
cudaError_t mlp_make_acc_tmap(void* tmap_out, const MlpDims& d, float* acc_row);
// W1 slice of a bf16 copy of the parameters, as a TMA descriptor (boxes of 128 rows x 64 columns).
cudaError_t mlp_make_shadow_tmap(void* tmap_out, const MlpDims& d, __nv_bfloat16* shadow);
// Step 1 + update of the W1 slice straight from the pooled operands of the set's nb micro-batches (slots): the
// weighted average is (sum_j X_j^T dZ_j) / B.  tm_*: descriptors from mlp_make_acc_tmap (x_in, x_out, v: fp32 vectors)
// and mlp_make_shadow_tmap (bf16 copy of x_out, or nullptr).  Needs d_hidden % 128 == 0.  max_ctas > 0 caps the grid.
cudaError_t launch_mlp_sync_w1(const MlpDims& d, const MlpScratch& s, const MlpPool& pool, const MlpSlots& slots, int nb,
                               const void* tm_x_in, const void* tm_x_out, const void* tm_v, const void* tm_shadow,
                               float B, float lr, float mu, float wd, float lambda_dc, float disp_scale, int max_ctas,
                               cudaStream_t stream, bool chained);
// The same step for the rest of the vector (b1, W2, b2) from the pooled per-micro-batch partials; also moves the
// set's device counters cnt[0..W) into log_row and clears them.  x_in, x_out, v, shadow_out: whole flat vectors.
cudaError_t launch_mlp_sync_small(const MlpDims& d, const MlpPool& pool, const MlpSlots& slots, int nb, const float* x_in,
                                  float* x_out, float* v, __nv_bfloat16* shadow_out, float B, float lr, float mu, float wd,
                                  float lambda_dc, float disp_scale, int32_t* cnt, int32_t* log_row, int W, cudaStream_t stream,
                                  bool chained);
// The gradient of a call is enqueued in three parts so that the caller can put them on different streams:
//   cast:  the only part that reads the caller's x_dev / y_dev (bf16 copies and labels into this scratch set);
//   front: forward GEMM, loss, layer-2 backward (writes dzt of this scratch set; adds db2, db1, dW2 into
//          acc_row; bumps cnt);   dw1: the dW1 GEMM, which reads xtb/dzt and adds into the W1 slice.
// shadow: bf16 copy of the published parameters (same flat layout), shadow_idx: which of the two copies it is.
// x_pub: the fp32 parameters.  variant: the ABS_K_MLP_DW1 bit mask of abs_set_launch (0 = dW1 kernel chosen per
// call; 4, 8 force one).  x_is_bf16: the caller's X holds bf16 values (copied as they are) instead of fp32.
// mark(user, kernel_class, -1 - part, stream) is called before a kernel (part: its ordinal within the class for
// one call -- forward class: 0 cast, 1 forward GEMM, 2 bias / ReLU / logits), mark(user, kernel_class, n, stream)
// after its n launches.
typedef void (*MlpMark)(void* user, int kernel_class, int n, cudaStream_t stream);
// pool (ABS_FLAG_MLP_DEFER): the cast writes into pool slots slot0.. instead of the scratch set's; the front kernels
// read them there (pool_slot0..), leave bf16(dZ)^T and the micro-batches' db1 | dW2 | db2 there and add nothing to
// acc_row; cnt is then the counter array of the whole set, and micro-batch j bumps cnt[workers->w[j]], atomically.
// x_devs / y_devs: the caller's buffers of the nb micro-batches (one pointer each; they need not be adjacent).
cudaError_t launch_mlp_cast(const MlpDims& d, const MlpScratch& s, int slot0, int nb, const void* const* x_devs, bool x_is_bf16,
                            const int32_t* const* y_devs, const MlpPool* pool, cudaStream_t stream, bool chained, MlpMark mark,
                            void* user);
cudaError_t launch_mlp_front(const MlpDims& d, const MlpScratch& s, const float* x_pub, const __nv_bfloat16* shadow,
                             int shadow_idx, int nb, bool store, float* acc_row, int32_t* cnt, const MlpPool* pool,
                             int pool_slot0, const MlpWorkers* workers, int variant, cudaStream_t stream, int chain, MlpMark mark,
                             void* user);
// Bias / W2 part of the rows of workers first_worker .. first_worker + n_workers - 1 of one accumulator set from the
// pooled per-micro-batch partials: row = (keep_mask bit ? row : 0) + sum of the partials of the worker's slots
// (owners[q] = worker of slots.s[q]), in list order.
cudaError_t launch_mlp_gather_small(const MlpDims& d, const MlpPool& pool, const MlpSlots& slots, const uint8_t* owners, int n,
                                    int first_worker, int n_workers, unsigned long long keep_mask, float* acc_set,
                                    size_t row_stride, cudaStream_t stream, bool chained);
// nb: a call may carry up to kMlpMaxBatch micro-batches (x_dev [nb][mb][d_in], y_dev [nb][mb]): the front kernels
// take them as an extra grid dimension, and ONE dW1 launch contracts them with K = 64 nb (the accumulator slice is
// read and written once).
// store: the accumulator row holds nothing yet (the worker's first gradient of the iteration): front and dw1
// store their results instead of adding them, and dw1 does not read the accumulator slice at all.
// pool: the operands are those of a deferred-operand pool, micro-batch j in slot slots->s[j] (nb <= kMlpMaxSlots);
// nullptr: slots 0..nb-1 of the scratch set (nb <= kMlpMaxBatch).
cudaError_t launch_mlp_dw1(const MlpDims& d, const MlpScratch& s, const MlpPool* pool, const MlpSlots* slots, float* acc_row,
                           const void* acc_tmap, int nb, bool store, int variant, cudaStream_t stream, bool chained,
                           MlpMark mark, void* user);

}  // namespace abs_sgd
