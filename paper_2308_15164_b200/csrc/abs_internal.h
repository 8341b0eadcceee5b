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

// ---- Step 2: acc_row[j] += g[j], cnt[0] += 1 (Algorithm 1, Step 2) ------------------------
// grad_dtype: ABS_GRAD_F32 / ABS_GRAD_BF16.  P = number of valid elements in g.
cudaError_t launch_accumulate(float* acc_row, const void* g, uint32_t grad_dtype, size_t P, int32_t* cnt,
                              int ctas_per_sm, int num_sms, cudaStream_t stream);

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
};
cudaError_t launch_sync(const SyncArgs& a, int ctas_per_sm, int num_sms, cudaStream_t stream);

// bf16 copy of an fp32 vector (n multiple of 4): used once at init for the MLP weight shadow.
cudaError_t launch_cast_bf16(const float* src, __nv_bfloat16* dst, size_t n, int num_sms, cudaStream_t stream);

// ---- MLP micro-batch gradient (Step 2 with the gradient computed on the device) ----------
struct MlpDims {
    int d_in, d_hidden, d_out, mb;
};
struct alignas(64) TmapBytes {   // storage for one CUtensorMap (encoded on the host, passed by value to kernels)
    unsigned char b[128];
};
struct MlpScratch {      // device pointers carved from the workspace (all hidden-major, see mlp.cu)
    __nv_bfloat16* xb;   // [mb][d_in]            bf16(X)
    __nv_bfloat16* xtb;  // [d_in][mb]            bf16(X)^T: K-major A operand of dW1
    float* zpart;        // [split][d_hidden][mb] split-K partial sums of the forward GEMM
    float* zt;           // [d_hidden][mb]        pre-activations Z^T (fp32)
    __nv_bfloat16* hbt;  // [d_hidden][mb]        bf16(relu(Z))^T
    __nv_bfloat16* dzt;  // [d_hidden][mb]        bf16(dZ)^T: K-major B operand of dW1
    float* lpart;        // [chunks][mb][16]      partial logits
    float* dl;           // [mb][16]              dL (fp32)
    __nv_bfloat16* dlb;  // [mb][16]              bf16(dL)
    int* status;         // device status word: ABS_ETIMEOUT if a bounded wait ran out
    TmapBytes tmap_xt, tmap_dzt;   // dW1 operands
    TmapBytes tmap_xb, tmap_w1[2]; // forward GEMM operands (W1 of each bf16 shadow copy)
};
size_t mlp_scratch_bytes(const MlpDims& d);
// Lays the scratch out at `base` (1024-B aligned) and encodes the operand TMA descriptors (host call).
cudaError_t mlp_scratch_init(MlpScratch* s, const MlpDims& d, void* base, __nv_bfloat16* shadow0,
                             __nv_bfloat16* shadow1, const char** err);
// TMA descriptor of the W1 slice of one worker's accumulator row (fp32 [d_in][d_hidden]).
cudaError_t mlp_make_acc_tmap(void* tmap_out, const MlpDims& d, float* acc_row);
// Enqueues the whole micro-batch gradient; adds into acc_row (flat MLP layout) and bumps cnt.
// shadow: bf16 copy of the published parameters (same flat layout).  x_pub: the fp32 parameters.
// shadow_idx: which of the two shadow copies `shadow` is.  variant: bit 0 = dW1 epilogue by TMA reduce-add
// (else TMA load + add + TMA store); bit 1 = forward GEMM on CUDA cores (cross-check of the tcgen05 one).
// mark(user, kernel_class, 0) is called before a kernel group, mark(user, kernel_class, n) after n launches.
cudaError_t launch_mlp_grad(const MlpDims& d, const MlpScratch& s, const float* x_pub,
                            const __nv_bfloat16* shadow, int shadow_idx, const float* x_dev, const int32_t* y_dev,
                            float* acc_row, const void* acc_tmap, int32_t* cnt, int variant, cudaStream_t stream,
                            void (*mark)(void* user, int kernel_class, int n), void* user);

}  // namespace abs_sgd
