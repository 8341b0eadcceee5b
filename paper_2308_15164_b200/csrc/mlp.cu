// Gradient of one reference batch (Algorithm 1, Step 2) for the 2-layer ReLU MLP with mean
// softmax cross-entropy, accumulated into a worker's buffer.
//
// Per micro-batch X [mb=64, d_in], y [64]; flat parameters W1 [d_in, d_h], b1, W2 [d_h, d_out], b2:
//   Z = bf16(X) bf16(W1) + b1          H = relu(Z)            L = bf16(H) bf16(W2) + b2
//   dL = (softmax(L) - onehot(y)) / mb
//   dW2 = bf16(H)^T bf16(dL)     db2 = sum_rows dL     dH = bf16(dL) bf16(W2)^T
//   dZ = dH * [Z > 0]            db1 = sum_rows dZ     dW1 = bf16(X)^T bf16(dZ)
// Products of bf16 operands are accumulated in fp32; everything else is fp32.
//
// Layout choice: every intermediate is kept HIDDEN-MAJOR ([d_h][mb], i.e. transposed), because
// that makes both operands of the one large contraction, dW1 = X^T dZ (M = d_in, N = d_h,
// K = mb = 64), K-major: A = X^T stored [d_in][64], B = dZ^T stored [d_h][64].  A 64-element
// bf16 row is exactly one 128-byte swizzle row, so each operand tile is one TMA box.
//
// Kernels (five launches per call of 1..4 micro-batches; only the first reads the caller's buffers, the
// others may run on another stream):
//   k_cast_x        X fp32 -> bf16 in both orientations
//   (k_fwd_fused    k_fwd1_tcgen05 + k_fwd2 in one kernel: the K splits of a hidden tile form a thread-block cluster
//                   and are added up through distributed shared memory; same bits, selectable)
//   k_fwd1_tcgen05  Z^T partials = W1^T X^T, split over d_in, on tcgen05 (W1 as an MN-major operand)
//   (k_fwd1         the same on CUDA cores, kept as a cross-check selectable through abs_set_launch)
//   k_fwd2          Z = sum of partials + b1, bf16(H), partial logits per 32 hidden units; the last CTA of
//                   each group of 8 ("last CTA done" ticket) sums the group's partial logits in a fixed order
//   k_bwd           every CTA: logits = sum of group partials + b2, softmax, dL (CTA 0: db2 += ...); then
//                   dH, dZ, bf16(dZ)^T, db1 += ..., dW2 += ..., b_i += 1
//   dW1 = X^T dZ on the 5th-gen tensor cores (TMEM accumulator), one of (chosen per call, see launch_mlp_dw1):
//   k_dw1_ring      persistent, warp-specialised, K-batched: operand ring in shared memory, two TMEM
//                   accumulators, finished tiles leave by TMA store (a worker's first gradient of an iteration)
//                   or TMA reduce-add; 128 x 64 or 128 x 128 tiles
//   k_dw1_regs      one 128 x 64 tile per CTA, the accumulator tile prefetched into registers, K-batched
//   k_dw1_tcgen05   one tile per CTA, the accumulator tile by TMA load / add in shared memory / TMA store
//                   (or TMA reduce-add); the first version, kept selectable
#include <cuda.h>

#include <cstdio>

#include "abs_internal.h"

namespace abs_sgd {

namespace {

constexpr int kMB = 64;          // samples per micro-batch = K of the dW1 contraction
constexpr int kOutPad = 16;      // logits / dL rows are padded to 16 columns
constexpr int kSplitK = 4;       // forward GEMM: d_in is split into at most this many partial sums
constexpr int kHB = 32;          // hidden units per CTA in k_fwd2 / k_bwd
constexpr int kGroup = 8;        // CTAs per first-level group of the logit reduction
constexpr int kMaxBatch = kMlpMaxBatch;   // micro-batches one call may carry (grid dimension of the front kernels)

__device__ __forceinline__ float bf16_to_f(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b) {
    __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&p);
}

// --------------------------------------------------------------------------------------------
// X [64][d_in] fp32  ->  xb [64][d_in] bf16  and  xtb [d_in][64] bf16.   CTA: 16 columns.
// Also copies the labels, so that the caller's buffers are read by this kernel only (the rest of
// the gradient may run on another stream after the caller's stream has moved on).
// --------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_cast_x(const float* __restrict__ x, const int32_t* __restrict__ y,
                                                __nv_bfloat16* __restrict__ xb, __nv_bfloat16* __restrict__ xtb,
                                                int32_t* __restrict__ ycopy, int d_in) {
    __shared__ __nv_bfloat16 tile[16][kMB + 8];
    const int c0 = blockIdx.x * 16;
    if (blockIdx.x == 0 && threadIdx.x < kMB) ycopy[blockIdx.y * kMB + threadIdx.x] = y[blockIdx.y * kMB + threadIdx.x];
    x += (size_t)blockIdx.y * kMB * d_in;      // micro-batch blockIdx.y of the call
    xb += (size_t)blockIdx.y * kMB * d_in;
    xtb += (size_t)blockIdx.y * d_in * kMB;
    {
        const int r = threadIdx.x / 4, q = threadIdx.x % 4;
        const float4 v = *reinterpret_cast<const float4*>(x + (size_t)r * d_in + c0 + 4 * q);
        uint2 pk;
        pk.x = pack_bf16x2(v.x, v.y);
        pk.y = pack_bf16x2(v.z, v.w);
        *reinterpret_cast<uint2*>(xb + (size_t)r * d_in + c0 + 4 * q) = pk;
        tile[4 * q + 0][r] = __float2bfloat16_rn(v.x);
        tile[4 * q + 1][r] = __float2bfloat16_rn(v.y);
        tile[4 * q + 2][r] = __float2bfloat16_rn(v.z);
        tile[4 * q + 3][r] = __float2bfloat16_rn(v.w);
    }
    __syncthreads();
    {
        const int c = threadIdx.x / 16, r4 = (threadIdx.x % 16) * 4;
        uint2 pk = *reinterpret_cast<const uint2*>(&tile[c][r4]);
        *reinterpret_cast<uint2*>(xtb + (size_t)(c0 + c) * kMB + r4) = pk;
    }
}

// --------------------------------------------------------------------------------------------
// Forward GEMM, CUDA cores (cross-check):  zpart[s][h][r] = sum_{k in split s} W1b[k][h] * xb[r][k]
// CTA tile: 64 hidden x 64 samples, 256 threads, 4x4 outputs per thread; gridDim.y = number of splits.
// --------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_fwd1(const __nv_bfloat16* __restrict__ w1b, const __nv_bfloat16* __restrict__ xb,
                                              float* __restrict__ zpart, int d_in, int d_h) {
    constexpr int KT = 32;
    __shared__ float sw[KT][64 + 4];   // [k][h]
    __shared__ float sx[KT][64 + 4];   // [k][r]
    const int h0 = blockIdx.x * 64;
    const int s = blockIdx.y;
    xb += (size_t)blockIdx.z * kMB * d_in;                   // micro-batch blockIdx.z of the call
    zpart += (size_t)blockIdx.z * kSplitK * d_h * kMB;
    const int k_per = d_in / (int)gridDim.y;
    const int kbeg = s * k_per, kend = kbeg + k_per;
    const int th = threadIdx.x / 16, tr = threadIdx.x % 16;   // 16 x 16 threads, 4 h x 4 r each
    float acc[4][4] = {};
    for (int k0 = kbeg; k0 < kend; k0 += KT) {
        for (int e = threadIdx.x; e < KT * 64; e += 256) {
            const int k = e / 64, h = e % 64;
            sw[k][h] = bf16_to_f(w1b[(size_t)(k0 + k) * d_h + h0 + h]);
        }
        for (int e = threadIdx.x; e < KT * 64; e += 256) {
            const int r = e / KT, k = e % KT;
            sx[k][r] = bf16_to_f(xb[(size_t)r * d_in + k0 + k]);
        }
        __syncthreads();
#pragma unroll 8
        for (int k = 0; k < KT; ++k) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = sw[k][th * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = sx[k][tr * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
    float* out = zpart + (size_t)s * d_h * kMB;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float4 v = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
        *reinterpret_cast<float4*>(out + (size_t)(h0 + th * 4 + i) * kMB + tr * 4) = v;
    }
}

// --------------------------------------------------------------------------------------------
// k_fwd2: per CTA 32 hidden units x 64 samples.
//   phase 1 (thread = sample r, 8 hidden units): Z = sum_s zpart + b1 ; hb = bf16(relu(Z)) -> hbt
//   phase 2 (thread = sample r, 4 logits):        partial logits of these 32 hidden units -> lpart[cta]
//   tail: the last CTA of each group of 8 sums the group's partials (fixed order) -> gpart[group].
//         The remaining sum over the groups is cheap (n_groups x 4 KB) and is done by every CTA of k_bwd.
// tickets[0 .. n_groups) are the group tickets: all zero on entry and reset before exit.
// --------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_fwd2(const float* zpart, int nsplit, const float* __restrict__ b1,
                                              const __nv_bfloat16* __restrict__ w2b, __nv_bfloat16* hbt,
                                              float* lpart, float* gpart, unsigned int* tickets, int d_h, int d_out) {
    __shared__ float sh[kHB][kMB + 1];
    __shared__ float sw2[kHB][kOutPad];
    __shared__ unsigned int s_last;
    const int h_beg = blockIdx.x * kHB;
    const int n_cta = gridDim.x;
    {   // micro-batch blockIdx.y of the call: its own slices of every scratch array
        const int j = blockIdx.y, n_groups = (n_cta + kGroup - 1) / kGroup;
        zpart += (size_t)j * kSplitK * d_h * kMB;
        hbt += (size_t)j * d_h * kMB;
        lpart += (size_t)j * n_cta * kMB * kOutPad;
        gpart += (size_t)j * n_groups * kMB * kOutPad;
        tickets += (size_t)j * n_groups;
    }

    for (int e = threadIdx.x; e < kHB * kOutPad; e += 256) {
        const int hl = e / kOutPad, o = e % kOutPad;
        sw2[hl][o] = o < d_out ? bf16_to_f(w2b[(size_t)(h_beg + hl) * d_out + o]) : 0.f;
    }
    {
        const int r = threadIdx.x % kMB, g = threadIdx.x / kMB;
        float z[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) z[j] = b1[h_beg + g * 8 + j];
        for (int s = 0; s < nsplit; ++s)
#pragma unroll
            for (int j = 0; j < 8; ++j) z[j] += zpart[((size_t)s * d_h + h_beg + g * 8 + j) * kMB + r];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const __nv_bfloat16 hb = __float2bfloat16_rn(z[j] > 0.f ? z[j] : 0.f);
            hbt[(size_t)(h_beg + g * 8 + j) * kMB + r] = hb;
            sh[g * 8 + j][r] = bf16_to_f(hb);
        }
    }
    __syncthreads();
    {
        const int r = threadIdx.x / 4, og = threadIdx.x % 4;
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll 8
        for (int hl = 0; hl < kHB; ++hl) {
            const float hv = sh[hl][r];
            a0 = fmaf(hv, sw2[hl][4 * og + 0], a0);
            a1 = fmaf(hv, sw2[hl][4 * og + 1], a1);
            a2 = fmaf(hv, sw2[hl][4 * og + 2], a2);
            a3 = fmaf(hv, sw2[hl][4 * og + 3], a3);
        }
        reinterpret_cast<float4*>(lpart)[(size_t)blockIdx.x * (kMB * kOutPad / 4) + threadIdx.x] = make_float4(a0, a1, a2, a3);
    }
    // ---- first level: last CTA of the group reduces the group's partial logits
    const int group = blockIdx.x / kGroup;
    const int g_first = group * kGroup;
    const int g_count = min(kGroup, n_cta - g_first);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = (atomicAdd(&tickets[group], 1u) == (unsigned)(g_count - 1));
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int c = 0; c < g_count; ++c) {
            const float4 v = __ldcg(reinterpret_cast<const float4*>(lpart) + (size_t)(g_first + c) * (kMB * kOutPad / 4) + threadIdx.x);
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        reinterpret_cast<float4*>(gpart)[(size_t)group * (kMB * kOutPad / 4) + threadIdx.x] = acc;
    }
    if (threadIdx.x == 0) tickets[group] = 0u;   // ready for the next launch
}

// --------------------------------------------------------------------------------------------
// k_bwd: per CTA 32 hidden units x 64 samples.
//   prologue (every CTA, identical result): logits = sum over groups of gpart + b2 (fixed order);
//            dL = (softmax - onehot)/mb, 4 lanes per sample row (max and sum by shuffles); CTA 0 also adds
//            db2 = sum_r dL
//   phase 1 (thread = sample r, 8 hidden units): dH = sum_o bf16(dL)[r][o] W2b[h][o]; dZ = dH * [H > 0]
//            (H > 0 exactly when Z > 0); dzt[h][r] = bf16(dZ)
//   phase 2 (thread = hidden unit, 2 outputs): dW2[h][o] += sum_r bf16(H)[h][r] bf16(dL)[r][o],
//            db1[h] += sum_r dZ[h][r]   (fixed summation order over r)
// --------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_bwd(const __nv_bfloat16* hbt, const float* gpart, int n_groups,
                                             const float* __restrict__ b2, const int32_t* y,
                                             const __nv_bfloat16* __restrict__ w2b, __nv_bfloat16* dzt, float* bpart,
                                             unsigned int* tickets_b, float* acc_b1, float* acc_w2, float* acc_b2,
                                             int32_t* cnt, int d_h, int d_out, int store) {
    __shared__ float sdl[kMB][kOutPad + 1];     // bf16(dL) as float
    __shared__ float sdl32[kMB][kOutPad + 1];   // dL unrounded (CTA 0: db2)
    __shared__ float sw2[kHB][kOutPad];
    __shared__ float sh[kHB][kMB + 1];
    __shared__ float sdz[kHB][kMB + 1];
    __shared__ unsigned int s_last;
    const int h_beg = blockIdx.x * kHB;
    const int jb = blockIdx.y, nb = gridDim.y;       // micro-batch of this CTA, micro-batches in the call
    hbt += (size_t)jb * d_h * kMB;
    dzt += (size_t)jb * d_h * kMB;
    gpart += (size_t)jb * n_groups * kMB * kOutPad;
    y += (size_t)jb * kMB;
    const int r = threadIdx.x % kMB, g = threadIdx.x / kMB;
    float hv[8];                                     // issued first: independent of the logit sums below
#pragma unroll
    for (int j = 0; j < 8; ++j) hv[j] = bf16_to_f(hbt[(size_t)(h_beg + g * 8 + j) * kMB + r]);
    {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int c = 0; c < n_groups; ++c) {
            const float4 v = reinterpret_cast<const float4*>(gpart)[(size_t)c * (kMB * kOutPad / 4) + threadIdx.x];
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        // softmax and dL on the registers that hold the sums: 4 adjacent lanes share a sample row
        const int rr = threadIdx.x / 4, og = threadIdx.x % 4;
        float l[4] = {acc.x, acc.y, acc.z, acc.w};
        float mx = -INFINITY;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int o = 4 * og + j;
            l[j] = o < d_out ? l[j] + b2[o] : -INFINITY;
            mx = fmaxf(mx, l[j]);
        }
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        float den = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            l[j] = (4 * og + j) < d_out ? expf(l[j] - mx) : 0.f;
            den += l[j];
        }
        den += __shfl_xor_sync(0xffffffffu, den, 1);
        den += __shfl_xor_sync(0xffffffffu, den, 2);
        const int yr = y[rr];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int o = 4 * og + j;
            const float gl = o < d_out ? (l[j] / den - (o == yr ? 1.f : 0.f)) * (1.0f / kMB) : 0.f;
            sdl32[rr][o] = gl;
            sdl[rr][o] = bf16_to_f(__float2bfloat16_rn(gl));
        }
    }
    for (int e = threadIdx.x; e < kHB * kOutPad; e += 256) {
        const int hl = e / kOutPad, o = e % kOutPad;
        sw2[hl][o] = o < d_out ? bf16_to_f(w2b[(size_t)(h_beg + hl) * d_out + o]) : 0.f;
    }
    __syncthreads();
    float db2 = 0.f;                                 // CTA column 0, thread o < d_out: sum_r dL[r][o]
    if (blockIdx.x == 0 && threadIdx.x < d_out)
        for (int rr = 0; rr < kMB; ++rr) db2 += sdl32[rr][threadIdx.x];
    {
        float dl[kOutPad];
#pragma unroll
        for (int o = 0; o < kOutPad; ++o) dl[o] = sdl[r][o];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int hl = g * 8 + j;
            float dh = 0.f;
#pragma unroll
            for (int o = 0; o < kOutPad; ++o) dh = fmaf(dl[o], sw2[hl][o], dh);
            const float dz = hv[j] > 0.f ? dh : 0.f;
            dzt[(size_t)(h_beg + hl) * kMB + r] = __float2bfloat16_rn(dz);
            sh[hl][r] = hv[j];
            sdz[hl][r] = dz;
        }
    }
    __syncthreads();
    {
        const int hl = threadIdx.x / 8, slot = threadIdx.x % 8;   // dW2 outputs `slot` and `slot + 8`; slot 0 also db1
        float a = 0.f, b = 0.f, c = 0.f;
#pragma unroll 8
        for (int rr = 0; rr < kMB; ++rr) {
            const float h = sh[hl][rr];
            a = fmaf(h, sdl[rr][slot], a);
            b = fmaf(h, sdl[rr][slot + 8], b);
            if (slot == 0) c += sdz[hl][rr];
        }
        const int h = h_beg + hl;
        if (nb > 1) {
            // Several micro-batches add into the same accumulator entries: every CTA parks its partial sums, and
            // the last of the nb CTAs of this hidden chunk ("last CTA done" ticket) adds them up in micro-batch
            // order and does the one read-modify-write -- a fixed summation order, no atomics on the data.
            float* mine = bpart + ((size_t)(jb * gridDim.x + blockIdx.x) * 4) * 256;
            mine[threadIdx.x] = a; mine[256 + threadIdx.x] = b; mine[512 + threadIdx.x] = c; mine[768 + threadIdx.x] = db2;
            __threadfence();
            __syncthreads();
            if (threadIdx.x == 0) s_last = (atomicAdd(&tickets_b[blockIdx.x], 1u) == (unsigned)(nb - 1));
            __syncthreads();
            if (!s_last) return;
            __threadfence();
            a = b = c = db2 = 0.f;
            for (int q = 0; q < nb; ++q) {
                const float* p = bpart + ((size_t)(q * gridDim.x + blockIdx.x) * 4) * 256;
                a += __ldcg(p + threadIdx.x); b += __ldcg(p + 256 + threadIdx.x);
                c += __ldcg(p + 512 + threadIdx.x); db2 += __ldcg(p + 768 + threadIdx.x);
            }
            if (threadIdx.x == 0) tickets_b[blockIdx.x] = 0u;
        }
        if (store) {   // a worker's first gradient of the iteration: the slices hold nothing yet
            if (slot < d_out) acc_w2[(size_t)h * d_out + slot] = a;
            if (slot + 8 < d_out) acc_w2[(size_t)h * d_out + slot + 8] = b;
            if (slot == 0) acc_b1[h] = c;
            if (blockIdx.x == 0 && threadIdx.x < d_out) acc_b2[threadIdx.x] = db2;
        } else {
            if (slot < d_out) acc_w2[(size_t)h * d_out + slot] += a;
            if (slot + 8 < d_out) acc_w2[(size_t)h * d_out + slot + 8] += b;
            if (slot == 0) acc_b1[h] += c;
            if (blockIdx.x == 0 && threadIdx.x < d_out) acc_b2[threadIdx.x] += db2;
        }
        if (blockIdx.x == 0 && threadIdx.x == 0) cnt[0] += nb;   // M_t^i += nb * M_r
    }
}

// ============================================================================================
// tcgen05 / TMA / mbarrier helpers
// ============================================================================================
constexpr uint32_t kSpinLimit = 1u << 22;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Bounded wait: gives up after kSpinLimit polls and reports failure instead of hanging.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    const uint32_t addr = smem_u32(bar);
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
            : "=r"(ok) : "r"(addr), "r"(parity) : "memory");
        if (ok) return true;
    }
    return false;
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* tm, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* tm, const void* src, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(tm)), "r"(smem_u32(src)), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* tm, const void* src, int x, int y) {
    asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(tm)), "r"(smem_u32(src)), "r"(x), "r"(y) : "memory");
}

// Shared-memory matrix descriptor for a K-major bf16 tile stored as 128-byte rows with the
// 128-byte swizzle (what a TMA box of 64 bf16 x rows produces): 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_k_sw128(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);          // start address
    d |= (uint64_t)1 << 16;                               // leading-dim byte offset (unused with swizzle)
    d |= (uint64_t)(1024 >> 4) << 32;                     // stride-dim byte offset: 8 rows x 128 B
    d |= (uint64_t)1 << 46;                               // descriptor version (sm_100)
    d |= (uint64_t)2 << 61;                               // 128-byte swizzle
    return d;
}
// Same for an MN-major tile: a TMA box of 64 MN-elements x 64 k (128-byte rows, 128-byte swizzle).
// Groups of 8 k-rows are 1024 bytes apart (stride offset); the next 64-wide MN block is `lbo_bytes` away.
__device__ __forceinline__ uint64_t umma_desc_mn_sw128(uint32_t smem_addr, uint32_t lbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);
    d |= (uint64_t)(lbo_bytes >> 4) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Instruction descriptor: D = f32, A = B = bf16, both K-major (set bit 15 for an MN-major A), M x N tile.
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int M, int N) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
        " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld_32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
// Adds the 32 TMEM values of one row into that row of a swizzled [128][32] fp32 panel in shared
// memory (row = 128 bytes; 16-byte chunk j sits at position j ^ (row % 8), as the TMA box wrote it).
template <bool kAdd>
__device__ __forceinline__ void panel_row_update(float* panel, int row, const uint32_t (&v)[32]) {
    float4* prow = reinterpret_cast<float4*>(panel + row * 32);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        float4* q = prow + (j ^ (row & 7));
        float4 d = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]), __uint_as_float(v[4 * j + 2]),
                               __uint_as_float(v[4 * j + 3]));
        if (kAdd) {
            const float4 c = *q;
            d.x += c.x; d.y += c.y; d.z += c.z; d.w += c.w;
        }
        *q = d;
    }
}

// ============================================================================================
// dW1 = X^T dZ on tcgen05.  One CTA per 128 x kDwN output tile; K = 64 = four UMMA steps.
// ============================================================================================
constexpr int kTileM = 128;
constexpr int kDwN = 64;
constexpr int kPanels = kDwN / 32;

struct DwSmem {
    alignas(1024) uint8_t a[kTileM * 128];            // A tile  [128 m][64 k] bf16, swizzled rows
    alignas(1024) uint8_t b[kDwN * 128];              // B tile  [kDwN n][64 k] bf16
    alignas(1024) float c[kPanels][kTileM * 32];      // accumulator tile as column panels [128][32] fp32, swizzled rows
    alignas(8) uint64_t bar_ab;
    uint64_t bar_c;
    uint64_t bar_mma;
    uint32_t tmem_base;
    uint32_t failed;
};

template <bool kReduce>
__global__ void __launch_bounds__(128) k_dw1_tcgen05(const __grid_constant__ CUtensorMap tm_xt,
                                                     const __grid_constant__ CUtensorMap tm_dzt,
                                                     const __grid_constant__ CUtensorMap tm_acc, int store,
                                                     int* status) {
    // store != 0: the accumulator slice is known to hold nothing yet (a worker's first gradient of the
    // iteration): the tile is not read, the product is stored instead of added.
    extern __shared__ uint8_t smem_raw[];
    DwSmem& s = *reinterpret_cast<DwSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x / 32;
    const bool load_c = !kReduce && !store;
    const int n0 = blockIdx.x * kDwN;     // hidden offset
    const int m0 = blockIdx.y * kTileM;   // input-feature offset

    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s.tmem_base)), "r"(kDwN) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (threadIdx.x == 0) {
        mbar_init(&s.bar_ab, 1);
        mbar_init(&s.bar_c, 1);
        mbar_init(&s.bar_mma, 1);
        s.failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s.tmem_base;

    if (threadIdx.x == 0) {
        mbar_expect_tx(&s.bar_ab, kTileM * 128 + kDwN * 128);
        tma_load_2d(s.a, &tm_xt, 0, m0, &s.bar_ab);
        tma_load_2d(s.b, &tm_dzt, 0, n0, &s.bar_ab);
        if (load_c) {   // the accumulator tile streams in while the MMA runs
            mbar_expect_tx(&s.bar_c, kTileM * kDwN * 4);
#pragma unroll
            for (int p = 0; p < kPanels; ++p) tma_load_2d(s.c[p], &tm_acc, n0 + p * 32, m0, &s.bar_c);
        }
        if (mbar_wait(&s.bar_ab, 0)) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint64_t da = umma_desc_k_sw128(smem_u32(s.a));
            const uint64_t db = umma_desc_k_sw128(smem_u32(s.b));
            constexpr uint32_t idesc = umma_idesc_bf16(kTileM, kDwN);
#pragma unroll
            for (int k = 0; k < kMB / 16; ++k)   // K advances by 16 bf16 = 32 bytes: +2 in the address field
                umma_bf16(tmem, da + 2 * k, db + 2 * k, idesc, k > 0);
            umma_commit(&s.bar_mma);
        } else {
            s.failed = 1;
        }
    }
    __syncwarp();

    bool ok = mbar_wait(&s.bar_mma, 0);
    if (load_c) ok = mbar_wait(&s.bar_c, 0) && ok;
    ok = __all_sync(0xffffffffu, ok);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (ok) {
        const int row = threadIdx.x;                    // TMEM lane = output row
#pragma unroll 1
        for (int p = 0; p < kPanels; ++p) {
            uint32_t v[32];
            tmem_ld_32(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)(p * 32), v);
            if (load_c) panel_row_update<true>(s.c[p], row, v);
            else panel_row_update<false>(s.c[p], row, v);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // smem writes -> visible to the TMA engine
    } else {
        s.failed = 1;
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x == 0) {
        if (!s.failed) {
#pragma unroll
            for (int p = 0; p < kPanels; ++p) {
                if (kReduce && !store) tma_reduce_add_2d(&tm_acc, s.c[p], n0 + p * 32, m0);
                else tma_store_2d(&tm_acc, s.c[p], n0 + p * 32, m0);
            }
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            // shared memory may be released once the engine has read it; the global writes complete on their own
            asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        } else {
            atomicExch(status, ABS_ETIMEOUT);
            // give copies that may still be in flight a bounded chance to land before smem is released
            mbar_wait(&s.bar_ab, 0);
            if (load_c) mbar_wait(&s.bar_c, 0);
        }
    }
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kDwN) : "memory");
    }
}

// ============================================================================================
// dW1 with a register-prefetched accumulator tile, optionally K-batched.  Same tile as
// k_dw1_tcgen05, but the fp32 accumulator tile never goes through TMA: every thread loads its
// 8 float4 of the tile with plain coalesced loads at kernel entry (all in flight while the
// operands arrive and the MMAs run), the TMEM result is transposed through a padded shared-memory
// tile, and the sums go back with coalesced stores.
// K batching: the operands of nb (1..kMaxBatch) micro-batches are stacked along K, so one launch
// computes  acc += sum_j X_j^T dZ_j  (K = 64 nb) and the accumulator slice is read and written once
// for nb micro-batches instead of nb times -- the kernel is bound by that traffic, not by the MMAs.
// Operand j lives at row offset j*d_in (X^T) / j*d_h (dZ^T) of the stacked operand tensors.
// 256 threads: warps 0-3 read TMEM columns 0..31 of their lane quarter, warps 4-7 columns 32..63.
// ============================================================================================
constexpr int kDwPitch = kDwN + 4;   // floats per row of the staging tile (pitch 272 B: conflict-free float4 rows)
constexpr int kDwOperandBytes = kTileM * 128 + kDwN * 128;   // A tile 16 KB + B tile 8 KB per micro-batch
constexpr int kDwStagingBytes = kTileM * kDwPitch * 4;       // 34 KB

// Dynamic shared memory: [operands of nb micro-batches | reused as the staging tile once the MMAs are done]
// followed by this control block.
struct DwRegCtl {
    alignas(8) uint64_t bar_ab;
    uint64_t bar_mma;
    uint32_t tmem_base;
    uint32_t failed;
};
__host__ __device__ constexpr int dw_regs_buf_bytes(int nb) {
    return (nb * kDwOperandBytes > kDwStagingBytes ? nb * kDwOperandBytes : kDwStagingBytes + 1023) / 1024 * 1024;
}

__global__ void __launch_bounds__(256) k_dw1_regs(const __grid_constant__ CUtensorMap tm_xt,
                                                  const __grid_constant__ CUtensorMap tm_dzt, float* acc_w1, int d_in,
                                                  int ld, int nb, int store, int* status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* buf = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    DwRegCtl& s = *reinterpret_cast<DwRegCtl*>(buf + dw_regs_buf_bytes(nb));
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int n0 = blockIdx.x * kDwN, m0 = blockIdx.y * kTileM;
    constexpr int kC4 = kDwN / 4;                   // float4 per tile row
    constexpr int kPer = kTileM * kC4 / 256;        // float4 per thread (8)

    // accumulator tile -> registers, coalesced (a warp covers 32 consecutive float4 = 2 rows of 256 B)
    float4* gbase = reinterpret_cast<float4*>(acc_w1 + (size_t)m0 * ld + n0);
    const size_t ld4 = (size_t)ld / 4;
    float4 c[kPer];
#pragma unroll
    for (int k = 0; k < kPer; ++k) {
        const int e = threadIdx.x + 256 * k;
        c[k] = store ? make_float4(0.f, 0.f, 0.f, 0.f) : gbase[(size_t)(e / kC4) * ld4 + (e % kC4)];   // store: see k_dw1_tcgen05
    }

    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s.tmem_base)), "r"(kDwN) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (threadIdx.x == 0) {
        mbar_init(&s.bar_ab, 1);
        mbar_init(&s.bar_mma, 1);
        s.failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s.tmem_base;

    if (threadIdx.x == 0) {
        mbar_expect_tx(&s.bar_ab, nb * kDwOperandBytes);
        for (int j = 0; j < nb; ++j) {
            tma_load_2d(buf + j * kDwOperandBytes, &tm_xt, 0, j * d_in + m0, &s.bar_ab);
            tma_load_2d(buf + j * kDwOperandBytes + kTileM * 128, &tm_dzt, 0, j * ld + n0, &s.bar_ab);
        }
        if (mbar_wait(&s.bar_ab, 0)) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            constexpr uint32_t idesc = umma_idesc_bf16(kTileM, kDwN);
            for (int j = 0; j < nb; ++j) {
                const uint32_t a0 = smem_u32(buf + j * kDwOperandBytes);
                const uint64_t da = umma_desc_k_sw128(a0), db = umma_desc_k_sw128(a0 + kTileM * 128);
#pragma unroll
                for (int k = 0; k < kMB / 16; ++k) umma_bf16(tmem, da + 2 * k, db + 2 * k, idesc, (j > 0 || k > 0));
            }
            umma_commit(&s.bar_mma);
        } else {
            s.failed = 1;
        }
    }
    __syncwarp();

    bool ok = mbar_wait(&s.bar_mma, 0);
    ok = __all_sync(0xffffffffu, ok);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (ok) {
        const int q = warp % 4, half = warp / 4;
        const int row = q * 32 + lane;
        uint32_t v[32];
        tmem_ld_32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(half * 32), v);
        float4* drow = reinterpret_cast<float4*>(reinterpret_cast<float*>(buf) + row * kDwPitch + half * 32);
#pragma unroll
        for (int j = 0; j < 8; ++j)
            drow[j] = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]), __uint_as_float(v[4 * j + 2]),
                                  __uint_as_float(v[4 * j + 3]));
    } else {
        s.failed = 1;
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (!*reinterpret_cast<volatile uint32_t*>(&s.failed)) {
#pragma unroll
        for (int k = 0; k < kPer; ++k) {
            const int e = threadIdx.x + 256 * k;
            const float4 d = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(buf) + (e / kC4) * kDwPitch + (e % kC4) * 4);
            float4 o = c[k];
            o.x += d.x; o.y += d.y; o.z += d.z; o.w += d.w;
            gbase[(size_t)(e / kC4) * ld4 + (e % kC4)] = o;
        }
    } else if (threadIdx.x == 0) {
        atomicExch(status, ABS_ETIMEOUT);
        mbar_wait(&s.bar_ab, 0);   // bounded chance for the operand copies to land before smem is released
    }
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kDwN) : "memory");
    }
}

// ============================================================================================
// dW1, persistent warp-specialised version, K-batched.  One CTA per SM walks over its share of
// the 128 x 64 output tiles (hidden index fastest, so neighbouring CTAs share the X^T tile in L2):
//   warp 0 (one lane)   TMA producer: one ring slot = the operands {A, B} of one micro-batch of one
//                       tile; the slots of the next tiles fill while the current one is computed
//   warp 1 (one lane)   MMA issuer: 4 nb x tcgen05.mma per tile into one of two TMEM accumulators;
//                       each slot is handed back by a tcgen05.commit on its `empty` barrier
//   warps 2..5          epilogue: tcgen05.ld -> registers (the accumulator is free again), write the
//                       tile into one of kRingC swizzled staging tiles, then ONE thread issues the TMA
//                       store (store mode) or TMA reduce-add (fp32 add done by the memory system)
// The accumulator slice never passes through the SM on its way in: no CTA ever waits for DRAM, the
// only loads are the (L2-resident) bf16 operands.
// ============================================================================================
// kN = 64: 128 x 64 tiles (1536 of them at 3072 x 4096: even shares for 148 CTAs); kN = 128: 128 x 128 tiles, a
// third less operand traffic per output element -- the choice for K-batched calls, which are bound by it.
// kLight: half the operand slots and one outgoing staging tile (104 / 96 KB instead of 208 / 224 KB), so that a
// forward-GEMM CTA of another worker's call fits on the same SM.  Alone on the GPU the deep form is faster
// (K = 256: 20.5 against 24.7 us); with several workers' calls in flight the light forms are (16.5 -> 15.6 us per
// micro-batch with batch calls), because forward and dW1 CTAs then run side by side instead of taking turns.
template <int kN, bool kLight = false>
struct DwRingCfg {
    static constexpr int kSlotBytes = kTileM * 128 + kN * 128;   // [A 128 x 64 | B kN x 64] bf16
    static constexpr int kOps = kLight ? (kN == 64 ? 3 : 2) : (kN == 64 ? 6 : 5);   // operand slots
    static constexpr int kC = kLight ? 1 : 2;                    // outgoing staging tiles of 32 KB (128 x 64 fp32)
};

template <int kN, bool kLight = false>
struct DwRingSmem {
    alignas(1024) uint8_t op[DwRingCfg<kN, kLight>::kOps][DwRingCfg<kN, kLight>::kSlotBytes];   // swizzled 128-byte rows
    alignas(1024) float c[DwRingCfg<kN, kLight>::kC][kTileM * kDwN];   // two [128][32] fp32 column panels each, swizzled rows
    alignas(8) uint64_t op_full[DwRingCfg<kN, kLight>::kOps];
    uint64_t op_empty[DwRingCfg<kN, kLight>::kOps];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint32_t tmem_base;
    uint32_t failed;
    uint32_t stop[2];
};

template <int kN, bool kLight = false>
__global__ void __launch_bounds__(192) k_dw1_ring(const __grid_constant__ CUtensorMap tm_xt,
                                                  const __grid_constant__ CUtensorMap tm_dzt,
                                                  const __grid_constant__ CUtensorMap tm_acc, int n_tiles_n, int n_tiles,
                                                  int d_in, int ld, int nb, int store, int* status) {
    constexpr int kRingOps = DwRingCfg<kN, kLight>::kOps, kSlotBytes = DwRingCfg<kN, kLight>::kSlotBytes;
    constexpr int kRingC = DwRingCfg<kN, kLight>::kC;
    constexpr int kHalves = kN / kDwN;               // the epilogue works on 64-column pieces of the tile
    extern __shared__ uint8_t smem_raw[];
    DwRingSmem<kN, kLight>& s = *reinterpret_cast<DwRingSmem<kN, kLight>*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int my_tiles = (n_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;

    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s.tmem_base)), "r"(2 * kN) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (threadIdx.x == 0) {
        for (int i = 0; i < kRingOps; ++i) {
            mbar_init(&s.op_full[i], 1);
            mbar_init(&s.op_empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&s.acc_full[i], 1);
            mbar_init(&s.acc_empty[i], 128);
        }
        s.failed = 0;
        s.stop[0] = s.stop[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s.tmem_base;

    if (warp == 0) {
        if (lane == 0) {                             // ---- TMA producer
            int q = 0;                               // running slot count
            for (int i = 0; i < my_tiles && !s.failed; ++i) {
                const int t = (int)blockIdx.x + i * (int)gridDim.x;
                const int n0 = (t % n_tiles_n) * kN, m0 = (t / n_tiles_n) * kTileM;
                for (int j = 0; j < nb; ++j, ++q) {
                    const int st = q % kRingOps;
                    if (q >= kRingOps && !mbar_wait(&s.op_empty[st], ((q / kRingOps) - 1) & 1)) { s.failed = 1; break; }
                    mbar_expect_tx(&s.op_full[st], kSlotBytes);
                    tma_load_2d(s.op[st], &tm_xt, 0, j * d_in + m0, &s.op_full[st]);
#pragma unroll
                    for (int b = 0; b < kHalves; ++b)   // 64-row boxes, 8 KB apart: one K-major B operand of kN rows
                        tma_load_2d(s.op[st] + kTileM * 128 + b * (kDwN * 128), &tm_dzt, 0, j * ld + n0 + b * kDwN, &s.op_full[st]);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {                             // ---- MMA issuer
            constexpr uint32_t idesc = umma_idesc_bf16(kTileM, kN);
            int q = 0;
            bool ok = true;
            for (int i = 0; i < my_tiles && ok; ++i) {
                const int ab = i & 1;
                if (i >= 2 && !mbar_wait(&s.acc_empty[ab], ((i / 2) - 1) & 1)) { ok = false; break; }
                for (int j = 0; j < nb; ++j, ++q) {
                    const int st = q % kRingOps;
                    if (!mbar_wait(&s.op_full[st], (q / kRingOps) & 1)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a0 = smem_u32(s.op[st]);
                    const uint64_t da = umma_desc_k_sw128(a0), db = umma_desc_k_sw128(a0 + kTileM * 128);
#pragma unroll
                    for (int k = 0; k < kMB / 16; ++k) umma_bf16(tmem + ab * kN, da + 2 * k, db + 2 * k, idesc, (j > 0 || k > 0));
                    umma_commit(&s.op_empty[st]);    // the slot is free once these MMAs have read it
                }
                if (ok) umma_commit(&s.acc_full[ab]);
            }
            if (!ok) s.failed = 1;
        }
    } else {                                         // ---- epilogue warps 2..5
        const int qd = warp % 4;                     // TMEM lane quarter this warp may access
        const int row = qd * 32 + lane;
        const bool leader = (threadIdx.x == 64);
        bool stopped = false;
        for (int i = 0; i < my_tiles && !stopped; ++i) {
            const int ab = i & 1;
            bool ok = mbar_wait(&s.acc_full[ab], (i / 2) & 1);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) s.failed = 1;
            const int t = (int)blockIdx.x + i * (int)gridDim.x;
            const int n0 = (t % n_tiles_n) * kN, m0 = (t / n_tiles_n) * kTileM;
#pragma unroll 1
            for (int hh = 0; hh < kHalves; ++hh) {
                const int e = i * kHalves + hh, ci = e % kRingC;
                uint32_t v0[32], v1[32];
                if (ok) {
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    tmem_ld_32(tmem + ((uint32_t)(qd * 32) << 16) + (uint32_t)(ab * kN + hh * kDwN), v0);
                    tmem_ld_32(tmem + ((uint32_t)(qd * 32) << 16) + (uint32_t)(ab * kN + hh * kDwN + 32), v1);
                    if (hh == kHalves - 1) {         // the accumulator is in registers: the next tile may use it
                        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                        mbar_arrive(&s.acc_empty[ab]);
                    }
                }
                // Every epilogue warp reaches both barriers of a step (also after a failed wait); the leader
                // samples the failure flag before the first one and all four warps act on that one sample after
                // it, so they leave the loop together.  Before it, the leader also makes sure that the TMA
                // operation which last read staging tile ci has finished reading.
                if (leader) {
                    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(kRingC - 1) : "memory");
                    s.stop[e & 1] = *reinterpret_cast<volatile uint32_t*>(&s.failed);
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (*reinterpret_cast<volatile uint32_t*>(&s.stop[e & 1])) { stopped = true; break; }
                panel_row_update<false>(s.c[ci], row, v0);
                panel_row_update<false>(s.c[ci] + kTileM * 32, row, v1);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // smem writes -> visible to the TMA engine
                asm volatile("bar.sync 1, 128;" ::: "memory");
                if (leader) {
#pragma unroll
                    for (int p = 0; p < kPanels; ++p) {
                        if (store) tma_store_2d(&tm_acc, s.c[ci] + p * (kTileM * 32), n0 + hh * kDwN + p * 32, m0);
                        else tma_reduce_add_2d(&tm_acc, s.c[ci] + p * (kTileM * 32), n0 + hh * kDwN + p * 32, m0);
                    }
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
            }
        }
        if (leader) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
    }
    __syncwarp();
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x == 0 && s.failed) {
        atomicExch(status, ABS_ETIMEOUT);
        for (int i = 0; i < kRingOps; ++i) mbar_wait(&s.op_full[i], 0);   // bounded chance for copies in flight to land
    }
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(2 * kN) : "memory");
    }
}

// ============================================================================================
// Forward GEMM on tcgen05:  zpart[s][h][r] = sum_{k in split s} W1b[k][h] * xb[r][k]
//   D [M = 128 hidden][N = 64 samples] += A B^T with
//   A = W1b^T tile: stored [k][h] with h contiguous, i.e. an MN-major operand.  A TMA box of
//       64 h x 64 k (128-byte rows, 128-byte swizzle) is exactly the canonical MN-major layout:
//       8-k-row groups 1024 B apart (stride offset), the two 64-wide h blocks of the tile one box
//       (8192 B) apart (leading offset).  One UMMA step (K = 16) consumes two 8-k groups: +2048 B.
//   B = xb tile [64 samples][64 k], K-major as in the dW1 kernel.
//       The NB micro-batches of a call are stacked along N (N = 64 NB <= 256): one 64 x 64 box
//       each, 8192 B apart -- the same 8-row groups 1024 B apart, so one descriptor covers them
//       and the weights are streamed once per call, not once per micro-batch.
// One CTA per (128-hidden tile, K split); a ring of TMA -> MMA stages streams the weights
// once.  Warp 0 lane 0 issues TMA, warp 1 lane 0 issues MMAs, all four warps store D.
// ============================================================================================
// kLight: 2 - 3 stages (72 - 96 KB) instead of 4 - 6, so that a dW1 CTA of another worker's call fits beside it.
template <int NB, bool kLight = false>
struct FwdCfg {
    static constexpr int kStages = kLight ? (NB <= 2 ? 3 : 2) : (NB <= 2 ? 6 : (NB == 3 ? 5 : 4));   // <= 200 KB of stages
    static constexpr int kStageBytes = 2 * 8192 + NB * 8192;              // two A boxes + NB B boxes
    static constexpr int kTmemCols = NB == 1 ? 64 : (NB == 2 ? 128 : 256);   // power of two >= 64 NB
};

template <int NB, bool kLight = false>
struct FwdSmem {
    alignas(1024) uint8_t stage[FwdCfg<NB, kLight>::kStages][FwdCfg<NB, kLight>::kStageBytes];   // [A h0..63 | A h64..127 | B x NB]
    alignas(8) uint64_t full[FwdCfg<NB, kLight>::kStages];
    uint64_t empty[FwdCfg<NB, kLight>::kStages];
    uint64_t done;
    uint32_t tmem_base;
    uint32_t failed;
};

template <int NB, bool kLight = false>
__global__ void __launch_bounds__(128) k_fwd1_tcgen05(const __grid_constant__ CUtensorMap tm_w1,
                                                      const __grid_constant__ CUtensorMap tm_xb, float* __restrict__ zpart,
                                                      int d_in, int d_h, int* status) {
    constexpr int kFwdStages = FwdCfg<NB, kLight>::kStages, kFwdStageBytes = FwdCfg<NB, kLight>::kStageBytes;
    constexpr int kTmemCols = FwdCfg<NB, kLight>::kTmemCols;
    extern __shared__ uint8_t smem_raw[];
    FwdSmem<NB, kLight>& s = *reinterpret_cast<FwdSmem<NB, kLight>*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int h0 = blockIdx.x * 128;
    const int split = blockIdx.y;
    const int k_per = d_in / (int)gridDim.y;
    const int kbeg = split * k_per;
    const int nk = k_per / 64;                       // pipeline steps of 64 k

    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s.tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (threadIdx.x == 0) {
        for (int i = 0; i < kFwdStages; ++i) {
            mbar_init(&s.full[i], 1);
            mbar_init(&s.empty[i], 1);
        }
        mbar_init(&s.done, 1);
        s.failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s.tmem_base;

    if (warp == 0 && lane == 0) {                    // ---- TMA producer
        for (int kb = 0; kb < nk; ++kb) {
            const int st = kb % kFwdStages;
            if (kb >= kFwdStages && !mbar_wait(&s.empty[st], ((kb / kFwdStages) - 1) & 1)) { s.failed = 1; break; }
            mbar_expect_tx(&s.full[st], kFwdStageBytes);
            const int k0 = kbeg + kb * 64;
            tma_load_2d(s.stage[st], &tm_w1, h0, k0, &s.full[st]);
            tma_load_2d(s.stage[st] + 8192, &tm_w1, h0 + 64, k0, &s.full[st]);
#pragma unroll
            for (int jb = 0; jb < NB; ++jb)          // rows jb*64.. of the stacked xb
                tma_load_2d(s.stage[st] + 16384 + jb * 8192, &tm_xb, k0, jb * kMB, &s.full[st]);
        }
    } else if (warp == 1 && lane == 0) {             // ---- MMA issuer
        constexpr uint32_t idesc = umma_idesc_bf16(128, 64 * NB) | (1u << 15);   // A is MN-major
        bool ok = true;
        for (int kb = 0; kb < nk && ok; ++kb) {
            const int st = kb % kFwdStages;
            ok = mbar_wait(&s.full[st], (kb / kFwdStages) & 1);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a0 = smem_u32(s.stage[st]);
            const uint64_t db = umma_desc_k_sw128(a0 + 16384);
#pragma unroll
            for (int k = 0; k < 4; ++k)
                umma_bf16(tmem, umma_desc_mn_sw128(a0 + k * 2048, 8192), db + 2 * k, idesc, (kb > 0 || k > 0));
            umma_commit(&s.empty[st]);               // frees the stage once these MMAs have read it
        }
        if (ok) umma_commit(&s.done);
        else s.failed = 1;
    }
    __syncwarp();

    bool ok = mbar_wait(&s.done, 0);
    ok = __all_sync(0xffffffffu, ok);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (ok) {
        // A thread holds one hidden unit's row (TMEM lane), 32 columns per load; stored directly, a warp
        // would write 32 rows x 16 bytes per instruction.  Each warp turns its 32 x 32 block round through
        // shared memory (stage 0 is free: every load has landed and every MMA has completed; pitch 36
        // floats: conflict-free both ways) and stores 4 rows x 128 contiguous bytes per instruction.
        constexpr int kPitch = 36;
        float* tr = reinterpret_cast<float*>(s.stage[0]) + warp * 32 * kPitch;
#pragma unroll 1
        for (int p = 0; p < 2 * NB; ++p) {           // 32 accumulator columns = half a micro-batch per step
            uint32_t v[32];
            tmem_ld_32(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)(p * 32), v);
#pragma unroll
            for (int j = 0; j < 8; ++j)
                *reinterpret_cast<float4*>(tr + lane * kPitch + 4 * j) =
                    make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]), __uint_as_float(v[4 * j + 2]),
                                __uint_as_float(v[4 * j + 3]));
            __syncwarp();
            float* out = zpart + (((size_t)(p >> 1) * kSplitK + split) * d_h + h0 + warp * 32) * kMB + (p & 1) * 32;
#pragma unroll
            for (int it = 0; it < 8; ++it) {
                const int row = it * 4 + lane / 8, c4 = (lane % 8) * 4;
                *reinterpret_cast<float4*>(out + (size_t)row * kMB + c4) = *reinterpret_cast<const float4*>(tr + row * kPitch + c4);
            }
            __syncwarp();
        }
    } else if (threadIdx.x == 0) {
        atomicExch(status, ABS_ETIMEOUT);
        // bounded chance for copies still in flight to land before shared memory is released
        for (int i = 0; i < kFwdStages; ++i) mbar_wait(&s.full[i], 0);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

// ============================================================================================
// Forward, fused:  k_fwd1_tcgen05 + k_fwd2 in one kernel.  The CTAs that hold the K splits of one
// 128-hidden tile form a thread-block cluster (1 x nsplit x 1).  Each runs the same TMA -> MMA
// pipeline as k_fwd1_tcgen05, then parks its partial accumulator [128][64 NB] in its own shared
// memory (the pipeline stages are free by then); after a cluster barrier, CTA rank q adds up rows
// [q 128/nsplit, (q+1) 128/nsplit) of all nsplit partials through distributed shared memory, in
// rank order (fixed summation order), and does k_fwd2's work for those hidden units: bias, ReLU,
// bf16 H -> hbt, partial logits -> lpart, group ticket -> gpart.  The split-K partials never
// leave the SMs (k_fwd1_tcgen05 writes and k_fwd2 re-reads 4 bytes x nsplit per element of Z).
// ============================================================================================
__device__ __forceinline__ float4 ld_dsmem_f4(uint32_t local_addr, uint32_t rank) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(remote));
    return v;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

template <int NB>
__global__ void __launch_bounds__(128) k_fwd_fused(const __grid_constant__ CUtensorMap tm_w1,
                                                   const __grid_constant__ CUtensorMap tm_xb, const float* __restrict__ b1,
                                                   const __nv_bfloat16* __restrict__ w2b, __nv_bfloat16* hbt, float* lpart,
                                                   float* gpart, unsigned int* tickets, int d_in, int d_h, int d_out,
                                                   int* status) {
    constexpr int kFwdStages = FwdCfg<NB>::kStages, kFwdStageBytes = FwdCfg<NB>::kStageBytes;
    constexpr int kTmemCols = FwdCfg<NB>::kTmemCols;
    constexpr int kPitch = 64 * NB + 4;              // floats per row of the parked partial (conflict-free float4 rows)
    static_assert(128 * kPitch * 4 <= kFwdStages * kFwdStageBytes, "the parked partial must fit into the stages");
    extern __shared__ uint8_t smem_raw[];
    FwdSmem<NB>& s = *reinterpret_cast<FwdSmem<NB>*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    __shared__ float sh[kHB][kMB + 1];
    __shared__ float sw2[kHB][kOutPad];
    __shared__ unsigned int s_last[2 * kMaxBatch];
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int h0 = blockIdx.x * 128;
    const int nsplit = gridDim.y;                    // = cluster size
    const int split = blockIdx.y;
    const int k_per = d_in / nsplit;
    const int kbeg = split * k_per;
    const int nk = k_per / 64;                       // pipeline steps of 64 k
    uint32_t rank;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));

    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s.tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (threadIdx.x == 0) {
        for (int i = 0; i < kFwdStages; ++i) {
            mbar_init(&s.full[i], 1);
            mbar_init(&s.empty[i], 1);
        }
        mbar_init(&s.done, 1);
        s.failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s.tmem_base;

    if (warp == 0 && lane == 0) {                    // ---- TMA producer
        for (int kb = 0; kb < nk; ++kb) {
            const int st = kb % kFwdStages;
            if (kb >= kFwdStages && !mbar_wait(&s.empty[st], ((kb / kFwdStages) - 1) & 1)) { s.failed = 1; break; }
            mbar_expect_tx(&s.full[st], kFwdStageBytes);
            const int k0 = kbeg + kb * 64;
            tma_load_2d(s.stage[st], &tm_w1, h0, k0, &s.full[st]);
            tma_load_2d(s.stage[st] + 8192, &tm_w1, h0 + 64, k0, &s.full[st]);
#pragma unroll
            for (int jb = 0; jb < NB; ++jb)
                tma_load_2d(s.stage[st] + 16384 + jb * 8192, &tm_xb, k0, jb * kMB, &s.full[st]);
        }
    } else if (warp == 1 && lane == 0) {             // ---- MMA issuer
        constexpr uint32_t idesc = umma_idesc_bf16(128, 64 * NB) | (1u << 15);   // A is MN-major
        bool ok = true;
        for (int kb = 0; kb < nk && ok; ++kb) {
            const int st = kb % kFwdStages;
            ok = mbar_wait(&s.full[st], (kb / kFwdStages) & 1);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a0 = smem_u32(s.stage[st]);
            const uint64_t db = umma_desc_k_sw128(a0 + 16384);
#pragma unroll
            for (int k = 0; k < 4; ++k)
                umma_bf16(tmem, umma_desc_mn_sw128(a0 + k * 2048, 8192), db + 2 * k, idesc, (kb > 0 || k > 0));
            umma_commit(&s.empty[st]);
        }
        if (ok) umma_commit(&s.done);
        else s.failed = 1;
    }
    __syncwarp();

    bool ok = mbar_wait(&s.done, 0);
    ok = __all_sync(0xffffffffu, ok);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    float* red = reinterpret_cast<float*>(s.stage[0]);   // every load has landed, every MMA has completed
    if (ok) {
        const int row = warp * 32 + lane;            // TMEM lane = hidden unit within the tile
#pragma unroll 1
        for (int p = 0; p < 2 * NB; ++p) {
            uint32_t v[32];
            tmem_ld_32(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)(p * 32), v);
#pragma unroll
            for (int j = 0; j < 8; ++j)
                *reinterpret_cast<float4*>(red + row * kPitch + p * 32 + 4 * j) =
                    make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]), __uint_as_float(v[4 * j + 2]),
                                __uint_as_float(v[4 * j + 3]));
        }
    } else if (threadIdx.x == 0) {
        atomicExch(status, ABS_ETIMEOUT);
        for (int i = 0; i < kFwdStages; ++i) mbar_wait(&s.full[i], 0);   // bounded chance for copies in flight to land
    }
    __syncwarp();
    // From here on every CTA of the cluster takes the same path (also after a failed wait: its numbers are
    // then meaningless and the status word says so), so that both cluster barriers and every ticket are met.
    cluster_sync_all();
    {
        const int rows_per_rank = 128 / nsplit, n_chunk = rows_per_rank / kHB;   // 32 (64) rows = 1 (2) chunks of 32
        const int n_cta2 = d_h / kHB, n_groups = (n_cta2 + kGroup - 1) / kGroup; // chunk = what one k_fwd2 CTA handles
        const uint32_t red_addr = smem_u32(red);
        for (int ch = 0; ch < n_chunk; ++ch) {
            const int hl0 = (int)rank * rows_per_rank + ch * kHB;                 // first tile row of the chunk
            const int cta2 = (h0 + hl0) / kHB;
            for (int e = threadIdx.x; e < kHB * kOutPad; e += 128) {
                const int hl = e / kOutPad, o = e % kOutPad;
                sw2[hl][o] = o < d_out ? bf16_to_f(w2b[(size_t)(h0 + hl0 + hl) * d_out + o]) : 0.f;
            }
#pragma unroll 1
            for (int jb = 0; jb < NB; ++jb) {
                // Z = sum over the K splits (rank order) + b1 ; H = bf16(relu(Z)) -> hbt and sh.
                // All 4 x nsplit remote loads of a thread are issued before the first add.
                float4 part[4][kSplitK];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int hl = threadIdx.x / 16 + 8 * k, r4 = (threadIdx.x % 16) * 4;
                    const uint32_t off = red_addr + (uint32_t)(((hl0 + hl) * kPitch + jb * kMB + r4) * 4);
#pragma unroll
                    for (int sp = 0; sp < kSplitK; ++sp)
                        if (sp < nsplit) part[k][sp] = ld_dsmem_f4(off, (uint32_t)sp);
                }
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int hl = threadIdx.x / 16 + 8 * k, r4 = (threadIdx.x % 16) * 4;
                    const int h = h0 + hl0 + hl;
                    const float bias = b1[h];
                    float4 z = make_float4(bias, bias, bias, bias);
#pragma unroll
                    for (int sp = 0; sp < kSplitK; ++sp)
                        if (sp < nsplit) { z.x += part[k][sp].x; z.y += part[k][sp].y; z.z += part[k][sp].z; z.w += part[k][sp].w; }
                    const __nv_bfloat16 q0 = __float2bfloat16_rn(z.x > 0.f ? z.x : 0.f), q1 = __float2bfloat16_rn(z.y > 0.f ? z.y : 0.f);
                    const __nv_bfloat16 q2 = __float2bfloat16_rn(z.z > 0.f ? z.z : 0.f), q3 = __float2bfloat16_rn(z.w > 0.f ? z.w : 0.f);
                    uint2 pk;
                    pk.x = (uint32_t)__bfloat16_as_ushort(q0) | ((uint32_t)__bfloat16_as_ushort(q1) << 16);
                    pk.y = (uint32_t)__bfloat16_as_ushort(q2) | ((uint32_t)__bfloat16_as_ushort(q3) << 16);
                    *reinterpret_cast<uint2*>(hbt + ((size_t)jb * d_h + h) * kMB + r4) = pk;
                    sh[hl][r4 + 0] = bf16_to_f(q0); sh[hl][r4 + 1] = bf16_to_f(q1);
                    sh[hl][r4 + 2] = bf16_to_f(q2); sh[hl][r4 + 3] = bf16_to_f(q3);
                }
                __syncthreads();
                {   // partial logits of these 32 hidden units: thread = (sample r, 8 of the 16 padded outputs)
                    const int r = threadIdx.x / 2, og = threadIdx.x % 2;
                    float a[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll 8
                    for (int hl = 0; hl < kHB; ++hl) {
                        const float hv = sh[hl][r];
#pragma unroll
                        for (int j = 0; j < 8; ++j) a[j] = fmaf(hv, sw2[hl][8 * og + j], a[j]);
                    }
                    float4* dst = reinterpret_cast<float4*>(lpart + ((size_t)jb * n_cta2 + cta2) * (kMB * kOutPad)) + r * 4 + og * 2;
                    dst[0] = make_float4(a[0], a[1], a[2], a[3]);
                    dst[1] = make_float4(a[4], a[5], a[6], a[7]);
                }
                __syncthreads();                     // sh is rewritten by the next micro-batch
            }
            __syncthreads();                         // sw2 is rewritten by the next chunk
        }
        // ---- group tickets (one per chunk and micro-batch), as in k_fwd2
        __threadfence();
        __syncthreads();
        const int n_units = n_chunk * NB;
        if ((int)threadIdx.x < n_units) {
            const int ch = threadIdx.x / NB, jb = threadIdx.x % NB;
            const int cta2 = (h0 + (int)rank * rows_per_rank + ch * kHB) / kHB;
            const int group = cta2 / kGroup, g_count = min(kGroup, n_cta2 - group * kGroup);
            s_last[threadIdx.x] = (atomicAdd(&tickets[(size_t)jb * n_groups + group], 1u) == (unsigned)(g_count - 1));
        }
        __syncthreads();
        for (int u = 0; u < n_units; ++u) {
            if (!s_last[u]) continue;
            __threadfence();
            const int ch = u / NB, jb = u % NB;
            const int cta2 = (h0 + (int)rank * rows_per_rank + ch * kHB) / kHB;
            const int group = cta2 / kGroup, g_first = group * kGroup, g_count = min(kGroup, n_cta2 - g_first);
            const float4* lp = reinterpret_cast<const float4*>(lpart + (size_t)jb * n_cta2 * (kMB * kOutPad));
            float4* gp = reinterpret_cast<float4*>(gpart + ((size_t)jb * n_groups + group) * (kMB * kOutPad));
            for (int i = threadIdx.x; i < kMB * kOutPad / 4; i += 128) {
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int c = 0; c < g_count; ++c) {
                    const float4 v = __ldcg(lp + (size_t)(g_first + c) * (kMB * kOutPad / 4) + i);
                    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
                }
                gp[i] = acc;
            }
            if (threadIdx.x == 0) tickets[(size_t)jb * n_groups + group] = 0u;   // ready for the next launch
        }
    }
    cluster_sync_all();                              // nobody leaves while its shared memory may still be read
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

template <int NB>
cudaError_t fwd_fused_set_attr() {
    return cudaFuncSetAttribute(k_fwd_fused<NB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(FwdSmem<NB>) + 1024);
}
// Launch with the nsplit CTAs of a hidden tile as one thread-block cluster.
template <int NB>
cudaError_t fwd_fused_launch(int n_tiles, int nsplit, cudaStream_t stream, const CUtensorMap& tw, const CUtensorMap& tx,
                             const float* b1, const __nv_bfloat16* w2b, __nv_bfloat16* hbt, float* lpart, float* gpart,
                             unsigned int* tickets, int d_in, int d_h, int d_out, int* status) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_tiles, nsplit, 1);
    cfg.blockDim = dim3(128, 1, 1);
    cfg.dynamicSmemBytes = sizeof(FwdSmem<NB>) + 1024;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1;
    attr[0].val.clusterDim.y = nsplit;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, k_fwd_fused<NB>, tw, tx, b1, w2b, hbt, lpart, gpart, tickets, d_in, d_h, d_out, status);
}

template <int NB>
cudaError_t fwd1_set_attr() {
    cudaError_t e = cudaFuncSetAttribute(k_fwd1_tcgen05<NB, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)sizeof(FwdSmem<NB, false>) + 1024);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(k_fwd1_tcgen05<NB, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)sizeof(FwdSmem<NB, true>) + 1024);
}
template <int NB>
void fwd1_launch(dim3 grid, cudaStream_t stream, bool light, const CUtensorMap& tw, const CUtensorMap& tx, float* zpart,
                 int d_in, int d_h, int* status) {
    if (light)
        k_fwd1_tcgen05<NB, true><<<grid, 128, sizeof(FwdSmem<NB, true>) + 1024, stream>>>(tw, tx, zpart, d_in, d_h, status);
    else
        k_fwd1_tcgen05<NB, false><<<grid, 128, sizeof(FwdSmem<NB, false>) + 1024, stream>>>(tw, tx, zpart, d_in, d_h, status);
}

// ---- host helpers --------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// 2-D row-major tensor [rows][cols] of `esize`-byte elements, box [box_rows][box_cols], 128-B swizzle.
bool encode_2d(CUtensorMap* tm, CUtensorMapDataType dt, int esize, void* base, uint64_t rows, uint64_t cols,
               uint32_t box_rows, uint32_t box_cols) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * (uint64_t)esize};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return enc(tm, dt, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// One description of the scratch layout, used for sizing (base == nullptr) and for carving.
size_t layout_scratch(MlpScratch* s, const MlpDims& d, char* base) {
    size_t o = 0;
    auto take = [&](size_t b) { char* at = base ? base + o : nullptr; o = align_up(o + b, 1024); return at; };
    const int n_cta = d.d_hidden / kHB;
    const int n_groups = (n_cta + kGroup - 1) / kGroup;
    char* xb = take((size_t)kMaxBatch * kMB * d.d_in * 2);
    char* xtb = take((size_t)kMaxBatch * d.d_in * kMB * 2);
    char* zpart = take((size_t)kMaxBatch * kSplitK * d.d_hidden * kMB * 4);
    char* hbt = take((size_t)kMaxBatch * d.d_hidden * kMB * 2);
    char* dzt = take((size_t)kMaxBatch * d.d_hidden * kMB * 2);
    char* lpart = take((size_t)kMaxBatch * n_cta * kMB * kOutPad * 4);
    char* gpart = take((size_t)kMaxBatch * n_groups * kMB * kOutPad * 4);
    char* bpart = take((size_t)kMaxBatch * n_cta * 4 * 256 * 4);
    char* ycopy = take((size_t)kMaxBatch * kMB * 4);
    char* tickets = take((size_t)(kMaxBatch * n_groups + n_cta) * 4);   // k_fwd2 group tickets, then k_bwd chunk tickets
    char* status = take(256);
    if (s) {
        s->xb = reinterpret_cast<__nv_bfloat16*>(xb);
        s->xtb = reinterpret_cast<__nv_bfloat16*>(xtb);
        s->zpart = reinterpret_cast<float*>(zpart);
        s->hbt = reinterpret_cast<__nv_bfloat16*>(hbt);
        s->dzt = reinterpret_cast<__nv_bfloat16*>(dzt);
        s->lpart = reinterpret_cast<float*>(lpart);
        s->gpart = reinterpret_cast<float*>(gpart);
        s->tickets = reinterpret_cast<unsigned int*>(tickets);
        s->tickets_b = reinterpret_cast<unsigned int*>(tickets) + kMaxBatch * n_groups;
        s->bpart = reinterpret_cast<float*>(bpart);
        s->ycopy = reinterpret_cast<int32_t*>(ycopy);
        s->status = reinterpret_cast<int*>(status);
        s->zero_from = tickets;
        s->zero_bytes = (size_t)(status + 256 - tickets);
    }
    return o;
}

}  // namespace

size_t mlp_scratch_bytes(const MlpDims& d) { return layout_scratch(nullptr, d, nullptr); }

cudaError_t mlp_scratch_init(MlpScratch* s, const MlpDims& d, void* base, __nv_bfloat16* shadow0,
                             __nv_bfloat16* shadow1, const char** err) {
    layout_scratch(s, d, static_cast<char*>(base));
    static_assert(sizeof(CUtensorMap) == sizeof(TmapBytes), "tensor map size");
    // the operands of up to kMaxBatch micro-batches are stacked: micro-batch j at rows [j*d_in, (j+1)*d_in) of X^T
    // and [j*d_h, (j+1)*d_h) of dZ^T
    if (!encode_2d(reinterpret_cast<CUtensorMap*>(&s->tmap_xt), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, s->xtb,
                   (uint64_t)kMaxBatch * d.d_in, kMB, kTileM, kMB) ||
        !encode_2d(reinterpret_cast<CUtensorMap*>(&s->tmap_dzt), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, s->dzt,
                   (uint64_t)kMaxBatch * d.d_hidden, kMB, kDwN, kMB)) {
        *err = "cuTensorMapEncodeTiled failed for the dW1 operands";
        return cudaErrorInvalidValue;
    }
    // forward GEMM operands: W1 (bf16 shadow, [d_in][d_hidden]) in 64 x 64 boxes, xb [mb][d_in] in 64 x 64 boxes
    if (!encode_2d(reinterpret_cast<CUtensorMap*>(&s->tmap_w1[0]), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, shadow0, d.d_in,
                   d.d_hidden, 64, 64) ||
        !encode_2d(reinterpret_cast<CUtensorMap*>(&s->tmap_w1[1]), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, shadow1, d.d_in,
                   d.d_hidden, 64, 64) ||
        !encode_2d(reinterpret_cast<CUtensorMap*>(&s->tmap_xb), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, s->xb,
                   (uint64_t)kMaxBatch * kMB, d.d_in, kMB, 64)) {
        *err = "cuTensorMapEncodeTiled failed for the forward GEMM operands";
        return cudaErrorInvalidValue;
    }
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&s->num_sms, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(k_dw1_ring<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(DwRingSmem<64, false>) + 1024);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(k_dw1_ring<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(DwRingSmem<128, false>) + 1024);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(k_dw1_ring<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(DwRingSmem<64, true>) + 1024);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(k_dw1_ring<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(DwRingSmem<128, true>) + 1024);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(k_dw1_regs, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 dw_regs_buf_bytes(kMaxBatch) + (int)sizeof(DwRegCtl) + 1024);
    if (e == cudaSuccess)
        e = fwd1_set_attr<1>();
        if (e == cudaSuccess) e = fwd1_set_attr<2>();
        if (e == cudaSuccess) e = fwd1_set_attr<3>();
        if (e == cudaSuccess) e = fwd1_set_attr<4>();
        if (e == cudaSuccess) e = fwd_fused_set_attr<1>();
        if (e == cudaSuccess) e = fwd_fused_set_attr<2>();
        if (e == cudaSuccess) e = fwd_fused_set_attr<3>();
        if (e == cudaSuccess) e = fwd_fused_set_attr<4>();
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(k_dw1_tcgen05<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(DwSmem) + 1024);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(k_dw1_tcgen05<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(DwSmem) + 1024);
    if (e != cudaSuccess) *err = "cudaFuncSetAttribute(tcgen05 kernels)";
    return e;
}

cudaError_t mlp_make_acc_tmap(void* tmap_out, const MlpDims& d, float* acc_row) {
    // W1 slice of a worker's accumulator: [d_in][d_hidden] fp32 at offset 0 of the flat row.
    return encode_2d(reinterpret_cast<CUtensorMap*>(tmap_out), CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, acc_row, d.d_in,
                     d.d_hidden, kTileM, 32)
               ? cudaSuccess
               : cudaErrorInvalidValue;
}

cudaError_t launch_mlp_cast(const MlpDims& d, const MlpScratch& s, int slot0, int nb, const float* x_dev, const int32_t* y_dev,
                            cudaStream_t stream, MlpMark mark, void* user) {
    mark(user, ABS_K_MLP_FWD, 0, stream);
    // micro-batch j of the call goes to slot slot0 + j of the scratch set
    k_cast_x<<<dim3(d.d_in / 16, nb), 256, 0, stream>>>(x_dev, y_dev, s.xb + (size_t)slot0 * kMB * d.d_in,
                                                        s.xtb + (size_t)slot0 * d.d_in * kMB, s.ycopy + slot0 * kMB, d.d_in);
    return cudaGetLastError();
}

cudaError_t launch_mlp_front(const MlpDims& d, const MlpScratch& s, const float* x_pub, const __nv_bfloat16* shadow,
                             int shadow_idx, int nb, bool store, float* acc_row, int32_t* cnt, int variant,
                             cudaStream_t stream, MlpMark mark, void* user) {
    const size_t o_b1 = (size_t)d.d_in * d.d_hidden, o_w2 = o_b1 + d.d_hidden, o_b2 = o_w2 + (size_t)d.d_hidden * d.d_out;
    cudaError_t e;
    const unsigned n_cta = d.d_hidden / kHB;
    const bool light = (variant & kMlpLightBit) != 0;

    // every K split must be a whole number of 64-wide pipeline steps (d_in is a multiple of 128)
    const int nsplit = (d.d_in % (64 * kSplitK) == 0) ? kSplitK : 2;
    const CUtensorMap* tw = reinterpret_cast<const CUtensorMap*>(&s.tmap_w1[shadow_idx]);
    const CUtensorMap* tx = reinterpret_cast<const CUtensorMap*>(&s.tmap_xb);
    if ((variant & 64) && !(variant & 2)) {
        // one kernel: forward GEMM, split-K sum through the cluster's shared memory, bias / ReLU / logits.  Same
        // bits as the two-kernel path; measured slower when several workers' calls overlap (its 128 CTAs keep a
        // whole SM's shared memory each while 128 threads do the epilogue work), so it is not the default.
        const int n_tiles = d.d_hidden / 128;
        const float* b1 = x_pub + o_b1;
        const __nv_bfloat16* w2b = shadow + o_w2;
        switch (nb) {
            case 1: e = fwd_fused_launch<1>(n_tiles, nsplit, stream, *tw, *tx, b1, w2b, s.hbt, s.lpart, s.gpart, s.tickets, d.d_in, d.d_hidden, d.d_out, s.status); break;
            case 2: e = fwd_fused_launch<2>(n_tiles, nsplit, stream, *tw, *tx, b1, w2b, s.hbt, s.lpart, s.gpart, s.tickets, d.d_in, d.d_hidden, d.d_out, s.status); break;
            case 3: e = fwd_fused_launch<3>(n_tiles, nsplit, stream, *tw, *tx, b1, w2b, s.hbt, s.lpart, s.gpart, s.tickets, d.d_in, d.d_hidden, d.d_out, s.status); break;
            default: e = fwd_fused_launch<4>(n_tiles, nsplit, stream, *tw, *tx, b1, w2b, s.hbt, s.lpart, s.gpart, s.tickets, d.d_in, d.d_hidden, d.d_out, s.status); break;
        }
        if (e != cudaSuccess) return e;
    } else {
        if (variant & 2) {
            k_fwd1<<<dim3(d.d_hidden / 64, nsplit, nb), 256, 0, stream>>>(shadow, s.xb, s.zpart, d.d_in, d.d_hidden);
        } else {
            const dim3 grid(d.d_hidden / 128, nsplit);
            switch (nb) {                                // the nb micro-batches are stacked along N of one GEMM
                case 1: fwd1_launch<1>(grid, stream, light, *tw, *tx, s.zpart, d.d_in, d.d_hidden, s.status); break;
                case 2: fwd1_launch<2>(grid, stream, light, *tw, *tx, s.zpart, d.d_in, d.d_hidden, s.status); break;
                case 3: fwd1_launch<3>(grid, stream, light, *tw, *tx, s.zpart, d.d_in, d.d_hidden, s.status); break;
                default: fwd1_launch<4>(grid, stream, light, *tw, *tx, s.zpart, d.d_in, d.d_hidden, s.status); break;
            }
        }
        k_fwd2<<<dim3(n_cta, nb), 256, 0, stream>>>(s.zpart, nsplit, x_pub + o_b1, shadow + o_w2, s.hbt, s.lpart, s.gpart,
                                                    s.tickets, d.d_hidden, d.d_out);
    }
    mark(user, ABS_K_MLP_FWD, ((variant & 64) && !(variant & 2)) ? 2 : 3, stream);   // launches of the group, the cast included
    if ((e = cudaGetLastError()) != cudaSuccess) return e;

    mark(user, ABS_K_MLP_BWD, 0, stream);
    const int n_groups = (n_cta + kGroup - 1) / kGroup;
    k_bwd<<<dim3(n_cta, nb), 256, 0, stream>>>(s.hbt, s.gpart, n_groups, x_pub + o_b2, s.ycopy, shadow + o_w2, s.dzt, s.bpart,
                                               s.tickets_b, acc_row + o_b1, acc_row + o_w2, acc_row + o_b2, cnt, d.d_hidden,
                                               d.d_out, store ? 1 : 0);
    mark(user, ABS_K_MLP_BWD, 1, stream);
    return cudaGetLastError();
}

cudaError_t launch_mlp_dw1(const MlpDims& d, const MlpScratch& s, float* acc_row, const void* acc_tmap, int nb, bool store,
                           int variant, cudaStream_t stream, MlpMark mark, void* user) {
    const int st = store ? 1 : 0;
    const bool light = (variant & kMlpLightBit) != 0;
    mark(user, ABS_K_MLP_DW1, 0, stream);
    const dim3 grid(d.d_hidden / kDwN, d.d_in / kTileM);
    const CUtensorMap* ta = reinterpret_cast<const CUtensorMap*>(&s.tmap_xt);
    const CUtensorMap* tb = reinterpret_cast<const CUtensorMap*>(&s.tmap_dzt);
    const CUtensorMap* tc = reinterpret_cast<const CUtensorMap*>(acc_tmap);
    // Which kernel: bits 4 (ring), 8 (register prefetch), 16 (TMA load + add + store), 1 (TMA reduce-add) force
    // one; otherwise the measured best for the case: the persistent ring kernel when the tile is stored (it
    // never reads the accumulator) and for K-batched adds, the register-prefetch kernel for single adds.
    int kind = (variant & 4) ? 4 : (variant & 8) ? 8 : (variant & 16) ? 16 : (variant & 1) ? 1 : 0;
    if (kind == 0) kind = (store || nb > 1) ? 4 : 8;
    if ((kind == 16 || kind == 1) && nb > 1) kind = 8;   // the one-tile-per-CTA TMA kernels are not K-batched
    if (kind == 4) {
        if (nb > 1 && !(variant & 32)) {   // K-batched: 128 x 128 tiles (bit 5 keeps 128 x 64)
            const int n_tiles_n = d.d_hidden / 128, n_tiles = n_tiles_n * (d.d_in / kTileM);
            const int ctas = n_tiles < s.num_sms ? n_tiles : s.num_sms;
            if (light)
                k_dw1_ring<128, true><<<ctas, 192, sizeof(DwRingSmem<128, true>) + 1024, stream>>>(*ta, *tb, *tc, n_tiles_n, n_tiles,
                                                                                                 d.d_in, d.d_hidden, nb, st, s.status);
            else
                k_dw1_ring<128, false><<<ctas, 192, sizeof(DwRingSmem<128, false>) + 1024, stream>>>(*ta, *tb, *tc, n_tiles_n, n_tiles,
                                                                                                   d.d_in, d.d_hidden, nb, st, s.status);
        } else {
            const int n_tiles_n = d.d_hidden / kDwN, n_tiles = n_tiles_n * (d.d_in / kTileM);
            const int ctas = n_tiles < s.num_sms ? n_tiles : s.num_sms;
            if (light)
                k_dw1_ring<64, true><<<ctas, 192, sizeof(DwRingSmem<64, true>) + 1024, stream>>>(*ta, *tb, *tc, n_tiles_n, n_tiles,
                                                                                               d.d_in, d.d_hidden, nb, st, s.status);
            else
                k_dw1_ring<64, false><<<ctas, 192, sizeof(DwRingSmem<64, false>) + 1024, stream>>>(*ta, *tb, *tc, n_tiles_n, n_tiles,
                                                                                                 d.d_in, d.d_hidden, nb, st, s.status);
        }
    } else if (kind == 8) {
        const size_t smem = dw_regs_buf_bytes(nb) + sizeof(DwRegCtl) + 1024;
        k_dw1_regs<<<grid, 256, smem, stream>>>(*ta, *tb, acc_row, d.d_in, d.d_hidden, nb, st, s.status);
    } else if (kind == 1) {
        k_dw1_tcgen05<true><<<grid, 128, sizeof(DwSmem) + 1024, stream>>>(*ta, *tb, *tc, st, s.status);
    } else {
        k_dw1_tcgen05<false><<<grid, 128, sizeof(DwSmem) + 1024, stream>>>(*ta, *tb, *tc, st, s.status);
    }
    mark(user, ABS_K_MLP_DW1, 1, stream);
    return cudaGetLastError();
}

}  // namespace abs_sgd
