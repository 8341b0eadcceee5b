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
// Kernels (five launches per call of 1..4 micro-batches, chained by programmatic dependent launch; only the
// first reads the caller's buffers, the others may run on another stream):
//   k_cast_x        X (fp32 or bf16) -> bf16 in both orientations, labels copied
//   k_fwd1_tcgen05  Z^T partials = W1^T X^T, split over d_in, on tcgen05 (W1 as an MN-major operand)
//   k_fwd2          Z = sum of partials + b1, bf16(H), partial logits per 32 hidden units; the last CTA of
//                   each group of 8 ("last CTA done" ticket) sums the group's partial logits in a fixed order
//   k_bwd           every CTA: logits = sum of group partials + b2, softmax, dL (CTA 0: db2 += ...); then
//                   dH, dZ, bf16(dZ)^T, db1 += ..., dW2 += ..., b_i += 1
//   dW1 = X^T dZ on the 5th-gen tensor cores (TMEM accumulator), one of (chosen per call, see launch_mlp_dw1):
//   k_dw1_ring      persistent, warp-specialised, K-batched: operand ring in shared memory, two TMEM
//                   accumulators, finished tiles leave by TMA store (a worker's first gradient of an iteration)
//                   or TMA reduce-add; 128 x 64 or 128 x 128 tiles
//   k_dw1_regs      one 128 x 64 tile per CTA, the accumulator tile prefetched into registers, K-batched
// Deferred mode (all gradients of an iteration are evaluated at the same x_t, so the sums may be formed late): a
// call stops after k_bwd and leaves bf16(X)^T, bf16(dZ)^T and its db1 | dW2 | db2 in pool slots; then
//   k_sync_w1            Step 1 + update of the W1 slice: ONE contraction over all pooled micro-batches of the
//                        iteration, the update as its epilogue (no accumulator row involved)
//   k_sync_small_pooled  the same step for b1, W2, b2 from the pooled partials
//   k_gather_small, k_dw1_ring over a slot list: the rows themselves, when somebody needs them
#include <cuda.h>

#include <cstdio>

#include "abs_internal.h"
#include "bulk_copy.cuh"

namespace abs_sgd {

namespace {

constexpr int kMB = 64;          // samples per micro-batch = K of the dW1 contraction
constexpr int kOutPad = 16;      // logits / dL rows are padded to 16 columns
constexpr int kSplitK = 4;       // forward GEMM: d_in is split into at most this many partial sums (stride of zpart)
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
struct CastList {          // the caller's buffers of the micro-batches of a call (contiguous or not)
    const void* x[kMlpMaxBatch];
    const int32_t* y[kMlpMaxBatch];
};
template <bool kBf16In>   // the caller's X already holds bf16 values: copied (and transposed) as they are
__global__ void __launch_bounds__(256) k_cast_x(const __grid_constant__ CastList in,
                                                __nv_bfloat16* __restrict__ xb, __nv_bfloat16* __restrict__ xtb,
                                                int32_t* __restrict__ ycopy, int d_in) {
    __shared__ __nv_bfloat16 tile[16][kMB + 8];
    const int c0 = blockIdx.x * 16;
    pdl_wait();
    pdl_trigger();
    const void* x_in = in.x[blockIdx.y];                     // micro-batch blockIdx.y of the call
    if (blockIdx.x == 0 && threadIdx.x < kMB) ycopy[blockIdx.y * kMB + threadIdx.x] = in.y[blockIdx.y][threadIdx.x];
    const size_t mb_off = (size_t)blockIdx.y * kMB * d_in;
    xb += mb_off;
    xtb += (size_t)blockIdx.y * d_in * kMB;
    {
        const int r = threadIdx.x / 4, q = threadIdx.x % 4;
        const size_t at = (size_t)r * d_in + c0 + 4 * q;
        uint2 pk;
        if (kBf16In) {
            pk = *reinterpret_cast<const uint2*>(static_cast<const __nv_bfloat16*>(x_in) + at);
        } else {
            const float4 v = *reinterpret_cast<const float4*>(static_cast<const float*>(x_in) + at);
            pk.x = pack_bf16x2(v.x, v.y);
            pk.y = pack_bf16x2(v.z, v.w);
        }
        *reinterpret_cast<uint2*>(xb + at) = pk;
        tile[4 * q + 0][r] = __ushort_as_bfloat16((unsigned short)(pk.x & 0xFFFFu));
        tile[4 * q + 1][r] = __ushort_as_bfloat16((unsigned short)(pk.x >> 16));
        tile[4 * q + 2][r] = __ushort_as_bfloat16((unsigned short)(pk.y & 0xFFFFu));
        tile[4 * q + 3][r] = __ushort_as_bfloat16((unsigned short)(pk.y >> 16));
    }
    __syncthreads();
    {
        const int c = threadIdx.x / 16, r4 = (threadIdx.x % 16) * 4;
        uint2 pk = *reinterpret_cast<const uint2*>(&tile[c][r4]);
        *reinterpret_cast<uint2*>(xtb + (size_t)(c0 + c) * kMB + r4) = pk;
    }
}

// --------------------------------------------------------------------------------------------
// k_fwd2: per CTA 32 hidden units x 64 samples.
//   phase 1 (thread = sample r, 8 hidden units): Z = sum_s zpart + b1 ; hb = bf16(relu(Z)) -> hbt
//   phase 2 (thread = sample r, 4 logits):        partial logits of these 32 hidden units -> lpart[cta]
//   tail: the last CTA of each group of 8 sums the group's partials (fixed order) -> gpart[group]; the last group
//         to finish sums the group partials (fixed order), adds b2 and forms dL once for the micro-batch -> dlbuf.
// tickets[0 .. n_groups) are the group tickets, tickets2[0] the second level's: all zero on entry, reset before exit.
// --------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_fwd2(const float* zpart, int nsplit, const float* __restrict__ b1,
                                              const __nv_bfloat16* __restrict__ w2b, __nv_bfloat16* hbt,
                                              float* lpart, float* gpart, unsigned int* tickets, int d_h, int d_out,
                                              const float* __restrict__ b2, const int32_t* y, float* dlbuf,
                                              unsigned int* tickets2) {
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
        y += (size_t)j * kMB;
        dlbuf += (size_t)j * 2 * kMB * kOutPad;
        tickets2 += j;
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
        // up to here only parameters were read (published before the call started); zpart comes from the
        // forward GEMM just ahead on the stream
        pdl_wait();
        pdl_trigger();
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
    // ---- second level: the last group to finish sums the group partials (fixed order), adds b2 and forms
    //      dL = (softmax - onehot) / mb once for the micro-batch: dlbuf[0] unrounded (db2), dlbuf[1] rounded to bf16.
    //      (Every k_bwd CTA used to do this for itself: n_groups x 4 KB of L2 reads per CTA.)
    const int n_groups = (n_cta + kGroup - 1) / kGroup;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = (atomicAdd(tickets2, 1u) == (unsigned)(n_groups - 1));
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int c = 0; c < n_groups; ++c) {
            const float4 v = __ldcg(reinterpret_cast<const float4*>(gpart) + (size_t)c * (kMB * kOutPad / 4) + threadIdx.x);
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
        float gl[4], gb[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int o = 4 * og + j;
            gl[j] = o < d_out ? (l[j] / den - (o == yr ? 1.f : 0.f)) * (1.0f / kMB) : 0.f;
            gb[j] = bf16_to_f(__float2bfloat16_rn(gl[j]));
        }
        reinterpret_cast<float4*>(dlbuf)[threadIdx.x] = make_float4(gl[0], gl[1], gl[2], gl[3]);
        reinterpret_cast<float4*>(dlbuf + kMB * kOutPad)[threadIdx.x] = make_float4(gb[0], gb[1], gb[2], gb[3]);
    }
    if (threadIdx.x == 0) *tickets2 = 0u;
}

// --------------------------------------------------------------------------------------------
// k_bwd: per CTA 32 hidden units x 64 samples.
//   prologue: dL = (softmax - onehot)/mb of the micro-batch as k_fwd2's last CTA left it (unrounded and rounded
//            to bf16); CTA 0 also adds db2 = sum_r dL
//   phase 1 (thread = sample r, 8 hidden units): dH = sum_o bf16(dL)[r][o] W2b[h][o]; dZ = dH * [H > 0]
//            (H > 0 exactly when Z > 0); dzt[h][r] = bf16(dZ)
//   phase 2 (thread = hidden unit, 2 outputs): dW2[h][o] += sum_r bf16(H)[h][r] bf16(dL)[r][o],
//            db1[h] += sum_r dZ[h][r]   (fixed summation order over r)
// --------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_bwd(const __nv_bfloat16* hbt, const float* dlbuf,
                                             const __nv_bfloat16* __restrict__ w2b, __nv_bfloat16* dzt, float* bpart,
                                             unsigned int* tickets_b, float* acc_b1, float* acc_w2, float* acc_b2,
                                             int32_t* cnt, int d_h, int d_out, int store, float* part, size_t part_stride,
                                             MlpWorkers wk) {
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
    const int r = threadIdx.x % kMB, g = threadIdx.x / kMB;
    for (int e = threadIdx.x; e < kHB * kOutPad; e += 256) {   // parameters: published before the call started
        const int hl = e / kOutPad, o = e % kOutPad;
        sw2[hl][o] = o < d_out ? bf16_to_f(w2b[(size_t)(h_beg + hl) * d_out + o]) : 0.f;
    }
    pdl_wait();                                      // hbt and dL come from k_fwd2, just ahead on the stream
    pdl_trigger();
    float hv[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) hv[j] = bf16_to_f(hbt[(size_t)(h_beg + g * 8 + j) * kMB + r]);
    {   // dL of the micro-batch, formed once by k_fwd2: [0] unrounded (db2), [1] rounded to bf16
        const float* dl = dlbuf + (size_t)jb * 2 * kMB * kOutPad;
        const int rr = threadIdx.x / 4, og = threadIdx.x % 4;
        const float4 a = reinterpret_cast<const float4*>(dl)[threadIdx.x];
        const float4 b = reinterpret_cast<const float4*>(dl + kMB * kOutPad)[threadIdx.x];
        sdl32[rr][4 * og + 0] = a.x; sdl32[rr][4 * og + 1] = a.y; sdl32[rr][4 * og + 2] = a.z; sdl32[rr][4 * og + 3] = a.w;
        sdl[rr][4 * og + 0] = b.x; sdl[rr][4 * og + 1] = b.y; sdl[rr][4 * og + 2] = b.z; sdl[rr][4 * og + 3] = b.w;
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
        if (part) {
            // Deferred form: nothing is added to the row here.  Every micro-batch leaves its own db1 | dW2 | db2 (laid
            // out like the row behind W1) in its pool slot; k_gather_small adds them up, in slot order, when the
            // iteration ends -- so calls of one worker need no order among themselves.
            float* mine = part + (size_t)jb * part_stride;
            if (slot < d_out) mine[d_h + (size_t)h * d_out + slot] = a;
            if (slot + 8 < d_out) mine[d_h + (size_t)h * d_out + slot + 8] = b;
            if (slot == 0) mine[h] = c;
            if (blockIdx.x == 0 && threadIdx.x < d_out) mine[d_h + (size_t)d_h * d_out + threadIdx.x] = db2;
            // M_t^i += M_r for the worker this micro-batch belongs to (cnt: the set's counters; a gathered group may
            // hold micro-batches of several workers)
            if (blockIdx.x == 0 && threadIdx.x == 0) atomicAdd(cnt + wk.w[jb], 1);
            return;
        }
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

// --------------------------------------------------------------------------------------------
// k_gather_small (ABS_FLAG_MLP_DEFER): the bias / W2 part of worker rows from the per-micro-batch partials that
// k_bwd left in the pool.  Worker w = first_worker + blockIdx.y:
//     row_w[o_small + t] = (keep_w ? row_w[o_small + t] : 0) + sum over the slots owned by w, in list order, of part[slot][t]
// Workers without slots in the list are left alone.
// --------------------------------------------------------------------------------------------
struct GatherList {
    MlpSlots slots;                  // pool slots, in contraction order
    uint8_t owner[kMlpMaxSlots];     // worker that owns each of them
};
__global__ void __launch_bounds__(256) k_gather_small(const float* __restrict__ part, size_t part_stride,
                                                      const __grid_constant__ GatherList gl, int n, int first_worker,
                                                      unsigned long long keep_mask, float* acc, size_t row_stride,
                                                      size_t o_small, int n_small) {
    const int w = first_worker + blockIdx.y;
    pdl_wait();
    pdl_trigger();
    bool any = false;
    for (int q = 0; q < n; ++q) any = any || gl.owner[q] == w;
    if (!any) return;
    float* row = acc + (size_t)w * row_stride + o_small;
    const bool keep = (keep_mask >> w) & 1ull;
    for (int t = blockIdx.x * 256 + threadIdx.x; t < n_small; t += gridDim.x * 256) {
        float a = keep ? row[t] : 0.f;
        for (int q = 0; q < n; ++q)
            if (gl.owner[q] == w) a += part[(size_t)gl.slots.s[q] * part_stride + t];
        row[t] = a;
    }
}

// ============================================================================================
// tcgen05 / TMA / mbarrier helpers
// ============================================================================================
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* tm, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
// Same with an L2 cache policy (createpolicy) for the loaded lines.
__device__ __forceinline__ void tma_load_2d_hint(void* dst, const CUtensorMap* tm, int x, int y, uint64_t* bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(policy) : "memory");
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
// 16 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld_16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
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
// dW1 = X^T dZ on tcgen05, 128 x 64 output tiles; one micro-batch is K = 64 = four UMMA steps.
// ============================================================================================
constexpr int kTileM = 128;
constexpr int kDwN = 64;
constexpr int kPanels = kDwN / 32;

// ============================================================================================
// dW1 with a register-prefetched accumulator tile, optionally K-batched.  One CTA per tile; the fp32
// accumulator tile never goes through TMA: every thread loads its 8 float4 of the tile with plain
// coalesced loads at kernel entry (all in flight while the kernel ahead on the stream finishes, the
// operands arrive and the MMAs run), the TMEM result is transposed through a padded shared-memory
// tile, and the sums go back with coalesced stores.
// K batching: the operands of nb (1..kMaxBatch) micro-batches are stacked along K, so one launch
// computes  acc += sum_j X_j^T dZ_j  (K = 64 nb) and the accumulator slice is read and written once
// for nb micro-batches instead of nb times -- the kernel is bound by that traffic, not by the MMAs.
// Operand j lives in slot sl.s[j] of the stacked operand tensors: row offset slot*d_in (X^T) / slot*d_h (dZ^T).
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
                                                  const __grid_constant__ CUtensorMap tm_dzt,
                                                  const __grid_constant__ MlpSlots sl, float* acc_w1, int d_in, int ld,
                                                  int nb, int store, int* status) {
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
        // store: the slice holds nothing yet (a worker's first gradient of the iteration), so it is not read.
        // These loads stand in front of pdl_wait(): the slice was last written by a kernel at least two places
        // ahead on this stream (the previous dW1 of this worker) or by work ordered before the whole call.
        c[k] = store ? make_float4(0.f, 0.f, 0.f, 0.f) : gbase[(size_t)(e / kC4) * ld4 + (e % kC4)];
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
    pdl_wait();      // dzt comes from k_bwd, just ahead on the stream
    pdl_trigger();

    if (threadIdx.x == 0) {
        mbar_expect_tx(&s.bar_ab, nb * kDwOperandBytes);
        for (int j = 0; j < nb; ++j) {
            tma_load_2d(buf + j * kDwOperandBytes, &tm_xt, 0, (int)sl.s[j] * d_in + m0, &s.bar_ab);
            tma_load_2d(buf + j * kDwOperandBytes + kTileM * 128, &tm_dzt, 0, (int)sl.s[j] * ld + n0, &s.bar_ab);
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
                                                  const __grid_constant__ CUtensorMap tm_acc,
                                                  const __grid_constant__ MlpSlots sl, int n_tiles_n, int n_tiles,
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
    pdl_wait();      // dzt comes from k_bwd, just ahead on the stream
    pdl_trigger();

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
                    const int slot = (int)sl.s[j];   // where micro-batch j of the contraction sits in the stacked operands
                    tma_load_2d(s.op[st], &tm_xt, 0, slot * d_in + m0, &s.op_full[st]);
#pragma unroll
                    for (int b = 0; b < kHalves; ++b)   // 64-row boxes, 8 KB apart: one K-major B operand of kN rows
                        tma_load_2d(s.op[st] + kTileM * 128 + b * (kDwN * 128), &tm_dzt, 0, slot * ld + n0 + b * kDwN, &s.op_full[st]);
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
// Step 1 + update for the W1 slice straight from the pooled dW1 operands (ABS_FLAG_MLP_DEFER).
// When no accumulator row's W1 slice was written during the iteration, sum_i G_t^i restricted to W1 is
// sum over ALL micro-batches of the iteration of X_j^T dZ_j: one contraction with K = 64 B, whose tiles feed
// the update directly -- the slices are never written, read or cleared:
//     g = (sum_j X_j^T dZ_j) * (1 / B);  Eq. 6;  + wd x;  v = mu v + g;  x' = x - lr v;  bf16(x') -> shadow
// Same roles as k_dw1_ring with 128 x 128 tiles (warp 0: operand TMA producer, warp 1: MMA issuer, two TMEM
// accumulators).  The eight epilogue warps take a finished tile in four panels of 32 columns: the x and v
// panels ([128][32] fp32, swizzled rows) arrive by TMA in a ring of kStepE stages whose loads the epilogue's own
// leader thread issues two panels ahead (self-paced: the operand producer never waits for the epilogue and
// cannot be what the epilogue waits for); each thread updates its row in place, the bf16 copy goes into a
// [128][64] panel shared by two steps, and the leader sends everything back with TMA stores.
// HBM traffic: 18 bytes per W1 element (x, v read; x', v, bf16 x' written) + the operands once (they stay in
// L2 between tiles), against (8 W_act + 18) for the row-based step plus 4 W_act for the contractions.
// ============================================================================================
constexpr int kStepE = 3;        // epilogue stages: [x panel 16 KB | v panel 16 KB]
constexpr int kStepEpiThreads = 256;   // eight epilogue warps: two per TMEM lane quarter, 16 columns of a panel each
constexpr int kPanelBytes = kTileM * 32 * 4;
// kN: tile width.  128: three operand slots of 32 KB.  256 (d_hidden a multiple of 256): two slots of 48 KB -- the
// same bytes in flight, a quarter less operand traffic from L2 per output element (the X^T tile serves twice the
// columns), all 512 TMEM columns for the two accumulators.
template <int kN>
struct StepCfg {
    static constexpr int kOps = kN == 128 ? 3 : 2;
    static constexpr int kSlotBytes = kTileM * 128 + kN * 128;
    static constexpr int kPP = kN / 32;              // epilogue panels per tile
};

template <int kN>
struct StepSmem {
    alignas(1024) uint8_t op[StepCfg<kN>::kOps][StepCfg<kN>::kSlotBytes];
    alignas(1024) uint8_t ep[kStepE][2 * kPanelBytes];
    alignas(1024) uint8_t sh[2][kTileM * 128];          // bf16 copy, [128 rows][64 columns], swizzled 128-byte rows
    alignas(8) uint64_t op_full[StepCfg<kN>::kOps];
    uint64_t op_empty[StepCfg<kN>::kOps];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint64_t ep_full[kStepE];
    uint32_t tmem_base;
    uint32_t failed;
    uint32_t stop[2];
};

struct W1StepCoef {
    float inv_B;         // 1 / B, B = sum_i b_i of the set
    float lr, mu, wd, lambda_dc, disp_scale;
};

template <int kN>
__global__ void __launch_bounds__(64 + kStepEpiThreads) k_sync_w1(const __grid_constant__ CUtensorMap tm_xt,
                                                 const __grid_constant__ CUtensorMap tm_dzt,
                                                 const __grid_constant__ CUtensorMap tm_x_in,
                                                 const __grid_constant__ CUtensorMap tm_x_out,
                                                 const __grid_constant__ CUtensorMap tm_v,
                                                 const __grid_constant__ CUtensorMap tm_shadow,
                                                 const __grid_constant__ MlpSlots sl, int n_tiles_n, int n_tiles, int d_in,
                                                 int ld, int nb, W1StepCoef cf, int has_shadow, int* status) {
    extern __shared__ uint8_t smem_raw[];
    constexpr int kStepOps = StepCfg<kN>::kOps, kStepSlotBytes = StepCfg<kN>::kSlotBytes, kPP = StepCfg<kN>::kPP;
    constexpr int kStepN = kN;
    StepSmem<kN>& s = *reinterpret_cast<StepSmem<kN>*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int my_tiles = (n_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    const int my_panels = my_tiles * (kN / 32);

    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s.tmem_base)), "r"(2 * kStepN) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (threadIdx.x == 0) {
        for (int i = 0; i < kStepOps; ++i) {
            mbar_init(&s.op_full[i], 1);
            mbar_init(&s.op_empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&s.acc_full[i], 1);
            mbar_init(&s.acc_empty[i], kStepEpiThreads);
        }
        for (int i = 0; i < kStepE; ++i) mbar_init(&s.ep_full[i], 1);
        s.failed = 0;
        s.stop[0] = s.stop[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s.tmem_base;
    pdl_wait();      // the operands come from the gradient kernels, x and v from the previous step
    pdl_trigger();

    if (warp == 0) {
        if (lane == 0) {                             // ---- operand producer
            int q = 0;
            for (int i = 0; i < my_tiles && !s.failed; ++i) {
                const int t = (int)blockIdx.x + i * (int)gridDim.x;
                const int n0 = (t % n_tiles_n) * kStepN, m0 = (t / n_tiles_n) * kTileM;
                for (int j = 0; j < nb; ++j, ++q) {
                    const int st = q % kStepOps;
                    if (q >= kStepOps && !mbar_wait(&s.op_empty[st], ((q / kStepOps) - 1) & 1)) { s.failed = 1; break; }
                    mbar_expect_tx(&s.op_full[st], kStepSlotBytes);
                    const int slot = (int)sl.s[j];
                    tma_load_2d(s.op[st], &tm_xt, 0, slot * d_in + m0, &s.op_full[st]);
                    tma_load_2d(s.op[st] + kTileM * 128, &tm_dzt, 0, slot * ld + n0, &s.op_full[st]);   // one box of kN rows
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {                             // ---- MMA issuer
            constexpr uint32_t idesc = umma_idesc_bf16(kTileM, kStepN);
            int q = 0;
            bool ok = true;
            for (int i = 0; i < my_tiles && ok; ++i) {
                const int ab = i & 1;
                if (i >= 2 && !mbar_wait(&s.acc_empty[ab], ((i / 2) - 1) & 1)) { ok = false; break; }
                for (int j = 0; j < nb; ++j, ++q) {
                    const int st = q % kStepOps;
                    if (!mbar_wait(&s.op_full[st], (q / kStepOps) & 1)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a0 = smem_u32(s.op[st]);
                    const uint64_t da = umma_desc_k_sw128(a0), db = umma_desc_k_sw128(a0 + kTileM * 128);
#pragma unroll
                    for (int k = 0; k < kMB / 16; ++k) umma_bf16(tmem + ab * kStepN, da + 2 * k, db + 2 * k, idesc, (j > 0 || k > 0));
                    umma_commit(&s.op_empty[st]);
                }
                if (ok) umma_commit(&s.acc_full[ab]);
            }
            if (!ok) s.failed = 1;
        }
    } else {                                         // ---- epilogue warps 2..9
        // A warp may read the TMEM lanes of its quarter (warp % 4) only; warps 2-5 take columns 0..15 of a panel,
        // warps 6-9 columns 16..31, so every scheduler of the SM has two warps to issue from.
        const int qd = warp % 4, half = (warp - 2) / 4;
        const int row = qd * 32 + lane;
        const int sw = row & 7;
        const bool leader = (threadIdx.x == 64);
        auto panel_coords = [&](int e, int* col, int* m0) {
            const int t = (int)blockIdx.x + (e / kPP) * (int)gridDim.x;
            *col = (t % n_tiles_n) * kStepN + (e % kPP) * 32;
            *m0 = (t / n_tiles_n) * kTileM;
        };
        auto load_panels = [&](int e) {              // leader only: x and v panels of step e into stage e % kStepE
            int col, m0;
            panel_coords(e, &col, &m0);
            const int st = e % kStepE;
            mbar_expect_tx(&s.ep_full[st], 2 * kPanelBytes);
            tma_load_2d(s.ep[st], &tm_x_in, col, m0, &s.ep_full[st]);
            tma_load_2d(s.ep[st] + kPanelBytes, &tm_v, col, m0, &s.ep_full[st]);
        };
        if (leader)
            for (int e = 0; e < kStepE - 1 && e < my_panels; ++e) load_panels(e);
        const float c_dc = -cf.lambda_dc * cf.disp_scale;
        bool stopped = false;
        for (int e = 0; e < my_panels && !stopped; ++e) {
            const int i = e / kPP, p = e % kPP, ab = i & 1, st = e % kStepE;
            bool ok = true;
            if (p == 0) ok = mbar_wait(&s.acc_full[ab], (i / 2) & 1);
            ok = mbar_wait(&s.ep_full[st], (e / kStepE) & 1) && ok;
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) s.failed = 1;
            if (ok) {
                uint32_t acc[16];
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                tmem_ld_16(tmem + ((uint32_t)(qd * 32) << 16) + (uint32_t)(ab * kStepN + p * 32 + half * 16), acc);
                if (p == kPP - 1) {                  // the accumulator is in registers: the tile after next may use it
                    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                    mbar_arrive(&s.acc_empty[ab]);
                }
                float4* xrow = reinterpret_cast<float4*>(s.ep[st]) + row * 8;
                float4* vrow = reinterpret_cast<float4*>(s.ep[st] + kPanelBytes) + row * 8;
                uint8_t* shrow = s.sh[(e >> 1) & 1] + row * 128;
                float4 x[4], v[4];
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    const int j = half * 4 + jj;     // 16-byte chunk of the panel row
                    x[jj] = xrow[j ^ sw];
                    v[jj] = vrow[j ^ sw];
                }
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    const int j = half * 4 + jj;
                    float gx = __uint_as_float(acc[4 * jj]) * cf.inv_B, gy = __uint_as_float(acc[4 * jj + 1]) * cf.inv_B;
                    float gz = __uint_as_float(acc[4 * jj + 2]) * cf.inv_B, gw = __uint_as_float(acc[4 * jj + 3]) * cf.inv_B;
                    if (cf.lambda_dc != 0.0f) {      // Eq. 6 with x_t - x_{t-1} = -disp_scale * v
                        gx += c_dc * gx * gx * v[jj].x; gy += c_dc * gy * gy * v[jj].y;
                        gz += c_dc * gz * gz * v[jj].z; gw += c_dc * gw * gw * v[jj].w;
                    }
                    gx += cf.wd * x[jj].x; gy += cf.wd * x[jj].y; gz += cf.wd * x[jj].z; gw += cf.wd * x[jj].w;
                    v[jj].x = cf.mu * v[jj].x + gx; v[jj].y = cf.mu * v[jj].y + gy;
                    v[jj].z = cf.mu * v[jj].z + gz; v[jj].w = cf.mu * v[jj].w + gw;
                    x[jj].x -= cf.lr * v[jj].x; x[jj].y -= cf.lr * v[jj].y; x[jj].z -= cf.lr * v[jj].z; x[jj].w -= cf.lr * v[jj].w;
                    xrow[j ^ sw] = x[jj];
                    vrow[j ^ sw] = v[jj];
                    // columns 4j..4j+3 of panel p = bf16 elements (p & 1) * 32 + 4j.. of the 64-column copy row
                    uint2 pk;
                    pk.x = pack_bf16x2(x[jj].x, x[jj].y);
                    pk.y = pack_bf16x2(x[jj].z, x[jj].w);
                    const int chunk = (p & 1) * 4 + (j >> 1);
                    *reinterpret_cast<uint2*>(shrow + ((chunk ^ sw) << 4) + ((j & 1) << 3)) = pk;
                }
            }
            if (leader) s.stop[e & 1] = *reinterpret_cast<volatile uint32_t*>(&s.failed);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // smem writes -> visible to the TMA engine
            asm volatile("bar.sync 1, %0;" ::"n"(kStepEpiThreads) : "memory");
            if (*reinterpret_cast<volatile uint32_t*>(&s.stop[e & 1])) { stopped = true; break; }
            if (leader) {
                int col, m0;
                panel_coords(e, &col, &m0);
                tma_store_2d(&tm_x_out, s.ep[st], col, m0);
                tma_store_2d(&tm_v, s.ep[st] + kPanelBytes, col, m0);
                if ((p & 1) && has_shadow) tma_store_2d(&tm_shadow, s.sh[(e >> 1) & 1], col - 32, m0);
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                // the stores of step e-1 have read their stage: it takes the panels of step e + kStepE - 1
                asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                if (e + kStepE - 1 < my_panels) load_panels(e + kStepE - 1);
            }
        }
        if (leader) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
    }
    __syncwarp();
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x == 0 && s.failed) {
        atomicExch(status, ABS_ETIMEOUT);
        for (int i = 0; i < kStepOps; ++i) mbar_wait(&s.op_full[i], 0);   // bounded chance for copies in flight to land
        for (int i = 0; i < kStepE; ++i) mbar_wait(&s.ep_full[i], 0);
    }
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(2 * kStepN) : "memory");
    }
}

// The bias / W2 part of the same step (everything behind W1 in the flat vector), straight from the pooled
// per-micro-batch partials: sum_i G_t^i restricted to that part is the sum over all slots of db1 | dW2 | db2, added
// here in slot order, then the same update.  One thread per parameter; CTA 0 also moves the device counters b_i of
// the set into the consumed-count log and clears them (nothing in this step reads them: B comes from the host).
__global__ void __launch_bounds__(256) k_sync_small_pooled(const float* __restrict__ part, size_t part_stride,
                                                           const __grid_constant__ MlpSlots sl, int n,
                                                           const float* x_in, float* x_out, float* v,
                                                           __nv_bfloat16* shadow, int n_small, W1StepCoef cf, int32_t* cnt,
                                                           int32_t* log_row, int W) {
    const int t = blockIdx.x * 256 + threadIdx.x;
    pdl_wait();
    pdl_trigger();
    if (t < n_small) {
        float sum = 0.f;
        for (int q = 0; q < n; ++q) sum += part[(size_t)sl.s[q] * part_stride + t];
        float g = sum * cf.inv_B;
        float vv = v[t], x = x_in[t];
        if (cf.lambda_dc != 0.0f) g += (-cf.lambda_dc * cf.disp_scale) * g * g * vv;   // Eq. 6
        g += cf.wd * x;
        vv = cf.mu * vv + g;
        x -= cf.lr * vv;
        v[t] = vv;
        x_out[t] = x;
        if (shadow) shadow[t] = __float2bfloat16_rn(x);
    }
    if (blockIdx.x == 0 && threadIdx.x < W) {
        log_row[threadIdx.x] = cnt[threadIdx.x];
        cnt[threadIdx.x] = 0;
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
    static constexpr int kStageBytes = 2 * 8192 + NB * 8192;              // two A boxes + NB B boxes
    // <= 200 KB of stages (deep) / about 100 KB (light; 160 KB for more than four micro-batches)
    static constexpr int kStages = kLight ? (NB <= 2 ? 3 : 2) : (NB <= 2 ? 6 : (NB == 3 ? 5 : (NB == 4 ? 4 : (NB <= 6 ? 3 : 2))));
    static constexpr int kTmemCols = NB == 1 ? 64 : (NB == 2 ? 128 : (NB <= 4 ? 256 : 512));   // power of two >= 64 NB
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
                                                      int d_in, int d_h, int xb_row0, int* status) {
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
    pdl_wait();      // xb comes from k_cast_x, just ahead (possibly on another stream, then ordered by an event)
    pdl_trigger();

    if (warp == 0 && lane == 0) {                    // ---- TMA producer
        // The bf16 weights (2 bytes per W1 element, 25 MB at 3072 x 4096) are read by every gradient call of the
        // iteration: their lines are marked evict-last, so that they tend to stay in the 126 MB L2 between calls
        // while the accumulator traffic of the dW1 kernels streams through (measured: 31.4 -> 31.0 us per micro-batch
        // with single calls, 15.5 -> 15.3 batched; marking the accumulator traffic evict-first on top cost 7 %
        // with single calls -- a worker's stored slice is partly still cached when its next gradient is added).
        uint64_t pol_w1;
        asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_w1));
        for (int kb = 0; kb < nk; ++kb) {
            const int st = kb % kFwdStages;
            if (kb >= kFwdStages && !mbar_wait(&s.empty[st], ((kb / kFwdStages) - 1) & 1)) { s.failed = 1; break; }
            mbar_expect_tx(&s.full[st], kFwdStageBytes);
            const int k0 = kbeg + kb * 64;
            tma_load_2d_hint(s.stage[st], &tm_w1, h0, k0, &s.full[st], pol_w1);
            tma_load_2d_hint(s.stage[st] + 8192, &tm_w1, h0 + 64, k0, &s.full[st], pol_w1);
#pragma unroll
            for (int jb = 0; jb < NB; ++jb)          // rows xb_row0 + jb*64.. of the stacked xb
                tma_load_2d(s.stage[st] + 16384 + jb * 8192, &tm_xb, k0, xb_row0 + jb * kMB, &s.full[st]);
        }
    } else if (warp == 1 && lane == 0) {             // ---- MMA issuer
        // N of one instruction is at most 256: the first four micro-batches go into TMEM columns 0..255, the
        // others (NB > 4) into columns 256.. with a second instruction per K step.
        constexpr int kN0 = NB <= 4 ? 64 * NB : 256, kN1 = NB <= 4 ? 0 : 64 * (NB - 4);
        constexpr uint32_t idesc = umma_idesc_bf16(128, kN0) | (1u << 15);   // A is MN-major
        constexpr uint32_t idesc1 = umma_idesc_bf16(128, kN1 > 0 ? kN1 : 64) | (1u << 15);
        bool ok = true;
        for (int kb = 0; kb < nk && ok; ++kb) {
            const int st = kb % kFwdStages;
            ok = mbar_wait(&s.full[st], (kb / kFwdStages) & 1);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a0 = smem_u32(s.stage[st]);
            const uint64_t db = umma_desc_k_sw128(a0 + 16384);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                umma_bf16(tmem, umma_desc_mn_sw128(a0 + k * 2048, 8192), db + 2 * k, idesc, (kb > 0 || k > 0));
                if (kN1 > 0)
                    umma_bf16(tmem + 256, umma_desc_mn_sw128(a0 + k * 2048, 8192), umma_desc_k_sw128(a0 + 16384 + 4 * 8192) + 2 * k,
                              idesc1, (kb > 0 || k > 0));
            }
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

template <int NB>
cudaError_t fwd1_set_attr() {
    cudaError_t e = cudaFuncSetAttribute(k_fwd1_tcgen05<NB, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)sizeof(FwdSmem<NB, false>) + 1024);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(k_fwd1_tcgen05<NB, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)sizeof(FwdSmem<NB, true>) + 1024);
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
    char* dlbuf = take((size_t)kMaxBatch * 2 * kMB * kOutPad * 4);
    char* tickets = take((size_t)(kMaxBatch * n_groups + n_cta + kMaxBatch) * 4);   // k_fwd2 group tickets, k_bwd chunk tickets, k_fwd2 second level
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
        s->tickets2 = reinterpret_cast<unsigned int*>(tickets) + kMaxBatch * n_groups + n_cta;
        s->dlbuf = reinterpret_cast<float*>(dlbuf);
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
    if (e == cudaSuccess) e = fwd1_set_attr<1>();
    if (e == cudaSuccess) e = fwd1_set_attr<2>();
    if (e == cudaSuccess) e = fwd1_set_attr<3>();
    if (e == cudaSuccess) e = fwd1_set_attr<4>();
    if (e == cudaSuccess) e = fwd1_set_attr<5>();
    if (e == cudaSuccess) e = fwd1_set_attr<6>();
    if (e == cudaSuccess) e = fwd1_set_attr<7>();
    if (e == cudaSuccess) e = fwd1_set_attr<8>();
    if (e != cudaSuccess) *err = "cudaFuncSetAttribute(tcgen05 kernels)";
    return e;
}

namespace {
size_t pool_part_stride(const MlpDims& d) {   // floats per slot: db1 | dW2 | db2, padded to whole 128-byte lines
    return align_up((size_t)d.d_hidden + (size_t)d.d_hidden * d.d_out + d.d_out, 32);
}
}  // namespace

size_t mlp_pool_bytes(const MlpDims& d, int cap) {
    return 2 * align_up((size_t)cap * d.d_in * kMB * 2, 1024) + align_up((size_t)cap * d.d_hidden * kMB * 2, 1024) +
           align_up((size_t)cap * kMB * 4, 1024) + align_up((size_t)cap * pool_part_stride(d) * 4, 1024);
}

cudaError_t mlp_pool_init(MlpPool* p, const MlpDims& d, int cap, void* base) {
    p->cap = cap;
    char* at = static_cast<char*>(base);
    p->xtb = reinterpret_cast<__nv_bfloat16*>(at);
    at += align_up((size_t)cap * d.d_in * kMB * 2, 1024);
    p->dzt = reinterpret_cast<__nv_bfloat16*>(at);
    at += align_up((size_t)cap * d.d_hidden * kMB * 2, 1024);
    p->xb = reinterpret_cast<__nv_bfloat16*>(at);
    at += align_up((size_t)cap * d.d_in * kMB * 2, 1024);
    p->ycopy = reinterpret_cast<int32_t*>(at);
    at += align_up((size_t)cap * kMB * 4, 1024);
    p->part = reinterpret_cast<float*>(at);
    p->part_stride = pool_part_stride(d);
    if (!encode_2d(reinterpret_cast<CUtensorMap*>(&p->tmap_xb), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, p->xb, (uint64_t)cap * kMB,
                   d.d_in, kMB, 64) ||
        !encode_2d(reinterpret_cast<CUtensorMap*>(&p->tmap_dzt128), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, p->dzt,
                   (uint64_t)cap * d.d_hidden, kMB, 128, kMB) ||
        (d.d_hidden % 256 == 0 &&
         !encode_2d(reinterpret_cast<CUtensorMap*>(&p->tmap_dzt256), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, p->dzt,
                    (uint64_t)cap * d.d_hidden, kMB, 256, kMB)))
        return cudaErrorInvalidValue;
    // same boxes as the scratch sets' operands: slot j at rows [j*d_in, (j+1)*d_in) of X^T, [j*d_h, (j+1)*d_h) of dZ^T
    if (!encode_2d(reinterpret_cast<CUtensorMap*>(&p->tmap_xt), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, p->xtb,
                   (uint64_t)cap * d.d_in, kMB, kTileM, kMB) ||
        !encode_2d(reinterpret_cast<CUtensorMap*>(&p->tmap_dzt), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, p->dzt,
                   (uint64_t)cap * d.d_hidden, kMB, kDwN, kMB))
        return cudaErrorInvalidValue;
    return cudaSuccess;
}

cudaError_t launch_mlp_gather_small(const MlpDims& d, const MlpPool& pool, const MlpSlots& slots, const uint8_t* owners, int n,
                                    int first_worker, int n_workers, unsigned long long keep_mask, float* acc_set,
                                    size_t row_stride, cudaStream_t stream, bool chained) {
    if (n < 1 || n > kMlpMaxSlots || n_workers < 1) return cudaErrorInvalidValue;
    GatherList gl;
    gl.slots = slots;
    for (int q = 0; q < kMlpMaxSlots; ++q) gl.owner[q] = q < n ? owners[q] : (uint8_t)255;
    const int n_small = d.d_hidden + d.d_hidden * d.d_out + d.d_out;
    const size_t o_small = (size_t)d.d_in * d.d_hidden;
    const float* part = pool.part;
    return launch_kernel(k_gather_small, dim3((n_small + 255) / 256, n_workers), 256, 0, stream, chained, part, pool.part_stride, gl, n,
                         first_worker, keep_mask, acc_set, row_stride, o_small, n_small);
}

cudaError_t mlp_make_shadow_tmap(void* tmap_out, const MlpDims& d, __nv_bfloat16* shadow) {
    // W1 slice of a bf16 copy of the parameters: [d_in][d_hidden] bf16, boxes of 128 rows x 64 columns
    return encode_2d(reinterpret_cast<CUtensorMap*>(tmap_out), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, shadow, d.d_in, d.d_hidden,
                     kTileM, 64)
               ? cudaSuccess
               : cudaErrorInvalidValue;
}

cudaError_t launch_mlp_sync_small(const MlpDims& d, const MlpPool& pool, const MlpSlots& slots, int nb, const float* x_in,
                                  float* x_out, float* v, __nv_bfloat16* shadow_out, float B, float lr, float mu, float wd,
                                  float lambda_dc, float disp_scale, int32_t* cnt, int32_t* log_row, int W, cudaStream_t stream,
                                  bool chained) {
    if (nb < 1 || nb > kMlpMaxSlots) return cudaErrorInvalidValue;
    const size_t w1 = (size_t)d.d_in * d.d_hidden;
    const int n_small = d.d_hidden + d.d_hidden * d.d_out + d.d_out;
    const W1StepCoef cf{1.0f / B, lr, mu, wd, lambda_dc, disp_scale};
    const float* part = pool.part;
    const float* xi = x_in + w1;
    return launch_kernel(k_sync_small_pooled, (n_small + 255) / 256, 256, 0, stream, chained, part, pool.part_stride, slots, nb, xi,
                         x_out + w1, v + w1, shadow_out ? shadow_out + w1 : nullptr, n_small, cf, cnt, log_row, W);
}

namespace {
template <int kN>
cudaError_t sync_w1_launch(const MlpDims& d, const MlpScratch& s, const TmapBytes& tm_a, const TmapBytes& tm_b, const MlpSlots& slots,
                           int nb, const void* tm_x_in, const void* tm_x_out, const void* tm_v, const void* tm_shadow,
                           const W1StepCoef& cf, int max_ctas, cudaStream_t stream, bool chained) {
    static bool opted_in[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !opted_in[dev]) {
        e = cudaFuncSetAttribute(k_sync_w1<kN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(StepSmem<kN>) + 1024);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) opted_in[dev] = true;
    }
    const int n_tiles_n = d.d_hidden / kN, n_tiles = n_tiles_n * (d.d_in / kTileM);
    int ctas = n_tiles < s.num_sms ? n_tiles : s.num_sms;
    if (max_ctas > 0 && ctas > max_ctas) ctas = max_ctas;
    const CUtensorMap& shadow_map = *reinterpret_cast<const CUtensorMap*>(tm_shadow ? tm_shadow : tm_x_out);
    return launch_kernel(k_sync_w1<kN>, ctas, 64 + kStepEpiThreads, sizeof(StepSmem<kN>) + 1024, stream, chained,
                         *reinterpret_cast<const CUtensorMap*>(&tm_a), *reinterpret_cast<const CUtensorMap*>(&tm_b),
                         *reinterpret_cast<const CUtensorMap*>(tm_x_in), *reinterpret_cast<const CUtensorMap*>(tm_x_out),
                         *reinterpret_cast<const CUtensorMap*>(tm_v), shadow_map, slots, n_tiles_n, n_tiles, d.d_in, d.d_hidden, nb,
                         cf, tm_shadow ? 1 : 0, s.status);
}
}  // namespace

cudaError_t launch_mlp_sync_w1(const MlpDims& d, const MlpScratch& s, const MlpPool& pool, const MlpSlots& slots, int nb,
                               const void* tm_x_in, const void* tm_x_out, const void* tm_v, const void* tm_shadow,
                               float B, float lr, float mu, float wd, float lambda_dc, float disp_scale, int max_ctas,
                               cudaStream_t stream, bool chained) {
    if (nb < 1 || nb > kMlpMaxSlots || d.d_hidden % 128 != 0) return cudaErrorInvalidValue;
    const W1StepCoef cf{1.0f / B, lr, mu, wd, lambda_dc, disp_scale};
    // 128 x 256 tiles where the layer allows them and there are enough of them to go round
    if (d.d_hidden % 256 == 0 && max_ctas != -128)
        return sync_w1_launch<256>(d, s, pool.tmap_xt, pool.tmap_dzt256, slots, nb, tm_x_in, tm_x_out, tm_v, tm_shadow, cf, max_ctas,
                                   stream, chained);
    return sync_w1_launch<128>(d, s, pool.tmap_xt, pool.tmap_dzt128, slots, nb, tm_x_in, tm_x_out, tm_v, tm_shadow, cf,
                               max_ctas < 0 ? 0 : max_ctas, stream, chained);
}

cudaError_t mlp_make_acc_tmap(void* tmap_out, const MlpDims& d, float* acc_row) {
    // W1 slice of a worker's accumulator: [d_in][d_hidden] fp32 at offset 0 of the flat row.
    return encode_2d(reinterpret_cast<CUtensorMap*>(tmap_out), CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, acc_row, d.d_in,
                     d.d_hidden, kTileM, 32)
               ? cudaSuccess
               : cudaErrorInvalidValue;
}

cudaError_t launch_mlp_cast(const MlpDims& d, const MlpScratch& s, int slot0, int nb, const void* const* x_devs, bool x_is_bf16,
                            const int32_t* const* y_devs, const MlpPool* pool, cudaStream_t stream, bool chained, MlpMark mark,
                            void* user) {
    if (nb < 1 || nb > kMaxBatch) return cudaErrorInvalidValue;
    CastList in{};
    for (int j = 0; j < nb; ++j) {
        in.x[j] = x_devs[j];
        in.y[j] = y_devs[j];
    }
    mark(user, ABS_K_MLP_FWD, -1, stream);   // part 0 of the forward class: the cast
    // micro-batch j of the call goes to slot slot0 + j of the scratch set, or of the pool
    __nv_bfloat16* xb = (pool ? pool->xb : s.xb) + (size_t)slot0 * kMB * d.d_in;
    __nv_bfloat16* xtb = (pool ? pool->xtb : s.xtb) + (size_t)slot0 * d.d_in * kMB;
    int32_t* yc = (pool ? pool->ycopy : s.ycopy) + slot0 * kMB;
    const dim3 grid(d.d_in / 16, nb);
    const cudaError_t e = x_is_bf16 ? launch_kernel(k_cast_x<true>, grid, 256, 0, stream, chained, in, xb, xtb, yc, d.d_in)
                                    : launch_kernel(k_cast_x<false>, grid, 256, 0, stream, chained, in, xb, xtb, yc, d.d_in);
    mark(user, ABS_K_MLP_FWD, 1, stream);
    return e;
}

template <int NB>
cudaError_t fwd1_launch(dim3 grid, cudaStream_t stream, bool chained, bool light, const CUtensorMap& tw, const CUtensorMap& tx,
                        float* zpart, int d_in, int d_h, int xb_row0, int* status) {
    if (light)
        return launch_kernel(k_fwd1_tcgen05<NB, true>, grid, 128, sizeof(FwdSmem<NB, true>) + 1024, stream, chained, tw, tx, zpart,
                             d_in, d_h, xb_row0, status);
    return launch_kernel(k_fwd1_tcgen05<NB, false>, grid, 128, sizeof(FwdSmem<NB, false>) + 1024, stream, chained, tw, tx, zpart,
                         d_in, d_h, xb_row0, status);
}

cudaError_t launch_mlp_front(const MlpDims& d, const MlpScratch& s, const float* x_pub, const __nv_bfloat16* shadow,
                             int shadow_idx, int nb, bool store, float* acc_row, int32_t* cnt, const MlpPool* pool,
                             int pool_slot0, const MlpWorkers* workers, int variant, cudaStream_t stream, int chain, MlpMark mark,
                             void* user) {
    const size_t o_b1 = (size_t)d.d_in * d.d_hidden, o_w2 = o_b1 + d.d_hidden, o_b2 = o_w2 + (size_t)d.d_hidden * d.d_out;
    cudaError_t e;
    const unsigned n_cta = d.d_hidden / kHB;
    const bool light = (variant & kMlpLightBit) != 0;

    // every K split must be a whole number of 64-wide pipeline steps (d_in is a multiple of 128).  Eight splits (256
    // CTAs, two per SM) measured slower than four: 34.7 against 33.4 us per micro-batch, 16.7 against 15.5 batched.
    // A call of several micro-batches has enough MMA work per CTA with two splits, and every split costs the
    // call 2 x 1 MB of partial sums per micro-batch (measured, batch calls of up to 4 / 8: 14.5 -> 13.8 / 13.0 -> 12.3 us
    // per micro-batch; with ABS_FLAG_MLP_DEFER 9.5 -> 9.0 / 9.5 -> 8.8; one split was no better than two).
    int nsplit = nb == 1 ? kSplitK : 2;
    while (nsplit > 1 && d.d_in % (64 * nsplit) != 0) nsplit /= 2;
    const CUtensorMap& tw = *reinterpret_cast<const CUtensorMap*>(&s.tmap_w1[shadow_idx]);
    const CUtensorMap& tx = *reinterpret_cast<const CUtensorMap*>(pool ? &pool->tmap_xb : &s.tmap_xb);
    const int xb_row0 = pool ? pool_slot0 * kMB : 0;
    const dim3 grid(d.d_hidden / 128, nsplit);
    mark(user, ABS_K_MLP_FWD, -2, stream);       // part 1: the forward GEMM
    switch (nb) {                                // the nb micro-batches are stacked along N of one GEMM
        case 1: e = fwd1_launch<1>(grid, stream, (chain & kChainFwd1) != 0, light, tw, tx, s.zpart, d.d_in, d.d_hidden, xb_row0, s.status); break;
        case 2: e = fwd1_launch<2>(grid, stream, (chain & kChainFwd1) != 0, light, tw, tx, s.zpart, d.d_in, d.d_hidden, xb_row0, s.status); break;
        case 3: e = fwd1_launch<3>(grid, stream, (chain & kChainFwd1) != 0, light, tw, tx, s.zpart, d.d_in, d.d_hidden, xb_row0, s.status); break;
        case 4: e = fwd1_launch<4>(grid, stream, (chain & kChainFwd1) != 0, light, tw, tx, s.zpart, d.d_in, d.d_hidden, xb_row0, s.status); break;
        case 5: e = fwd1_launch<5>(grid, stream, (chain & kChainFwd1) != 0, light, tw, tx, s.zpart, d.d_in, d.d_hidden, xb_row0, s.status); break;
        case 6: e = fwd1_launch<6>(grid, stream, (chain & kChainFwd1) != 0, light, tw, tx, s.zpart, d.d_in, d.d_hidden, xb_row0, s.status); break;
        case 7: e = fwd1_launch<7>(grid, stream, (chain & kChainFwd1) != 0, light, tw, tx, s.zpart, d.d_in, d.d_hidden, xb_row0, s.status); break;
        case 8: e = fwd1_launch<8>(grid, stream, (chain & kChainFwd1) != 0, light, tw, tx, s.zpart, d.d_in, d.d_hidden, xb_row0, s.status); break;
        default: return cudaErrorInvalidValue;
    }
    mark(user, ABS_K_MLP_FWD, 1, stream);
    if (e != cudaSuccess) return e;
    mark(user, ABS_K_MLP_FWD, -3, stream);       // part 2: bias, ReLU, partial logits
    const float* zp = s.zpart;
    const float* b1 = x_pub + o_b1;
    const __nv_bfloat16* w2b = shadow + o_w2;
    const float* b2 = x_pub + o_b2;
    const int32_t* yc = pool ? pool->ycopy + (size_t)pool_slot0 * kMB : s.ycopy;
    e = launch_kernel(k_fwd2, dim3(n_cta, nb), 256, 0, stream, (chain & kChainFwd2) != 0, zp, nsplit, b1, w2b, s.hbt, s.lpart, s.gpart, s.tickets,
                      d.d_hidden, d.d_out, b2, yc, s.dlbuf, s.tickets2);
    mark(user, ABS_K_MLP_FWD, 1, stream);
    if (e != cudaSuccess) return e;

    mark(user, ABS_K_MLP_BWD, -1, stream);
    const __nv_bfloat16* hbt = s.hbt;
    const float* dlbuf = s.dlbuf;
    __nv_bfloat16* dzt = pool ? pool->dzt + (size_t)pool_slot0 * d.d_hidden * kMB : s.dzt;
    float* part = pool ? pool->part + (size_t)pool_slot0 * pool->part_stride : nullptr;
    const size_t part_stride = pool ? pool->part_stride : 0;
    e = launch_kernel(k_bwd, dim3(n_cta, nb), 256, 0, stream, (chain & kChainBwd) != 0, hbt, dlbuf, w2b, dzt, s.bpart,
                      s.tickets_b, acc_row + o_b1, acc_row + o_w2, acc_row + o_b2, cnt, d.d_hidden, d.d_out, store ? 1 : 0, part,
                      part_stride, workers ? *workers : MlpWorkers{});
    mark(user, ABS_K_MLP_BWD, 1, stream);
    return e;
}

template <int kN, bool kLight>
cudaError_t dw1_ring_launch(const MlpDims& d, const MlpScratch& s, const CUtensorMap& ta, const CUtensorMap& tb,
                            const CUtensorMap& tc, const MlpSlots& sl, int nb, int st, cudaStream_t stream, bool chained) {
    const int n_tiles_n = d.d_hidden / kN, n_tiles = n_tiles_n * (d.d_in / kTileM);
    const int ctas = n_tiles < s.num_sms ? n_tiles : s.num_sms;
    return launch_kernel(k_dw1_ring<kN, kLight>, ctas, 192, sizeof(DwRingSmem<kN, kLight>) + 1024, stream, chained, ta, tb, tc,
                         sl, n_tiles_n, n_tiles, d.d_in, d.d_hidden, nb, st, s.status);
}

cudaError_t launch_mlp_dw1(const MlpDims& d, const MlpScratch& s, const MlpPool* pool, const MlpSlots* slots, float* acc_row,
                           const void* acc_tmap, int nb, bool store, int variant, cudaStream_t stream, bool chained,
                           MlpMark mark, void* user) {
    const int st = store ? 1 : 0;
    const bool light = (variant & kMlpLightBit) != 0;
    if (nb < 1 || nb > (pool ? kMlpMaxSlots : kMaxBatch) || (pool && !slots)) return cudaErrorInvalidValue;
    mark(user, ABS_K_MLP_DW1, -1, stream);
    const CUtensorMap& ta = *reinterpret_cast<const CUtensorMap*>(pool ? &pool->tmap_xt : &s.tmap_xt);
    const CUtensorMap& tb = *reinterpret_cast<const CUtensorMap*>(pool ? &pool->tmap_dzt : &s.tmap_dzt);
    const CUtensorMap& tc = *reinterpret_cast<const CUtensorMap*>(acc_tmap);
    MlpSlots sl;
    if (pool) {
        sl = *slots;
    } else {
        for (int j = 0; j < kMlpMaxSlots; ++j) sl.s[j] = (uint16_t)(j < kMaxBatch ? j : 0);
    }
    // Which kernel: bit 4 (ring) or 8 (register prefetch) forces one; otherwise the measured best for the case: the
    // persistent ring kernel when the tile is stored (it never reads the accumulator) and for K-batched adds, the
    // register-prefetch kernel for single adds.
    int kind = (variant & 4) ? 4 : (variant & 8) ? 8 : 0;
    if (kind == 0) kind = (store || nb > 1) ? 4 : 8;
    if (nb > kMaxBatch) kind = 4;          // the register-prefetch kernel holds every operand in shared memory at once
    cudaError_t e;
    if (kind == 4) {
        if (nb > 1 && !(variant & 32))     // K-batched: 128 x 128 tiles (bit 32 keeps 128 x 64)
            e = light ? dw1_ring_launch<128, true>(d, s, ta, tb, tc, sl, nb, st, stream, chained)
                      : dw1_ring_launch<128, false>(d, s, ta, tb, tc, sl, nb, st, stream, chained);
        else
            e = light ? dw1_ring_launch<64, true>(d, s, ta, tb, tc, sl, nb, st, stream, chained)
                      : dw1_ring_launch<64, false>(d, s, ta, tb, tc, sl, nb, st, stream, chained);
    } else {
        const size_t smem = dw_regs_buf_bytes(nb) + sizeof(DwRegCtl) + 1024;
        e = launch_kernel(k_dw1_regs, dim3(d.d_hidden / kDwN, d.d_in / kTileM), 256, smem, stream, chained, ta, tb, sl, acc_row,
                          d.d_in, d.d_hidden, nb, st, s.status);
    }
    mark(user, ABS_K_MLP_DW1, 1, stream);
    return e;
}

}  // namespace abs_sgd
