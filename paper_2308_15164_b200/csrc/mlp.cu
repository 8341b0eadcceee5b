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
// Kernels (all on the caller's stream):
//   k_cast_x      X fp32 -> bf16 in both orientations
//   k_fwd1_tcgen05  Z^T partials = W1^T X^T, split over d_in, on tcgen05 (W1 as an MN-major operand)
//   (k_fwd1         the same on CUDA cores, kept as a cross-check selectable through abs_set_launch)
//   k_fwd2        Z = sum of partials + b1, gate, bf16(H), per-chunk partial logits
//   k_loss        logits, softmax, dL, db2 += ...
//   k_bwd         dH, dZ, db1 += ..., dW2 += ..., bf16(dZ)^T, b_i += 1
//   k_dw1_tcgen05 dW1 tile = A B^T on the 5th-gen tensor cores (TMEM accumulator); epilogue
//                 adds the tile into the worker's accumulator slice via TMA load / TMA store.
#include <cuda.h>

#include <cstdio>

#include "abs_internal.h"

namespace abs_sgd {

namespace {

constexpr int kMB = 64;          // samples per micro-batch = K of the dW1 contraction
constexpr int kOutPad = 16;      // logits / dL rows are padded to 16 columns
constexpr int kSplitK = 4;       // forward GEMM: d_in is split into this many partial sums
constexpr int kChunkH = 128;     // hidden units per CTA in k_fwd2 (partial-logit chunk)

__device__ __forceinline__ float bf16_to_f(__nv_bfloat16 v) { return __bfloat162float(v); }

// --------------------------------------------------------------------------------------------
// X [64][d_in] fp32  ->  xb [64][d_in] bf16  and  xtb [d_in][64] bf16
// --------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_cast_x(const float* __restrict__ x, __nv_bfloat16* __restrict__ xb,
                                                __nv_bfloat16* __restrict__ xtb, int d_in) {
    __shared__ __nv_bfloat16 tile[kMB][64 + 2];
    const int c0 = blockIdx.x * 64;
    for (int e = threadIdx.x; e < kMB * 64; e += 256) {
        const int r = e / 64, c = e % 64;
        const __nv_bfloat16 v = __float2bfloat16_rn(x[(size_t)r * d_in + c0 + c]);
        xb[(size_t)r * d_in + c0 + c] = v;
        tile[r][c] = v;
    }
    __syncthreads();
    for (int e = threadIdx.x; e < kMB * 64; e += 256) {
        const int c = e / 64, r = e % 64;
        xtb[(size_t)(c0 + c) * kMB + r] = tile[r][c];
    }
}

// --------------------------------------------------------------------------------------------
// Forward GEMM, CUDA cores:  zpart[s][h][r] = sum_{k in split s} W1b[k][h] * xb[r][k]
// CTA tile: 64 hidden x 64 samples, 256 threads, 4x4 outputs per thread.
// --------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_fwd1(const __nv_bfloat16* __restrict__ w1b, const __nv_bfloat16* __restrict__ xb,
                                              float* __restrict__ zpart, int d_in, int d_h) {
    constexpr int KT = 32;
    __shared__ float sw[KT][64 + 4];   // [k][h]
    __shared__ float sx[KT][64 + 4];   // [k][r]
    const int h0 = blockIdx.x * 64;
    const int s = blockIdx.y;
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
// Z = sum_s zpart + b1 ; gate ; bf16(H) ; partial logits of this chunk of hidden units.
// CTA: kChunkH hidden units; 256 threads = 4 groups of 64 samples.
// --------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_fwd2(const float* __restrict__ zpart, const float* __restrict__ b1,
                                              const __nv_bfloat16* __restrict__ w2b, float* __restrict__ zt,
                                              __nv_bfloat16* __restrict__ hbt, float* __restrict__ lpart, int d_h,
                                              int d_out, int nsplit) {
    __shared__ float red[4][kMB][kOutPad];
    const int r = threadIdx.x % kMB, grp = threadIdx.x / kMB;
    const int h_beg = blockIdx.x * kChunkH;
    float l[kOutPad];
#pragma unroll
    for (int o = 0; o < kOutPad; ++o) l[o] = 0.f;
    for (int h = h_beg + grp; h < h_beg + kChunkH; h += 4) {
        float z = 0.f;
        for (int s = 0; s < nsplit; ++s) z += zpart[((size_t)s * d_h + h) * kMB + r];
        z += b1[h];
        zt[(size_t)h * kMB + r] = z;
        const __nv_bfloat16 hb = __float2bfloat16_rn(z > 0.f ? z : 0.f);
        hbt[(size_t)h * kMB + r] = hb;
        const float hf = bf16_to_f(hb);
        for (int o = 0; o < d_out; ++o) l[o] = fmaf(hf, bf16_to_f(w2b[(size_t)h * d_out + o]), l[o]);
    }
#pragma unroll
    for (int o = 0; o < kOutPad; ++o) red[grp][r][o] = l[o];
    __syncthreads();
    for (int e = threadIdx.x; e < kMB * kOutPad; e += 256) {
        const int rr = e / kOutPad, o = e % kOutPad;
        lpart[((size_t)blockIdx.x * kMB + rr) * kOutPad + o] = (red[0][rr][o] + red[1][rr][o]) + (red[2][rr][o] + red[3][rr][o]);
    }
}

// --------------------------------------------------------------------------------------------
// One CTA: logits = sum of chunk partials + b2 ; softmax ; dL = (p - onehot)/mb ; db2 += sum_r dL.
// --------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kMB) k_loss(const float* __restrict__ lpart, int n_chunks, const float* __restrict__ b2,
                                              const int32_t* __restrict__ y, float* __restrict__ dl,
                                              __nv_bfloat16* __restrict__ dlb, float* acc_b2, int d_out) {
    __shared__ float sdl[kMB][kOutPad];
    const int r = threadIdx.x;
    float l[kOutPad];
    float mx = -INFINITY;
    for (int o = 0; o < d_out; ++o) {
        float s = 0.f;
        for (int c = 0; c < n_chunks; ++c) s += lpart[((size_t)c * kMB + r) * kOutPad + o];
        l[o] = s + b2[o];
        mx = fmaxf(mx, l[o]);
    }
    float den = 0.f;
    for (int o = 0; o < d_out; ++o) {
        l[o] = expf(l[o] - mx);
        den += l[o];
    }
    const int yr = y[r];
    for (int o = 0; o < kOutPad; ++o) {
        float g = 0.f;
        if (o < d_out) g = (l[o] / den - (o == yr ? 1.f : 0.f)) * (1.0f / kMB);
        dl[r * kOutPad + o] = g;
        dlb[r * kOutPad + o] = __float2bfloat16_rn(g);
        sdl[r][o] = g;
    }
    __syncthreads();
    if (r < d_out) {
        float s = 0.f;
        for (int rr = 0; rr < kMB; ++rr) s += sdl[rr][r];
        acc_b2[r] += s;
    }
}

// --------------------------------------------------------------------------------------------
// Backward through layer 2 and the ReLU, hidden-major.  CTA: 8 hidden units, 64 threads each.
//   dH[r][h] = sum_o bf16(dL)[r][o] * W2b[h][o] ; dZ = dH * [Z > 0] ; dzt[h][r] = bf16(dZ)
//   db1[h] += sum_r dZ ; dW2[h][o] += sum_r bf16(H)[h][r] * bf16(dL)[r][o] ; b_i += 1
// --------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(512) k_bwd(const float* __restrict__ zt, const __nv_bfloat16* __restrict__ hbt,
                                             const __nv_bfloat16* __restrict__ dlb, const __nv_bfloat16* __restrict__ w2b,
                                             __nv_bfloat16* __restrict__ dzt, float* acc_b1, float* acc_w2, int32_t* cnt,
                                             int d_out) {
    __shared__ float sdl[kMB][kOutPad];
    __shared__ float red[8][2][kOutPad + 1];
    for (int e = threadIdx.x; e < kMB * kOutPad; e += 512) sdl[e / kOutPad][e % kOutPad] = bf16_to_f(dlb[e]);
    __syncthreads();
    const int r = threadIdx.x % kMB, g = threadIdx.x / kMB;
    const int h = blockIdx.x * 8 + g;
    float dh = 0.f;
    for (int o = 0; o < d_out; ++o) dh = fmaf(sdl[r][o], bf16_to_f(w2b[(size_t)h * d_out + o]), dh);
    const float dz = zt[(size_t)h * kMB + r] > 0.f ? dh : 0.f;
    dzt[(size_t)h * kMB + r] = __float2bfloat16_rn(dz);
    const float hf = bf16_to_f(hbt[(size_t)h * kMB + r]);
    // reductions over the 64 samples: values [0, d_out) are dW2[h][o], value d_out is db1[h]
    float vals[kOutPad + 1];
#pragma unroll
    for (int o = 0; o < kOutPad; ++o) vals[o] = o < d_out ? hf * sdl[r][o] : 0.f;
    vals[kOutPad] = dz;
#pragma unroll
    for (int o = 0; o <= kOutPad; ++o) {
        float v = vals[o];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
        vals[o] = v;
    }
    const int half = (threadIdx.x % kMB) / 32;
    if (threadIdx.x % 32 == 0)
#pragma unroll
        for (int o = 0; o <= kOutPad; ++o) red[g][half][o] = vals[o];
    __syncthreads();
    if (r <= kOutPad) {
        const float s = red[g][0][r] + red[g][1][r];
        if (r < d_out) acc_w2[(size_t)h * d_out + r] += s;
        else if (r == kOutPad) acc_b1[h] += s;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) cnt[0] += 1;   // M_t^i += M_r
}

// ============================================================================================
// dW1 = X^T dZ on tcgen05.  One CTA per 128 x 128 output tile; K = 64 = four UMMA steps.
// ============================================================================================
constexpr int kTileM = 128, kTileN = 128;
constexpr uint32_t kSpinLimit = 1u << 22;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
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
// Instruction descriptor: D = f32, A = B = bf16, both K-major, M x N tile.
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int M, int N) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

struct DwSmem {
    alignas(1024) uint8_t a[kTileM * 128];        // A tile  [128 m][64 k] bf16, swizzled rows
    alignas(1024) uint8_t b[kTileN * 128];        // B tile  [128 n][64 k] bf16
    alignas(1024) float c[4][kTileM * 32];        // accumulator tile as 4 column panels [128][32] fp32, swizzled rows
    alignas(8) uint64_t bar_ab;
    uint64_t bar_c;
    uint64_t bar_mma;
    uint32_t tmem_base;
    uint32_t failed;
};

template <bool kReduce>
__global__ void __launch_bounds__(128) k_dw1_tcgen05(const __grid_constant__ CUtensorMap tm_xt,
                                                     const __grid_constant__ CUtensorMap tm_dzt,
                                                     const __grid_constant__ CUtensorMap tm_acc, int* status) {
    extern __shared__ uint8_t smem_raw[];
    DwSmem& s = *reinterpret_cast<DwSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int n0 = blockIdx.x * kTileN;   // hidden offset
    const int m0 = blockIdx.y * kTileM;   // input-feature offset

    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s.tmem_base)), "r"(kTileN) : "memory");
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
        mbar_expect_tx(&s.bar_ab, kTileM * 128 + kTileN * 128);
        tma_load_2d(s.a, &tm_xt, 0, m0, &s.bar_ab);
        tma_load_2d(s.b, &tm_dzt, 0, n0, &s.bar_ab);
        if (!kReduce) {   // the accumulator tile streams in while the MMA runs
            mbar_expect_tx(&s.bar_c, kTileM * kTileN * 4);
#pragma unroll
            for (int p = 0; p < 4; ++p) tma_load_2d(s.c[p], &tm_acc, n0 + p * 32, m0, &s.bar_c);
        }
        if (mbar_wait(&s.bar_ab, 0)) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint64_t da = umma_desc_k_sw128(smem_u32(s.a));
            const uint64_t db = umma_desc_k_sw128(smem_u32(s.b));
            constexpr uint32_t idesc = umma_idesc_bf16(kTileM, kTileN);
#pragma unroll
            for (int k = 0; k < kMB / 16; ++k) {
                const uint32_t accumulate = k > 0;
                // advancing K by 16 bf16 = 32 bytes inside the swizzled row: +2 in the address field
                asm volatile(
                    "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                    " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
                    ::"r"(tmem), "l"(da + 2 * k), "l"(db + 2 * k), "r"(idesc), "r"(accumulate) : "memory");
            }
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&s.bar_mma)) : "memory");
        } else {
            s.failed = 1;
        }
    }
    __syncwarp();

    bool ok = mbar_wait(&s.bar_mma, 0);
    if (!kReduce) ok = mbar_wait(&s.bar_c, 0) && ok;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (ok) {
        const int row = threadIdx.x;                    // TMEM lane = output row
#pragma unroll 1
        for (int p = 0; p < 4; ++p) {
            uint32_t v[32];
            const uint32_t taddr = tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)(p * 32);
            asm volatile(
                "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
                  "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
                  "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
                  "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                : "r"(taddr) : "memory");
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            // panel p: row `row` is 128 bytes; 16-byte chunk j sits at position j ^ (row % 8)
            float4* prow = reinterpret_cast<float4*>(s.c[p] + row * 32);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                float4* q = prow + (j ^ (row & 7));
                float4 d = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                       __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
                if (!kReduce) {
                    const float4 c = *q;
                    d.x += c.x; d.y += c.y; d.z += c.z; d.w += c.w;
                }
                *q = d;
            }
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
            for (int p = 0; p < 4; ++p) {
                if (kReduce) tma_reduce_add_2d(&tm_acc, s.c[p], n0 + p * 32, m0);
                else tma_store_2d(&tm_acc, s.c[p], n0 + p * 32, m0);
            }
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        } else {
            atomicExch(status, ABS_ETIMEOUT);
            // give copies that may still be in flight a bounded chance to land before smem is released
            mbar_wait(&s.bar_ab, 0);
            if (!kReduce) mbar_wait(&s.bar_c, 0);
        }
    }
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTileN) : "memory");
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
// One CTA per (128-hidden tile, K split); a kFwdStages-deep TMA -> MMA pipeline streams the
// weights once.  Warp 0 lane 0 issues TMA, warp 1 lane 0 issues MMAs, all four warps store D.
// ============================================================================================
constexpr int kFwdStages = 6;
constexpr int kFwdStageBytes = 2 * 8192 + 8192;   // two A boxes + one B box

__device__ __forceinline__ uint64_t umma_desc_mn_sw128(uint32_t smem_addr, uint32_t lbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);
    d |= (uint64_t)(lbo_bytes >> 4) << 16;                // leading-dim byte offset: next 64-wide MN block
    d |= (uint64_t)(1024 >> 4) << 32;                     // stride-dim byte offset: next group of 8 k-rows
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

struct FwdSmem {
    alignas(1024) uint8_t stage[kFwdStages][kFwdStageBytes];   // [A h0..63 | A h64..127 | B]
    alignas(8) uint64_t full[kFwdStages];
    uint64_t empty[kFwdStages];
    uint64_t done;
    uint32_t tmem_base;
    uint32_t failed;
};

__global__ void __launch_bounds__(128) k_fwd1_tcgen05(const __grid_constant__ CUtensorMap tm_w1,
                                                      const __grid_constant__ CUtensorMap tm_xb, float* __restrict__ zpart,
                                                      int d_in, int d_h, int* status) {
    extern __shared__ uint8_t smem_raw[];
    FwdSmem& s = *reinterpret_cast<FwdSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int h0 = blockIdx.x * 128;
    const int split = blockIdx.y;
    const int k_per = d_in / (int)gridDim.y;
    const int kbeg = split * k_per;
    const int nk = k_per / 64;                       // pipeline steps of 64 k

    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s.tmem_base)), "r"(64) : "memory");
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
            tma_load_2d(s.stage[st] + 16384, &tm_xb, k0, 0, &s.full[st]);
        }
    } else if (warp == 1 && lane == 0) {             // ---- MMA issuer
        constexpr uint32_t idesc = umma_idesc_bf16(128, 64) | (1u << 15);   // A is MN-major
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
                const uint64_t da = umma_desc_mn_sw128(a0 + k * 2048, 8192);
                const uint32_t accumulate = (kb > 0 || k > 0);
                asm volatile(
                    "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                    " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
                    ::"r"(tmem), "l"(da), "l"(db + 2 * k), "r"(idesc), "r"(accumulate) : "memory");
            }
            // frees the stage for the producer once these MMAs have read it
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&s.empty[st])) : "memory");
        }
        if (ok) asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&s.done)) : "memory");
        else s.failed = 1;
    }
    __syncwarp();

    bool ok = mbar_wait(&s.done, 0);
    ok = __all_sync(0xffffffffu, ok);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (ok) {
        const int h = h0 + threadIdx.x;               // TMEM lane = hidden unit
        float* out = zpart + ((size_t)split * d_h + h) * kMB;
#pragma unroll 1
        for (int p = 0; p < 2; ++p) {
            uint32_t v[32];
            const uint32_t taddr = tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)(p * 32);
            asm volatile(
                "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
                  "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
                  "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
                  "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                : "r"(taddr) : "memory");
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
            for (int j = 0; j < 8; ++j)
                *reinterpret_cast<float4*>(out + p * 32 + 4 * j) =
                    make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]), __uint_as_float(v[4 * j + 2]),
                                __uint_as_float(v[4 * j + 3]));
        }
    } else if (threadIdx.x == 0) {
        atomicExch(status, ABS_ETIMEOUT);
        // bounded chance for copies still in flight to land before shared memory is released
        for (int i = 0; i < kFwdStages; ++i) mbar_wait(&s.full[i], 0);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(64) : "memory");
    }
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

}  // namespace

size_t mlp_scratch_bytes(const MlpDims& d) {
    size_t o = 0;
    auto take = [&](size_t b) { o = align_up(o + b, 1024); };
    take((size_t)kMB * d.d_in * 2);                 // xb
    take((size_t)d.d_in * kMB * 2);                 // xtb
    take((size_t)kSplitK * d.d_hidden * kMB * 4);   // zpart
    take((size_t)d.d_hidden * kMB * 4);             // zt
    take((size_t)d.d_hidden * kMB * 2);             // hbt
    take((size_t)d.d_hidden * kMB * 2);             // dzt
    take((size_t)(d.d_hidden / kChunkH) * kMB * kOutPad * 4);   // lpart
    take((size_t)kMB * kOutPad * 4);                // dl
    take((size_t)kMB * kOutPad * 2);                // dlb
    take(256);                                      // status word
    return o;
}

cudaError_t mlp_scratch_init(MlpScratch* s, const MlpDims& d, void* base, __nv_bfloat16* shadow0,
                             __nv_bfloat16* shadow1, const char** err) {
    char* p = static_cast<char*>(base);
    size_t o = 0;
    auto take = [&](size_t b) { char* at = p + o; o = align_up(o + b, 1024); return at; };
    s->xb = reinterpret_cast<__nv_bfloat16*>(take((size_t)kMB * d.d_in * 2));
    s->xtb = reinterpret_cast<__nv_bfloat16*>(take((size_t)d.d_in * kMB * 2));
    s->zpart = reinterpret_cast<float*>(take((size_t)kSplitK * d.d_hidden * kMB * 4));
    s->zt = reinterpret_cast<float*>(take((size_t)d.d_hidden * kMB * 4));
    s->hbt = reinterpret_cast<__nv_bfloat16*>(take((size_t)d.d_hidden * kMB * 2));
    s->dzt = reinterpret_cast<__nv_bfloat16*>(take((size_t)d.d_hidden * kMB * 2));
    s->lpart = reinterpret_cast<float*>(take((size_t)(d.d_hidden / kChunkH) * kMB * kOutPad * 4));
    s->dl = reinterpret_cast<float*>(take((size_t)kMB * kOutPad * 4));
    s->dlb = reinterpret_cast<__nv_bfloat16*>(take((size_t)kMB * kOutPad * 2));
    s->status = reinterpret_cast<int*>(take(256));
    static_assert(sizeof(CUtensorMap) == sizeof(TmapBytes), "tensor map size");
    if (!encode_2d(reinterpret_cast<CUtensorMap*>(&s->tmap_xt), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, s->xtb, d.d_in, kMB,
                   kTileM, kMB) ||
        !encode_2d(reinterpret_cast<CUtensorMap*>(&s->tmap_dzt), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, s->dzt, d.d_hidden,
                   kMB, kTileN, kMB)) {
        *err = "cuTensorMapEncodeTiled failed for the dW1 operands";
        return cudaErrorInvalidValue;
    }
    // forward GEMM operands: W1 (bf16 shadow, [d_in][d_hidden]) in 64 x 64 boxes, xb [mb][d_in] in 64 x 64 boxes
    if (!encode_2d(reinterpret_cast<CUtensorMap*>(&s->tmap_w1[0]), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, shadow0, d.d_in,
                   d.d_hidden, 64, 64) ||
        !encode_2d(reinterpret_cast<CUtensorMap*>(&s->tmap_w1[1]), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, shadow1, d.d_in,
                   d.d_hidden, 64, 64) ||
        !encode_2d(reinterpret_cast<CUtensorMap*>(&s->tmap_xb), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, s->xb, kMB, d.d_in, kMB,
                   64)) {
        *err = "cuTensorMapEncodeTiled failed for the forward GEMM operands";
        return cudaErrorInvalidValue;
    }
    cudaError_t e0 = cudaFuncSetAttribute(k_fwd1_tcgen05, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)sizeof(FwdSmem) + 1024);
    if (e0 != cudaSuccess) {
        *err = "cudaFuncSetAttribute(forward kernel)";
        return e0;
    }
    cudaError_t e = cudaFuncSetAttribute(k_dw1_tcgen05<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)sizeof(DwSmem) + 1024);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(k_dw1_tcgen05<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(DwSmem) + 1024);
    if (e != cudaSuccess) *err = "cudaFuncSetAttribute(dW1 kernel)";
    return e;
}

cudaError_t mlp_make_acc_tmap(void* tmap_out, const MlpDims& d, float* acc_row) {
    // W1 slice of a worker's accumulator: [d_in][d_hidden] fp32 at offset 0 of the flat row.
    return encode_2d(reinterpret_cast<CUtensorMap*>(tmap_out), CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, acc_row, d.d_in,
                     d.d_hidden, kTileM, 32)
               ? cudaSuccess
               : cudaErrorInvalidValue;
}

cudaError_t launch_mlp_grad(const MlpDims& d, const MlpScratch& s, const float* x_pub, const __nv_bfloat16* shadow,
                            int shadow_idx, const float* x_dev, const int32_t* y_dev, float* acc_row, const void* acc_tmap,
                            int32_t* cnt, int variant, cudaStream_t stream, void (*mark)(void*, int, int), void* user) {
    const size_t o_b1 = (size_t)d.d_in * d.d_hidden, o_w2 = o_b1 + d.d_hidden, o_b2 = o_w2 + (size_t)d.d_hidden * d.d_out;
    const int n_chunks = d.d_hidden / kChunkH;
    cudaError_t e;

    mark(user, ABS_K_MLP_FWD, 0);
    k_cast_x<<<d.d_in / 64, 256, 0, stream>>>(x_dev, s.xb, s.xtb, d.d_in);
    // every K split must be a whole number of 64-wide pipeline steps (d_in is a multiple of 128)
    const int nsplit = (d.d_in % (64 * kSplitK) == 0) ? kSplitK : 2;
    if (variant & 2) {
        k_fwd1<<<dim3(d.d_hidden / 64, nsplit), 256, 0, stream>>>(shadow, s.xb, s.zpart, d.d_in, d.d_hidden);
    } else {
        const CUtensorMap* tw = reinterpret_cast<const CUtensorMap*>(&s.tmap_w1[shadow_idx]);
        const CUtensorMap* tx = reinterpret_cast<const CUtensorMap*>(&s.tmap_xb);
        k_fwd1_tcgen05<<<dim3(d.d_hidden / 128, nsplit), 128, sizeof(FwdSmem) + 1024, stream>>>(*tw, *tx, s.zpart, d.d_in,
                                                                                           d.d_hidden, s.status);
    }
    k_fwd2<<<n_chunks, 256, 0, stream>>>(s.zpart, x_pub + o_b1, shadow + o_w2, s.zt, s.hbt, s.lpart, d.d_hidden, d.d_out,
                                         nsplit);
    k_loss<<<1, kMB, 0, stream>>>(s.lpart, n_chunks, x_pub + o_b2, y_dev, s.dl, s.dlb, acc_row + o_b2, d.d_out);
    mark(user, ABS_K_MLP_FWD, 4);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;

    mark(user, ABS_K_MLP_BWD, 0);
    k_bwd<<<d.d_hidden / 8, 512, 0, stream>>>(s.zt, s.hbt, s.dlb, shadow + o_w2, s.dzt, acc_row + o_b1, acc_row + o_w2, cnt,
                                              d.d_out);
    mark(user, ABS_K_MLP_BWD, 1);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;

    mark(user, ABS_K_MLP_DW1, 0);
    const dim3 grid(d.d_hidden / kTileN, d.d_in / kTileM);
    const CUtensorMap* ta = reinterpret_cast<const CUtensorMap*>(&s.tmap_xt);
    const CUtensorMap* tb = reinterpret_cast<const CUtensorMap*>(&s.tmap_dzt);
    const CUtensorMap* tc = reinterpret_cast<const CUtensorMap*>(acc_tmap);
    if (variant & 1)
        k_dw1_tcgen05<true><<<grid, 128, sizeof(DwSmem) + 1024, stream>>>(*ta, *tb, *tc, s.status);
    else
        k_dw1_tcgen05<false><<<grid, 128, sizeof(DwSmem) + 1024, stream>>>(*ta, *tb, *tc, s.status);
    mark(user, ABS_K_MLP_DW1, 1);
    return cudaGetLastError();
}

}  // namespace abs_sgd
