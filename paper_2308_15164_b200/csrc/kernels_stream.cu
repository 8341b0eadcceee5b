// Streaming kernels of the delayed synchronous step (arXiv 2308.15164, Algorithm 1).
//
//   k_accumulate_*  Step 2:  G_t^i += g ;  b_i += 1      (k_accumulate_multi_*: n gradients in one pass)
//   k_sync          Step 1 + Eq. 6 + "Update parameters", fused:
//                     B = sum_i b_i ;  Gbar = (sum_i G_{t-1}^i) / B ;  compensation ;
//                     g = Gbar + wd*x ; v = mu*v + g ; x' = x - lr*v ;
//                     G_{t-1}^i <- 0 ; b_i <- 0 (after logging them)
//   k_sync_global   the same step when the workers sit on several GPUs: each rank's launch handles a slice of
//                   the vector over all ranks' rows (peer pointers) and writes x' to every rank
//
// Both are pure HBM streams (about 1 flop per 4 bytes), so the design goal is bytes in flight:
// 128-bit accesses, all independent loads of a thread issued before the first use, and one pass
// over every byte (each accumulator element is read once and overwritten with zero by the same
// thread that read it).  Launch shape: measured on B200, one tile per CTA (a grid of thousands
// of 256-thread CTAs) beats a persistent grid of 148 x k CTAs by 5-10 % for the accumulate kernels
// and for the fused step with up to 4 workers, so that is their default; the fused step with more
// workers runs its chunked form on a persistent grid (see launch_sync).  abs_set_launch overrides.
#include "abs_internal.h"

namespace abs_sgd {

namespace {

constexpr int kBlock = 256;

// Read-once global loads: bypass L1, mark evict-first in L2.
__device__ __forceinline__ float4 ld_stream(const float4* p) {
    float4 r;
    asm volatile("ld.global.cs.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w) : "l"(p));
    return r;
}
__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 r;
    asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}
__device__ __forceinline__ void st_stream(float4* p, float4 v) {
    asm volatile("st.global.cs.v4.f32 [%0], {%1,%2,%3,%4};" ::"l"(p), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// ------------------------------------------------------------------------------------------
// Step 2, fp32 gradient: 12 bytes per parameter (read g, read acc, write acc).
// ------------------------------------------------------------------------------------------
template <int U, bool kOverwrite>
__global__ void __launch_bounds__(kBlock) k_accumulate_f32(float* acc, const float* __restrict__ g,
                                                           unsigned long long n_vec, unsigned long long P,
                                                           int32_t* cnt) {
    float4* acc4 = reinterpret_cast<float4*>(acc);
    const float4* g4 = reinterpret_cast<const float4*>(g);
    const unsigned long long tile = (unsigned long long)kBlock * U;
    pdl_wait();      // the row may have been written by the kernel just ahead on the stream
    pdl_trigger();
    for (unsigned long long base = blockIdx.x * tile; base < n_vec; base += gridDim.x * tile) {
        float4 a[U], b[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const unsigned long long idx = base + (unsigned long long)u * kBlock + threadIdx.x;
            if (idx < n_vec) {
                b[u] = ld_stream(g4 + idx);
                if (!kOverwrite) a[u] = acc4[idx];
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const unsigned long long idx = base + (unsigned long long)u * kBlock + threadIdx.x;
            if (idx < n_vec) {
                if (kOverwrite) {
                    a[u] = b[u];
                } else {
                    a[u].x += b[u].x; a[u].y += b[u].y; a[u].z += b[u].z; a[u].w += b[u].w;
                }
                st_stream(acc4 + idx, a[u]);
            }
        }
    }
    if (blockIdx.x == 0) {
        const unsigned long long j = n_vec * 4 + threadIdx.x;   // ragged tail (P % 4 elements)
        if (j < P) acc[j] = kOverwrite ? g[j] : acc[j] + g[j];
        if (threadIdx.x == 0) cnt[0] += 1;                      // M_t^i += M_r
    }
}

// ------------------------------------------------------------------------------------------
// Step 2, bf16 gradient: 10 bytes per parameter.  One 128-bit load carries 8 gradients.
// ------------------------------------------------------------------------------------------
template <int U, bool kOverwrite>
__global__ void __launch_bounds__(kBlock) k_accumulate_bf16(float* acc, const uint16_t* __restrict__ g,
                                                            unsigned long long n_vec8, unsigned long long P,
                                                            int32_t* cnt) {
    float4* acc4 = reinterpret_cast<float4*>(acc);
    const uint4* g8 = reinterpret_cast<const uint4*>(g);
    const unsigned long long tile = (unsigned long long)kBlock * U;
    pdl_wait();
    pdl_trigger();
    for (unsigned long long base = blockIdx.x * tile; base < n_vec8; base += gridDim.x * tile) {
        float4 a0[U], a1[U];
        uint4 b[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const unsigned long long idx = base + (unsigned long long)u * kBlock + threadIdx.x;
            if (idx < n_vec8) {
                b[u] = ld_stream(g8 + idx);
                if (!kOverwrite) {
                    a0[u] = acc4[2 * idx];
                    a1[u] = acc4[2 * idx + 1];
                } else {
                    a0[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                    a1[u] = a0[u];
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const unsigned long long idx = base + (unsigned long long)u * kBlock + threadIdx.x;
            if (idx < n_vec8) {
                a0[u].x += bf16_lo(b[u].x); a0[u].y += bf16_hi(b[u].x);
                a0[u].z += bf16_lo(b[u].y); a0[u].w += bf16_hi(b[u].y);
                a1[u].x += bf16_lo(b[u].z); a1[u].y += bf16_hi(b[u].z);
                a1[u].z += bf16_lo(b[u].w); a1[u].w += bf16_hi(b[u].w);
                st_stream(acc4 + 2 * idx, a0[u]);
                st_stream(acc4 + 2 * idx + 1, a1[u]);
            }
        }
    }
    if (blockIdx.x == 0) {
        const unsigned long long j = n_vec8 * 8 + threadIdx.x;  // ragged tail (P % 8 elements)
        if (j < P) acc[j] = (kOverwrite ? 0.f : acc[j]) + __uint_as_float((uint32_t)g[j] << 16);
        if (threadIdx.x == 0) cnt[0] += 1;
    }
}

// ------------------------------------------------------------------------------------------
// Step 2 for n gradients of one worker in one pass:  G_t^i += g_0 + ... (added one after the
// other, in that order, exactly as n single launches would) ;  b_i += n.  The accumulator row
// is read and written once instead of n times: (4 n + 8) bytes per parameter (fp32 gradients;
// 2 n + 8 for bf16) instead of 12 n (10 n).
// ------------------------------------------------------------------------------------------
template <int U, int MAXN, bool kOverwrite>   // n <= MAXN
__global__ void __launch_bounds__(kBlock) k_accumulate_multi_f32(float* acc, GradList gl, int n, unsigned long long n_vec,
                                                                 unsigned long long P, int32_t* cnt) {
    float4* acc4 = reinterpret_cast<float4*>(acc);
    const unsigned long long tile = (unsigned long long)kBlock * U;
    pdl_wait();
    pdl_trigger();
    for (unsigned long long base = blockIdx.x * tile; base < n_vec; base += gridDim.x * tile) {
        float4 a[U], b[U][MAXN];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const unsigned long long idx = base + (unsigned long long)u * kBlock + threadIdx.x;
            if (idx < n_vec) {
#pragma unroll
                for (int k = 0; k < MAXN; ++k)
                    if (k < n) b[u][k] = ld_stream(static_cast<const float4*>(gl.p[k]) + idx);
                if (!kOverwrite) a[u] = acc4[idx];
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const unsigned long long idx = base + (unsigned long long)u * kBlock + threadIdx.x;
            if (idx < n_vec) {
                if (kOverwrite) a[u] = b[u][0];
#pragma unroll
                for (int k = kOverwrite ? 1 : 0; k < MAXN; ++k)
                    if (k < n) { a[u].x += b[u][k].x; a[u].y += b[u][k].y; a[u].z += b[u][k].z; a[u].w += b[u][k].w; }
                st_stream(acc4 + idx, a[u]);
            }
        }
    }
    if (blockIdx.x == 0) {
        const unsigned long long j = n_vec * 4 + threadIdx.x;   // ragged tail (P % 4 elements)
        if (j < P) {
            float t = kOverwrite ? static_cast<const float*>(gl.p[0])[j] : acc[j];
            for (int k = kOverwrite ? 1 : 0; k < n; ++k) t += static_cast<const float*>(gl.p[k])[j];
            acc[j] = t;
        }
        if (threadIdx.x == 0) cnt[0] += n;                      // M_t^i += n M_r
    }
}

template <int U, int MAXN, bool kOverwrite>   // n <= MAXN
__global__ void __launch_bounds__(kBlock) k_accumulate_multi_bf16(float* acc, GradList gl, int n, unsigned long long n_vec8,
                                                                  unsigned long long P, int32_t* cnt) {
    float4* acc4 = reinterpret_cast<float4*>(acc);
    const unsigned long long tile = (unsigned long long)kBlock * U;
    pdl_wait();
    pdl_trigger();
    for (unsigned long long base = blockIdx.x * tile; base < n_vec8; base += gridDim.x * tile) {
        uint4 b[U][MAXN];
        float4 a0[U], a1[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const unsigned long long idx = base + (unsigned long long)u * kBlock + threadIdx.x;
            if (idx < n_vec8) {
#pragma unroll
                for (int k = 0; k < MAXN; ++k)
                    if (k < n) b[u][k] = ld_stream(static_cast<const uint4*>(gl.p[k]) + idx);
                a0[u] = make_float4(0.f, 0.f, 0.f, 0.f);   // 0 + g = g: storing is adding to zero
                a1[u] = a0[u];
                if (!kOverwrite) {
                    a0[u] = acc4[2 * idx];
                    a1[u] = acc4[2 * idx + 1];
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const unsigned long long idx = base + (unsigned long long)u * kBlock + threadIdx.x;
            if (idx < n_vec8) {
#pragma unroll
                for (int k = 0; k < MAXN; ++k)
                    if (k < n) {
                        a0[u].x += bf16_lo(b[u][k].x); a0[u].y += bf16_hi(b[u][k].x);
                        a0[u].z += bf16_lo(b[u][k].y); a0[u].w += bf16_hi(b[u][k].y);
                        a1[u].x += bf16_lo(b[u][k].z); a1[u].y += bf16_hi(b[u][k].z);
                        a1[u].z += bf16_lo(b[u][k].w); a1[u].w += bf16_hi(b[u][k].w);
                    }
                st_stream(acc4 + 2 * idx, a0[u]);
                st_stream(acc4 + 2 * idx + 1, a1[u]);
            }
        }
    }
    if (blockIdx.x == 0) {
        const unsigned long long j = n_vec8 * 8 + threadIdx.x;  // ragged tail (P % 8 elements)
        if (j < P) {
            float t = kOverwrite ? 0.f : acc[j];
            for (int k = 0; k < n; ++k) t += __uint_as_float((uint32_t) static_cast<const uint16_t*>(gl.p[k])[j] << 16);
            acc[j] = t;
        }
        if (threadIdx.x == 0) cnt[0] += n;
    }
}

// ------------------------------------------------------------------------------------------
// Step 1 + update, fused.  (8*W_act + 16) bytes per parameter, W_act = #{i : b_i > 0}:
// read W_act accumulators + x + v, write x' + v + W_act zeros.  Rows of idle workers
// (b_i = 0) are neither read nor rewritten.  WT > 0 (used for W <= 4): W known at compile time, all
// loads of a vector are issued before the first add; WT == 0: any W, in chunks of 8 rows.
// ------------------------------------------------------------------------------------------
struct UpdateCoef {
    float lr, mu, wd, lambda_dc;
    float disp_scale;   // x_t - x_{t-1} = -disp_scale * v   (0 when the previous step was a no-op)
};
// Returns the squared norm of the four averaged-gradient components (before Eq. 6 and weight decay).
__device__ __forceinline__ float update_vec(float4& x, float4& v, const float4 s, const float Bf,
                                            const UpdateCoef& a) {
    float gx = __fdiv_rn(s.x, Bf), gy = __fdiv_rn(s.y, Bf), gz = __fdiv_rn(s.z, Bf), gw = __fdiv_rn(s.w, Bf);
    const float n2 = gx * gx + gy * gy + gz * gz + gw * gw;
    if (a.lambda_dc != 0.0f) {   // Eq. 6 with x_t - x_{t-1} = -disp_scale * v
        const float c = -a.lambda_dc * a.disp_scale;
        gx += c * gx * gx * v.x; gy += c * gy * gy * v.y; gz += c * gz * gz * v.z; gw += c * gw * gw * v.w;
    }
    gx += a.wd * x.x; gy += a.wd * x.y; gz += a.wd * x.z; gw += a.wd * x.w;
    v.x = a.mu * v.x + gx; v.y = a.mu * v.y + gy; v.z = a.mu * v.z + gz; v.w = a.mu * v.w + gw;
    x.x -= a.lr * v.x; x.y -= a.lr * v.y; x.z -= a.lr * v.z; x.w -= a.lr * v.w;
    return n2;
}

__device__ __forceinline__ void store_shadow(__nv_bfloat16* shadow, unsigned long long idx, const float4 x) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(x.x, x.y);
    __nv_bfloat162 hi = __floats2bfloat162_rn(x.z, x.w);
    uint2 pk;
    pk.x = *reinterpret_cast<uint32_t*>(&lo);
    pk.y = *reinterpret_cast<uint32_t*>(&hi);
    reinterpret_cast<uint2*>(shadow)[idx] = pk;
}

template <int WT, int U, bool kNorm>
__global__ void __launch_bounds__(kBlock) k_sync(const SyncArgs a) {
    __shared__ int s_cnt[kMaxW];
    __shared__ double s_norm[kBlock / 32];
    float norm_acc = 0.f;   // kNorm: this thread's share of |Gbar|^2 (a handful of vectors)
    const int W = WT > 0 ? WT : a.W;
    pdl_wait();      // counters and rows come from the accumulate kernels ahead on the stream
    pdl_trigger();
    if (threadIdx.x < W) s_cnt[threadIdx.x] = a.cnt[threadIdx.x];
    __syncthreads();
    long long B = 0;
    unsigned long long active = 0;
    for (int i = 0; i < W; ++i) {
        B += s_cnt[i];
        if (s_cnt[i] > 0) active |= 1ull << i;
    }
    const float Bf = (float)B;
    const UpdateCoef uc{a.lr, a.mu, a.wd, a.lambda_dc, a.disp_scale};

    const float4* xin = reinterpret_cast<const float4*>(a.x_in);
    float4* xout = reinterpret_cast<float4*>(a.x_out);
    float4* v4 = reinterpret_cast<float4*>(a.v);
    float4* acc4 = reinterpret_cast<float4*>(a.acc);
    const unsigned long long rs = a.row_stride / 4;
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    const unsigned long long tile = (unsigned long long)kBlock * U;

    if (B > 0) {
        for (unsigned long long base = blockIdx.x * tile; base < a.n_vec; base += gridDim.x * tile) {
            if constexpr (WT > 0) {
                float4 r[U][WT], x[U], v[U];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const unsigned long long idx = base + (unsigned long long)u * kBlock + threadIdx.x;
                    if (idx < a.n_vec) {
#pragma unroll
                        for (int i = 0; i < WT; ++i)
                            if ((active >> i) & 1) r[u][i] = ld_stream(acc4 + i * rs + idx);
                        x[u] = ld_stream(xin + idx);
                        v[u] = ld_stream(v4 + idx);
                    }
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const unsigned long long idx = base + (unsigned long long)u * kBlock + threadIdx.x;
                    if (idx < a.n_vec) {
                        float4 s = zero;
#pragma unroll
                        for (int i = 0; i < WT; ++i)      // fixed worker order
                            if ((active >> i) & 1) {
                                s.x += r[u][i].x; s.y += r[u][i].y; s.z += r[u][i].z; s.w += r[u][i].w;
                            }
                        norm_acc += update_vec(x[u], v[u], s, Bf, uc);
                        st_stream(xout + idx, x[u]);
                        st_stream(v4 + idx, v[u]);
                        if (a.shadow) store_shadow(a.shadow, idx, x[u]);
#pragma unroll
                        for (int i = 0; i < WT; ++i)
                            if (a.zero_acc && ((active >> i) & 1)) st_stream(acc4 + i * rs + idx, zero);
                    }
                }
            } else {
                const unsigned long long idx = base + threadIdx.x;   // U == 1 in the generic path
                if (idx < a.n_vec) {
                    float4 x = ld_stream(xin + idx), v = ld_stream(v4 + idx);
                    float4 s = zero;
                    for (int i0 = 0; i0 < W; i0 += 8) {
                        float4 r[8];
#pragma unroll
                        for (int c = 0; c < 8; ++c)
                            if (i0 + c < W && ((active >> (i0 + c)) & 1)) r[c] = ld_stream(acc4 + (i0 + c) * rs + idx);
#pragma unroll
                        for (int c = 0; c < 8; ++c)
                            if (i0 + c < W && ((active >> (i0 + c)) & 1)) {
                                s.x += r[c].x; s.y += r[c].y; s.z += r[c].z; s.w += r[c].w;
                                if (a.zero_acc) st_stream(acc4 + (i0 + c) * rs + idx, zero);
                            }
                    }
                    norm_acc += update_vec(x, v, s, Bf, uc);
                    st_stream(xout + idx, x);
                    st_stream(v4 + idx, v);
                    if (a.shadow) store_shadow(a.shadow, idx, x);
                }
            }
        }
    } else if (a.x_out != a.x_in) {
        // Nothing to apply (sum_i b_i = 0): x_{t+1} = x_t, v unchanged.  The host normally
        // skips the launch in this case; kept so the kernel is correct on its own.
        for (unsigned long long idx = blockIdx.x * (unsigned long long)kBlock + threadIdx.x; idx < a.n_vec;
             idx += (unsigned long long)gridDim.x * kBlock) {
            const float4 x = xin[idx];
            xout[idx] = x;
            if (a.shadow) store_shadow(a.shadow, idx, x);
        }
    }

    if constexpr (kNorm) {
        // |Gbar|^2: per-thread fp32 share -> warp sum in fp64 by shuffles -> one fp64 partial per CTA, in a slot
        // of its own; the last CTA adds the slots in a fixed order, so the figure is reproducible run to run.
        double w = (double)norm_acc;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) w += __shfl_xor_sync(0xFFFFFFFFu, w, o);
        if ((threadIdx.x & 31) == 0) s_norm[threadIdx.x >> 5] = w;
        __syncthreads();
        if (threadIdx.x == 0) {
            double c = 0.0;
            for (int k = 0; k < kBlock / 32; ++k) c += s_norm[k];
            a.norm_part[blockIdx.x] = c;
        }
    }

    // The last CTA to finish logs the consumed b_i and clears the device counters (every CTA
    // read them before taking its ticket).
    __shared__ unsigned int s_last;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const unsigned int t = atomicAdd(a.ticket, 1u);
        s_last = (t == gridDim.x - 1) ? 1u : 0u;
        if (t == gridDim.x - 1) {
            for (int i = 0; i < W; ++i) {
                a.log_row[i] = s_cnt[i];
                a.cnt[i] = 0;
            }
            *a.ticket = 0u;
        }
    }
    if constexpr (kNorm) {
        __syncthreads();
        if (s_last) {   // every other CTA's partial was written (and fenced) before it took its ticket
            __threadfence();
            double c = 0.0;
            for (unsigned k = threadIdx.x; k < gridDim.x; k += kBlock) c += __ldcg(a.norm_part + k);
            __shared__ double s_all[kBlock];
            s_all[threadIdx.x] = c;
            __syncthreads();
            if (threadIdx.x == 0) {
                double tot = 0.0;
                for (int k = 0; k < kBlock; ++k) tot += s_all[k];
                *a.norm_out = B > 0 ? tot : 0.0;
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
// Step 1 when the workers live on G GPUs (the paper's setting: "global synchronization" of G_{t-1}^i and
// M_{t-1}^i between workers).  One kernel per rank does what a reduce-scatter, the update and an all-gather
// would do as three passes: rank r owns the vectors [vec_lo, vec_hi); for each of them it loads the element of
// every worker row of every rank (local rows from HBM, the peers' rows through NVLink peer mappings), sums them
// in global worker order (rank-major, so the result equals the one-GPU kernel on G * W_local rows bit for bit),
// updates x and its slice of v, stores x_{t+1} into every rank's output buffer and writes zeros over the
// elements it consumed.  Every accumulator byte crosses HBM once and NVLink at most once; x_{t+1} crosses
// NVLink once per peer.  No CTA waits for another rank: the caller orders the launches with two stream-ordered
// collectives (all b_i exchanged before, a barrier after).
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kBlock) k_sync_global(const GlobalSyncArgs a) {
    __shared__ int s_cnt[kMaxW];
    __shared__ float4* s_row[kMaxW];
    const int R = a.G * a.W_local;                    // rows in global worker order: j = q * W_local + i
    pdl_wait();
    pdl_trigger();
    if (threadIdx.x < R) {
        const int q = threadIdx.x / a.W_local, i = threadIdx.x - q * a.W_local;
        s_cnt[threadIdx.x] = a.cnt_all[threadIdx.x];
        s_row[threadIdx.x] = reinterpret_cast<float4*>(a.acc[q] + (unsigned long long)i * a.row_stride);
    }
    const int applied_before = *a.applied;
    __syncthreads();
    long long B = 0;
    unsigned long long active = 0;
    for (int j = 0; j < R; ++j) {
        B += s_cnt[j];
        if (s_cnt[j] > 0) active |= 1ull << j;
    }
    const float Bf = (float)B;
    const UpdateCoef uc{a.lr, a.mu, a.wd, a.lambda_dc, applied_before ? a.disp_scale : 0.0f};
    const float4* xin = reinterpret_cast<const float4*>(a.x_in);
    float4* v4 = reinterpret_cast<float4*>(a.v);
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);

    for (unsigned long long idx = a.vec_lo + blockIdx.x * (unsigned long long)kBlock + threadIdx.x; idx < a.vec_hi;
         idx += (unsigned long long)gridDim.x * kBlock) {
        float4 x = ld_stream(xin + idx);
        if (B > 0) {
            float4 v = ld_stream(v4 + idx);
            float4 s = zero;
            for (int j0 = 0; j0 < R; j0 += 8) {
                float4 r[8];
#pragma unroll
                for (int c = 0; c < 8; ++c)
                    if (j0 + c < R && ((active >> (j0 + c)) & 1)) r[c] = ld_stream(s_row[j0 + c] + idx);
#pragma unroll
                for (int c = 0; c < 8; ++c)
                    if (j0 + c < R && ((active >> (j0 + c)) & 1)) {
                        s.x += r[c].x; s.y += r[c].y; s.z += r[c].z; s.w += r[c].w;
                        if (a.zero_acc) st_stream(s_row[j0 + c] + idx, zero);
                    }
            }
            update_vec(x, v, s, Bf, uc);
            st_stream(v4 + idx, v);
        }
        // sum_i b_i = 0: x_{t+1} = x_t on every rank, v untouched
        for (int q = 0; q < a.G; ++q) {
            st_stream(reinterpret_cast<float4*>(a.x_out[q]) + idx, x);
            if (a.shadow[q]) store_shadow(a.shadow[q], idx, x);
        }
    }
    __threadfence_system();   // the peers' copies of this slice are complete before the kernel counts as done

    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned int t = atomicAdd(a.ticket, 1u);
        if (t == gridDim.x - 1) {
            for (int j = 0; j < R; ++j) a.log_row[j] = s_cnt[j];
            *a.applied = B > 0 ? 1 : 0;
            *a.ticket = 0u;
        }
    }
}

__global__ void k_global_counts(int32_t* gcnt, int32_t* cnt, int own_lo, int W_local, int n_total) {
    pdl_wait();
    pdl_trigger();
    const int j = threadIdx.x;
    if (j >= n_total) return;
    const bool own = j >= own_lo && j < own_lo + W_local;
    gcnt[j] = own ? cnt[j - own_lo] : 0;
    if (own) cnt[j - own_lo] = 0;
}

__global__ void __launch_bounds__(kBlock) k_cast_bf16(const float4* __restrict__ src, __nv_bfloat16* dst,
                                                      unsigned long long n_vec) {
    pdl_wait();
    pdl_trigger();
    for (unsigned long long idx = blockIdx.x * (unsigned long long)kBlock + threadIdx.x; idx < n_vec;
         idx += (unsigned long long)gridDim.x * kBlock)
        store_shadow(dst, idx, src[idx]);
}

inline unsigned grid_for(unsigned long long n_items, int per_cta, int ctas_per_sm, int num_sms) {
    unsigned long long tiles = (n_items + per_cta - 1) / per_cta;
    if (tiles == 0) tiles = 1;
    if (ctas_per_sm > 0) {
        const unsigned long long cap = (unsigned long long)ctas_per_sm * num_sms;
        if (tiles > cap) tiles = cap;
    }
    if (tiles > 0x7FFFFFFFull) tiles = 0x7FFFFFFFull;
    return (unsigned)tiles;
}

template <int WT, int U>
cudaError_t launch_sync_t(const SyncArgs& a, int ctas_per_sm, int num_sms, cudaStream_t stream, bool chained) {
    const unsigned grid = grid_for(a.n_vec, kBlock * U, ctas_per_sm, num_sms);
    if (a.norm_out) {
        if (grid > a.norm_slots) return cudaErrorInvalidValue;
        return launch_kernel(k_sync<WT, U, true>, grid, kBlock, 0, stream, chained, a);
    }
    return launch_kernel(k_sync<WT, U, false>, grid, kBlock, 0, stream, chained, a);
}

}  // namespace

cudaError_t launch_accumulate(float* acc_row, const void* g, uint32_t grad_dtype, size_t P, int32_t* cnt, bool overwrite,
                              int ctas_per_sm, int num_sms, cudaStream_t stream, bool chained) {
    constexpr int U = 4;
    if (ctas_per_sm == 0) ctas_per_sm = -1;   // measured: one tile per CTA beats a persistent grid
    const unsigned long long P_ = P;
    if (grad_dtype == ABS_GRAD_F32) {
        const unsigned long long n_vec = P / 4;
        const unsigned grid = grid_for(n_vec, kBlock * U, ctas_per_sm, num_sms);
        const float* gf = static_cast<const float*>(g);
        return launch_kernel(overwrite ? k_accumulate_f32<U, true> : k_accumulate_f32<U, false>, grid, kBlock, 0, stream,
                             chained, acc_row, gf, n_vec, P_, cnt);
    }
    const unsigned long long n_vec8 = P / 8;
    const unsigned grid = grid_for(n_vec8, kBlock * U, ctas_per_sm, num_sms);
    const uint16_t* gb = static_cast<const uint16_t*>(g);
    return launch_kernel(overwrite ? k_accumulate_bf16<U, true> : k_accumulate_bf16<U, false>, grid, kBlock, 0, stream,
                         chained, acc_row, gb, n_vec8, P_, cnt);
}

cudaError_t launch_accumulate_multi(float* acc_row, const GradList& gl, int n, uint32_t grad_dtype, size_t P, int32_t* cnt,
                                    bool overwrite, int ctas_per_sm, int num_sms, cudaStream_t stream, bool chained) {
    if (ctas_per_sm == 0) ctas_per_sm = -1;
    const unsigned long long P_ = P;
    if (grad_dtype == ABS_GRAD_F32) {
        const unsigned long long n_vec = P / 4;
        if (n <= 4) {   // few gradients: two vectors per thread keep enough loads in flight
            const unsigned grid = grid_for(n_vec, kBlock * 2, ctas_per_sm, num_sms);
            return launch_kernel(overwrite ? k_accumulate_multi_f32<2, 4, true> : k_accumulate_multi_f32<2, 4, false>, grid, kBlock,
                                 0, stream, chained, acc_row, gl, n, n_vec, P_, cnt);
        }
        if (n <= 6) {
            const unsigned grid = grid_for(n_vec, kBlock * 2, ctas_per_sm, num_sms);
            return launch_kernel(overwrite ? k_accumulate_multi_f32<2, 6, true> : k_accumulate_multi_f32<2, 6, false>, grid, kBlock,
                                 0, stream, chained, acc_row, gl, n, n_vec, P_, cnt);
        }
        const unsigned grid = grid_for(n_vec, kBlock, ctas_per_sm, num_sms);
        return launch_kernel(overwrite ? k_accumulate_multi_f32<1, 8, true> : k_accumulate_multi_f32<1, 8, false>, grid, kBlock, 0,
                             stream, chained, acc_row, gl, n, n_vec, P_, cnt);
    }
    const unsigned long long n_vec8 = P / 8;
    if (n <= 4) {
        const unsigned grid = grid_for(n_vec8, kBlock * 2, ctas_per_sm, num_sms);
        return launch_kernel(overwrite ? k_accumulate_multi_bf16<2, 4, true> : k_accumulate_multi_bf16<2, 4, false>, grid, kBlock, 0,
                             stream, chained, acc_row, gl, n, n_vec8, P_, cnt);
    }
    const unsigned grid = grid_for(n_vec8, kBlock, ctas_per_sm, num_sms);
    return launch_kernel(overwrite ? k_accumulate_multi_bf16<1, 8, true> : k_accumulate_multi_bf16<1, 8, false>, grid, kBlock, 0,
                         stream, chained, acc_row, gl, n, n_vec8, P_, cnt);
}

cudaError_t launch_sync(const SyncArgs& a, int ctas_per_sm, int num_sms, cudaStream_t stream, bool chained) {
    // The bulk-copy kernel (sync_tma.cu) gives the same bits; which form is faster depends on W and on whether
    // the step runs alone or beside the next iteration's accumulate kernels (pipelined mode).  Measured on a B200
    // (P = 25.6 M, every W from 2 to 24):
    //   alone: bulk copy ahead by 1 - 8 % for W = 5 - 7 and 9 - 17, behind by 3 - 10 % for W <= 4, by 3 % for W = 8
    //     and W >= 18;
    //   overlapped (whole pipelined iterations, two micro-batches per worker): bulk copy ahead by 2 - 6 % for
    //     W = 5 - 21, level for W = 3, 4, behind for W = 2 and for W >= 22 (two stages of 100 KiB are too few).
    // Each table lists the W where the bulk-copy form is the default; -2 asks for it wherever it can run.
    constexpr unsigned kBulkAlone = (0x7u << 5) | (0x1FFu << 9);          // 5 - 7, 9 - 17
    constexpr unsigned kBulkOverlapped = 0x1FFFFu << 5;                   // 5 - 21
    const bool bulk_default = a.W < 32 && (((a.overlapped ? kBulkOverlapped : kBulkAlone) >> a.W) & 1u);
    const bool long_enough = a.n_vec >= (1ull << 18);   // short vectors are launch-bound: keep the lighter kernel
    if (!a.plain_only && (ctas_per_sm == -2 || (ctas_per_sm == 0 && bulk_default && long_enough && !a.norm_out))) {
        const cudaError_t e = launch_sync_tma(a, num_sms, stream, chained);
        if (e != cudaErrorNotSupported) return e;
        ctas_per_sm = 0;
    }
    // Measured on B200 (kernel alone, accumulators far larger than L2, GB/s on (8 W + 16) P bytes):
    //   W <= 4   compile-time W, every load of a vector in flight at once, one tile per CTA: 6.2 - 6.5 TB/s
    //            (W = 1: two vectors per thread);
    //   W >= 5   rows in chunks of 8 (at most 10 loads in flight per thread, 2 CTAs resident per SM).  With
    //            compile-time W the same kernels fell to 4.4 - 4.9 TB/s (W = 5..12) and 2.9 TB/s (W = 16: 142
    //            registers, one CTA per SM).  Up to W = 24 a persistent grid of exactly the resident CTAs is
    //            best (5.4 - 6.25 TB/s against 4.3 - 6.0 with one tile per CTA); beyond, a tile already takes
    //            long enough and one tile per CTA wins again (6.2 - 6.4 TB/s).
    if (a.W > 4) {
        if (ctas_per_sm == 0) ctas_per_sm = a.W <= 24 ? 2 : -1;
        return launch_sync_t<0, 1>(a, ctas_per_sm, num_sms, stream, chained);
    }
    if (ctas_per_sm == 0) ctas_per_sm = -1;
    switch (a.W) {
        case 1: return launch_sync_t<1, 2>(a, ctas_per_sm, num_sms, stream, chained);
        case 2: return launch_sync_t<2, 1>(a, ctas_per_sm, num_sms, stream, chained);
        case 3: return launch_sync_t<3, 1>(a, ctas_per_sm, num_sms, stream, chained);
        default: return launch_sync_t<4, 1>(a, ctas_per_sm, num_sms, stream, chained);
    }
}

cudaError_t launch_sync_global(const GlobalSyncArgs& a, int ctas_per_sm, int num_sms, cudaStream_t stream, bool chained) {
    // Chunked rows like the one-GPU kernel for W > 4.  Default grid: 6 CTAs per SM (3 are resident at 74
    // registers), never more CTAs than the slice has tiles.  Measured with all ranks on one B200: 2 to 8 per SM
    // differ by a few per cent, one tile per CTA is 25 - 40 % slower.
    const unsigned long long n = a.vec_hi > a.vec_lo ? a.vec_hi - a.vec_lo : 0;
    if (ctas_per_sm == 0) ctas_per_sm = 6;
    const unsigned grid = grid_for(n, kBlock, ctas_per_sm, num_sms);
    return launch_kernel(k_sync_global, grid, kBlock, 0, stream, chained, a);
}

cudaError_t launch_global_counts(int32_t* gcnt, int32_t* cnt, int own_lo, int W_local, int n_total, cudaStream_t stream) {
    k_global_counts<<<1, kMaxW, 0, stream>>>(gcnt, cnt, own_lo, W_local, n_total);
    return cudaGetLastError();
}

cudaError_t launch_cast_bf16(const float* src, __nv_bfloat16* dst, size_t n, int num_sms, cudaStream_t stream) {
    const unsigned long long n_vec = n / 4;
    const unsigned grid = grid_for(n_vec, kBlock, 8, num_sms);
    k_cast_bf16<<<grid, kBlock, 0, stream>>>(reinterpret_cast<const float4*>(src), dst, n_vec);
    return cudaGetLastError();
}

}  // namespace abs_sgd
