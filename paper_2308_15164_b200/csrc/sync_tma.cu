// Fused Step 1 + update (same arithmetic as k_sync in kernels_stream.cu), with the rows moved by the bulk-copy
// engine instead of by the threads' own loads and stores.  Three roles per CTA, coupled by mbarriers only:
//
//   loader  (one thread)    for every 4 KiB tile of the vector: one cp.async.bulk per active accumulator row
//                           plus x and v into a shared-memory stage; completion is counted on the stage's
//                           "full" barrier;
//   workers (128 threads)   wait for "full", sum the rows of the stage in worker order, update x and v in place
//                           in shared memory (two float4 per thread), write the bf16 copy, arrive on "done";
//   sender  (one thread)    waits for "done", sends the stage out with cp.async.bulk stores -- x', v', the bf16
//                           copy, and a constant tile of zeros over every row that was read -- and hands the
//                           stage back to the loader ("empty") once the engine has read it; with three stages
//                           or more it does so one tile late, so that it never waits for the engine's queue.
//
// The threads never touch global memory, the register count does not grow with the number of workers, and
// 2 - 4 stages of (W + 2) x 4 KiB per CTA keep 85 - 180 KiB per SM in flight.  Every wait on an mbarrier is
// bounded: on a time-out the thread records ABS_ETIMEOUT in the status word and raises the CTA's abort flag, every
// role stops taking tiles, the loader waits (bounded) for the copies it armed, and the CTA returns.
#include "abs_internal.h"
#include "bulk_copy.cuh"

namespace abs_sgd {

namespace {

constexpr int kTileElems = 1024;               // floats of one row per stage
constexpr int kTileBytes = kTileElems * 4;
constexpr int kConsumers = 128;
constexpr int kLoaderTid = kConsumers, kSenderTid = kConsumers + 32;
constexpr int kThreads = kConsumers + 64;
constexpr int kMaxStages = 4;
constexpr int kCtlBytes = 256;

struct Ctl {
    uint64_t full[kMaxStages], empty[kMaxStages], done[kMaxStages];
    int abort;
};
static_assert(sizeof(Ctl) <= kCtlBytes, "control block");

// global -> shared, bytes and both addresses multiples of 16; read-once data: evict-first in L2
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src, uint32_t bytes, uint64_t* bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(smem_u32(dst_smem)), "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy) : "memory");
}
__device__ __forceinline__ void bulk_store(void* dst, const void* src_smem, uint32_t bytes, uint64_t policy) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;"
                 ::"l"(dst), "r"(smem_u32(src_smem)), "r"(bytes), "l"(policy) : "memory");
}

__device__ __forceinline__ uint32_t pack2(float a, float b) {
    __nv_bfloat162 t = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&t);
}

// lazy: a stage goes back to the producer one tile later (after the NEXT tile's stores have been issued), so that
// the consumers never sit waiting for the copy engine to get round to reading a stage; needs three stages or more.
__global__ void __launch_bounds__(kThreads) k_sync_tma(const SyncArgs a, const int n_stages, const int lazy) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ int s_cnt[kMaxW];
    Ctl* ctl = reinterpret_cast<Ctl*>(smem);
    float4* zero_tile = reinterpret_cast<float4*>(smem + kCtlBytes);
    unsigned char* stage0 = smem + kCtlBytes + kTileBytes;
    const int W = a.W;
    const size_t stage_bytes = (size_t)(W + 2) * kTileBytes + kTileBytes / 2;
    const int tid = threadIdx.x;

    for (int i = tid; i < kTileElems / 4; i += kThreads) zero_tile[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (tid == 0) {
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(&ctl->full[s], 1);
            mbar_init(&ctl->empty[s], 1);
            mbar_init(&ctl->done[s], kConsumers);
        }
        ctl->abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the zero tile is read by the copy engine
    pdl_wait();      // set-up above overlaps the tail of the kernel ahead on the stream; its counters and rows are read below
    pdl_trigger();
    if (tid < W) s_cnt[tid] = a.cnt[tid];
    __syncthreads();

    long long B = 0;
    unsigned long long active = 0;
    for (int i = 0; i < W; ++i) {
        B += s_cnt[i];
        if (s_cnt[i] > 0) active |= 1ull << i;
    }
    const unsigned long long n_elems = a.n_vec * 4;
    const unsigned long long n_tiles = (n_elems + kTileElems - 1) / kTileElems;
    volatile int* abort_flag = &ctl->abort;

    if (B > 0) {
        if (tid == kLoaderTid) {
            uint64_t pol;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
            const int n_act = __popcll(active);
            int it = 0;
            for (unsigned long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it) {
                const int s = it % n_stages, use = it / n_stages;
                if (*abort_flag) break;
                if (use > 0 && !mbar_wait(&ctl->empty[s], (uint32_t)((use - 1) & 1))) {
                    *abort_flag = 1;
                    if (a.status) *a.status = ABS_ETIMEOUT;
                    break;
                }
                const unsigned long long e0 = tile * kTileElems;
                const uint32_t elems = (uint32_t)(n_elems - e0 < (unsigned long long)kTileElems ? n_elems - e0 : kTileElems);
                const uint32_t bytes = elems * 4;
                unsigned char* base = stage0 + (size_t)s * stage_bytes;
                mbar_expect_tx(&ctl->full[s], bytes * (uint32_t)(n_act + 2));
                for (int i = 0; i < W; ++i)
                    if ((active >> i) & 1)
                        bulk_load(base + (size_t)i * kTileBytes, a.acc + (size_t)i * a.row_stride + e0, bytes, &ctl->full[s], pol);
                bulk_load(base + (size_t)W * kTileBytes, a.x_in + e0, bytes, &ctl->full[s], pol);
                bulk_load(base + (size_t)(W + 1) * kTileBytes, a.v + e0, bytes, &ctl->full[s], pol);
            }
            // Nothing armed by this thread may still be landing when the CTA ends: in a run without time-outs
            // the workers have waited for every one of these phases already.
            for (int s = 0; s < n_stages && s < it; ++s) {
                const int last_use = (it - 1 - s) / n_stages;
                mbar_wait(&ctl->full[s], (uint32_t)(last_use & 1));
            }
        } else if (tid == kSenderTid) {
            uint64_t pol;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
            int it = 0;
            int held = -1;   // lazy: the stage whose stores were issued last and that is not released yet
            for (unsigned long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it) {
                const int s = it % n_stages, use = it / n_stages;
                if (*abort_flag) break;
                if (!mbar_wait(&ctl->done[s], (uint32_t)(use & 1))) {
                    *abort_flag = 1;
                    if (a.status) *a.status = ABS_ETIMEOUT;
                    break;
                }
                const unsigned long long e0 = tile * kTileElems;
                const uint32_t elems = (uint32_t)(n_elems - e0 < (unsigned long long)kTileElems ? n_elems - e0 : kTileElems);
                const uint32_t bytes = elems * 4;
                unsigned char* base = stage0 + (size_t)s * stage_bytes;
                bulk_store(a.x_out + e0, base + (size_t)W * kTileBytes, bytes, pol);
                bulk_store(a.v + e0, base + (size_t)(W + 1) * kTileBytes, bytes, pol);
                if (a.shadow) bulk_store(a.shadow + e0, base + (size_t)(W + 2) * kTileBytes, bytes / 2, pol);
                if (a.zero_acc)
                    for (int i = 0; i < W; ++i)
                        if ((active >> i) & 1) bulk_store(a.acc + (size_t)i * a.row_stride + e0, zero_tile, bytes, pol);
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                if (lazy) {
                    asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");   // all but this tile's group
                    if (held >= 0) mbar_arrive(&ctl->empty[held]);
                    held = s;
                } else {
                    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the stage has been read out
                    mbar_arrive(&ctl->empty[s]);
                }
            }
            asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // everything read and written
        } else if (tid < kConsumers) {
            const float Bf = (float)B;
            int it = 0;
            for (unsigned long long tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it) {
                const int s = it % n_stages, use = it / n_stages;
                if (*abort_flag) break;
                if (!mbar_wait(&ctl->full[s], (uint32_t)(use & 1))) {
                    *abort_flag = 1;
                    if (a.status) *a.status = ABS_ETIMEOUT;
                    break;
                }
                const unsigned long long e0 = tile * kTileElems;
                const uint32_t elems = (uint32_t)(n_elems - e0 < (unsigned long long)kTileElems ? n_elems - e0 : kTileElems);
                unsigned char* base = stage0 + (size_t)s * stage_bytes;
                float4* xs = reinterpret_cast<float4*>(base + (size_t)W * kTileBytes);
                float4* vs = reinterpret_cast<float4*>(base + (size_t)(W + 1) * kTileBytes);
                uint2* sh = reinterpret_cast<uint2*>(base + (size_t)(W + 2) * kTileBytes);
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int j = tid + h * kConsumers;
                    if ((uint32_t)j * 4 < elems) {
                        float4 x = xs[j], v = vs[j];
                        float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
                        for (int i = 0; i < W; ++i)                    // fixed worker order
                            if ((active >> i) & 1) {
                                const float4 r = reinterpret_cast<const float4*>(base + (size_t)i * kTileBytes)[j];
                                sum.x += r.x; sum.y += r.y; sum.z += r.z; sum.w += r.w;
                            }
                        float gx = __fdiv_rn(sum.x, Bf), gy = __fdiv_rn(sum.y, Bf), gz = __fdiv_rn(sum.z, Bf), gw = __fdiv_rn(sum.w, Bf);
                        if (a.lambda_dc != 0.0f) {   // Eq. 6 with x_t - x_{t-1} = -disp_scale * v
                            const float c = -a.lambda_dc * a.disp_scale;
                            gx += c * gx * gx * v.x; gy += c * gy * gy * v.y; gz += c * gz * gz * v.z; gw += c * gw * gw * v.w;
                        }
                        gx += a.wd * x.x; gy += a.wd * x.y; gz += a.wd * x.z; gw += a.wd * x.w;
                        v.x = a.mu * v.x + gx; v.y = a.mu * v.y + gy; v.z = a.mu * v.z + gz; v.w = a.mu * v.w + gw;
                        x.x -= a.lr * v.x; x.y -= a.lr * v.y; x.z -= a.lr * v.z; x.w -= a.lr * v.w;
                        xs[j] = x;
                        vs[j] = v;
                        if (a.shadow) sh[j] = make_uint2(pack2(x.x, x.y), pack2(x.z, x.w));
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // these writes -> visible to the copy engine
                mbar_arrive(&ctl->done[s]);
            }
        }
    } else if (a.x_out != a.x_in) {
        // sum_i b_i = 0: x_{t+1} = x_t, v unchanged (the host normally skips the launch)
        const float4* xin = reinterpret_cast<const float4*>(a.x_in);
        float4* xout = reinterpret_cast<float4*>(a.x_out);
        for (unsigned long long idx = blockIdx.x * (unsigned long long)kThreads + tid; idx < a.n_vec;
             idx += (unsigned long long)gridDim.x * kThreads) {
            const float4 x = xin[idx];
            xout[idx] = x;
            if (a.shadow) reinterpret_cast<uint2*>(a.shadow)[idx] = make_uint2(pack2(x.x, x.y), pack2(x.z, x.w));
        }
    }

    // The last CTA to finish logs the consumed b_i and clears the device counters.
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        const unsigned int t = atomicAdd(a.ticket, 1u);
        if (t == gridDim.x - 1) {
            for (int i = 0; i < W; ++i) {
                a.log_row[i] = s_cnt[i];
                a.cnt[i] = 0;
            }
            *a.ticket = 0u;
        }
    }
}

// Waits, with the same bounded polling loop, for an mbarrier that nothing ever completes, and reports the
// time-out the way the pipeline above does.  `polls` keeps the whole kernel to well under a second.
__global__ void k_bounded_wait_selftest(int* status, uint32_t polls) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (!mbar_wait(&bar, 0u, polls)) *status = ABS_ETIMEOUT;
    }
}

}  // namespace

cudaError_t launch_bounded_wait_selftest(int* status, cudaStream_t stream) {
    k_bounded_wait_selftest<<<1, 32, 0, stream>>>(status, 1u << 12);
    return cudaGetLastError();
}

cudaError_t launch_sync_tma(const SyncArgs& a, int num_sms, cudaStream_t stream, bool chained) {
    if (a.W < 1 || a.W > kSyncTmaMaxW || a.norm_out) return cudaErrorNotSupported;
    const size_t stage_bytes = (size_t)(a.W + 2) * kTileBytes + kTileBytes / 2;
    const size_t fixed = kCtlBytes + kTileBytes;
    // Three stages or more let a stage be released lazily (see the kernel).  The stages of all CTAs of an SM
    // together stay below 200 KiB: configurations that take (nearly) all of an SM's shared memory measured 5 - 12 %
    // slower beside other kernels (W = 10, 11: four stages against three; W = 14, 15: three against two; W = 6: two
    // CTAs of three against one of four) and no faster alone.  Two CTAs per SM when three stages each fit into that
    // budget, else one CTA with up to four stages.
    const size_t budget_sm = 200 * 1024, whole = 224 * 1024;
    int ctas = 2;
    if (2 * (fixed + 3 * stage_bytes) > budget_sm) ctas = 1;
    int stages = (int)((budget_sm / ctas - fixed) / stage_bytes);
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 2) stages = 2;
    if (a.tma_one_cta > 0) {   // the caller wants room left on the SM for another kernel's CTA
        ctas = 1;
        stages = a.tma_one_cta > kMaxStages ? kMaxStages : a.tma_one_cta;
        while (stages > 2 && fixed + (size_t)stages * stage_bytes > budget_sm / 2 + stage_bytes) --stages;
        if (stages < 2) stages = 2;
    }
    if (fixed + (size_t)stages * stage_bytes > whole) return cudaErrorNotSupported;
    const int lazy = stages >= 3 ? 1 : 0;
    const size_t smem = fixed + (size_t)stages * stage_bytes;
    // the opt-in to large dynamic shared memory is per device: once each
    static bool opted_in[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !opted_in[dev]) {
        e = cudaFuncSetAttribute(k_sync_tma, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)whole);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) opted_in[dev] = true;
    }
    const unsigned long long n_tiles = (a.n_vec * 4 + kTileElems - 1) / kTileElems;
    unsigned long long grid = (unsigned long long)num_sms * ctas;
    if (grid > n_tiles) grid = n_tiles;
    if (grid == 0) grid = 1;
    return launch_kernel(k_sync_tma, (unsigned)grid, kThreads, smem, stream, chained, a, stages, lazy);
}

}  // namespace abs_sgd
