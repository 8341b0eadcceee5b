// abs_sync_step_noalloc: the fused weighted-reduce / momentum-SGD / clear kernel applied to
// buffers the caller owns, for callers that cannot allocate device memory.
//
// Who that is: code that lives inside somebody else's memory budget -- an extension running
// under a framework that has already reserved the whole GPU for its own pool, a job whose
// device memory was carved up front by a launcher, or a latency-critical loop where the
// implicit device-wide synchronisation of cudaMalloc / cudaFree is not acceptable.  Such a
// caller can hand over its parameter, momentum and accumulator buffers, but it has no way to
// provide the few words of working memory the kernel needs next to them (the "last CTA done"
// ticket and the log of consumed micro-batch counts).  Here that working memory is a small
// array that is part of the library image itself.
#include <mutex>

#include "abs_internal.h"

namespace {

// Working memory of the kernel: word 0 is the CTA ticket (must be zero when a launch starts),
// words 64..127 receive the b_i the step consumed (at most ABS_MAX_WORKERS of them).
// 1 KiB, resident on every GPU that loads this library until the process exits.
constexpr int kScratchWords = 256;
static __device__ __align__(256) unsigned int g_noalloc_scratch[kScratchWords];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned int* g_scratch_addr[kMaxDevices] = {nullptr};   // device address of the array, per device
int g_num_sms[kMaxDevices] = {0};

// In host code the name g_noalloc_scratch is only a handle; the address a kernel can use has
// to be asked for, once per device, with that device current.
cudaError_t scratch_for_current_device(unsigned int** out, int* num_sms) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
        unsigned int* p = nullptr;
        e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_noalloc_scratch);
        if (e != cudaSuccess) return e;
        int sms = 0;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        g_scratch_addr[dev] = p;
        g_num_sms[dev] = sms;
    }
    *out = g_scratch_addr[dev];
    *num_sms = g_num_sms[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" int abs_sync_step_noalloc(float* x_dev, float* v_dev, float* acc_dev, uint64_t row_stride, uint64_t P,
                                     uint32_t W, int32_t* cnt_dev, float lr, float momentum, float weight_decay,
                                     void* stream) {
    if (!x_dev || !v_dev || !acc_dev || !cnt_dev) return ABS_EINVAL;
    if (W == 0 || P == 0) return ABS_EINVAL;
    if (W > ABS_MAX_WORKERS) return ABS_ELIMIT;   // the built-in working memory logs at most 64 counts
    if ((P & 3) || (row_stride & 3) || row_stride < P) return ABS_EINVAL;
    if ((reinterpret_cast<uintptr_t>(x_dev) | reinterpret_cast<uintptr_t>(v_dev) | reinterpret_cast<uintptr_t>(acc_dev)) & 15)
        return ABS_EINVAL;
    if (reinterpret_cast<uintptr_t>(cnt_dev) & 3) return ABS_EINVAL;
    // The built-in array and the launch belong to the CURRENT device: the caller's buffers must live there too.
    // (A query of the pointer's attributes allocates nothing.)
    {
        int dev = -1;
        if (cudaGetDevice(&dev) != cudaSuccess) return ABS_ECUDA;
        const void* bufs[4] = {x_dev, v_dev, acc_dev, cnt_dev};
        for (const void* b : bufs) {
            cudaPointerAttributes at{};
            if (cudaPointerGetAttributes(&at, b) != cudaSuccess) { cudaGetLastError(); return ABS_EINVAL; }
            if ((at.type != cudaMemoryTypeDevice && at.type != cudaMemoryTypeManaged) || (at.type == cudaMemoryTypeDevice && at.device != dev))
                return ABS_EINVAL;
        }
    }

    unsigned int* scratch = nullptr;
    int num_sms = 0;
    if (scratch_for_current_device(&scratch, &num_sms) != cudaSuccess) return ABS_ECUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // The array keeps whatever the previous call left; the ticket has to start at zero.
    if (cudaMemsetAsync(scratch, 0, sizeof(unsigned int), s) != cudaSuccess) return ABS_ECUDA;

    abs_sgd::SyncArgs a{};
    a.x_in = x_dev;
    a.x_out = x_dev;
    a.v = v_dev;
    a.acc = acc_dev;
    a.row_stride = row_stride;
    a.n_vec = P / 4;
    a.W = static_cast<int>(W);
    a.cnt = cnt_dev;
    a.log_row = reinterpret_cast<int32_t*>(scratch + 64);
    a.ticket = scratch;
    a.lr = lr;
    a.mu = momentum;
    a.wd = weight_decay;
    a.lambda_dc = 0.0f;
    a.disp_scale = 0.0f;
    a.shadow = nullptr;
    a.zero_acc = 1;
    // Always the load/store form of the kernel: its bulk-copy form has bounded waits whose time-out is reported
    // through a context (abs_check), which this entry point does not have.
    a.plain_only = 1;
    return abs_sgd::launch_sync(a, 0, num_sms, s, false) == cudaSuccess ? ABS_OK : ABS_ECUDA;
}
