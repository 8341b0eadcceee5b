// Host side of the C ABI: state machine of Algorithm 1 (arXiv 2308.15164), workspace carving,
// argument checks, stream ordering of Step 1 against Step 2, kernel launches.
#include <cuda.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <string>
#include <unordered_set>
#include <vector>

#include "abs_internal.h"

using namespace abs_sgd;

namespace {

constexpr uint32_t kMagic = 0xAB55D6D0u;
constexpr size_t kMaxSpans = 1u << 20;

struct TimedLaunch {
    int kernel_class;
    cudaEvent_t start, stop;
    cudaStream_t stream;
    int part;
};

size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Layout {
    size_t P_pad = 0;
    size_t off_x[2] = {0, 0}, off_v = 0, off_acc = 0, off_cnt = 0, off_ticket = 0, off_log = 0, off_gcnt = 0;
    size_t off_shadow[2] = {0, 0}, off_mlp = 0, off_stage[2] = {0, 0}, off_norm_part = 0, off_norm_log = 0;
    size_t off_pool[2] = {0, 0};
    int pool_cap = 0;
    size_t norm_slots = 0;
    size_t total = 0;
};

bool config_ok(const abs_config* c, std::string* why) {
    auto fail = [&](const char* m) { if (why) *why = m; return false; };
    if (!c) return fail("config is NULL");
    if (c->P == 0) return fail("P must be > 0");
    if (c->W == 0 || c->W > ABS_MAX_WORKERS) return fail("W must be in 1..64");
    if (c->grad_dtype != ABS_GRAD_F32 && c->grad_dtype != ABS_GRAD_BF16) return fail("unknown grad_dtype");
    if (c->flags & ~(ABS_FLAG_PIPELINED | ABS_FLAG_MLP | ABS_FLAG_HOST_INPUT | ABS_FLAG_OVERWRITE_FIRST | ABS_FLAG_MLP_COALESCE |
                     ABS_FLAG_GRAD_NORM | ABS_FLAG_MLP_X_BF16 | ABS_FLAG_MLP_DEFER))
        return fail("unknown flag bits");
    if ((c->flags & ABS_FLAG_MLP_DEFER) && !(c->flags & ABS_FLAG_MLP)) return fail("ABS_FLAG_MLP_DEFER needs ABS_FLAG_MLP");
    if ((c->flags & ABS_FLAG_MLP_COALESCE) && !(c->flags & ABS_FLAG_MLP)) return fail("ABS_FLAG_MLP_COALESCE needs ABS_FLAG_MLP");
    if ((c->flags & ABS_FLAG_MLP_X_BF16) && !(c->flags & ABS_FLAG_MLP)) return fail("ABS_FLAG_MLP_X_BF16 needs ABS_FLAG_MLP");
    if (!std::isfinite(c->lr) || !std::isfinite(c->momentum) || !std::isfinite(c->weight_decay) ||
        !std::isfinite(c->lambda_dc))
        return fail("lr, momentum, weight_decay and lambda_dc must be finite");
    if ((c->flags & ABS_FLAG_PIPELINED) && c->stream_acc == c->stream_sync)
        return fail("pipelined mode needs two different streams");
    if (c->flags & ABS_FLAG_MLP) {
        if (c->mlp_in == 0 || c->mlp_in % 128 || c->mlp_hidden == 0 || c->mlp_hidden % 128)
            return fail("mlp_in and mlp_hidden must be positive multiples of 128");
        if (c->mlp_out == 0 || c->mlp_out > 16) return fail("mlp_out must be in 1..16");
        if (c->mlp_mb != 64) return fail("mlp_mb must be 64");
        const uint64_t need = (uint64_t)c->mlp_in * c->mlp_hidden + c->mlp_hidden +
                              (uint64_t)c->mlp_hidden * c->mlp_out + c->mlp_out;
        if (need != c->P) return fail("P does not match the MLP layer sizes");
    }
    return true;
}

Layout make_layout(const abs_config& c) {
    Layout L;
    L.P_pad = round_up(c.P, kPadElems);
    const bool pipe = c.flags & ABS_FLAG_PIPELINED;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = round_up(o + bytes, 4096); return at; };
    L.off_x[0] = take(L.P_pad * 4);
    L.off_x[1] = pipe ? take(L.P_pad * 4) : L.off_x[0];
    L.off_v = take(L.P_pad * 4);
    L.off_acc = take((size_t)2 * c.W * L.P_pad * 4);
    L.off_cnt = take((size_t)2 * kMaxW * 4);
    L.off_ticket = take(256);
    L.off_log = take((size_t)kLogDepth * kMaxW * 4);
    L.off_gcnt = take((size_t)(kMaxW + 64) * 4);   // multi-GPU mode: exchanged b_i of all ranks + "previous step applied" word
    if (c.flags & ABS_FLAG_MLP) {
        L.off_shadow[0] = take(L.P_pad * 2);
        L.off_shadow[1] = pipe ? take(L.P_pad * 2) : L.off_shadow[0];
        MlpDims d{(int)c.mlp_in, (int)c.mlp_hidden, (int)c.mlp_out, (int)c.mlp_mb};
        L.off_mlp = take((size_t)kMlpSets * mlp_scratch_bytes(d));
        if (c.flags & ABS_FLAG_MLP_DEFER) {
            // room for 16 micro-batches per worker and iteration before the operands are contracted early
            L.pool_cap = (int)std::min<uint32_t>(std::max<uint32_t>(16 * c.W, 32), kMlpMaxSlots);
            L.off_pool[0] = take(mlp_pool_bytes(d, L.pool_cap));
            L.off_pool[1] = take(mlp_pool_bytes(d, L.pool_cap));
        }
    }
    if (c.flags & ABS_FLAG_HOST_INPUT) {
        const size_t es = c.grad_dtype == ABS_GRAD_BF16 ? 2 : 4;
        L.off_stage[0] = take(L.P_pad * es);
        L.off_stage[1] = take(L.P_pad * es);
    }
    if (c.flags & ABS_FLAG_GRAD_NORM) {
        L.norm_slots = L.P_pad / 1024 + 1;            // one per CTA of the fused step's largest grid
        L.off_norm_part = take(L.norm_slots * 8);
        L.off_norm_log = take((size_t)kLogDepth * 8);
    }
    L.total = o;
    return L;
}

// Multi-GPU mode: rank r owns the float4 vectors [lo, hi) of the padded flat vector -- equal runs of whole
// 256-vector tiles, the last rank(s) take what is left (possibly nothing).
void slice_vectors(size_t P_pad, uint32_t G, uint32_t r, unsigned long long* lo, unsigned long long* hi) {
    const unsigned long long n_vec = P_pad / 4;
    const unsigned long long per = ((n_vec + G - 1) / G + 255) / 256 * 256;
    *lo = std::min(n_vec, per * r);
    *hi = std::min(n_vec, *lo + per);
}

std::mutex g_live_mu;
std::unordered_set<abs_ctx*> g_live;
thread_local std::string g_init_error;

}  // namespace

struct abs_ctx {
    uint32_t magic = kMagic;
    abs_config cfg{};
    Layout L;
    char* ws = nullptr;
    cudaStream_t s_acc = nullptr, s_sync = nullptr, s_copy = nullptr;
    bool pipelined = false, mlp = false;
    int device = 0, num_sms = 148;

    // logical state of Algorithm 1 (host mirror)
    std::vector<int32_t> h_cnt;   // [2][W]
    uint32_t cur = 0;
    uint64_t t = 0;

    // execution state
    int pub = 0;                  // which x buffer holds the published parameters
    bool pending = false;         // pipelined: a fused kernel launched on s_sync is not yet published
    int pending_out = 0;          // buffer it writes
    float lr_now = 0.f;
    float lr_prev_call = 0.f;     // learning rate in effect at the previous abs_sync_step call
    float disp_scale = 0.f;       // lr of the step that produced the newest x (0 after a no-op)
    cudaEvent_t ev_acc_done = nullptr, ev_sync_done = nullptr, ev_aux = nullptr;
    cudaEvent_t ev_stage_free[2] = {nullptr, nullptr}, ev_stage_full[2] = {nullptr, nullptr};
    bool stage_used[2] = {false, false};
    int stage_next = 0;
    int ctas_per_sm[ABS_K_COUNT] = {0, 0, 0, 0, 0, 0};
    // consecutive kernels of a stream are chained by programmatic dependent launch (abs_set_launch(ABS_K_CHAIN, 1): off)
    bool chained() const { return ctas_per_sm[ABS_K_CHAIN] == 0; }
    // the gradient kernels of the MLP: which of them are chained (kChain* bits); nb = micro-batches of the call
    int mlp_chain(bool serial, int nb) const {
        if (!chained()) return 0;
        // Measured (3072-4096-10, W = 4): with every kernel of a call alone on the GPU the whole chain gains (55 -> 50 us
        // per single call, 73 -> 69 per batch call).  With several workers' calls in flight the gaps are filled by the
        // other workers' kernels anyway, and a forward or dW1 CTA that is resident early only holds shared memory and
        // TMEM another worker's kernel could use: there only the two small kernels of single calls are chained
        // (33.4 -> 32.2 us per micro-batch; K-batched calls measured best with none: 15.5 against 15.7 - 16.1).
        if (serial || cfg.W == 1) return kChainCast | kChainFwd1 | kChainFwd2 | kChainBwd | kChainDw1;
        return nb == 1 ? (kChainFwd2 | kChainBwd) : 0;
    }
    bool x_bf16() const { return (cfg.flags & ABS_FLAG_MLP_X_BF16) != 0; }
    MlpDims mlp_dims{0, 0, 0, 0};
    // The paper's workers compute concurrently: the gradient kernels of worker i run on internal stream
    // i % n_wstreams (calls of one worker stay in order: its accumulator is added to in call order), each call
    // in its own scratch set, taken round-robin.
    MlpScratch mlp_scratch[kMlpSets]{};
    cudaStream_t s_w[kMlpStreams] = {};
    // The dW1 GEMM of a call runs on a second stream of the worker, at the lowest priority: the worker's next call
    // (forward, loss, backward: short, latency-bound kernels that only touch the bias / W2 slices of the row)
    // overlaps it, and the short kernels of every worker get free CTA slots before the HBM-bound GEMMs, whose
    // thousands of CTAs would otherwise keep them queueing (timeline with four workers' calls in flight: a 3 us
    // cast kernel took 23 us on average, `k_fwd2` 23 against 5).  Measured on 3072-4096-10, W = 4: single calls
    // 31.1 -> 30.0 us per micro-batch, batch calls 15.4 -> 14.6.
    cudaStream_t s_d[kMlpStreams] = {};
    cudaEvent_t ev_front[kMlpStreams] = {};        // front kernels of the newest call on s_w[k] have finished
    int n_wstreams = 0;
    cudaEvent_t ev_fork = nullptr;                 // stream_acc -> worker stream (re-recorded per call)
    cudaEvent_t ev_set_done[kMlpSets] = {};        // last use of a scratch set has finished
    cudaEvent_t ev_w_done[kMlpStreams] = {};       // newest call enqueued on a worker stream has finished
    bool set_used[kMlpSets] = {};
    bool w_outstanding[kMlpStreams] = {};          // enqueued since stream_acc last waited for that stream
    int mlp_set_next = 0;
    // ABS_FLAG_MLP_COALESCE: single calls of a worker wait, already cast into consecutive slots of one scratch
    // set, until four have gathered (or something needs the accumulator), then run as one batch call.
    bool coalesce = false;
    int pend_n[kMaxW] = {};        // micro-batches of worker i waiting (0..kMlpGatherMax)
    int pend_set[kMaxW] = {};      // scratch set that holds them
    bool pend_first[kMaxW] = {};   // they open the worker's iteration (the row holds nothing yet)
    bool set_reserved[kMlpSets] = {};
    int n_reserved = 0;
    uint64_t pend_age[kMaxW] = {}; // order in which the pending groups were opened
    uint64_t pend_clock = 0;
    std::vector<TmapBytes> acc_tmaps;   // [2][W]: TMA descriptor of each accumulator row's W1 slice
    // ABS_FLAG_MLP_DEFER: the dW1 operands of every gradient call of an iteration stay in the accumulator set's
    // operand pool; a worker's dW1 = sum_j X_j^T dZ_j is contracted in ONE launch (K = 64 b_i) when the iteration
    // ends, when something reads or adds to its accumulator row, or when the pool is full.
    bool defer = false;
    MlpPool pool[2]{};
    int pool_n[2] = {0, 0};                   // slots handed out (bump allocation; back to 0 when the iteration ends)
    std::vector<int16_t> pool_owner[2];       // worker whose micro-batch sits in the slot; -1: none (contracted, or never used)
    // In this mode a call adds nothing to its worker's row, so calls need no order among themselves: call after call
    // takes the next of the kMlpStreams internal streams (and that stream's scratch set), whoever the worker is.
    int rr_stream = 0;
    // ... and ABS_FLAG_MLP_COALESCE gathers single calls into one group whoever their workers are
    int grp_n = 0, grp_pool0 = 0;
    MlpWorkers grp_workers{};
    bool d_outstanding[kMlpStreams] = {};     // contractions enqueued on s_d[k] since stream_acc last waited for it
    cudaEvent_t ev_d_done[kMlpStreams] = {};
    bool w1_touched[2][kMaxW] = {};           // the row's W1 slice has been written in the set's current iteration
    // A set whose iteration ended with every W1 slice untouched is not contracted row by row: its fused step forms
    // the weighted average of the W1 slice straight from the pooled operands (k_sync_w1) and runs the row-based
    // kernel on the rest of the vector only.
    bool fused_pending[2] = {false, false};
    MlpSlots fused_slots[2]{};
    int fused_n[2] = {0, 0};
    TmapBytes tm_x[2]{}, tm_v{}, tm_shadow[2]{};   // W1 slices of the parameter buffers, the momentum and the bf16 copies

    // multi-GPU mode (abs_global_*): every rank's workspace as mapped in this process
    uint32_t n_ranks = 0, rank = 0;
    char* peer_ws[kMaxRanks] = {};
    int global_phase = 0;         // 0 = idle, 1 = after abs_global_begin, 2 = after abs_global_step
    float global_prev_lr = 0.f;   // rate of the previous abs_global_step

    // bookkeeping
    uint64_t launches = 0;
    bool profiling = false;
    std::vector<TimedLaunch> timed;
    std::vector<cudaEvent_t> ev_pool;
    bool timeline_on = false;         // abs_profile(ctx, 2): the spans of the timed launches are kept as well
    cudaEvent_t ev_origin = nullptr;  // time zero of the timeline (recorded on stream_acc when it was switched on)
    std::vector<abs_span> spans;
    uint64_t stat_n[ABS_K_COUNT] = {0};
    double stat_ms[ABS_K_COUNT] = {0};
    std::string err;

    float* x(int k) const { return reinterpret_cast<float*>(ws + L.off_x[k]); }
    float* v() const { return reinterpret_cast<float*>(ws + L.off_v); }
    float* acc(uint32_t set, uint32_t i) const {
        return reinterpret_cast<float*>(ws + L.off_acc) + ((size_t)set * cfg.W + i) * L.P_pad;
    }
    int32_t* cnt(uint32_t set, uint32_t i) const { return reinterpret_cast<int32_t*>(ws + L.off_cnt) + set * kMaxW + i; }
    unsigned int* ticket() const { return reinterpret_cast<unsigned int*>(ws + L.off_ticket); }
    int32_t* log_row(uint64_t step) const {
        return reinterpret_cast<int32_t*>(ws + L.off_log) + (step % kLogDepth) * kMaxW;
    }
    __nv_bfloat16* shadow(int k) const { return reinterpret_cast<__nv_bfloat16*>(ws + L.off_shadow[k]); }
    double* norm_part() const { return reinterpret_cast<double*>(ws + L.off_norm_part); }
    double* norm_log(uint64_t step) const { return reinterpret_cast<double*>(ws + L.off_norm_log) + step % kLogDepth; }
    bool grad_norm() const { return (cfg.flags & ABS_FLAG_GRAD_NORM) != 0; }
    int32_t* gcnt() const { return reinterpret_cast<int32_t*>(ws + L.off_gcnt); }
    int* applied_word() const { return reinterpret_cast<int*>(ws + L.off_gcnt) + kMaxW; }
};

namespace {

bool live(abs_ctx* c) {
    if (!c) return false;
    std::lock_guard<std::mutex> g(g_live_mu);
    return g_live.count(c) != 0 && c->magic == kMagic;
}

int cuda_fail(abs_ctx* c, cudaError_t e, const char* what) {
    char buf[256];
    snprintf(buf, sizeof buf, "%s: %s", what, cudaGetErrorString(e));
    c->err = buf;
    return ABS_ECUDA;
}
#define CK(call)                                                   \
    do {                                                           \
        cudaError_t e__ = (call);                                  \
        if (e__ != cudaSuccess) return cuda_fail(c, e__, #call);   \
    } while (0)

int invalid(abs_ctx* c, const char* msg) {
    c->err = msg;
    return ABS_EINVAL;
}

cudaEvent_t take_event(abs_ctx* c) {
    if (!c->ev_pool.empty()) {
        cudaEvent_t e = c->ev_pool.back();
        c->ev_pool.pop_back();
        return e;
    }
    cudaEvent_t e = nullptr;
    if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
    return e;
}

// Brackets a launch with an event pair when profiling is on.
struct Timed {
    abs_ctx* c;
    cudaStream_t s;
    cudaEvent_t stop = nullptr;
    Timed(abs_ctx* c_, int kernel_class, cudaStream_t s_) : c(c_), s(s_) {
        if (!c->profiling) return;
        cudaEvent_t start = take_event(c);
        stop = take_event(c);
        if (!start || !stop) { stop = nullptr; return; }
        cudaEventRecord(start, s);
        c->timed.push_back({kernel_class, start, stop, s, 0});
    }
    ~Timed() {
        if (stop) cudaEventRecord(stop, s);
    }
};

int stream_index(const abs_ctx* c, cudaStream_t s) {
    if (s == c->s_acc) return 0;
    if (s == c->s_sync) return 1;
    for (int k = 0; k < c->n_wstreams; ++k) {
        if (s == c->s_w[k]) return 2 + k;
        if (s == c->s_d[k]) return 2 + kMlpStreams + k;
    }
    return -1;
}

int collect_timings(abs_ctx* c) {
    for (auto& tl : c->timed) {
        CK(cudaEventSynchronize(tl.stop));
        float ms = 0.f;
        CK(cudaEventElapsedTime(&ms, tl.start, tl.stop));
        c->stat_n[tl.kernel_class] += 1;
        c->stat_ms[tl.kernel_class] += ms;
        if (c->timeline_on && c->ev_origin && c->spans.size() < kMaxSpans) {
            float t0 = 0.f;
            CK(cudaEventElapsedTime(&t0, c->ev_origin, tl.start));
            c->spans.push_back({tl.kernel_class, stream_index(c, tl.stream), tl.part, t0 * 1e3f, (t0 + ms) * 1e3f});
        }
        c->ev_pool.push_back(tl.start);
        c->ev_pool.push_back(tl.stop);
    }
    c->timed.clear();
    return ABS_OK;
}

void mlp_mark(void* user, int kernel_class, int n, cudaStream_t stream);

int flush_all(abs_ctx* c);
int flush_worker(abs_ctx* c, uint32_t worker);
int settle_all(abs_ctx* c);
int contract_pending_sets(abs_ctx* c);

// stream_acc waits (on the device) for every gradient kernel enqueued so far on the worker streams (waiting
// micro-batch groups are started and pooled dW1 operands contracted first).
// `stream` waits (on the device) for everything enqueued so far on the internal streams.  Per-call mode records
// ev_w_done behind every call; deferred mode records here, once per wait instead of once per call.
int wait_for_workers(abs_ctx* c, cudaStream_t stream, bool clear) {
    for (int k = 0; k < c->n_wstreams; ++k) {
        if (c->w_outstanding[k]) {
            if (c->defer) CK(cudaEventRecord(c->ev_w_done[k], c->s_w[k]));
            CK(cudaStreamWaitEvent(stream, c->ev_w_done[k], 0));
            if (clear) c->w_outstanding[k] = false;
        }
        if (c->d_outstanding[k]) {
            CK(cudaEventRecord(c->ev_d_done[k], c->s_d[k]));
            CK(cudaStreamWaitEvent(stream, c->ev_d_done[k], 0));
            if (clear) c->d_outstanding[k] = false;
        }
    }
    return ABS_OK;
}

int join_workers(abs_ctx* c) {
    if (int rc = settle_all(c)) return rc;
    return wait_for_workers(c, c->s_acc, true);
}

// Launch the fused Step-1 kernel on `set`, reading x[in] and writing x[out], on `stream`.
int launch_fused(abs_ctx* c, uint32_t set, int in, int out, uint64_t log_step, cudaStream_t stream) {
    SyncArgs a{};
    a.x_in = c->x(in);
    a.x_out = c->x(out);
    a.v = c->v();
    a.acc = c->acc(set, 0);
    a.row_stride = c->L.P_pad;
    a.n_vec = c->L.P_pad / 4;
    a.W = (int)c->cfg.W;
    a.cnt = c->cnt(set, 0);
    a.log_row = c->log_row(log_step);
    a.ticket = c->ticket();
    a.lr = c->lr_now;
    a.mu = c->cfg.momentum;
    a.wd = c->cfg.weight_decay;
    a.lambda_dc = c->cfg.lambda_dc;
    a.disp_scale = c->disp_scale;
    a.shadow = c->mlp ? c->shadow(out) : nullptr;
    a.zero_acc = (c->cfg.flags & ABS_FLAG_OVERWRITE_FIRST) ? 0 : 1;
    a.status = reinterpret_cast<int*>(c->ticket() + 2);
    a.overlapped = c->pipelined ? 1 : 0;
    if (c->grad_norm()) {
        a.norm_part = c->norm_part();
        a.norm_out = c->norm_log(log_step);
        a.norm_slots = (unsigned int)c->L.norm_slots;
    }
    // Beside the MLP's gradient kernels (pipelined mode) the bulk-copy form is the better neighbour: it holds six
    // warps per SM instead of every thread slot.  Measured on the 3072-4096-10 workload with batch calls: 16.9
    // against 17.5 us per micro-batch, although alone on the GPU it is the slower one at W = 4.  There it runs
    // as one CTA per SM with four stages (110 KB at W = 4) instead of two CTAs with three (168 KB), so that a
    // forward-GEMM or dW1 CTA still fits on the SM (single calls 32.4 -> 32.0 us, batch calls 15.8 -> 15.4; with
    // ABS_FLAG_MLP_DEFER 17.1 -> 16.6 and 14.9 -> 14.2 for gathered calls).
    int shape = c->ctas_per_sm[ABS_K_SYNC];
    if (shape == 0 && c->mlp && c->pipelined) {
        shape = -2;
        a.tma_one_cta = 4;
    }
    if (c->fused_pending[set]) {
        // Weighted average and update straight from the set's pool: the bias / W2 part from the per-micro-batch
        // partials (a small kernel, which also logs and clears the counters), the W1 slice from the dW1 operands.
        // No accumulator row is read or written.
        float B = 0.f;
        for (uint32_t i = 0; i < c->cfg.W; ++i) B += (float)c->h_cnt[(size_t)set * c->cfg.W + i];
        {
            Timed tm(c, ABS_K_SYNC, stream);
            CK(launch_mlp_sync_small(c->mlp_dims, c->pool[set], c->fused_slots[set], c->fused_n[set], a.x_in, a.x_out, a.v, a.shadow,
                                     B, a.lr, a.mu, a.wd, a.lambda_dc, a.disp_scale, a.cnt, a.log_row, (int)c->cfg.W, stream,
                                     c->chained()));
            CK(launch_mlp_sync_w1(c->mlp_dims, c->mlp_scratch[0], c->pool[set], c->fused_slots[set], c->fused_n[set], &c->tm_x[in],
                                  &c->tm_x[out], &c->tm_v, &c->tm_shadow[out], B, a.lr, a.mu, a.wd, a.lambda_dc, a.disp_scale,
                                  c->ctas_per_sm[ABS_K_MLP_BWD] == 2 ? -128 : 0, stream, c->chained()));
        }
        c->launches += 2;
        c->fused_pending[set] = false;
        for (int q = 0; q < c->pool_n[set]; ++q) c->pool_owner[set][q] = -1;
        c->pool_n[set] = 0;
        return ABS_OK;
    }
    {
        Timed tm(c, ABS_K_SYNC, stream);
        CK(launch_sync(a, shape, c->num_sms, stream, c->chained()));
    }
    c->launches += 1;
    return ABS_OK;
}

// Next scratch set that no pending group holds; stream_acc waits (on the device) for its previous user.
int take_scratch_set(abs_ctx* c, bool serial, int* out) {
    int set = c->mlp_set_next;
    for (int tries = 0; tries < kMlpSets && c->set_reserved[set]; ++tries) set = (set + 1) % kMlpSets;
    c->mlp_set_next = (set + 1) % kMlpSets;
    if (!serial && c->set_used[set]) CK(cudaStreamWaitEvent(c->s_acc, c->ev_set_done[set], 0));
    *out = set;
    return ABS_OK;
}

// Forward, loss, backward and dW1 of the n micro-batches that sit, cast, in slots 0..n-1 of scratch set `set`
// (ABS_FLAG_MLP_DEFER: in pool slots pool0.. of the current accumulator set, and without the dW1), on an internal
// stream, which first waits for everything enqueued on stream_acc so far, the casts included.
int run_mlp_group(abs_ctx* c, uint32_t worker, int set, int n, bool first, int pool0, const MlpWorkers* mixed = nullptr) {
    int k = (int)(worker % (uint32_t)c->n_wstreams);
    int variant = c->ctas_per_sm[ABS_K_MLP_DW1];
    const bool serial = c->ctas_per_sm[ABS_K_MLP_FWD] == 1;
    // With several workers' calls in flight the forward GEMM and the ring dW1 kernel run in their light
    // shared-memory configurations (a CTA of each fits on one SM); alone, the deep pipelines are faster.
    if (!serial && c->cfg.W > 1 && !(variant & 128)) variant |= kMlpLightBit;
    if (c->defer) {
        // The next internal stream and its own scratch set (calls on one stream are ordered, so the set needs no
        // guard); what crosses streams -- bf16(X), labels, the dW1 operands, the small partial gradients -- sits
        // in the call's pool slots.  The call ends with k_bwd.
        k = serial ? 0 : c->rr_stream;
        if (!serial) c->rr_stream = (c->rr_stream + 1) % c->n_wstreams;
        cudaStream_t s_run = serial ? c->s_acc : c->s_w[k];
        if (!serial) {
            CK(cudaEventRecord(c->ev_fork, c->s_acc));
            CK(cudaStreamWaitEvent(s_run, c->ev_fork, 0));
        }
        MlpWorkers wk{};
        for (int j = 0; j < n; ++j) wk.w[j] = mixed ? mixed->w[j] : (uint8_t)worker;
        CK(launch_mlp_front(c->mlp_dims, c->mlp_scratch[k], c->x(c->pub), c->shadow(c->pub), c->pub, n, first,
                            c->acc(c->cur, worker), c->cnt(c->cur, 0), &c->pool[c->cur], pool0, &wk, variant, s_run,
                            c->mlp_chain(serial, n), mlp_mark, c));
        for (int j = 0; j < n; ++j) c->pool_owner[c->cur][pool0 + j] = (int16_t)wk.w[j];
        if (!serial) c->w_outstanding[k] = true;
        return ABS_OK;
    }
    const MlpScratch& sc = c->mlp_scratch[set];
    cudaStream_t s_run = serial ? c->s_acc : c->s_w[k];
    if (!serial) {
        CK(cudaEventRecord(c->ev_fork, c->s_acc));
        CK(cudaStreamWaitEvent(s_run, c->ev_fork, 0));
    }
    CK(launch_mlp_front(c->mlp_dims, sc, c->x(c->pub), c->shadow(c->pub), c->pub, n, first, c->acc(c->cur, worker),
                        c->cnt(c->cur, worker), nullptr, 0, nullptr, variant, s_run, c->mlp_chain(serial, n), mlp_mark, c));
    cudaStream_t s_gemm = s_run;
    if (!serial) {   // dW1 on the worker's second (lowest-priority) stream, behind the front kernels of this call
        s_gemm = c->s_d[k];
        CK(cudaEventRecord(c->ev_front[k], s_run));
        CK(cudaStreamWaitEvent(s_gemm, c->ev_front[k], 0));
    }
    // On its own stream the kernel ahead of this dW1 is the worker's previous dW1, which writes the same slice:
    // never chained there (the register-prefetch kernel reads the slice in front of its wait).
    CK(launch_mlp_dw1(c->mlp_dims, sc, nullptr, nullptr, c->acc(c->cur, worker),
                      &c->acc_tmaps[(size_t)c->cur * c->cfg.W + worker], n, first, variant, s_gemm,
                      serial && (c->mlp_chain(serial, n) & kChainDw1) != 0, mlp_mark, c));
    c->w1_touched[c->cur][worker] = true;
    if (serial) {
        for (bool& u : c->set_used) u = false;
    } else {
        CK(cudaEventRecord(c->ev_set_done[set], s_gemm));
        CK(cudaEventRecord(c->ev_w_done[k], s_gemm));
        c->set_used[set] = true;
        c->w_outstanding[k] = true;
    }
    return ABS_OK;
}

// Runs the worker's waiting micro-batches (ABS_FLAG_MLP_COALESCE) as one group.
int flush_worker(abs_ctx* c, uint32_t worker) {
    const int n = c->pend_n[worker];
    if (n == 0) return ABS_OK;
    const int set = c->pend_set[worker];
    c->pend_n[worker] = 0;
    c->set_reserved[set] = false;
    c->n_reserved -= 1;
    return run_mlp_group(c, worker, set, n, c->pend_first[worker], 0);
}

int flush_all(abs_ctx* c) {
    if (c->grp_n > 0) {   // deferred mode: the one group of gathered single calls
        const int n = c->grp_n;
        c->grp_n = 0;
        if (int rc = run_mlp_group(c, c->grp_workers.w[0], 0, n, false, c->grp_pool0, &c->grp_workers)) return rc;
    }
    if (c->n_reserved == 0) return ABS_OK;
    for (;;) {   // oldest group first: the order does not change results (rows are independent), only timing
        int best = -1;
        for (uint32_t i = 0; i < c->cfg.W; ++i)
            if (c->pend_n[i] && (best < 0 || c->pend_age[i] < c->pend_age[best])) best = (int)i;
        if (best < 0) return ABS_OK;
        if (int rc = flush_worker(c, (uint32_t)best)) return rc;
    }
}

// ABS_FLAG_MLP_DEFER: dW1 of the worker's micro-batches waiting in the current set's operand pool, one launch
// (K = 64 per micro-batch), stored into -- or, if the W1 slice of its row was written earlier in the iteration,
// added to -- the accumulator row.  Runs behind the worker's front kernels, on its second stream.
int contract_worker(abs_ctx* c, uint32_t set, uint32_t worker) {
    MlpSlots sl{};
    uint8_t owners[kMlpMaxSlots];
    int n = 0;
    for (int q = 0; q < c->pool_n[set]; ++q)
        if (c->pool_owner[set][q] == (int16_t)worker) {
            owners[n] = (uint8_t)worker;
            sl.s[n++] = (uint16_t)q;
            c->pool_owner[set][q] = -1;
        }
    if (n == 0) return ABS_OK;
    const int k = (int)(worker % (uint32_t)c->n_wstreams);
    const bool serial = c->ctas_per_sm[ABS_K_MLP_FWD] == 1;
    int variant = c->ctas_per_sm[ABS_K_MLP_DW1];
    // light form beside the other workers' kernels, as for per-call dW1 (measured: batch calls 13.6 -> 13.1 us)
    if (!serial && c->cfg.W > 1 && !(variant & 128)) variant |= kMlpLightBit;
    cudaStream_t s_gemm = c->s_acc;
    if (!serial) {   // the worker's calls ran on any of the internal streams; stream_acc may have waited for some already
        s_gemm = c->s_d[k];
        CK(cudaEventRecord(c->ev_fork, c->s_acc));
        CK(cudaStreamWaitEvent(s_gemm, c->ev_fork, 0));
        for (int j = 0; j < c->n_wstreams; ++j)
            if (c->w_outstanding[j]) {
                CK(cudaEventRecord(c->ev_front[j], c->s_w[j]));
                CK(cudaStreamWaitEvent(s_gemm, c->ev_front[j], 0));
            }
    }
    const bool keep = c->w1_touched[set][worker];   // the row was written earlier in the iteration: add to it
    CK(launch_mlp_gather_small(c->mlp_dims, c->pool[set], sl, owners, n, (int)worker, 1, keep ? (1ull << worker) : 0ull,
                               c->acc(set, 0), c->L.P_pad, s_gemm, false));
    c->launches += 1;
    CK(launch_mlp_dw1(c->mlp_dims, c->mlp_scratch[0], &c->pool[set], &sl, c->acc(set, worker),
                      &c->acc_tmaps[(size_t)set * c->cfg.W + worker], n, !keep, variant, s_gemm, false, mlp_mark, c));
    c->w1_touched[set][worker] = true;
    if (!serial) c->d_outstanding[k] = true;
    return ABS_OK;
}

// Every gradient enqueued so far is on its way into the accumulator rows: waiting groups are started and
// (ABS_FLAG_MLP_DEFER) the pooled dW1 operands contracted.
int settle_all(abs_ctx* c) {
    if (int rc = flush_all(c)) return rc;
    if (!c->defer || c->fused_pending[c->cur]) return ABS_OK;   // (pending: the set's fused step works from the pool)
    for (uint32_t i = 0; i < c->cfg.W; ++i)
        if (int rc = contract_worker(c, c->cur, i)) return rc;
    return ABS_OK;
}

// A set that waits for its fused step with its W1 gradients still in pooled form (eager mode: until the next
// abs_sync_step) is needed row by row after all: contract it.
int contract_pending_sets(abs_ctx* c) {
    for (uint32_t set = 0; set < 2; ++set)
        if (c->fused_pending[set]) {
            c->fused_pending[set] = false;
            for (uint32_t i = 0; i < c->cfg.W; ++i)
                if (int rc = contract_worker(c, set, i)) return rc;
            c->pool_n[set] = 0;
        }
    return ABS_OK;
}

// End of the current set's iteration: its waiting groups are started, and its pooled dW1 operands are either left
// for the fused step (every W1 slice of the set untouched: the step then works from the operands, see
// fused_pending) or contracted into the rows.
int close_iteration(abs_ctx* c) {
    if (int rc = flush_all(c)) return rc;
    if (!c->defer) return ABS_OK;
    const uint32_t set = c->cur;
    bool fuse = c->n_ranks == 0 && !c->grad_norm() && c->mlp_dims.d_hidden % 128 == 0 && c->ctas_per_sm[ABS_K_MLP_BWD] != 1;
    for (uint32_t i = 0; i < c->cfg.W && fuse; ++i) fuse = !c->w1_touched[set][i];
    int n = 0;
    if (fuse) {
        for (int q = 0; q < c->pool_n[set]; ++q)
            if (c->pool_owner[set][q] >= 0) c->fused_slots[set].s[n++] = (uint16_t)q;
        fuse = n > 0;
    }
    if (!fuse) {
        if (int rc = settle_all(c)) return rc;
        c->pool_n[set] = 0;
        return ABS_OK;
    }
    c->fused_pending[set] = true;
    c->fused_n[set] = n;
    return ABS_OK;
}

// n consecutive free slots of the current set's operand pool.  A full pool is emptied first: everything in it is
// contracted, and stream_acc (so every later kernel that writes a slot) waits for those launches.
int take_pool_slots(abs_ctx* c, int n, int* slot0) {
    const uint32_t set = c->cur;
    if (c->pool_n[set] + n > c->pool[set].cap) {
        if (int rc = settle_all(c)) return rc;
        if (int rc = wait_for_workers(c, c->s_acc, true)) return rc;
        c->pool_n[set] = 0;
    }
    *slot0 = c->pool_n[set];
    c->pool_n[set] += n;
    return ABS_OK;
}

// The iteration of set `closing` has ended (its gradients are settled); `opening` starts a new one (its pool is
// empty: what it held was contracted, or consumed by its fused step, before the set could become current again).
void turn_sets(abs_ctx* c, uint32_t closing, uint32_t opening) {
    (void)closing;
    for (uint32_t i = 0; i < c->cfg.W; ++i) c->w1_touched[opening][i] = false;
}

// One micro-batch of `worker` joins its waiting group: cast now (the caller's buffers are free again once
// stream_acc has passed this point), everything else when the group runs.
int coalesce_one(abs_ctx* c, uint32_t worker, const void* x_dev, const int32_t* y_dev) {
    if (c->defer) {
        // Deferred calls are independent of their workers: ONE group gathers the next kMlpGatherMax single calls,
        // whoever makes them, in consecutive pool slots (slots a group leaves unused stay empty).  (Groups of eight
        // measured slower than groups of four: 10.8 against 10.1 us per micro-batch -- the forward GEMM of a group
        // starts later and the last group of an iteration holds the step back longer.)
        if (c->grp_n == 0)
            if (int rc = take_pool_slots(c, kMlpGatherMax, &c->grp_pool0)) return rc;
        CK(launch_mlp_cast(c->mlp_dims, c->mlp_scratch[0], c->grp_pool0 + c->grp_n, 1, &x_dev, c->x_bf16(), &y_dev, &c->pool[c->cur],
                           c->s_acc, (c->mlp_chain(false, 1) & kChainCast) != 0, mlp_mark, c));
        c->grp_workers.w[c->grp_n++] = (uint8_t)worker;
        c->h_cnt[(size_t)c->cur * c->cfg.W + worker] += 1;
        if (c->grp_n == kMlpGatherMax) return flush_all(c);
        return ABS_OK;
    }
    if (c->pend_n[worker] == 0) {
        {
            if (c->n_reserved >= kMlpSets / 2) {   // keep half of the scratch sets for groups that are running
                int oldest = -1;
                for (uint32_t i = 0; i < c->cfg.W; ++i)
                    if (c->pend_n[i] && (oldest < 0 || c->pend_age[i] < c->pend_age[oldest])) oldest = (int)i;
                if (int rc = flush_worker(c, (uint32_t)oldest)) return rc;
            }
            int set = 0;
            if (int rc = take_scratch_set(c, false, &set)) return rc;
            c->set_reserved[set] = true;
            c->pend_set[worker] = set;
        }
        c->n_reserved += 1;
        c->pend_first[worker] = c->h_cnt[(size_t)c->cur * c->cfg.W + worker] == 0;
        c->pend_age[worker] = ++c->pend_clock;
    }
    const int slot = c->pend_n[worker];
    CK(launch_mlp_cast(c->mlp_dims, c->mlp_scratch[c->pend_set[worker]], slot, 1, &x_dev, c->x_bf16(), &y_dev, nullptr, c->s_acc,
                       (c->mlp_chain(false, 1) & kChainCast) != 0, mlp_mark, c));
    c->pend_n[worker] = slot + 1;
    c->h_cnt[(size_t)c->cur * c->cfg.W + worker] += 1;
    if (c->pend_n[worker] == kMlpGatherMax) return flush_worker(c, worker);
    return ABS_OK;
}

}  // namespace

extern "C" {

size_t abs_workspace_bytes(const abs_config* cfg) {
    if (!config_ok(cfg, nullptr)) return 0;
    return make_layout(*cfg).total;
}

int abs_init(abs_ctx** out, const abs_config* cfg, void* workspace_dev, size_t workspace_bytes,
             const float* params0_dev) {
    g_init_error.clear();
    if (!out) { g_init_error = "out is NULL"; return ABS_EINVAL; }
    *out = nullptr;
    std::string why;
    if (!config_ok(cfg, &why)) { g_init_error = why; return ABS_EINVAL; }
    if (!workspace_dev || (reinterpret_cast<uintptr_t>(workspace_dev) & 255)) {
        g_init_error = "workspace must be non-NULL and 256-byte aligned";
        return ABS_EINVAL;
    }
    if (!params0_dev || (reinterpret_cast<uintptr_t>(params0_dev) & 15)) {
        g_init_error = "params0 must be non-NULL and 16-byte aligned";
        return ABS_EINVAL;
    }
    Layout L = make_layout(*cfg);
    if (workspace_bytes < L.total) { g_init_error = "workspace too small"; return ABS_ENOMEM; }

    abs_ctx* c = new abs_ctx();
    c->cfg = *cfg;
    c->L = L;
    c->ws = static_cast<char*>(workspace_dev);
    c->s_acc = static_cast<cudaStream_t>(cfg->stream_acc);
    c->s_sync = static_cast<cudaStream_t>(cfg->stream_sync);
    c->pipelined = cfg->flags & ABS_FLAG_PIPELINED;
    c->mlp = cfg->flags & ABS_FLAG_MLP;
    c->coalesce = cfg->flags & ABS_FLAG_MLP_COALESCE;
    c->defer = cfg->flags & ABS_FLAG_MLP_DEFER;
    c->h_cnt.assign((size_t)2 * cfg->W, 0);
    c->lr_now = cfg->lr;
    c->lr_prev_call = cfg->lr;

    auto bail = [&](cudaError_t e, const char* what) {
        cuda_fail(c, e, what);
        g_init_error = c->err;
        delete c;
        return ABS_ECUDA;
    };
    cudaError_t e;
    if ((e = cudaGetDevice(&c->device)) != cudaSuccess) return bail(e, "cudaGetDevice");
    if ((e = cudaDeviceGetAttribute(&c->num_sms, cudaDevAttrMultiProcessorCount, c->device)) != cudaSuccess)
        return bail(e, "cudaDeviceGetAttribute");
    if ((e = cudaEventCreateWithFlags(&c->ev_acc_done, cudaEventDisableTiming)) != cudaSuccess) return bail(e, "cudaEventCreate");
    if ((e = cudaEventCreateWithFlags(&c->ev_sync_done, cudaEventDisableTiming)) != cudaSuccess) return bail(e, "cudaEventCreate");
    if ((e = cudaEventCreateWithFlags(&c->ev_aux, cudaEventDisableTiming)) != cudaSuccess) return bail(e, "cudaEventCreate");
    if (cfg->flags & ABS_FLAG_HOST_INPUT) {
        if ((e = cudaStreamCreateWithFlags(&c->s_copy, cudaStreamNonBlocking)) != cudaSuccess) return bail(e, "cudaStreamCreate");
        for (int k = 0; k < 2; ++k) {
            if ((e = cudaEventCreateWithFlags(&c->ev_stage_free[k], cudaEventDisableTiming)) != cudaSuccess) return bail(e, "cudaEventCreate");
            if ((e = cudaEventCreateWithFlags(&c->ev_stage_full[k], cudaEventDisableTiming)) != cudaSuccess) return bail(e, "cudaEventCreate");
        }
    }

    // Algorithm 1, Initialization: G_{-1}^i = 0, counters 0, v = 0, x_0 = params0.
    const size_t state_bytes = L.off_gcnt + (size_t)(kMaxW + 64) * 4;
    if ((e = cudaMemsetAsync(c->ws, 0, state_bytes, c->s_acc)) != cudaSuccess) return bail(e, "cudaMemsetAsync");
    if ((e = cudaMemcpyAsync(c->x(0), params0_dev, cfg->P * 4, cudaMemcpyDeviceToDevice, c->s_acc)) != cudaSuccess)
        return bail(e, "cudaMemcpyAsync(params0)");
    if ((cfg->flags & ABS_FLAG_GRAD_NORM) &&
        (e = cudaMemsetAsync(c->ws + L.off_norm_log, 0, (size_t)kLogDepth * 8, c->s_acc)) != cudaSuccess)
        return bail(e, "cudaMemsetAsync");
    if (c->mlp) {
        c->mlp_dims = MlpDims{(int)cfg->mlp_in, (int)cfg->mlp_hidden, (int)cfg->mlp_out, (int)cfg->mlp_mb};
        const char* msg = nullptr;
        if ((e = cudaMemsetAsync(c->ws + L.off_shadow[0], 0, L.P_pad * 2, c->s_acc)) != cudaSuccess) return bail(e, "cudaMemsetAsync");
        if (c->pipelined && (e = cudaMemsetAsync(c->ws + L.off_shadow[1], 0, L.P_pad * 2, c->s_acc)) != cudaSuccess)
            return bail(e, "cudaMemsetAsync");
        const size_t one = mlp_scratch_bytes(c->mlp_dims);
        for (int k = 0; k < kMlpSets; ++k) {
            if ((e = mlp_scratch_init(&c->mlp_scratch[k], c->mlp_dims, c->ws + L.off_mlp + k * one, c->shadow(0), c->shadow(1),
                                      &msg)) != cudaSuccess)
                return bail(e, msg ? msg : "mlp_scratch_init");
            if ((e = cudaMemsetAsync(c->mlp_scratch[k].zero_from, 0, c->mlp_scratch[k].zero_bytes, c->s_acc)) != cudaSuccess)
                return bail(e, "cudaMemsetAsync");
            if ((e = cudaEventCreateWithFlags(&c->ev_set_done[k], cudaEventDisableTiming)) != cudaSuccess) return bail(e, "cudaEventCreate");
        }
        if (c->defer)
            for (int k = 0; k < 2; ++k) {
                if ((e = mlp_pool_init(&c->pool[k], c->mlp_dims, L.pool_cap, c->ws + L.off_pool[k])) != cudaSuccess)
                    return bail(e, "cuTensorMapEncodeTiled(operand pool)");
                c->pool_owner[k].assign((size_t)L.pool_cap, (int16_t)-1);
                if ((e = mlp_make_acc_tmap(&c->tm_x[k], c->mlp_dims, c->x(k))) != cudaSuccess ||
                    (e = mlp_make_shadow_tmap(&c->tm_shadow[k], c->mlp_dims, c->shadow(k))) != cudaSuccess ||
                    (e = mlp_make_acc_tmap(&c->tm_v, c->mlp_dims, c->v())) != cudaSuccess)
                    return bail(e, "cuTensorMapEncodeTiled(parameters)");
            }
        if ((e = cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming)) != cudaSuccess) return bail(e, "cudaEventCreate");
        c->n_wstreams = c->defer ? kMlpStreams : (int)std::min<uint32_t>(cfg->W, kMlpStreams);
        // Highest priority: the short, dependent gradient kernels get free CTA slots before the long HBM-bound
        // fused step that runs beside them on stream_sync and would otherwise fill every slot with its own CTAs.
        int prio_lo = 0, prio_hi = 0;
        if ((e = cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi)) != cudaSuccess) return bail(e, "cudaDeviceGetStreamPriorityRange");
        for (int k = 0; k < c->n_wstreams; ++k) {
            if ((e = cudaStreamCreateWithPriority(&c->s_w[k], cudaStreamNonBlocking, prio_hi)) != cudaSuccess) return bail(e, "cudaStreamCreate");
            if ((e = cudaStreamCreateWithPriority(&c->s_d[k], cudaStreamNonBlocking, prio_lo)) != cudaSuccess) return bail(e, "cudaStreamCreate");
            if ((e = cudaEventCreateWithFlags(&c->ev_w_done[k], cudaEventDisableTiming)) != cudaSuccess) return bail(e, "cudaEventCreate");
            if ((e = cudaEventCreateWithFlags(&c->ev_front[k], cudaEventDisableTiming)) != cudaSuccess) return bail(e, "cudaEventCreate");
            if ((e = cudaEventCreateWithFlags(&c->ev_d_done[k], cudaEventDisableTiming)) != cudaSuccess) return bail(e, "cudaEventCreate");
        }
        c->acc_tmaps.resize((size_t)2 * cfg->W);
        for (uint32_t set = 0; set < 2; ++set)
            for (uint32_t i = 0; i < cfg->W; ++i)
                if ((e = mlp_make_acc_tmap(&c->acc_tmaps[(size_t)set * cfg->W + i], c->mlp_dims, c->acc(set, i))) != cudaSuccess)
                    return bail(e, "cuTensorMapEncodeTiled(accumulator)");
        if ((e = launch_cast_bf16(c->x(0), c->shadow(0), L.P_pad, c->num_sms, c->s_acc)) != cudaSuccess)
            return bail(e, "launch_cast_bf16");
        c->launches += 1;
    }
    if (c->pipelined) {   // stream_sync must not start before the state is initialised
        if ((e = cudaEventRecord(c->ev_aux, c->s_acc)) != cudaSuccess) return bail(e, "cudaEventRecord");
        if ((e = cudaStreamWaitEvent(c->s_sync, c->ev_aux, 0)) != cudaSuccess) return bail(e, "cudaStreamWaitEvent");
    }
    {
        std::lock_guard<std::mutex> g(g_live_mu);
        g_live.insert(c);
    }
    *out = c;
    return ABS_OK;
}

int abs_accumulate(abs_ctx* c, uint32_t worker, const void* grad_dev) {
    if (!live(c)) return ABS_ESTATE;
    if (worker >= c->cfg.W) return invalid(c, "worker index out of range");
    if (!grad_dev || (reinterpret_cast<uintptr_t>(grad_dev) & 15)) return invalid(c, "gradient pointer must be non-NULL and 16-byte aligned");
    if (int rc = join_workers(c)) return rc;
    // overwrite-first mode: the row is not kept zeroed, so a worker's first micro-batch of an iteration stores
    const bool first = (c->cfg.flags & ABS_FLAG_OVERWRITE_FIRST) && c->h_cnt[(size_t)c->cur * c->cfg.W + worker] == 0;
    {
        Timed tm(c, ABS_K_ACCUMULATE, c->s_acc);
        CK(launch_accumulate(c->acc(c->cur, worker), grad_dev, c->cfg.grad_dtype, c->cfg.P, c->cnt(c->cur, worker), first,
                             c->ctas_per_sm[ABS_K_ACCUMULATE], c->num_sms, c->s_acc, c->chained()));
    }
    c->launches += 1;
    c->w1_touched[c->cur][worker] = true;
    c->h_cnt[(size_t)c->cur * c->cfg.W + worker] += 1;
    return ABS_OK;
}

int abs_accumulate_batch(abs_ctx* c, uint32_t worker, uint32_t n, const void* const* grads_dev) {
    if (!live(c)) return ABS_ESTATE;
    if (worker >= c->cfg.W) return invalid(c, "worker index out of range");
    if (n == 0 || n > (uint32_t)kMaxAccBatch) return invalid(c, "n must be in 1..8");
    if (!grads_dev) return invalid(c, "gradient pointer list is NULL");
    GradList gl{};
    for (uint32_t k = 0; k < n; ++k) {
        if (!grads_dev[k] || (reinterpret_cast<uintptr_t>(grads_dev[k]) & 15))
            return invalid(c, "every gradient pointer must be non-NULL and 16-byte aligned");
        gl.p[k] = grads_dev[k];
    }
    if (int rc = join_workers(c)) return rc;
    const bool first = (c->cfg.flags & ABS_FLAG_OVERWRITE_FIRST) && c->h_cnt[(size_t)c->cur * c->cfg.W + worker] == 0;
    {
        Timed tm(c, ABS_K_ACCUMULATE, c->s_acc);
        CK(launch_accumulate_multi(c->acc(c->cur, worker), gl, (int)n, c->cfg.grad_dtype, c->cfg.P, c->cnt(c->cur, worker),
                                   first, c->ctas_per_sm[ABS_K_ACCUMULATE], c->num_sms, c->s_acc, c->chained()));
    }
    c->launches += 1;
    c->w1_touched[c->cur][worker] = true;
    c->h_cnt[(size_t)c->cur * c->cfg.W + worker] += (int32_t)n;
    return ABS_OK;
}

int abs_accumulate_host(abs_ctx* c, uint32_t worker, const void* grad_host) {
    if (!live(c)) return ABS_ESTATE;
    if (!(c->cfg.flags & ABS_FLAG_HOST_INPUT)) return invalid(c, "context was created without ABS_FLAG_HOST_INPUT");
    if (worker >= c->cfg.W) return invalid(c, "worker index out of range");
    if (!grad_host) return invalid(c, "gradient pointer is NULL");
    if (int rc = join_workers(c)) return rc;
    const bool first = (c->cfg.flags & ABS_FLAG_OVERWRITE_FIRST) && c->h_cnt[(size_t)c->cur * c->cfg.W + worker] == 0;
    const int k = c->stage_next;
    c->stage_next ^= 1;
    const size_t es = c->cfg.grad_dtype == ABS_GRAD_BF16 ? 2 : 4;
    void* stage = c->ws + c->L.off_stage[k];
    // The copy of micro-batch n+1 overlaps the accumulate kernel of micro-batch n.
    if (c->stage_used[k]) CK(cudaStreamWaitEvent(c->s_copy, c->ev_stage_free[k], 0));
    CK(cudaMemcpyAsync(stage, grad_host, c->cfg.P * es, cudaMemcpyHostToDevice, c->s_copy));
    CK(cudaEventRecord(c->ev_stage_full[k], c->s_copy));
    CK(cudaStreamWaitEvent(c->s_acc, c->ev_stage_full[k], 0));
    {
        Timed tm(c, ABS_K_ACCUMULATE, c->s_acc);
        CK(launch_accumulate(c->acc(c->cur, worker), stage, c->cfg.grad_dtype, c->cfg.P, c->cnt(c->cur, worker), first,
                             c->ctas_per_sm[ABS_K_ACCUMULATE], c->num_sms, c->s_acc, c->chained()));
    }
    CK(cudaEventRecord(c->ev_stage_free[k], c->s_acc));
    c->stage_used[k] = true;
    c->launches += 1;
    c->w1_touched[c->cur][worker] = true;
    c->h_cnt[(size_t)c->cur * c->cfg.W + worker] += 1;
    return ABS_OK;
}

int abs_accumulate_mlp_list(abs_ctx* c, uint32_t worker, uint32_t n, const void* const* x_devs, const int32_t* const* y_devs) {
    if (!live(c)) return ABS_ESTATE;
    if (!c->mlp) return invalid(c, "context was created without ABS_FLAG_MLP");
    if (worker >= c->cfg.W) return invalid(c, "worker index out of range");
    if (n == 0 || n > (uint32_t)kMlpMaxBatch) return invalid(c, "n must be in 1..8");
    if (!x_devs || !y_devs) return invalid(c, "pointer list is NULL");
    for (uint32_t j = 0; j < n; ++j) {
        if (!x_devs[j] || (reinterpret_cast<uintptr_t>(x_devs[j]) & 15)) return invalid(c, "x pointer must be non-NULL and 16-byte aligned");
        if (!y_devs[j] || (reinterpret_cast<uintptr_t>(y_devs[j]) & 3)) return invalid(c, "y pointer must be non-NULL and 4-byte aligned");
    }
    const bool serial = c->ctas_per_sm[ABS_K_MLP_FWD] == 1;   // measurement aid: everything on stream_acc
    if (c->coalesce && n == 1 && !serial) return coalesce_one(c, worker, x_devs[0], y_devs[0]);
    if (int rc = flush_worker(c, worker)) return rc;           // the worker's row is added to in call order
    // Only the cast kernel reads the caller's buffers; it runs on stream_acc, in call order.  The rest of the
    // call (forward, loss, backward, dW1) runs on the worker's internal stream, so that the latency chains of
    // different workers overlap and the HBM-bound dW1 GEMMs fill the gaps of the small kernels.
    if (serial) {
        if (int rc = join_workers(c)) return rc;
    }
    int set = 0, pool0 = 0;
    if (c->defer) {
        if (int rc = take_pool_slots(c, (int)n, &pool0)) return rc;
    } else if (int rc = take_scratch_set(c, serial, &set)) {
        return rc;
    }
    // A worker's first gradient of an iteration finds its accumulator row empty (all zero, or -- with
    // ABS_FLAG_OVERWRITE_FIRST -- stale): it is stored, not added, and dW1 skips reading the 4 d_in d_hidden
    // bytes of the slice.  0 + g = g, so the default mode's results do not change.
    const bool first = c->h_cnt[(size_t)c->cur * c->cfg.W + worker] == 0;
    CK(launch_mlp_cast(c->mlp_dims, c->mlp_scratch[set], c->defer ? pool0 : 0, (int)n, x_devs, c->x_bf16(), y_devs,
                       c->defer ? &c->pool[c->cur] : nullptr, c->s_acc, (c->mlp_chain(serial, (int)n) & kChainCast) != 0, mlp_mark, c));
    if (int rc = run_mlp_group(c, worker, set, (int)n, first, pool0)) return rc;
    c->h_cnt[(size_t)c->cur * c->cfg.W + worker] += (int32_t)n;
    return ABS_OK;
}

int abs_accumulate_mlp_batch(abs_ctx* c, uint32_t worker, uint32_t n, const void* x_dev, const int32_t* y_dev) {
    if (!live(c)) return ABS_ESTATE;
    if (!c->mlp) return invalid(c, "context was created without ABS_FLAG_MLP");
    if (n == 0 || n > (uint32_t)kMlpMaxBatch) return invalid(c, "n must be in 1..8");
    if (!x_dev || (reinterpret_cast<uintptr_t>(x_dev) & 15)) return invalid(c, "x pointer must be non-NULL and 16-byte aligned");
    if (!y_dev || (reinterpret_cast<uintptr_t>(y_dev) & 3)) return invalid(c, "y pointer must be non-NULL and 4-byte aligned");
    // micro-batch j at x_dev + j * mb * mlp_in elements, y_dev + j * mb
    const void* xs[kMlpMaxBatch];
    const int32_t* ys[kMlpMaxBatch];
    const size_t es = c->x_bf16() ? 2 : 4;
    for (uint32_t j = 0; j < n; ++j) {
        xs[j] = static_cast<const char*>(x_dev) + (size_t)j * c->mlp_dims.mb * c->mlp_dims.d_in * es;
        ys[j] = y_dev + (size_t)j * c->mlp_dims.mb;
    }
    return abs_accumulate_mlp_list(c, worker, n, xs, ys);
}

int abs_accumulate_mlp(abs_ctx* c, uint32_t worker, const void* x_dev, const int32_t* y_dev) {
    return abs_accumulate_mlp_batch(c, worker, 1, x_dev, y_dev);
}

int abs_sync_step(abs_ctx* c) {
    if (!live(c)) return ABS_ESTATE;
    if (c->n_ranks != 0) return invalid(c, "context is in multi-GPU mode: end iterations with abs_global_begin / _step / _end");
    if (int rc = close_iteration(c)) return rc;   // every gradient of iteration t is under way before the iteration ends
    const uint32_t W = c->cfg.W;
    const uint32_t d = c->cur ^ 1;   // the delayed set (filled during iteration t-1)
    if (!c->pipelined) {
        // Step 1 on the delayed set, in place, on stream_acc: the gradient kernels still running on the
        // worker streams read the parameters it overwrites.
        if (int rc = join_workers(c)) return rc;
        int64_t B = 0;
        for (uint32_t i = 0; i < W; ++i) B += c->h_cnt[(size_t)d * W + i];
        if (B > 0) {
            // The learning rate travels with the gradients: the delayed set is applied with the
            // rate that was in effect when its iteration ended (same rule as pipelined mode,
            // where that kernel was already launched one call ago).
            const float lr_call = c->lr_now;
            c->lr_now = c->lr_prev_call;
            int rc = launch_fused(c, d, c->pub, c->pub, c->t, c->s_acc);
            c->lr_now = lr_call;
            if (rc != ABS_OK) return rc;
            c->disp_scale = c->lr_prev_call;
        } else {
            CK(cudaMemsetAsync(c->log_row(c->t), 0, kMaxW * 4, c->s_acc));
            if (c->grad_norm()) CK(cudaMemsetAsync(c->norm_log(c->t), 0, 8, c->s_acc));
            c->disp_scale = 0.f;
        }
    } else {
        // Publish x_{t+1}: the kernel launched one call ago (on the set of iteration t-1).
        if (c->pending) {
            CK(cudaStreamWaitEvent(c->s_acc, c->ev_sync_done, 0));
            c->pub = c->pending_out;
            c->pending = false;
        }
        // Launch Step 1 for the set just filled (iteration t); it is published by the next call.
        int64_t B = 0;
        for (uint32_t i = 0; i < W; ++i) B += c->h_cnt[(size_t)c->cur * W + i];
        CK(cudaEventRecord(c->ev_acc_done, c->s_acc));
        CK(cudaStreamWaitEvent(c->s_sync, c->ev_acc_done, 0));
        // Step 1 needs every gradient of iteration t; stream_acc does not: the workers go straight on with
        // iteration t+1 (other accumulator set, other parameter buffer), each behind its own previous call only.
        if (int rc = wait_for_workers(c, c->s_sync, false)) return rc;
        if (B > 0) {
            const int out = c->pub ^ 1;
            int rc = launch_fused(c, c->cur, c->pub, out, c->t + 1, c->s_sync);
            if (rc != ABS_OK) return rc;
            c->disp_scale = c->lr_now;
            c->pending_out = out;
        } else {
            CK(cudaMemsetAsync(c->log_row(c->t + 1), 0, kMaxW * 4, c->s_sync));
            if (c->grad_norm()) CK(cudaMemsetAsync(c->norm_log(c->t + 1), 0, 8, c->s_sync));
            c->disp_scale = 0.f;
            c->pending_out = c->pub;
        }
        CK(cudaEventRecord(c->ev_sync_done, c->s_sync));
        c->pending = true;
    }
    // Logical state (Algorithm 1: clear the consumed set, swap roles, t = t + 1).
    for (uint32_t i = 0; i < W; ++i) c->h_cnt[(size_t)d * W + i] = 0;
    turn_sets(c, c->cur, d);
    c->lr_prev_call = c->lr_now;
    c->cur = d;
    c->t += 1;
    return ABS_OK;
}

// ---- Step 1 across GPUs: one rank per GPU, this context holds the rank's W local workers ---------------
int abs_global_attach(abs_ctx* c, const abs_peer_table* peers) {
    if (!live(c)) return ABS_ESTATE;
    if (!peers) return invalid(c, "peer table is NULL");
    if (!c->pipelined) return invalid(c, "multi-GPU mode needs ABS_FLAG_PIPELINED (two parameter buffers)");
    if (peers->n_ranks == 0 || peers->n_ranks > ABS_MAX_RANKS) return invalid(c, "n_ranks must be in 1..16");
    if (peers->rank >= peers->n_ranks) return invalid(c, "rank out of range");
    if ((uint64_t)peers->n_ranks * c->cfg.W > ABS_MAX_WORKERS) return invalid(c, "n_ranks * W must not exceed 64");
    if (c->grad_norm()) return invalid(c, "ABS_FLAG_GRAD_NORM is not available in multi-GPU mode");
    if (c->t != 0 || c->n_ranks != 0) return invalid(c, "attach once, before the first step");
    for (uint32_t q = 0; q < peers->n_ranks; ++q) {
        void* p = peers->workspace_dev[q];
        if (!p || (reinterpret_cast<uintptr_t>(p) & 255)) return invalid(c, "peer workspace must be non-NULL and 256-byte aligned");
    }
    if (peers->workspace_dev[peers->rank] != c->ws) return invalid(c, "workspace_dev[rank] must be this context's own workspace");
    // A peer's workspace on another GPU is read and written by this GPU's kernel with plain loads and stores: that
    // needs peer access from this device to the peer's.  Mappings opened with abs_ipc_open have it already (the IPC
    // open enables it); plain pointers of another device of the same process get it here.
    for (uint32_t q = 0; q < peers->n_ranks; ++q) {
        if (q == peers->rank) continue;
        cudaPointerAttributes at{};
        if (cudaPointerGetAttributes(&at, peers->workspace_dev[q]) != cudaSuccess) { cudaGetLastError(); return invalid(c, "a peer workspace is not a device pointer known to this process"); }
        if (at.type != cudaMemoryTypeDevice) return invalid(c, "a peer workspace is not device memory");
        if (at.device == c->device) continue;
        int can = 0;
        CK(cudaDeviceCanAccessPeer(&can, c->device, at.device));
        if (!can) return invalid(c, "this GPU has no peer access to a peer workspace's GPU");
        int cur_dev = c->device;
        CK(cudaGetDevice(&cur_dev));
        if (cur_dev != c->device) CK(cudaSetDevice(c->device));   // peer access is granted to the current device
        const cudaError_t e = cudaDeviceEnablePeerAccess(at.device, 0);
        if (cur_dev != c->device) cudaSetDevice(cur_dev);
        if (e == cudaErrorPeerAccessAlreadyEnabled) cudaGetLastError();
        else if (e != cudaSuccess) return cuda_fail(c, e, "cudaDeviceEnablePeerAccess");
    }
    c->n_ranks = peers->n_ranks;
    c->rank = peers->rank;
    for (uint32_t q = 0; q < peers->n_ranks; ++q) c->peer_ws[q] = static_cast<char*>(peers->workspace_dev[q]);
    c->global_phase = 0;
    return ABS_OK;
}

int abs_global_begin(abs_ctx* c, int32_t** counts_dev, uint32_t* n_counts) {
    if (!live(c)) return ABS_ESTATE;
    if (c->n_ranks == 0) return invalid(c, "abs_global_attach has not been called");
    if (c->global_phase != 0) return invalid(c, "abs_global_begin / _step / _end must be called in that order");
    if (!counts_dev || !n_counts) return invalid(c, "output pointer is NULL");
    if (int rc = settle_all(c)) return rc;
    c->pool_n[c->cur] = 0;
    const uint32_t W = c->cfg.W;
    // Publish x_{t+1}: the kernels launched one call ago, on every rank, have all finished (ev_sync_done was
    // recorded behind the caller's closing barrier).
    if (c->pending) {
        CK(cudaStreamWaitEvent(c->s_acc, c->ev_sync_done, 0));
        c->pub = c->pending_out;
        c->pending = false;
    }
    CK(cudaEventRecord(c->ev_acc_done, c->s_acc));
    CK(cudaStreamWaitEvent(c->s_sync, c->ev_acc_done, 0));
    if (int rc = wait_for_workers(c, c->s_sync, false)) return rc;
    // This rank's b_i into its slots of the exchange vector (zeros elsewhere: the caller's sum over ranks then
    // is a gather); the device counters of the set are cleared here, the kernel reads the exchanged copy.
    CK(launch_global_counts(c->gcnt(), c->cnt(c->cur, 0), (int)(c->rank * W), (int)W, (int)(c->n_ranks * W), c->s_sync));
    c->launches += 1;
    *counts_dev = c->gcnt();
    *n_counts = c->n_ranks * W;
    c->global_phase = 1;
    return ABS_OK;
}

int abs_global_step(abs_ctx* c) {
    if (!live(c)) return ABS_ESTATE;
    if (c->n_ranks == 0) return invalid(c, "abs_global_attach has not been called");
    if (c->global_phase != 1) return invalid(c, "abs_global_begin / _step / _end must be called in that order");
    const uint32_t W = c->cfg.W, G = c->n_ranks;
    const int out = c->pub ^ 1;
    GlobalSyncArgs a{};
    a.x_in = c->x(c->pub);
    a.v = c->v();
    for (uint32_t q = 0; q < G; ++q) {
        char* ws = c->peer_ws[q];   // identical configuration on every rank: identical layout
        a.acc[q] = reinterpret_cast<float*>(ws + c->L.off_acc) + (size_t)c->cur * W * c->L.P_pad;
        a.x_out[q] = reinterpret_cast<float*>(ws + c->L.off_x[out]);
        a.shadow[q] = c->mlp ? reinterpret_cast<__nv_bfloat16*>(ws + c->L.off_shadow[out]) : nullptr;
    }
    a.row_stride = c->L.P_pad;
    slice_vectors(c->L.P_pad, G, c->rank, &a.vec_lo, &a.vec_hi);
    a.G = (int)G;
    a.W_local = (int)W;
    a.cnt_all = c->gcnt();
    a.log_row = c->log_row(c->t + 1);
    a.ticket = c->ticket();
    a.applied = c->applied_word();
    a.lr = c->lr_now;
    a.mu = c->cfg.momentum;
    a.wd = c->cfg.weight_decay;
    a.lambda_dc = c->cfg.lambda_dc;
    a.disp_scale = c->global_prev_lr;
    a.zero_acc = (c->cfg.flags & ABS_FLAG_OVERWRITE_FIRST) ? 0 : 1;
    {
        Timed tm(c, ABS_K_SYNC, c->s_sync);
        CK(launch_sync_global(a, c->ctas_per_sm[ABS_K_SYNC], c->num_sms, c->s_sync, c->chained()));
    }
    c->launches += 1;
    c->global_prev_lr = c->lr_now;
    c->pending_out = out;
    // Logical state (Algorithm 1: clear the consumed set, swap roles, t = t + 1).
    const uint32_t d = c->cur ^ 1;
    for (uint32_t i = 0; i < W; ++i) c->h_cnt[(size_t)d * W + i] = 0;
    turn_sets(c, c->cur, d);
    c->lr_prev_call = c->lr_now;
    c->cur = d;
    c->t += 1;
    c->global_phase = 2;
    return ABS_OK;
}

int abs_global_end(abs_ctx* c) {
    if (!live(c)) return ABS_ESTATE;
    if (c->n_ranks == 0) return invalid(c, "abs_global_attach has not been called");
    if (c->global_phase != 2) return invalid(c, "abs_global_begin / _step / _end must be called in that order");
    CK(cudaEventRecord(c->ev_sync_done, c->s_sync));
    c->pending = true;
    c->global_phase = 0;
    return ABS_OK;
}

int abs_global_slice(abs_ctx* c, uint64_t* first, uint64_t* count) {
    if (!live(c)) return ABS_ESTATE;
    if (c->n_ranks == 0) return invalid(c, "abs_global_attach has not been called");
    return abs_global_partition(c->cfg.P, c->n_ranks, c->rank, first, count);
}

int abs_global_partition(uint64_t P, uint32_t n_ranks, uint32_t rank, uint64_t* first, uint64_t* count) {
    if (P == 0 || n_ranks == 0 || n_ranks > ABS_MAX_RANKS || rank >= n_ranks) return ABS_EINVAL;
    unsigned long long lo = 0, hi = 0;
    slice_vectors(round_up(P, kPadElems), n_ranks, rank, &lo, &hi);
    const uint64_t e_lo = std::min<uint64_t>(lo * 4, P), e_hi = std::min<uint64_t>(hi * 4, P);
    if (first) *first = e_lo;
    if (count) *count = e_hi - e_lo;
    return ABS_OK;
}

// CUDA IPC plumbing for abs_global_attach when the ranks are separate processes.
int abs_ipc_export(const void* dev_ptr, void* handle_out, uint64_t* offset_out) {
    if (!dev_ptr || !handle_out || !offset_out) return ABS_EINVAL;
    static_assert(sizeof(cudaIpcMemHandle_t) == ABS_IPC_HANDLE_BYTES, "handle size");
    typedef CUresult (*GetRange)(CUdeviceptr*, size_t*, CUdeviceptr);
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuMemGetAddressRange", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn) return ABS_ECUDA;
    CUdeviceptr base = 0;
    size_t size = 0;
    if (reinterpret_cast<GetRange>(fn)(&base, &size, reinterpret_cast<CUdeviceptr>(dev_ptr)) != CUDA_SUCCESS) return ABS_ECUDA;
    cudaIpcMemHandle_t h;
    if (cudaIpcGetMemHandle(&h, reinterpret_cast<void*>(base)) != cudaSuccess) { cudaGetLastError(); return ABS_ECUDA; }
    memcpy(handle_out, &h, sizeof h);
    *offset_out = reinterpret_cast<CUdeviceptr>(dev_ptr) - base;
    return ABS_OK;
}

int abs_ipc_open(const void* handle, uint64_t offset, void** dev_ptr_out) {
    if (!handle || !dev_ptr_out) return ABS_EINVAL;
    cudaIpcMemHandle_t h;
    memcpy(&h, handle, sizeof h);
    void* base = nullptr;
    if (cudaIpcOpenMemHandle(&base, h, cudaIpcMemLazyEnablePeerAccess) != cudaSuccess) { cudaGetLastError(); return ABS_ECUDA; }
    *dev_ptr_out = static_cast<char*>(base) + offset;
    return ABS_OK;
}

int abs_ipc_close(void* dev_ptr, uint64_t offset) {
    if (!dev_ptr) return ABS_EINVAL;
    if (cudaIpcCloseMemHandle(static_cast<char*>(dev_ptr) - offset) != cudaSuccess) { cudaGetLastError(); return ABS_ECUDA; }
    return ABS_OK;
}

int abs_params(abs_ctx* c, const float** x_dev_out) {
    if (!live(c)) return ABS_ESTATE;
    if (!x_dev_out) return invalid(c, "output pointer is NULL");
    *x_dev_out = c->x(c->pub);
    return ABS_OK;
}

int abs_params_host(abs_ctx* c, float* dst_host) {
    if (!live(c)) return ABS_ESTATE;
    if (!dst_host) return invalid(c, "destination pointer is NULL");
    CK(cudaMemcpyAsync(dst_host, c->x(c->pub), c->cfg.P * 4, cudaMemcpyDeviceToHost, c->s_acc));
    CK(cudaStreamSynchronize(c->s_acc));
    return ABS_OK;
}

int abs_momentum(abs_ctx* c, const float** v_dev_out) {
    if (!live(c)) return ABS_ESTATE;
    if (!v_dev_out) return invalid(c, "output pointer is NULL");
    *v_dev_out = c->v();
    return ABS_OK;
}

int abs_accumulator(abs_ctx* c, uint32_t set, uint32_t worker, const float** acc_dev_out) {
    if (!live(c)) return ABS_ESTATE;
    if (set > 1 || worker >= c->cfg.W || !acc_dev_out) return invalid(c, "bad set / worker / output pointer");
    if (int rc = contract_pending_sets(c)) return rc;
    if (int rc = join_workers(c)) return rc;
    *acc_dev_out = c->acc(set, worker);
    return ABS_OK;
}

int abs_counters(abs_ctx* c, int32_t* cnt_host, uint32_t* cur, uint64_t* t) {
    if (!live(c)) return ABS_ESTATE;
    if (cnt_host) memcpy(cnt_host, c->h_cnt.data(), c->h_cnt.size() * sizeof(int32_t));
    if (cur) *cur = c->cur;
    if (t) *t = c->t;
    return ABS_OK;
}

int abs_consumed(abs_ctx* c, uint64_t step, int32_t* b_host) {
    if (!live(c)) return ABS_ESTATE;
    if (!b_host) return invalid(c, "output pointer is NULL");
    if (step >= c->t || c->t - step >= (uint64_t)kLogDepth) return invalid(c, "step is not in the logged window");
    if (c->pipelined) CK(cudaStreamSynchronize(c->s_sync));
    CK(cudaStreamSynchronize(c->s_acc));
    CK(cudaMemcpy(b_host, c->log_row(step), c->cfg.W * sizeof(int32_t), cudaMemcpyDeviceToHost));
    return ABS_OK;
}

int abs_global_consumed(abs_ctx* c, uint64_t step, int32_t* b_host) {
    if (!live(c)) return ABS_ESTATE;
    if (c->n_ranks == 0) return invalid(c, "abs_global_attach has not been called");
    if (!b_host) return invalid(c, "output pointer is NULL");
    if (step >= c->t || c->t - step >= (uint64_t)kLogDepth) return invalid(c, "step is not in the logged window");
    CK(cudaStreamSynchronize(c->s_sync));
    CK(cudaStreamSynchronize(c->s_acc));
    CK(cudaMemcpy(b_host, c->log_row(step), (size_t)c->n_ranks * c->cfg.W * sizeof(int32_t), cudaMemcpyDeviceToHost));
    return ABS_OK;
}

int abs_grad_norm2(abs_ctx* c, uint64_t step, double* out) {
    if (!live(c)) return ABS_ESTATE;
    if (!c->grad_norm()) return invalid(c, "context was created without ABS_FLAG_GRAD_NORM");
    if (c->n_ranks != 0) return invalid(c, "not available in multi-GPU mode");
    if (!out) return invalid(c, "output pointer is NULL");
    if (step >= c->t || c->t - step >= (uint64_t)kLogDepth) return invalid(c, "step is not in the logged window");
    if (c->pipelined) CK(cudaStreamSynchronize(c->s_sync));
    CK(cudaStreamSynchronize(c->s_acc));
    CK(cudaMemcpy(out, c->norm_log(step), sizeof(double), cudaMemcpyDeviceToHost));
    return ABS_OK;
}

int abs_step1_finished(abs_ctx* c, int* done) {
    if (!live(c)) return ABS_ESTATE;
    if (!done) return invalid(c, "output pointer is NULL");
    *done = 1;
    if (c->pipelined && c->pending) {
        const cudaError_t e = cudaEventQuery(c->ev_sync_done);
        if (e == cudaErrorNotReady) *done = 0;
        else if (e != cudaSuccess) return cuda_fail(c, e, "cudaEventQuery");
    }
    return ABS_OK;
}

int abs_set_lr(abs_ctx* c, float lr) {
    if (!live(c)) return ABS_ESTATE;
    if (!std::isfinite(lr)) return invalid(c, "lr must be finite");
    c->lr_now = lr;
    return ABS_OK;
}

int abs_wait(abs_ctx* c) {
    if (!live(c)) return ABS_ESTATE;
    if (int rc = join_workers(c)) return rc;
    if (c->pipelined) {
        CK(cudaEventRecord(c->ev_aux, c->s_sync));
        CK(cudaStreamWaitEvent(c->s_acc, c->ev_aux, 0));
    }
    return ABS_OK;
}

int abs_check(abs_ctx* c) {
    if (!live(c)) return ABS_ESTATE;
    if (int rc = settle_all(c)) return rc;
    if (c->pipelined) CK(cudaStreamSynchronize(c->s_sync));
    for (int k = 0; k < c->n_wstreams; ++k) {
        CK(cudaStreamSynchronize(c->s_w[k]));
        CK(cudaStreamSynchronize(c->s_d[k]));
    }
    CK(cudaStreamSynchronize(c->s_acc));
    {
        int st = 0;
        CK(cudaMemcpy(&st, c->ticket() + 2, sizeof(int), cudaMemcpyDeviceToHost));
        if (st != 0) {
            CK(cudaMemset(c->ticket() + 2, 0, sizeof(int)));   // reported once; the context stays usable
            c->err = "a bounded device-side wait ran out (fused step, bulk-copy kernel)";
            return ABS_ETIMEOUT;
        }
    }
    if (c->mlp) {
        int bad = 0;
        for (int k = 0; k < kMlpSets; ++k) {
            int st = 0;
            CK(cudaMemcpy(&st, c->mlp_scratch[k].status, sizeof(int), cudaMemcpyDeviceToHost));
            bad |= st;
        }
        if (bad != 0) {
            c->err = "a bounded device-side wait ran out (MLP dW1 kernel)";
            return ABS_ETIMEOUT;
        }
    }
    return ABS_OK;
}

// ---- checkpoint / resume ----------------------------------------------------------------------------
namespace {
struct StateHeader {
    uint32_t magic, version;
    abs_config cfg;            // stream fields zeroed
    uint64_t payload_bytes;    // workspace prefix that holds x, v, accumulators, counters, logs
    uint64_t t;
    uint32_t cur, n_ranks, rank;
    int32_t pub, pending, pending_out;
    float lr_now, lr_prev_call, disp_scale, global_prev_lr;
    int32_t h_cnt[2 * kMaxW];
};
constexpr uint32_t kStateMagic = 0x53534241u;   // "ABSS"

size_t state_payload_bytes(const abs_ctx* c) { return c->L.off_gcnt + (size_t)(kMaxW + 64) * 4; }

bool same_config(const abs_config& a, const abs_config& b) {
    return a.P == b.P && a.W == b.W && a.grad_dtype == b.grad_dtype && a.flags == b.flags && a.mlp_in == b.mlp_in &&
           a.mlp_hidden == b.mlp_hidden && a.mlp_out == b.mlp_out && a.mlp_mb == b.mlp_mb && a.momentum == b.momentum &&
           a.weight_decay == b.weight_decay && a.lambda_dc == b.lambda_dc;
}

// Everything enqueued so far has finished (waiting micro-batch groups are started first).
int drain(abs_ctx* c) {
    if (int rc = contract_pending_sets(c)) return rc;
    if (int rc = settle_all(c)) return rc;
    if (c->pipelined) CK(cudaStreamSynchronize(c->s_sync));
    for (int k = 0; k < c->n_wstreams; ++k) {
        CK(cudaStreamSynchronize(c->s_w[k]));
        CK(cudaStreamSynchronize(c->s_d[k]));
    }
    if (c->s_copy) CK(cudaStreamSynchronize(c->s_copy));
    CK(cudaStreamSynchronize(c->s_acc));
    if (c->pipelined) CK(cudaStreamSynchronize(c->s_sync));
    for (int k = 0; k < c->n_wstreams; ++k) c->w_outstanding[k] = c->d_outstanding[k] = false;
    return ABS_OK;
}
}  // namespace

size_t abs_state_bytes(abs_ctx* c) {
    if (!live(c)) return 0;
    return sizeof(StateHeader) + state_payload_bytes(c);
}

int abs_state_export(abs_ctx* c, void* dst_host, size_t bytes) {
    if (!live(c)) return ABS_ESTATE;
    if (!dst_host) return invalid(c, "destination pointer is NULL");
    if (bytes < sizeof(StateHeader) + state_payload_bytes(c)) return invalid(c, "buffer smaller than abs_state_bytes()");
    if (c->global_phase != 0) return invalid(c, "between abs_global_begin and abs_global_end");
    if (int rc = drain(c)) return rc;
    StateHeader h{};
    h.magic = kStateMagic;
    h.version = 1;
    h.cfg = c->cfg;
    h.cfg.stream_acc = h.cfg.stream_sync = nullptr;
    h.cfg.lr = 0.f;   // the rate in effect is saved below
    h.payload_bytes = state_payload_bytes(c);
    h.t = c->t;
    h.cur = c->cur;
    h.n_ranks = c->n_ranks;
    h.rank = c->rank;
    h.pub = c->pub;
    h.pending = c->pending ? 1 : 0;
    h.pending_out = c->pending_out;
    h.lr_now = c->lr_now;
    h.lr_prev_call = c->lr_prev_call;
    h.disp_scale = c->disp_scale;
    h.global_prev_lr = c->global_prev_lr;
    for (size_t k = 0; k < c->h_cnt.size(); ++k) h.h_cnt[k] = c->h_cnt[k];
    memcpy(dst_host, &h, sizeof h);
    CK(cudaMemcpy(static_cast<char*>(dst_host) + sizeof h, c->ws, h.payload_bytes, cudaMemcpyDeviceToHost));
    return ABS_OK;
}

int abs_state_import(abs_ctx* c, const void* src_host, size_t bytes) {
    if (!live(c)) return ABS_ESTATE;
    if (!src_host) return invalid(c, "source pointer is NULL");
    if (bytes < sizeof(StateHeader)) return invalid(c, "buffer smaller than a state header");
    StateHeader h;
    memcpy(&h, src_host, sizeof h);
    if (h.magic != kStateMagic || h.version != 1) return invalid(c, "not a state written by abs_state_export");
    if (!same_config(h.cfg, c->cfg)) return invalid(c, "the state was exported from a context with another configuration");
    if (h.payload_bytes != state_payload_bytes(c) || bytes < sizeof h + h.payload_bytes) return invalid(c, "state is truncated");
    if (h.n_ranks != c->n_ranks || h.rank != c->rank) return invalid(c, "the state belongs to another rank layout (abs_global_attach first)");
    if (c->global_phase != 0) return invalid(c, "between abs_global_begin and abs_global_end");
    if (h.cur > 1 || h.pub < 0 || h.pub > 1 || h.pending_out < 0 || h.pending_out > 1) return invalid(c, "state header is corrupt");
    if (int rc = drain(c)) return rc;
    CK(cudaMemcpy(c->ws, static_cast<const char*>(src_host) + sizeof h, h.payload_bytes, cudaMemcpyHostToDevice));
    c->t = h.t;
    c->cur = h.cur;
    c->pub = h.pub;
    c->pending = h.pending != 0;
    c->pending_out = h.pending_out;
    c->lr_now = h.lr_now;
    c->lr_prev_call = h.lr_prev_call;
    c->disp_scale = h.disp_scale;
    c->global_prev_lr = h.global_prev_lr;
    for (size_t k = 0; k < c->h_cnt.size(); ++k) c->h_cnt[k] = h.h_cnt[k];
    for (uint32_t set = 0; set < 2; ++set) {   // a row that has received gradients may hold some in its W1 slice
        c->pool_n[set] = 0;
        c->fused_pending[set] = false;
        for (uint32_t i = 0; i < c->cfg.W; ++i) c->w1_touched[set][i] = c->h_cnt[(size_t)set * c->cfg.W + i] > 0;
    }
    if (c->mlp) {   // the bf16 copies are a function of the parameters: rebuild them
        CK(launch_cast_bf16(c->x(0), c->shadow(0), c->L.P_pad, c->num_sms, c->s_acc));
        c->launches += 1;
        if (c->pipelined) {
            CK(launch_cast_bf16(c->x(1), c->shadow(1), c->L.P_pad, c->num_sms, c->s_acc));
            c->launches += 1;
        }
        CK(cudaStreamSynchronize(c->s_acc));
    }
    if (c->pipelined) CK(cudaEventRecord(c->ev_sync_done, c->s_sync));   // what "pending" waits for has happened
    return ABS_OK;
}

int abs_selftest_timeout(abs_ctx* c) {
    if (!live(c)) return ABS_ESTATE;
    CK(launch_bounded_wait_selftest(reinterpret_cast<int*>(c->ticket() + 2), c->s_acc));
    c->launches += 1;
    return ABS_OK;
}

int abs_set_launch(abs_ctx* c, int kernel_class, int ctas_per_sm) {
    if (!live(c)) return ABS_ESTATE;
    if (kernel_class < 0 || kernel_class >= ABS_K_COUNT || ctas_per_sm < (kernel_class == ABS_K_SYNC ? -2 : -1) ||
        ctas_per_sm > (kernel_class == ABS_K_MLP_DW1 ? 255 : 64))
        return invalid(c, "bad kernel class or CTA count");
    if (kernel_class == ABS_K_MLP_DW1 && ctas_per_sm > 0 && (ctas_per_sm & ~(4 | 8 | 32 | 128)))
        return invalid(c, "unknown bits in the ABS_K_MLP_DW1 mask");
    if (kernel_class == ABS_K_CHAIN && (ctas_per_sm < 0 || ctas_per_sm > 1)) return invalid(c, "ABS_K_CHAIN takes 0 or 1");
    if (kernel_class == ABS_K_MLP_FWD && (ctas_per_sm < 0 || ctas_per_sm > 1)) return invalid(c, "ABS_K_MLP_FWD takes 0 or 1");
    if (kernel_class == ABS_K_MLP_BWD && (ctas_per_sm < 0 || ctas_per_sm > 2)) return invalid(c, "ABS_K_MLP_BWD takes 0, 1 or 2");
    if (int rc = settle_all(c)) return rc;
    c->ctas_per_sm[kernel_class] = ctas_per_sm;
    return ABS_OK;
}

int abs_profile(abs_ctx* c, int enable) {
    if (!live(c)) return ABS_ESTATE;
    int rc = collect_timings(c);
    if (rc != ABS_OK) return rc;
    if (enable) {
        for (int k = 0; k < ABS_K_COUNT; ++k) { c->stat_n[k] = 0; c->stat_ms[k] = 0.0; }
        c->spans.clear();
    }
    c->profiling = enable != 0;
    c->timeline_on = enable == 2;
    if (c->timeline_on) {
        if (!c->ev_origin) CK(cudaEventCreate(&c->ev_origin));
        CK(cudaEventRecord(c->ev_origin, c->s_acc));
    }
    return ABS_OK;
}

int abs_profile_timeline(abs_ctx* c, abs_span* out, size_t capacity, size_t* n) {
    if (!live(c)) return ABS_ESTATE;
    if (!n) return invalid(c, "output pointer is NULL");
    int rc = collect_timings(c);
    if (rc != ABS_OK) return rc;
    *n = c->spans.size();
    if (out) {
        const size_t m = std::min(capacity, c->spans.size());
        for (size_t k = 0; k < m; ++k) out[k] = c->spans[k];
    }
    return ABS_OK;
}

int abs_kernel_stats(abs_ctx* c, int kernel_class, uint64_t* launches, double* total_ms) {
    if (!live(c)) return ABS_ESTATE;
    if (kernel_class < 0 || kernel_class >= ABS_K_COUNT) return invalid(c, "bad kernel class");
    int rc = collect_timings(c);
    if (rc != ABS_OK) return rc;
    if (launches) *launches = c->stat_n[kernel_class];
    if (total_ms) *total_ms = c->stat_ms[kernel_class];
    return ABS_OK;
}

uint64_t abs_launch_count(abs_ctx* c) { return live(c) ? c->launches : 0; }

const char* abs_last_error(abs_ctx* c) {
    if (!c) return g_init_error.c_str();
    if (!live(c)) return "context is not alive";
    return c->err.c_str();
}

int abs_destroy(abs_ctx* c) {
    if (!live(c)) return ABS_ESTATE;
    {
        std::lock_guard<std::mutex> g(g_live_mu);
        g_live.erase(c);
    }
    cudaStreamSynchronize(c->s_acc);
    if (c->pipelined) cudaStreamSynchronize(c->s_sync);
    if (c->s_copy) { cudaStreamSynchronize(c->s_copy); cudaStreamDestroy(c->s_copy); }
    for (int k = 0; k < c->n_wstreams; ++k)
        if (c->s_w[k]) { cudaStreamSynchronize(c->s_w[k]); cudaStreamDestroy(c->s_w[k]); }
    for (int k = 0; k < c->n_wstreams; ++k)
        if (c->s_d[k]) { cudaStreamSynchronize(c->s_d[k]); cudaStreamDestroy(c->s_d[k]); }
    for (cudaEvent_t e : c->ev_front) if (e) cudaEventDestroy(e);
    for (cudaEvent_t e : c->ev_d_done) if (e) cudaEventDestroy(e);
    for (cudaEvent_t e : c->ev_set_done) if (e) cudaEventDestroy(e);
    for (cudaEvent_t e : c->ev_w_done) if (e) cudaEventDestroy(e);
    if (c->ev_fork) cudaEventDestroy(c->ev_fork);
    if (c->ev_origin) cudaEventDestroy(c->ev_origin);
    for (auto& tl : c->timed) { cudaEventDestroy(tl.start); cudaEventDestroy(tl.stop); }
    for (auto e : c->ev_pool) cudaEventDestroy(e);
    for (cudaEvent_t e : {c->ev_acc_done, c->ev_sync_done, c->ev_aux, c->ev_stage_free[0], c->ev_stage_free[1],
                          c->ev_stage_full[0], c->ev_stage_full[1]})
        if (e) cudaEventDestroy(e);
    c->magic = 0;
    delete c;
    return ABS_OK;
}

}  // extern "C"

namespace {
// Called by the MLP launcher around each of its kernels: n = -1 - part before, n = launches made after.
void mlp_mark(void* user, int kernel_class, int n, cudaStream_t stream) {
    abs_ctx* c = static_cast<abs_ctx*>(user);
    if (n > 0) c->launches += (uint64_t)n;
    if (!c->profiling) return;
    if (n < 0) {
        cudaEvent_t start = take_event(c), stop = take_event(c);
        if (!start || !stop) return;
        cudaEventRecord(start, stream);
        c->timed.push_back({kernel_class, start, stop, stream, -1 - n});
    } else if (!c->timed.empty() && c->timed.back().kernel_class == kernel_class) {
        cudaEventRecord(c->timed.back().stop, stream);
    }
}
}  // namespace
