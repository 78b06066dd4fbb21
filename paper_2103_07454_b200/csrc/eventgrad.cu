// Host side of the C ABI declared in include/eventgrad.h: context, layout, tile tables,
// stream-ordered launches.  No decision of the step is taken on the host.
#include "../../include/eventgrad.h"

#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "eg_common.cuh"
#include "eg_fused.cuh"
#include "eg_fused_hops.cuh"
#include "eg_fused_pipe.cuh"
#include "eg_norm.cuh"
#include "eg_quant.cuh"
#include "eg_step_small.cuh"
#include "eg_topk.cuh"

using namespace eg;

namespace {

constexpr int kFusedVpt = EG_FUSED_VPT;               // float4 columns per thread
constexpr int kFusedTile = kThreads * 4 * kFusedVpt;  // elements per CTA of the fused kernel
using PipeLayout = PipeSmem<kPipeTile, kPipeStages>;
constexpr int kMomStages = 4;                         // four tiles per stage: same footprint as 5 x 3
using MomLayout = PipeSmem<kPipeTile, kMomStages, 4, false>;
static_assert(kFusedTile == kPipeTile, "both fused kernels share one tile table");
constexpr uint64_t kStateMagic = 0x4547535441544534ull;  // "EGSTATE4"

struct HostTiles {
    std::vector<int> tensor, length, seg_begin;
    std::vector<long long> offset;
};

struct DeviceTiles {
    int *tensor = nullptr, *length = nullptr, *seg_begin = nullptr;
    long long* offset = nullptr;
    int n_tiles = 0;
    TileTable view(unsigned int* err) const { return TileTable{tensor, offset, length, seg_begin, n_tiles, err}; }
};

}  // namespace

struct eg_ctx {
    int device = 0;
    int P = 0, T = 0, H = 1;
    eg_threshold_params thr{};
    eg_topk_params topk{};
    std::vector<int64_t> numel, offset, kcount, out_off;
    int64_t stride = 0, n_total = 0, out_stride = 0;
    int degree = 0;
    int hops = 1;
    DeviceTiles tiles_norm, tiles_fused;
    // device state
    float* xhat = nullptr;
    double *partials_norm = nullptr, *partials_fused = nullptr;
    SegState st{};
    Counters* ctr = nullptr;
    long long* step_k = nullptr;
    unsigned int* err = nullptr;
    long long *d_numel = nullptr, *d_kcount = nullptr, *d_out_off = nullptr;
    int* outbox_count = nullptr;
    TopkState tk{};
    double* cons_partials = nullptr;
    // host staging for eg_step_host
    float *stage_x = nullptr, *stage_g = nullptr;
    // bookkeeping
    std::vector<void*> allocs;
    bool carry = false, carried_valid = false;
    const float* carried_params = nullptr;
    cudaStream_t last_stream = nullptr;
    int last_cuda_error = 0;
    int last_launches = 0;
    size_t fused_smem = 0;
    int fused_kind = EG_FUSED_AUTO;
    // single-launch iteration for small problems (k_step_small)
    bool small_eligible = false;
    double* partials_small = nullptr;   // second buffer of carried partials
    int *small_arrived = nullptr, *small_done = nullptr;
    int2 *small_range_fused = nullptr, *small_range_norm = nullptr;   // per fused tile: its tensor's tiles
    int topk_coop_grid = 0;   // CTAs of the one-launch Top-K kernel; 0: use the ten single-phase launches
    int variant = 0;
    double cap_alpha = 0.0, cap_beta = 1.0;   // bound alpha*beta^k on the squared threshold
    double* cap_g = nullptr;                  // [2] device: g(k) at [k & 1], advanced by the kernels
    int sms = 148;                            // multiprocessors of the context's device
    int topk_grid = 0, topk_seg_grid = 0;     // CTAs of the Top-K tile / segment phases
    bool last_capturing = false;              // the most recent step was recorded into a graph
    // sub-range of the step that eg_step_masked launches (eg_step_host pipelines groups of
    // tensors); the default is everything
    std::vector<int> seg_begin_norm, seg_begin_fused;   // host copies, [T+1]
    int range_t0 = 0, range_tn = 0;                      // tn == 0: all tensors
    bool range_last = true;                              // the launch that ends the iteration
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    std::vector<cudaEvent_t> group_events;
    // intermittent delivery (two copies: sent = xhat, received = mailbox)
    bool async = false;
    float* mailbox = nullptr;
    uint8_t *pending = nullptr, *recv_valid = nullptr, *arrive = nullptr;
    unsigned long long* arrivals = nullptr;
    bool stepped = false;   // a step has run since creation / reset / import
    // heavy-ball momentum: velocity of every replica, laid out like the parameters
    bool momentum = false;
    double mu = 0.0;
    float* vel = nullptr;
    // optional per-kernel timing (events on the launching stream)
    bool timing = false;
    bool nvtx = false;      // EG_NVTX in the environment at eg_create: named ranges around the kernel groups
    int fused_waves = 1;    // EG_FUSED_WAVES in the environment at eg_create: CTAs of a walking pipelined kernel per resident slot
    int* ticket = nullptr;       // device: tile counter of the walking fused kernel
    // quantised messages (eg_set_quantisation)
    int quant_bits = 0;                  // 0: messages in full precision
    float* quant_tile_max = nullptr;     // [P][norm tiles]
    int* quant_exp = nullptr;            // [P*T] scale exponent of the last quantised message
    int fused_walk_max_p = 24;   // EG_FUSED_WALK_MAX_P: rings of up to this many replicas use the walking form
    bool topk_pdl = true;   // EG_TOPK_PDL=0 in the environment at eg_create: no dependent launches inside the Top-K sequence
    bool no_pdl = false;    // EG_NO_PDL in the environment at eg_create: every kernel starts after its predecessor has ended
    std::vector<cudaEvent_t> ev_pool;      // pairs
    std::vector<int> ev_kind;              // kernel group of every recorded pair
    size_t ev_used = 0;
};

namespace {

#define EG_CUDA(ctx, call)                                   \
    do {                                                     \
        cudaError_t e_ = (call);                             \
        if (e_ != cudaSuccess) {                             \
            (ctx)->last_cuda_error = (int)e_;                \
            return e_ == cudaErrorMemoryAllocation ? EG_ERR_OOM : EG_ERR_CUDA; \
        }                                                    \
    } while (0)

// Test hook (eg_debug_fail_allocation): the n-th device allocation from now on reports
// cudaErrorMemoryAllocation without calling the runtime; 0: off.
int g_fail_alloc_in = 0;

template <typename Tp>
eg_status dev_alloc(eg_ctx* c, Tp** out, size_t count, bool zero = true) {
    void* p = nullptr;
    const size_t bytes = (count ? count : 1) * sizeof(Tp);
    if (g_fail_alloc_in > 0 && --g_fail_alloc_in == 0) {
        c->last_cuda_error = (int)cudaErrorMemoryAllocation;
        return EG_ERR_OOM;
    }
    EG_CUDA(c, cudaMalloc(&p, bytes));
    c->allocs.push_back(p);
    if (zero) EG_CUDA(c, cudaMemset(p, 0, bytes));
    *out = static_cast<Tp*>(p);
    return EG_OK;
}

template <typename Tp>
eg_status upload(eg_ctx* c, Tp** out, const std::vector<Tp>& v) {
    eg_status s = dev_alloc(c, out, v.size(), false);
    if (s != EG_OK) return s;
    if (!v.empty()) EG_CUDA(c, cudaMemcpy(*out, v.data(), v.size() * sizeof(Tp), cudaMemcpyHostToDevice));
    return EG_OK;
}

HostTiles build_tiles(const std::vector<int64_t>& numel, const std::vector<int64_t>& offset, int tile) {
    HostTiles h;
    for (size_t t = 0; t < numel.size(); ++t) {
        h.seg_begin.push_back((int)h.tensor.size());
        for (int64_t b = 0; b < numel[t]; b += tile) {
            h.tensor.push_back((int)t);
            h.offset.push_back((long long)(offset[t] + b));
            h.length.push_back((int)std::min<int64_t>(tile, numel[t] - b));
        }
    }
    h.seg_begin.push_back((int)h.tensor.size());
    return h;
}

eg_status upload_tiles(eg_ctx* c, const HostTiles& h, DeviceTiles* d) {
    eg_status s;
    if ((s = upload(c, &d->tensor, h.tensor)) != EG_OK) return s;
    if ((s = upload(c, &d->length, h.length)) != EG_OK) return s;
    if ((s = upload(c, &d->seg_begin, h.seg_begin)) != EG_OK) return s;
    if ((s = upload(c, &d->offset, h.offset)) != EG_OK) return s;
    d->n_tiles = (int)h.tensor.size();
    return EG_OK;
}

int64_t topk_entries(int64_t n, uint32_t num, uint32_t den) {
    const unsigned long long prod = (unsigned long long)n * num;
    unsigned long long q = (prod + den - 1ull) / den;
    if (q < 1) q = 1;
    if (q > (unsigned long long)n) q = (unsigned long long)n;
    return (int64_t)q;
}

// The instantiation of the single-launch kernel for P replicas (nullptr: none).
const void* small_kernel(int P) {
    if (P <= 4) return (const void*)k_step_small<4>;
    if (P <= 8) return (const void*)k_step_small<8>;
    if (P <= kSmallMaxP) return (const void*)k_step_small<16>;
    return nullptr;
}

eg_status init_state(eg_ctx* c) {
    const size_t S = (size_t)c->P * c->T;
    std::vector<double> delta(S, c->thr.mode == EG_THRESH_FIXED ? c->thr.delta_fixed : c->thr.delta_init);
    EG_CUDA(c, cudaMemcpy(c->st.delta, delta.data(), S * sizeof(double), cudaMemcpyHostToDevice));
    EG_CUDA(c, cudaMemcpy(c->st.thr_used, delta.data(), S * sizeof(double), cudaMemcpyHostToDevice));
    EG_CUDA(c, cudaMemset(c->st.khat, 0, S * sizeof(long long)));
    EG_CUDA(c, cudaMemset(c->st.hist, 0, S * c->H * sizeof(double)));
    EG_CUDA(c, cudaMemset(c->st.hist_len, 0, S * sizeof(int)));
    EG_CUDA(c, cudaMemset(c->st.valid, 0, S));
    EG_CUDA(c, cudaMemset(c->st.flag, 0, S));
    EG_CUDA(c, cudaMemset(c->st.snap, 0, S));
    EG_CUDA(c, cudaMemset(c->st.sparse, 0, S));
    if (c->st.quant) {
        EG_CUDA(c, cudaMemset(c->st.quant, 0, S));
        EG_CUDA(c, cudaMemset(c->quant_exp, 0, S * sizeof(int)));
    }
    EG_CUDA(c, cudaMemset(c->st.norm, 0, S * sizeof(double)));
    EG_CUDA(c, cudaMemset(c->st.events, 0, S * sizeof(unsigned long long)));
    EG_CUDA(c, cudaMemset(c->st.sent_norm, 0, S * sizeof(double)));
    EG_CUDA(c, cudaMemset(c->ctr, 0, sizeof(Counters)));
    EG_CUDA(c, cudaMemset(c->step_k, 0, sizeof(long long)));
    EG_CUDA(c, cudaMemset(c->err, 0, sizeof(unsigned int)));
    EG_CUDA(c, cudaMemset(c->outbox_count, 0, S * sizeof(int)));
    if (c->st.sparse_steps) EG_CUDA(c, cudaMemset(c->st.sparse_steps, 0, 2 * sizeof(unsigned int)));
    EG_CUDA(c, cudaMemset(c->xhat, 0, (size_t)c->P * c->stride * sizeof(float)));
    if (c->topk.enabled) {
        EG_CUDA(c, cudaMemset(c->tk.hist, 0, S * kMaxBins * sizeof(unsigned int)));
        EG_CUDA(c, cudaMemset(c->tk.prefix, 0, S * sizeof(unsigned int)));
        EG_CUDA(c, cudaMemset(c->tk.remaining, 0, S * sizeof(unsigned int)));
        EG_CUDA(c, cudaMemset(c->tk.offcnt, 0, S * kOffBins * sizeof(unsigned int)));
        EG_CUDA(c, cudaMemset(c->tk.offsel, 0, S));
        EG_CUDA(c, cudaMemset(c->tk.redo, 0, S));
        EG_CUDA(c, cudaMemset(c->tk.redo_count, 0, sizeof(unsigned int)));
        EG_CUDA(c, cudaMemset(c->tk.redo_total, 0, sizeof(unsigned long long)));
        for (int l = 0; l < 2; ++l) EG_CUDA(c, cudaMemset(c->tk.list[l].plan, 0, sizeof(TopkPlan)));
    }
    if (c->async) {
        EG_CUDA(c, cudaMemset(c->mailbox, 0, (size_t)c->P * c->stride * sizeof(float)));
        EG_CUDA(c, cudaMemset(c->pending, 0, S));
        EG_CUDA(c, cudaMemset(c->recv_valid, 0, S));
        EG_CUDA(c, cudaMemset(c->arrive, 0, S));
        EG_CUDA(c, cudaMemset(c->arrivals, 0, sizeof(unsigned long long)));
    }
    if (c->small_arrived) {
        EG_CUDA(c, cudaMemset(c->small_arrived, 0, (size_t)c->T * sizeof(int)));
        EG_CUDA(c, cudaMemset(c->small_done, 0, sizeof(int)));
    }
    if (c->vel) EG_CUDA(c, cudaMemset(c->vel, 0, (size_t)c->P * c->stride * sizeof(float)));
    {
        const double g0[2] = {c->cap_alpha, c->cap_alpha};   // iteration 0 reads slot 0
        EG_CUDA(c, cudaMemcpy(c->cap_g, g0, sizeof(g0), cudaMemcpyHostToDevice));
    }
    c->carried_valid = false;
    c->stepped = false;
    return EG_OK;
}

// g(k) = alpha * beta^k as the kernels carry it: k multiplications, one rounding each.
double cap_term(double alpha, double beta, long long k) {
    double g = alpha;
    for (long long q = 0; q < k; ++q) g = g * beta;
    return g;
}

// Puts the term of iteration k where that iteration will read it.
eg_status upload_cap(eg_ctx* c, long long k) {
    const double g = cap_term(c->cap_alpha, c->cap_beta, k);
    EG_CUDA(c, cudaMemcpy(c->cap_g + (k & 1), &g, sizeof(g), cudaMemcpyHostToDevice));
    return EG_OK;
}

eg_status sync_and_check(eg_ctx* c) {
    EG_CUDA(c, cudaStreamSynchronize(c->last_stream));
    unsigned int e = 0;
    EG_CUDA(c, cudaMemcpy(&e, c->err, sizeof(e), cudaMemcpyDeviceToHost));
    return eg_status_of_error_word(e);
}

constexpr size_t kMaxTimedPairs = 1 << 15;

// Launch with the programmatic-serialization attribute: the kernel may begin while its
// predecessor in the stream finishes; it calls pdl_wait() before it depends on that kernel.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(bool overlap, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                       cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;   // per-kernel timing wants every kernel's duration to be its own
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Brackets one kernel group with a pair of events when timing is on.
struct TimedSection {
    eg_ctx* c;
    cudaStream_t stream;
    bool on, range;
    TimedSection(eg_ctx* ctx, cudaStream_t s, int kind) : c(ctx), stream(s), on(false), range(ctx->nvtx) {
        static const char* const kNames[EG_KERNEL_GROUPS] = {"eventgrad:norm", "eventgrad:decide",
                                                             "eventgrad:topk", "eventgrad:fused"};
        if (range) nvtxRangePushA(kNames[kind]);      // host-side range around the launches of the group
        if (!c->timing || c->ev_used >= kMaxTimedPairs) return;
        if (c->ev_pool.size() < 2 * (c->ev_used + 1)) {
            cudaEvent_t a, b;
            if (cudaEventCreate(&a) != cudaSuccess) return;
            if (cudaEventCreate(&b) != cudaSuccess) { cudaEventDestroy(a); return; }
            c->ev_pool.push_back(a);
            c->ev_pool.push_back(b);
        }
        if (c->ev_kind.size() <= c->ev_used) c->ev_kind.push_back(kind);
        c->ev_kind[c->ev_used] = kind;
        on = cudaEventRecord(c->ev_pool[2 * c->ev_used], stream) == cudaSuccess;
    }
    ~TimedSection() {
        if (on) {
            cudaEventRecord(c->ev_pool[2 * c->ev_used + 1], stream);
            ++c->ev_used;
        }
        if (range) nvtxRangePop();
    }
};

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

}  // namespace

// The staged general-neighbourhood kernel: prefetch distance chosen so that two CTAs fit an SM.
constexpr int kMaxStagedHops = 4;
template <int M> struct StagedDepth;
template <> struct StagedDepth<2> { static constexpr int D = 4; };
template <> struct StagedDepth<3> { static constexpr int D = 3; };
template <> struct StagedDepth<4> { static constexpr int D = 2; };

template <int M>
static cudaError_t raise_hops_staged(int P) {
    constexpr int D = StagedDepth<M>::D;
    cudaError_t e = cudaFuncSetAttribute(k_fused_hops_staged<true, M, D>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)HopsStaged<M, D>::bytes(P, true));
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(k_fused_hops_staged<false, M, D>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)HopsStaged<M, D>::bytes(P, false));
    return e;
}

template <int M>
static void launch_hops_staged_m(eg_ctx* c, bool carry, int grid, cudaStream_t stream, float* params,
                                 const float* grads, const uint8_t* valid, const TileTable& tf, float lr,
                                 double* partials, long long* step_k) {
    constexpr int D = StagedDepth<M>::D;
    const size_t smem = HopsStaged<M, D>::bytes(c->P, carry);
    if (carry)
        k_fused_hops_staged<true, M, D><<<grid, kThreads, smem, stream>>>(
            params, grads, c->xhat, c->st.snap, valid, tf, c->P, c->T, c->stride, lr, partials, step_k,
            c->variant);
    else
        k_fused_hops_staged<false, M, D><<<grid, kThreads, smem, stream>>>(
            params, grads, c->xhat, c->st.snap, valid, tf, c->P, c->T, c->stride, lr, partials, step_k,
            c->variant, c->async ? c->mailbox : nullptr, c->async ? c->arrive : nullptr);
}

static void launch_hops_staged(eg_ctx* c, bool carry, int grid, cudaStream_t stream, float* params,
                               const float* grads, const uint8_t* valid, const TileTable& tf, float lr,
                               double* partials, long long* step_k) {
    switch (c->hops) {
        case 2: launch_hops_staged_m<2>(c, carry, grid, stream, params, grads, valid, tf, lr, partials, step_k); break;
        case 3: launch_hops_staged_m<3>(c, carry, grid, stream, params, grads, valid, tf, lr, partials, step_k); break;
        default: launch_hops_staged_m<4>(c, carry, grid, stream, params, grads, valid, tf, lr, partials, step_k); break;
    }
}

extern "C" {

void eg_debug_fail_allocation(int nth) { g_fail_alloc_in = nth > 0 ? nth : 0; }

const char* eg_strerror(eg_status s) {
    switch (s) {
        case EG_OK: return "ok";
        case EG_ERR_INVALID: return "invalid argument";
        case EG_ERR_OOM: return "out of memory";
        case EG_ERR_CUDA: return "CUDA runtime error";
        case EG_ERR_STATE: return "call not allowed in this state";
        case EG_ERR_TIMEOUT: return "timeout";
        case EG_ERR_INTERNAL: return "device-side consistency check failed";
    }
    return "unknown status";
}

eg_status eg_status_of_error_word(unsigned int word) {
    if (word & kErrWaitTimeout) return EG_ERR_TIMEOUT;   // a bounded device-side wait gave up
    return word ? EG_ERR_INTERNAL : EG_OK;               // kErrBounds, kErrTopkSlot
}

int eg_debug_build(void) {
#ifdef EG_DEBUG
    return 1;
#else
    return 0;
#endif
}

int eg_last_cuda_error(const eg_ctx* ctx) { return ctx ? ctx->last_cuda_error : 0; }
int eg_last_launch_count(const eg_ctx* ctx) { return ctx ? ctx->last_launches : 0; }

void eg_destroy(eg_ctx* c) {
    if (!c) return;
    {
        DeviceGuard guard(c->device);
        cudaDeviceSynchronize();
        for (void* p : c->allocs) cudaFree(p);
        for (cudaEvent_t e : c->ev_pool) cudaEventDestroy(e);
        for (cudaEvent_t e : c->group_events) cudaEventDestroy(e);
        if (c->copy_in) cudaStreamDestroy(c->copy_in);
        if (c->copy_out) cudaStreamDestroy(c->copy_out);
    }
    delete c;
}

eg_status eg_create(eg_ctx** out, int topology, int P, const int64_t* layer_numel, int T,
                    const eg_threshold_params* thr, const eg_topk_params* topk) {
    if (!out) return EG_ERR_INVALID;
    *out = nullptr;
    if (topology < EG_TOPO_RING || topology >= kMaxHops || P < 1 || P > kMaxReplicas || T < 1 ||
        !layer_numel || !thr)
        return EG_ERR_INVALID;
    if (thr->mode != EG_THRESH_ADAPTIVE && thr->mode != EG_THRESH_FIXED) return EG_ERR_INVALID;
    if (thr->history_len < 1 || thr->history_len > kMaxHistory) return EG_ERR_INVALID;
    if (std::isnan(thr->horizon) || std::isnan(thr->delta_init) || std::isnan(thr->delta_fixed))
        return EG_ERR_INVALID;
    if (topk && topk->enabled && (topk->k_num == 0 || topk->k_den == 0)) return EG_ERR_INVALID;
    for (int t = 0; t < T; ++t)
        if (layer_numel[t] < 1 || layer_numel[t] > 0x7fffffffll) return EG_ERR_INVALID;

    eg_ctx* c = new (std::nothrow) eg_ctx();
    if (!c) return EG_ERR_OOM;
    eg_status s = EG_OK;
    auto fail = [&](eg_status code) { eg_destroy(c); return code; };
    if (cudaGetDevice(&c->device) != cudaSuccess) return fail(EG_ERR_CUDA);
    { const char* e = getenv("EG_NVTX"); c->nvtx = e && *e && *e != '0'; }
    { const char* e = getenv("EG_NO_PDL"); c->no_pdl = e && *e && *e != '0'; }
    { const char* e = getenv("EG_TOPK_PDL"); c->topk_pdl = !(e && *e == '0'); }
    { const char* e = getenv("EG_FUSED_WAVES"); if (e && atoi(e) > 0) c->fused_waves = atoi(e); }
    { const char* e = getenv("EG_FUSED_WALK_MAX_P"); if (e && *e) c->fused_walk_max_p = atoi(e); }
    c->P = P; c->T = T; c->H = thr->history_len; c->thr = *thr;
    if (topk) c->topk = *topk;
    if (cudaDeviceGetAttribute(&c->sms, cudaDevAttrMultiProcessorCount, c->device) != cudaSuccess || c->sms < 1)
        return fail(EG_ERR_CUDA);
    c->topk_grid = c->sms * kTopkCtasPerSm;       // the tile phases loop over the work list
    c->topk_seg_grid = c->sms * kTopkSegCtasPerSm;
    c->hops = topology + 1;                       // EG_TOPO_RING_HOPS(m) == m - 1
    c->degree = std::min(2 * c->hops, P - 1);     // distinct neighbours of every replica
    // layout: every tensor starts on a 128-byte boundary
    int64_t off = 0, koff = 0;
    for (int t = 0; t < T; ++t) {
        c->numel.push_back(layer_numel[t]);
        c->offset.push_back(off);
        off += (layer_numel[t] + 31) / 32 * 32;
        c->n_total += layer_numel[t];
        const int64_t kt = c->topk.enabled ? topk_entries(layer_numel[t], c->topk.k_num, c->topk.k_den) : 0;
        c->kcount.push_back(kt);
        c->out_off.push_back(koff);
        koff += kt;
    }
    c->stride = off;
    c->out_stride = koff;

    const size_t S = (size_t)P * T;
    {
        const HostTiles hn = build_tiles(c->numel, c->offset, kNormTile);
        const HostTiles hf = build_tiles(c->numel, c->offset, kFusedTile);
        c->seg_begin_norm = hn.seg_begin;
        c->seg_begin_fused = hf.seg_begin;
        if ((s = upload_tiles(c, hn, &c->tiles_norm)) != EG_OK) return fail(s);
        if ((s = upload_tiles(c, hf, &c->tiles_fused)) != EG_OK) return fail(s);
    }
    std::vector<long long> numel_ll(c->numel.begin(), c->numel.end());
    std::vector<long long> kcount_ll(c->kcount.begin(), c->kcount.end());
    std::vector<long long> out_off_ll(c->out_off.begin(), c->out_off.end());
    if ((s = upload(c, &c->d_numel, numel_ll)) != EG_OK) return fail(s);
    if ((s = upload(c, &c->d_kcount, kcount_ll)) != EG_OK) return fail(s);
    if ((s = upload(c, &c->d_out_off, out_off_ll)) != EG_OK) return fail(s);
#define EG_ALLOC(ptr, count)                                              \
    if ((s = dev_alloc(c, &(ptr), (size_t)(count))) != EG_OK) return fail(s)
    EG_ALLOC(c->xhat, (size_t)P * c->stride);
    EG_ALLOC(c->partials_norm, (size_t)P * c->tiles_norm.n_tiles);
    EG_ALLOC(c->partials_fused, (size_t)P * c->tiles_fused.n_tiles);
    EG_ALLOC(c->st.delta, S); EG_ALLOC(c->st.khat, S); EG_ALLOC(c->st.hist, S * c->H);
    EG_ALLOC(c->st.hist_len, S); EG_ALLOC(c->st.valid, S); EG_ALLOC(c->st.flag, S);
    EG_ALLOC(c->st.snap, S); EG_ALLOC(c->st.sparse, S); EG_ALLOC(c->st.norm, S);
    EG_ALLOC(c->st.thr_used, S); EG_ALLOC(c->st.events, S); EG_ALLOC(c->st.sent_norm, S);
    EG_ALLOC(c->ctr, 1); EG_ALLOC(c->step_k, 1); EG_ALLOC(c->err, 2); EG_ALLOC(c->cap_g, 2); EG_ALLOC(c->ticket, 1);
    EG_ALLOC(c->outbox_count, S);
    if (c->topk.enabled) EG_ALLOC(c->st.sparse_steps, 2);
    EG_ALLOC(c->cons_partials, (size_t)c->tiles_fused.n_tiles + 1);
    if (c->topk.enabled) {
        EG_ALLOC(c->tk.hist, S * kMaxBins);
        EG_ALLOC(c->tk.prefix, S); EG_ALLOC(c->tk.remaining, S);
        EG_ALLOC(c->tk.tile_count, (size_t)P * c->tiles_norm.n_tiles);
        EG_ALLOC(c->tk.tile_cand, (size_t)P * c->tiles_norm.n_tiles * kSubSlices);
        EG_ALLOC(c->tk.tile_sub, (size_t)P * c->tiles_norm.n_tiles * kSubSlices);
        EG_ALLOC(c->tk.ent, (size_t)P * c->stride);
        for (int l = 0; l < 2; ++l) {      // the sparse segments of an iteration; those selected again
            EG_ALLOC(c->tk.list[l].plan, 1);
            EG_ALLOC(c->tk.list[l].sp_seg, S);
            EG_ALLOC(c->tk.list[l].sp_begin, S + 1);
            EG_ALLOC(c->tk.list[l].cta_q, (size_t)c->topk_grid * kFine);
        }
        EG_ALLOC(c->tk.offcnt, S * kOffBins);
        EG_ALLOC(c->tk.offsel, S);
        EG_ALLOC(c->tk.redo, S);
        EG_ALLOC(c->tk.redo_count, 1);
        EG_ALLOC(c->tk.redo_total, 1);
        EG_ALLOC(c->tk.outbox, (size_t)P * c->out_stride);
        {
            // one cooperative launch needs all its CTAs resident at the same time
            int coop = 0, per_sm = 0;
            const int sms = c->sms;
            if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, c->device) == cudaSuccess && coop &&
                cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_topk_all, kThreads, 0) == cudaSuccess &&
                per_sm > 0)
                c->topk_coop_grid = std::min(per_sm, 4) * sms;
            // Measured: the single launch saves about 40 us in a step without sparse messages but
            // is about 20 % slower than the separate launches when most tensors send (it runs every
            // phase at the occupancy of the largest one), so it is used where launch overhead
            // is visible: small problems.  EG_TOPK_SEPARATE_LAUNCHES forces the separate launches.
            if ((long long)P * c->tiles_norm.n_tiles > 65536 || getenv("EG_TOPK_SEPARATE_LAUNCHES"))
                c->topk_coop_grid = 0;
        }
        {
            const cudaError_t e = cudaFuncSetAttribute(k_topk_collect, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                       (int)CollectSmem::kBytes);
            if (e != cudaSuccess) { c->last_cuda_error = (int)e; return fail(EG_ERR_CUDA); }
        }
        c->tk.out_off = c->d_out_off;
        c->tk.count = c->d_kcount;
        c->tk.numel = c->d_numel;
        {
            // safety margin of the guessed bin, in standard deviations of the sampled count; a
            // negative value makes the guess fail on purpose (exercises the exact repeat)
            const char* e = getenv("EG_TOPK_GUESS_MARGIN");
            c->tk.guess_margin = e && *e ? (float)atof(e) : 5.0f;
        }
        c->tk.out_stride = c->out_stride;
    }
#undef EG_ALLOC
    c->fused_smem = ((2 * (size_t)P + 15) & ~(size_t)15) + (size_t)P * kWarps * sizeof(double);
    if (c->fused_smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(k_fused<kFusedVpt, true>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c->fused_smem);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(k_fused<kFusedVpt, false>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c->fused_smem);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(k_fused_hops<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)c->fused_smem);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(k_fused_hops<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)c->fused_smem);
        if (e != cudaSuccess) { c->last_cuda_error = (int)e; return fail(EG_ERR_CUDA); }
    }
    if (c->hops >= 2 && c->hops <= kMaxStagedHops && P >= 2 * c->hops + 1) {
        const cudaError_t e = c->hops == 2 ? raise_hops_staged<2>(P)
                              : c->hops == 3 ? raise_hops_staged<3>(P) : raise_hops_staged<4>(P);
        if (e != cudaSuccess) { c->last_cuda_error = (int)e; return fail(EG_ERR_CUDA); }
    }
    {
        const int pipe_smem = (int)PipeLayout::bytes(P, true, kPipeConsumers / 32);
        cudaError_t e = cudaSuccess;
        auto raise = [&](const void* fn) {
            if (e == cudaSuccess)
                e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, pipe_smem);
        };
        raise((const void*)k_fused_pipe<kPipeTile, kPipeStages, kPipeConsumers, true>);
        raise((const void*)k_fused_pipe<kPipeTile, kPipeStages, kPipeConsumers, false>);
        raise((const void*)k_fused_pipe_general<kPipeTile, kPipeStages, kPipeConsumers, true, false>);
        raise((const void*)k_fused_pipe_general<kPipeTile, kPipeStages, kPipeConsumers, false, false>);
        raise((const void*)k_fused_pipe_general<kPipeTile, kPipeStages, kPipeConsumers, false, true>);
        if (e != cudaSuccess) { c->last_cuda_error = (int)e; return fail(EG_ERR_CUDA); }
    }
    {
        // one launch per iteration where a few hundred CTAs cover the whole parameter set
        // ... and all of them are resident at the same time (a second wave would double the latency)
        int max_smem = 0, per_sm = 0;
        const int sms = c->sms;
        const void* fn = small_kernel(P);
        if (fn && !c->topk.enabled && c->hops == 1 &&
            cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, c->device) == cudaSuccess &&
            small_smem_bytes(P) <= (size_t)max_smem &&
            cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)small_smem_bytes(P)) ==
                cudaSuccess &&
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, kThreads, small_smem_bytes(P)) ==
                cudaSuccess &&
            c->tiles_fused.n_tiles <= per_sm * sms) {
            if ((s = dev_alloc(c, &c->partials_small, (size_t)P * c->tiles_fused.n_tiles)) != EG_OK) return fail(s);
            if ((s = dev_alloc(c, &c->small_arrived, (size_t)T)) != EG_OK) return fail(s);
            if ((s = dev_alloc(c, &c->small_done, 1)) != EG_OK) return fail(s);
            std::vector<int2> rf, rn;
            for (int t = 0; t < T; ++t)
                for (int q = c->seg_begin_fused[t]; q < c->seg_begin_fused[t + 1]; ++q) {
                    rf.push_back(make_int2(c->seg_begin_fused[t], c->seg_begin_fused[t + 1]));
                    rn.push_back(make_int2(c->seg_begin_norm[t], c->seg_begin_norm[t + 1]));
                }
            if ((s = upload(c, &c->small_range_fused, rf)) != EG_OK) return fail(s);
            if ((s = upload(c, &c->small_range_norm, rn)) != EG_OK) return fail(s);
            c->small_eligible = true;
        }
    }
    if ((s = init_state(c)) != EG_OK) return fail(s);
    if (cudaDeviceSynchronize() != cudaSuccess) return fail(EG_ERR_CUDA);
    *out = c;
    return EG_OK;
}

eg_status eg_layout(const eg_ctx* c, int64_t* tensor_offset_host, int64_t* replica_stride_host) {
    if (!c) return EG_ERR_INVALID;
    if (tensor_offset_host) memcpy(tensor_offset_host, c->offset.data(), c->T * sizeof(int64_t));
    if (replica_stride_host) *replica_stride_host = c->stride;
    return EG_OK;
}

eg_status eg_topk_count(const eg_ctx* c, int t, int64_t* k_t_host) {
    if (!c || t < 0 || t >= c->T || !k_t_host) return EG_ERR_INVALID;
    *k_t_host = c->kcount[t];
    return EG_OK;
}

eg_status eg_topk_repeat_count(eg_ctx* c, uint64_t* repeats_host) {
    if (!c || !repeats_host) return EG_ERR_INVALID;
    DeviceGuard guard(c->device);
    eg_status s = sync_and_check(c);
    if (s != EG_OK) return s;
    unsigned long long v = 0;
    if (c->topk.enabled)
        EG_CUDA(c, cudaMemcpy(&v, c->tk.redo_total, sizeof(v), cudaMemcpyDeviceToHost));
    *repeats_host = v;
    return EG_OK;
}

eg_status eg_set_carry_norm(eg_ctx* c, int enabled) {
    if (!c) return EG_ERR_INVALID;
    c->carry = enabled != 0;
    c->carried_valid = false;
    return EG_OK;
}

eg_status eg_step(eg_ctx* c, float* params, const float* grads, float lr, void* stream_v) {
    return eg_step_masked(c, params, grads, lr, nullptr, stream_v);
}

eg_status eg_step_masked(eg_ctx* c, float* params, const float* grads, float lr,
                         const uint8_t* deliver_dev, void* stream_v) {
    if (!c || !params || !grads) return EG_ERR_INVALID;
    if (deliver_dev && !c->async) return EG_ERR_STATE;     // eg_enable_delivery_masks first
    if (c->async && (c->variant & kOwnLastSent)) return EG_ERR_STATE;
    if (((uintptr_t)params & 15u) || ((uintptr_t)grads & 15u)) return EG_ERR_INVALID;
    DeviceGuard guard(c->device);
    if (!guard.ok) return EG_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    // One stream at a time: moving to another stream is allowed only once the stream of the
    // previous call has run dry.  Nothing can be asked while a graph is being recorded (on the
    // new stream or on the previous one): the caller ends the recording before moving on.
    bool capturing = false;
    {
        cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(stream, &cs) != cudaSuccess) { (void)cudaGetLastError(); cs = cudaStreamCaptureStatusNone; }
        capturing = cs != cudaStreamCaptureStatusNone;
    }
    if (c->stepped && stream != c->last_stream && !c->last_capturing && !capturing) {
        const cudaError_t q = cudaStreamQuery(c->last_stream);
        if (q == cudaErrorNotReady) return EG_ERR_STATE;
        if (q != cudaSuccess) (void)cudaGetLastError();
    }
    c->last_capturing = capturing;
    c->last_stream = stream;
    int launches = 0;
    const TileTable tn_all = c->tiles_norm.view(c->err), tf_all = c->tiles_fused.view(c->err);
    const int S = c->P * c->T;
    // tensors [t0, t0 + tcount) of this launch and their tiles in both tile tables
    const int t0 = c->range_tn ? c->range_t0 : 0, tcount = c->range_tn ? c->range_tn : c->T;
    const int nb = c->seg_begin_norm[t0], ne = c->seg_begin_norm[t0 + tcount];
    const int fb = c->seg_begin_fused[t0], fe = c->seg_begin_fused[t0 + tcount];
    const bool whole = (tcount == c->T);
    // views of the tile tables that start at the first tile of the range (per-tile arrays and
    // the partial-sum arrays are shifted together, so the kernels index them as usual)
    TileTable tn = tn_all, tf = tf_all;
    tn.tensor += nb; tn.offset += nb; tn.length += nb;
    tf.tensor += fb; tf.offset += fb; tf.length += fb;
    const dim3 grid_norm(ne - nb, c->P);
    const int grid_fused = fe - fb;
    double* partials_norm = c->partials_norm + nb;
    double* partials_fused = c->partials_fused + fb;
    long long* step_k = c->range_last ? c->step_k : nullptr;
    if (!whole && (c->topk.enabled || c->async || c->hops > 1 || c->fused_kind == EG_FUSED_REGISTER ||
                   c->quant_bits != 0))
        return EG_ERR_STATE;

    // a1: || x - x_hat || partial sums, unless the previous step carried them over
    const bool carry = c->carry;
    const bool use_carried = carry && c->carried_valid && c->carried_params == params;
    if (!use_carried) {
        TimedSection ts(c, stream, EG_KERNEL_NORM);
        k_norm_partial<<<grid_norm, kThreads, 0, stream>>>(params, c->xhat, tn, c->stride, partials_norm,
                                                          c->variant);
        ++launches;
    }
    const bool small = c->fused_kind == EG_FUSED_AUTO && c->small_eligible && whole && !c->async &&
                       c->variant == 0 && !c->momentum && c->quant_bits == 0;
    // a2 + a6: decision, threshold update, counters
    DecideParams dp{c->P, c->T, c->H, c->thr.mode, c->thr.horizon, c->thr.force_first_event,
                    c->topk.enabled, c->degree, c->variant,
                    c->cap_alpha > 0.0 ? c->cap_g : nullptr, c->cap_beta, t0, tcount, c->err,
                    c->ticket, c->quant_bits};
    const double* partials = use_carried ? c->partials_fused : c->partials_norm;
    const TileTable& tp = use_carried ? tf_all : tn_all;
    if (small) {
        // decisions, snapshot, average, update and the next norms in one launch
        TimedSection ts(c, stream, EG_KERNEL_FUSED);
        SmallArgs sa{use_carried ? nullptr : c->partials_norm, tn_all.n_tiles,
                     {c->partials_fused, c->partials_small}, carry ? 1 : 0, c->small_range_fused,
                     c->small_range_norm, c->small_arrived, c->small_done};
#define EG_SMALL_ARGS params, grads, c->xhat, tf, c->P, c->stride, lr, sa, dp, c->st, c->d_numel, c->ctr, \
                      c->step_k, c->err
        if (c->P <= 4)
            k_step_small<4><<<grid_fused, kThreads, small_smem_bytes(c->P), stream>>>(EG_SMALL_ARGS);
        else if (c->P <= 8)
            k_step_small<8><<<grid_fused, kThreads, small_smem_bytes(c->P), stream>>>(EG_SMALL_ARGS);
        else
            k_step_small<16><<<grid_fused, kThreads, small_smem_bytes(c->P), stream>>>(EG_SMALL_ARGS);
#undef EG_SMALL_ARGS
        ++launches;
    } else {
        TimedSection ts(c, stream, EG_KERNEL_DECIDE);
        EG_CUDA(c, launch_pdl(!c->timing && !c->no_pdl, k_decide, dim3((c->P * tcount + kWarps - 1) / kWarps), dim3(kThreads), 0, stream,
                              partials, (const int*)tp.seg_begin, tp.n_tiles, dp, c->st,
                              (const long long*)c->d_numel, (const long long*)c->d_kcount, c->outbox_count,
                              c->ctr, (const long long*)c->step_k,
                              DeliveryState{deliver_dev, c->pending, c->recv_valid, c->arrive, c->arrivals,
                                            c->async ? 1 : 0}));
        ++launches;
    }
    // quantised messages: delivered into x_hat before the averaging kernel, like Top-K messages
    if (c->quant_bits != 0 && !small) {
        TimedSection ts(c, stream, EG_KERNEL_TOPK);
        QuantArgs qa{params, c->xhat, tn_all, c->P, c->T, c->stride, c->st.quant, c->quant_tile_max, c->quant_exp,
                     c->d_numel, c->topk.enabled ? c->st.sparse : nullptr,
                     c->topk.enabled ? c->d_kcount : nullptr, c->quant_bits, c->degree, c->ctr};
        const int walk_grid = c->sms * 8;
        k_quant_max<<<walk_grid, kThreads, 0, stream>>>(qa);
        k_quant_scale<<<(int)((S + kWarps - 1) / kWarps), kThreads, 0, stream>>>(qa);
        k_quant_apply<<<walk_grid, kThreads, 0, stream>>>(qa);
        launches += 3;
    }
    // a4: Top-K select / pack / deliver for the segments that send a sparse message
    if (c->topk.enabled && !small) {
        TimedSection ts(c, stream, EG_KERNEL_TOPK);
        TopkArgs ta{params, c->xhat, tn, S, c->T, c->stride, c->st.sparse, c->tk, c->err, c->st.sparse_steps,
                    c->step_k, c->topk_grid};
        const int tile_grid = c->topk_grid, seg_grid = c->topk_seg_grid;
        if (c->topk_coop_grid > 0) {
            void* args[] = {&ta};
            EG_CUDA(c, cudaLaunchCooperativeKernel((const void*)k_topk_all, dim3(c->topk_coop_grid),
                                                   dim3(kThreads), args, 0, stream));
            launches += 1;
        } else {
            // Fifteen launches, five of which (the exact repeat for segments whose guessed bin
            // did not work out) leave at once in an ordinary iteration.  They are dependent launches:
            // each waits on the device, first thing it does, for the kernel before it, and none
            // lets its successor in before it ends.
            const bool pdl = !c->timing && !c->no_pdl && c->topk_pdl;
            const dim3 one(1), tile_blocks(tile_grid), entry_blocks(tile_grid / kEntryShares), seg_blocks(seg_grid);
            const dim3 collect_blocks(tile_grid / kCollectShares);
            const dim3 threads(kThreads);
            EG_CUDA(c, launch_pdl(pdl, k_topk_plan, one, dim3(kPlanThreads), 0, stream, ta, 0));
            EG_CUDA(c, launch_pdl(pdl, k_topk_hist, tile_blocks, threads, 0, stream, ta, 0));
            EG_CUDA(c, launch_pdl(pdl, k_topk_guess, seg_blocks, threads, 0, stream, ta));
            EG_CUDA(c, launch_pdl(pdl, k_topk_collect, collect_blocks, dim3(kCollectThreads), (size_t)CollectSmem::kBytes, stream, ta, 0));
            EG_CUDA(c, launch_pdl(pdl, k_topk_resolve, seg_blocks, threads, 0, stream, ta, 0));
            EG_CUDA(c, launch_pdl(pdl, k_topk_plan, one, dim3(kPlanThreads), 0, stream, ta, 1));
            EG_CUDA(c, launch_pdl(pdl, k_topk_hist, tile_blocks, threads, 0, stream, ta, 1));
            EG_CUDA(c, launch_pdl(pdl, k_topk_pick, seg_blocks, threads, 0, stream, ta, 1, 0));
            EG_CUDA(c, launch_pdl(pdl, k_topk_collect, collect_blocks, dim3(kCollectThreads), (size_t)CollectSmem::kBytes, stream, ta, 1));
            EG_CUDA(c, launch_pdl(pdl, k_topk_resolve, seg_blocks, threads, 0, stream, ta, 1));
            EG_CUDA(c, launch_pdl(pdl, k_topk_digit2, entry_blocks, threads, 0, stream, ta));
            EG_CUDA(c, launch_pdl(pdl, k_topk_pick, seg_blocks, threads, 0, stream, ta, 0, 2));
            EG_CUDA(c, launch_pdl(pdl, k_topk_recount, entry_blocks, threads, 0, stream, ta));
            EG_CUDA(c, launch_pdl(pdl, k_topk_scan, seg_blocks, threads, 0, stream, ta));
            EG_CUDA(c, launch_pdl(pdl, k_topk_write, entry_blocks, threads, 0, stream, ta));
            launches += 15;
        }
    }
    // a3 + a5: dense snapshot, consensus average, SGD
    if (!small) {
        TimedSection ts(c, stream, EG_KERNEL_FUSED);
        const uint8_t* valid = c->async ? c->recv_valid : c->st.valid;   // whom the neighbours have heard from
        // Rings of few replicas: a CTA of the pipelined kernels lives for P replicas only, and filling
        // and draining its ring of stages is a large part of that (8 replicas: 6.0 TB/s against
        // 6.7 at 64).  There the kernels are launched as one CTA per resident slot, each walking
        // from tile to tile with its ring kept full across them; after its first tile a CTA takes
        // whatever tile a counter hands out next, so that tiles are begun in address order however
        // the CTAs drift (measured against one CTA per tile on ResNet-18: 8 replicas 6.0 -> 6.7
        // TB/s, 12 replicas -6 % time, 16 replicas -2.5 %, 24 equal, 32 and 48 replicas +1-2 %).
        const int pipe_stages = c->momentum ? kMomStages : kPipeStages;
        const bool walk = c->P >= pipe_stages && c->P <= c->fused_walk_max_p && !c->momentum;
        const int grid_pipe = walk ? std::min(grid_fused, c->sms * 3 * c->fused_waves) : grid_fused;
        int* ticket = walk ? c->ticket : nullptr;
        float* vel = c->momentum ? c->vel : nullptr;
        float* mailbox = c->async ? c->mailbox : nullptr;
        const uint8_t* arrive = c->async ? c->arrive : nullptr;
        // The plain general kernel serves what the specialised ones leave out: more neighbours on
        // small rings or with momentum, and the carried norm under intermittent delivery.
        const bool staged = c->hops > 1 && c->hops <= kMaxStagedHops && c->P >= 2 * c->hops + 1 &&
                            c->fused_kind != EG_FUSED_REGISTER && !c->momentum && !(c->async && carry);
        if (staged) {
            // rows staged through shared memory; the register kernel choice keeps the plain form
            launch_hops_staged(c, carry, grid_fused, stream, params, grads, valid, tf, lr, partials_fused, step_k);
        } else if (c->hops > 1 || (c->async && carry)) {
            if (carry)
                k_fused_hops<true><<<grid_fused, kThreads, c->fused_smem, stream>>>(
                    params, grads, c->xhat, c->st.snap, valid, tf, c->P, c->T, c->stride, lr,
                    partials_fused, step_k, c->variant, c->hops, mailbox, arrive, vel, c->mu);
            else
                k_fused_hops<false><<<grid_fused, kThreads, c->fused_smem, stream>>>(
                    params, grads, c->xhat, c->st.snap, valid, tf, c->P, c->T, c->stride, lr,
                    partials_fused, step_k, c->variant, c->hops, mailbox, arrive, vel, c->mu);
        } else if (c->async) {
            if (c->momentum)
                k_fused_pipe_general<kPipeTile, kMomStages, kPipeConsumers, false, true, true>
                    <<<grid_fused, kPipeThreads, MomLayout::bytes(c->P, false, kPipeConsumers / 32), stream>>>(
                    params, grads, c->xhat, c->st.snap, valid, tf, c->P, c->T, c->stride, lr,
                    partials_fused, step_k, c->err, grid_fused, c->variant, c->mailbox, c->arrive, nullptr, vel, c->mu);
            else
                k_fused_pipe_general<kPipeTile, kPipeStages, kPipeConsumers, false, true>
                    <<<grid_pipe, kPipeThreads, PipeLayout::bytes(c->P, false, kPipeConsumers / 32), stream>>>(
                    params, grads, c->xhat, c->st.snap, valid, tf, c->P, c->T, c->stride, lr,
                    partials_fused, step_k, c->err, grid_fused, c->variant, c->mailbox, c->arrive, ticket);
        } else if (c->fused_kind == EG_FUSED_REGISTER) {
            if (carry)
                k_fused<kFusedVpt, true><<<grid_fused, kThreads, c->fused_smem, stream>>>(
                    params, grads, c->xhat, c->st.snap, valid, tf, c->P, c->T, c->stride, lr,
                    partials_fused, step_k, c->variant, vel, c->mu);
            else
                k_fused<kFusedVpt, false><<<grid_fused, kThreads, c->fused_smem, stream>>>(
                    params, grads, c->xhat, c->st.snap, valid, tf, c->P, c->T, c->stride, lr,
                    partials_fused, step_k, c->variant, vel, c->mu);
        } else if (c->momentum) {
            const size_t smem = MomLayout::bytes(c->P, carry, kPipeConsumers / 32);
#define EG_MOM_ARGS params, grads, c->xhat, (const uint8_t*)c->st.snap, valid, tf, c->P, c->T, \
                    (long long)c->stride, lr, partials_fused, step_k, c->err, grid_fused
            if (c->variant == 0) {
                if (carry)
                    k_fused_pipe_momentum<kPipeTile, kMomStages, kPipeConsumers, true>
                        <<<grid_fused, kPipeThreads, smem, stream>>>(EG_MOM_ARGS, c->vel, c->mu);
                else
                    k_fused_pipe_momentum<kPipeTile, kMomStages, kPipeConsumers, false>
                        <<<grid_fused, kPipeThreads, smem, stream>>>(EG_MOM_ARGS, c->vel, c->mu);
            } else {
                if (carry)
                    k_fused_pipe_general<kPipeTile, kMomStages, kPipeConsumers, true, false, true>
                        <<<grid_fused, kPipeThreads, smem, stream>>>(EG_MOM_ARGS, c->variant, nullptr, nullptr,
                                                                      nullptr, c->vel, c->mu);
                else
                    k_fused_pipe_general<kPipeTile, kMomStages, kPipeConsumers, false, false, true>
                        <<<grid_fused, kPipeThreads, smem, stream>>>(EG_MOM_ARGS, c->variant, nullptr, nullptr,
                                                                      nullptr, c->vel, c->mu);
            }
#undef EG_MOM_ARGS
        } else {
            const size_t smem = PipeLayout::bytes(c->P, carry, kPipeConsumers / 32);
#define EG_PIPE_ARGS params, grads, c->xhat, (const uint8_t*)c->st.snap, valid, tf, c->P, c->T, \
                     (long long)c->stride, lr, partials_fused, step_k, c->err, grid_fused
            if (c->variant == 0) {
                // started while the kernel before it (the decision kernel, or the Top-K sequence)
                // drains: it waits on the device before it reads anything that kernel writes
                if (carry)
                    EG_CUDA(c, launch_pdl(!c->timing && !c->no_pdl, k_fused_pipe<kPipeTile, kPipeStages, kPipeConsumers, true>,
                                          dim3(grid_pipe), dim3(kPipeThreads), smem, stream, EG_PIPE_ARGS, ticket));
                else
                    EG_CUDA(c, launch_pdl(!c->timing && !c->no_pdl, k_fused_pipe<kPipeTile, kPipeStages, kPipeConsumers, false>,
                                          dim3(grid_pipe), dim3(kPipeThreads), smem, stream, EG_PIPE_ARGS, ticket));
            } else {
                if (carry)
                    k_fused_pipe_general<kPipeTile, kPipeStages, kPipeConsumers, true, false>
                        <<<grid_pipe, kPipeThreads, smem, stream>>>(EG_PIPE_ARGS, c->variant, nullptr, nullptr, ticket);
                else
                    k_fused_pipe_general<kPipeTile, kPipeStages, kPipeConsumers, false, false>
                        <<<grid_pipe, kPipeThreads, smem, stream>>>(EG_PIPE_ARGS, c->variant, nullptr, nullptr, ticket);
            }
#undef EG_PIPE_ARGS
        }
        ++launches;
    }
    c->carried_valid = carry && whole;
    c->carried_params = params;
    c->stepped = true;
    c->last_launches = launches;
    EG_CUDA(c, cudaGetLastError());
    return EG_OK;
}

eg_status eg_step_host(eg_ctx* c, float* params_host, const float* grads_host, float lr) {
    if (!c || !params_host || !grads_host) return EG_ERR_INVALID;
    DeviceGuard guard(c->device);
    if (!guard.ok) return EG_ERR_CUDA;
    const size_t bytes = (size_t)c->P * c->stride * sizeof(float);
    if (!c->stage_x) {
        eg_status s = dev_alloc(c, &c->stage_x, (size_t)c->P * c->stride, false);
        if (s != EG_OK) return s;
        if ((s = dev_alloc(c, &c->stage_g, (size_t)c->P * c->stride, false)) != EG_OK) return s;
    }
    cudaStream_t stream = c->last_stream;
    c->carried_valid = false;  // the parameters come from outside
    const bool pipelined = !c->topk.enabled && !c->async && c->hops == 1 && c->quant_bits == 0 &&
                           c->fused_kind != EG_FUSED_REGISTER && c->T >= 2;
    if (!pipelined) {
        EG_CUDA(c, cudaMemcpyAsync(c->stage_x, params_host, bytes, cudaMemcpyHostToDevice, stream));
        EG_CUDA(c, cudaMemcpyAsync(c->stage_g, grads_host, bytes, cudaMemcpyHostToDevice, stream));
        eg_status s = eg_step(c, c->stage_x, c->stage_g, lr, stream);
        if (s != EG_OK) return s;
        EG_CUDA(c, cudaMemcpyAsync(params_host, c->stage_x, bytes, cudaMemcpyDeviceToHost, stream));
        EG_CUDA(c, cudaStreamSynchronize(stream));
        c->carried_valid = false;
        return EG_OK;
    }
    // Tensors do not interact within a step, so the step is run group by group: while one group
    // of tensors is being computed, the next one is on its way in and the previous one on its
    // way out (the two directions of the host link work at the same time).
    constexpr int kGroups = 8;
    struct RangeReset {   // whatever happens below, later steps cover all tensors again
        eg_ctx* c;
        ~RangeReset() { c->range_t0 = 0; c->range_tn = 0; c->range_last = true; }
    } range_reset{c};
    if (!c->copy_in) {
        EG_CUDA(c, cudaStreamCreateWithFlags(&c->copy_in, cudaStreamNonBlocking));
        EG_CUDA(c, cudaStreamCreateWithFlags(&c->copy_out, cudaStreamNonBlocking));
        for (int q = 0; q < 2 * kGroups + 1; ++q) {
            cudaEvent_t e;
            EG_CUDA(c, cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
            c->group_events.push_back(e);
        }
    }
    // group boundaries at tensor starts, about equal numbers of elements
    int bounds[kGroups + 1];
    bounds[0] = 0;
    {
        int t = 0;
        for (int gidx = 1; gidx < kGroups; ++gidx) {
            const int64_t target = c->stride * gidx / kGroups;
            while (t < c->T && c->offset[t] < target) ++t;
            bounds[gidx] = std::max(bounds[gidx - 1], std::min(t, c->T));
        }
        bounds[kGroups] = c->T;
    }
    // the copies must not start before earlier work on the staging buffers has finished
    EG_CUDA(c, cudaEventRecord(c->group_events[2 * kGroups], stream));
    EG_CUDA(c, cudaStreamWaitEvent(c->copy_in, c->group_events[2 * kGroups], 0));
    eg_status status = EG_OK;
    int last_group = -1;
    for (int gidx = 0; gidx < kGroups; ++gidx)
        if (bounds[gidx + 1] > bounds[gidx]) last_group = gidx;
    const size_t pitch = (size_t)c->stride * sizeof(float);
    for (int gidx = 0; gidx < kGroups && status == EG_OK; ++gidx) {
        const int t0 = bounds[gidx], t1 = bounds[gidx + 1];
        if (t1 <= t0) continue;
        const int64_t e0 = c->offset[t0], e1 = (t1 < c->T) ? c->offset[t1] : c->stride;
        const size_t width = (size_t)(e1 - e0) * sizeof(float);
        EG_CUDA(c, cudaMemcpy2DAsync(c->stage_x + e0, pitch, params_host + e0, pitch, width, c->P,
                                     cudaMemcpyHostToDevice, c->copy_in));
        EG_CUDA(c, cudaMemcpy2DAsync(c->stage_g + e0, pitch, grads_host + e0, pitch, width, c->P,
                                     cudaMemcpyHostToDevice, c->copy_in));
        EG_CUDA(c, cudaEventRecord(c->group_events[2 * gidx], c->copy_in));
        EG_CUDA(c, cudaStreamWaitEvent(stream, c->group_events[2 * gidx], 0));
        c->range_t0 = t0;
        c->range_tn = t1 - t0;
        c->range_last = (gidx == last_group);
        status = eg_step(c, c->stage_x, c->stage_g, lr, stream);
        if (status != EG_OK) break;
        EG_CUDA(c, cudaEventRecord(c->group_events[2 * gidx + 1], stream));
        EG_CUDA(c, cudaStreamWaitEvent(c->copy_out, c->group_events[2 * gidx + 1], 0));
        EG_CUDA(c, cudaMemcpy2DAsync(params_host + e0, pitch, c->stage_x + e0, pitch, width, c->P,
                                     cudaMemcpyDeviceToHost, c->copy_out));
    }
    EG_CUDA(c, cudaStreamSynchronize(stream));
    EG_CUDA(c, cudaStreamSynchronize(c->copy_out));
    c->carried_valid = false;
    return status;
}

eg_status eg_stats(eg_ctx* c, uint64_t* messages_sent_host, uint64_t* bytes_sent_host) {
    if (!c) return EG_ERR_INVALID;
    DeviceGuard guard(c->device);
    eg_status s = sync_and_check(c);
    if (s != EG_OK) return s;
    Counters h{};
    EG_CUDA(c, cudaMemcpy(&h, c->ctr, sizeof(h), cudaMemcpyDeviceToHost));
    if (messages_sent_host) *messages_sent_host = h.messages;
    if (bytes_sent_host) *bytes_sent_host = h.bytes;
    return EG_OK;
}

eg_status eg_event_count(eg_ctx* c, uint64_t* events_host) {
    if (!c || !events_host) return EG_ERR_INVALID;
    DeviceGuard guard(c->device);
    eg_status s = sync_and_check(c);
    if (s != EG_OK) return s;
    Counters h{};
    EG_CUDA(c, cudaMemcpy(&h, c->ctr, sizeof(h), cudaMemcpyDeviceToHost));
    *events_host = h.events;
    return EG_OK;
}

eg_status eg_last_decisions(eg_ctx* c, uint8_t* flags_host, double* norms_host, double* thresholds_host) {
    if (!c) return EG_ERR_INVALID;
    DeviceGuard guard(c->device);
    eg_status s = sync_and_check(c);
    if (s != EG_OK) return s;
    const size_t S = (size_t)c->P * c->T;
    if (flags_host) EG_CUDA(c, cudaMemcpy(flags_host, c->st.flag, S, cudaMemcpyDeviceToHost));
    if (norms_host) EG_CUDA(c, cudaMemcpy(norms_host, c->st.norm, S * sizeof(double), cudaMemcpyDeviceToHost));
    if (thresholds_host)
        EG_CUDA(c, cudaMemcpy(thresholds_host, c->st.thr_used, S * sizeof(double), cudaMemcpyDeviceToHost));
    return EG_OK;
}

eg_status eg_thresholds(eg_ctx* c, double* delta_host, uint64_t* events_host) {
    if (!c) return EG_ERR_INVALID;
    DeviceGuard guard(c->device);
    eg_status s = sync_and_check(c);
    if (s != EG_OK) return s;
    const size_t S = (size_t)c->P * c->T;
    if (delta_host) EG_CUDA(c, cudaMemcpy(delta_host, c->st.delta, S * sizeof(double), cudaMemcpyDeviceToHost));
    if (events_host)
        EG_CUDA(c, cudaMemcpy(events_host, c->st.events, S * sizeof(uint64_t), cudaMemcpyDeviceToHost));
    return EG_OK;
}

eg_status eg_last_outbox(eg_ctx* c, int i, int t, int32_t* idx_host, float* val_host, int32_t* count_host) {
    if (!c || i < 0 || i >= c->P || t < 0 || t >= c->T || !count_host) return EG_ERR_INVALID;
    DeviceGuard guard(c->device);
    eg_status s = sync_and_check(c);
    if (s != EG_OK) return s;
    int n = 0;
    EG_CUDA(c, cudaMemcpy(&n, c->outbox_count + (size_t)i * c->T + t, sizeof(int), cudaMemcpyDeviceToHost));
    *count_host = n;
    if (n <= 0 || !c->topk.enabled) { *count_host = 0; return EG_OK; }
    std::vector<int2> buf((size_t)n);
    EG_CUDA(c, cudaMemcpy(buf.data(), c->tk.outbox + (size_t)i * c->out_stride + c->out_off[t],
                          (size_t)n * sizeof(int2), cudaMemcpyDeviceToHost));
    for (int q = 0; q < n; ++q) {
        if (idx_host) idx_host[q] = buf[q].x;
        if (val_host) memcpy(&val_host[q], &buf[q].y, 4);
    }
    return EG_OK;
}

eg_status eg_read_mailboxes(eg_ctx* c, float* xhat_host) {
    if (!c || !xhat_host) return EG_ERR_INVALID;
    DeviceGuard guard(c->device);
    eg_status s = sync_and_check(c);
    if (s != EG_OK) return s;
    EG_CUDA(c, cudaMemcpy(xhat_host, c->xhat, (size_t)c->P * c->stride * sizeof(float), cudaMemcpyDeviceToHost));
    return EG_OK;
}

eg_status eg_set_variant(eg_ctx* c, int own_term, int trigger_metric) {
    if (!c || (own_term != EG_OWN_CURRENT && own_term != EG_OWN_LAST_SENT) ||
        (trigger_metric != EG_TRIGGER_NORM_OF_CHANGE && trigger_metric != EG_TRIGGER_CHANGE_OF_NORM))
        return EG_ERR_INVALID;
    if (c->stepped) return EG_ERR_STATE;   // only before the first step (or after eg_reset)
    if (c->async && own_term == EG_OWN_LAST_SENT) return EG_ERR_STATE;
    c->variant = (own_term == EG_OWN_LAST_SENT ? kOwnLastSent : 0) |
                 (trigger_metric == EG_TRIGGER_CHANGE_OF_NORM ? kChangeOfNorm : 0);
    c->carried_valid = false;
    return EG_OK;
}

eg_status eg_enable_delivery_masks(eg_ctx* c) {
    if (!c) return EG_ERR_INVALID;
    if (c->async) return EG_OK;
    if (c->variant & kOwnLastSent) return EG_ERR_STATE;
    DeviceGuard guard(c->device);
    EG_CUDA(c, cudaStreamSynchronize(c->last_stream));
    const size_t S = (size_t)c->P * c->T, n = (size_t)c->P * c->stride;
    eg_status s;
    if ((s = dev_alloc(c, &c->mailbox, n, false)) != EG_OK) return s;
    if ((s = dev_alloc(c, &c->pending, S)) != EG_OK) return s;
    if ((s = dev_alloc(c, &c->recv_valid, S, false)) != EG_OK) return s;
    if ((s = dev_alloc(c, &c->arrive, S)) != EG_OK) return s;
    if ((s = dev_alloc(c, &c->arrivals, 1)) != EG_OK) return s;
    // everything sent so far has arrived
    EG_CUDA(c, cudaMemcpy(c->mailbox, c->xhat, n * sizeof(float), cudaMemcpyDeviceToDevice));
    EG_CUDA(c, cudaMemcpy(c->recv_valid, c->st.valid, S, cudaMemcpyDeviceToDevice));
    c->async = true;
    c->carried_valid = false;
    return EG_OK;
}

eg_status eg_read_received(eg_ctx* c, float* received_host) {
    if (!c || !received_host) return EG_ERR_INVALID;
    DeviceGuard guard(c->device);
    eg_status s = sync_and_check(c);
    if (s != EG_OK) return s;
    EG_CUDA(c, cudaMemcpy(received_host, c->async ? c->mailbox : c->xhat,
                          (size_t)c->P * c->stride * sizeof(float), cudaMemcpyDeviceToHost));
    return EG_OK;
}

eg_status eg_delivery_status(eg_ctx* c, uint8_t* pending_host, uint64_t* arrivals_host) {
    if (!c) return EG_ERR_INVALID;
    DeviceGuard guard(c->device);
    eg_status s = sync_and_check(c);
    if (s != EG_OK) return s;
    const size_t S = (size_t)c->P * c->T;
    if (pending_host) {
        if (c->async) EG_CUDA(c, cudaMemcpy(pending_host, c->pending, S, cudaMemcpyDeviceToHost));
        else memset(pending_host, 0, S);
    }
    if (arrivals_host) {
        unsigned long long a = 0;
        if (c->async) EG_CUDA(c, cudaMemcpy(&a, c->arrivals, sizeof(a), cudaMemcpyDeviceToHost));
        else {
            Counters h{};
            EG_CUDA(c, cudaMemcpy(&h, c->ctr, sizeof(h), cudaMemcpyDeviceToHost));
            a = h.events;   // synchronous delivery: every event arrived
        }
        *arrivals_host = a;
    }
    return EG_OK;
}

eg_status eg_selftest_wait_timeout(eg_ctx* c, void* stream_v) {
    if (!c) return EG_ERR_INVALID;
    DeviceGuard guard(c->device);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    c->last_stream = stream;
    // the result word sits next to the error word
    int* gave_up = reinterpret_cast<int*>(c->err) + 1;
    k_selftest_wait<<<1, 32, 0, stream>>>(c->err, 2000000ll /* about a millisecond */, gave_up);
    EG_CUDA(c, cudaGetLastError());
    EG_CUDA(c, cudaStreamSynchronize(stream));
    int h = 0;
    EG_CUDA(c, cudaMemcpy(&h, gave_up, sizeof(h), cudaMemcpyDeviceToHost));
    return h ? EG_OK : EG_ERR_INTERNAL;
}

eg_status eg_set_threshold_cap(eg_ctx* c, double alpha, double beta) {
    if (!c || std::isnan(alpha) || std::isnan(beta) || (alpha > 0.0 && !(beta > 0.0))) return EG_ERR_INVALID;
    DeviceGuard guard(c->device);
    if (!guard.ok) return EG_ERR_CUDA;
    // the sequence continues from the term of the iteration the device has reached
    EG_CUDA(c, cudaStreamSynchronize(c->last_stream));
    long long k = 0;
    EG_CUDA(c, cudaMemcpy(&k, c->step_k, sizeof(k), cudaMemcpyDeviceToHost));
    c->cap_alpha = alpha;
    c->cap_beta = beta;
    return upload_cap(c, k);
}

eg_status eg_set_fused_kernel(eg_ctx* c, int kind) {
    if (!c || (kind != EG_FUSED_PIPELINED && kind != EG_FUSED_REGISTER && kind != EG_FUSED_AUTO))
        return EG_ERR_INVALID;
    if (kind != c->fused_kind) c->carried_valid = false;   // the kernels keep their carried sums apart
    c->fused_kind = kind;
    return EG_OK;
}

eg_status eg_set_timing(eg_ctx* c, int enabled) {
    if (!c) return EG_ERR_INVALID;
    c->timing = enabled != 0;
    c->ev_used = 0;
    return EG_OK;
}

eg_status eg_kernel_times(eg_ctx* c, double* ms_host, uint64_t* sections_host) {
    if (!c || !ms_host || !sections_host) return EG_ERR_INVALID;
    DeviceGuard guard(c->device);
    EG_CUDA(c, cudaStreamSynchronize(c->last_stream));
    for (int q = 0; q < EG_KERNEL_GROUPS; ++q) { ms_host[q] = 0.0; sections_host[q] = 0; }
    for (size_t q = 0; q < c->ev_used; ++q) {
        float ms = 0.f;
        EG_CUDA(c, cudaEventElapsedTime(&ms, c->ev_pool[2 * q], c->ev_pool[2 * q + 1]));
        ms_host[c->ev_kind[q]] += (double)ms;
        sections_host[c->ev_kind[q]] += 1;
    }
    c->ev_used = 0;
    return EG_OK;
}

eg_status eg_set_quantisation(eg_ctx* c, int bits) {
    if (!c) return EG_ERR_INVALID;
    if (bits == 32) bits = 0;
    if (bits != 0 && (bits < 2 || bits > 16)) return EG_ERR_INVALID;
    if (c->stepped) return EG_ERR_STATE;            // only before the first step (or after eg_reset)
    DeviceGuard guard(c->device);
    if (!guard.ok) return EG_ERR_CUDA;
    if (bits != 0 && !c->st.quant) {
        const size_t S = (size_t)c->P * c->T;
        eg_status s;
        if ((s = dev_alloc(c, &c->st.quant, S)) != EG_OK) return s;
        if ((s = dev_alloc(c, &c->quant_exp, S)) != EG_OK) return s;
        if ((s = dev_alloc(c, &c->quant_tile_max, (size_t)c->P * c->tiles_norm.n_tiles)) != EG_OK) return s;
    }
    c->quant_bits = bits;
    // in a Top-K context the packing kernel turns the selected values into codes
    c->tk.quant = bits != 0 ? c->st.quant : nullptr;
    c->tk.qexp = bits != 0 ? c->quant_exp : nullptr;
    c->tk.quant_bits = bits;
    c->carried_valid = false;
    return EG_OK;
}

eg_status eg_last_quantised(eg_ctx* c, uint8_t* quantised_host, int32_t* exponents_host) {
    if (!c || !quantised_host || !exponents_host) return EG_ERR_INVALID;
    if (!c->st.quant) return EG_ERR_STATE;
    DeviceGuard guard(c->device);
    eg_status s = sync_and_check(c);
    if (s != EG_OK) return s;
    const size_t S = (size_t)c->P * c->T;
    EG_CUDA(c, cudaMemcpy(quantised_host, c->st.quant, S, cudaMemcpyDeviceToHost));
    EG_CUDA(c, cudaMemcpy(exponents_host, c->quant_exp, S * sizeof(int), cudaMemcpyDeviceToHost));
    return EG_OK;
}

eg_status eg_set_momentum(eg_ctx* c, int enabled, double mu) {
    if (!c) return EG_ERR_INVALID;
    if (!enabled) { c->momentum = false; c->carried_valid = false; return EG_OK; }
    if (!(mu >= 0.0 && mu < 1.0)) return EG_ERR_INVALID;
    DeviceGuard guard(c->device);
    if (!guard.ok) return EG_ERR_CUDA;
    if (!c->vel) {
        float* v = nullptr;
        const eg_status s = dev_alloc(c, &v, (size_t)c->P * c->stride);   // zeroed
        if (s != EG_OK) return s;
        const int smem = (int)MomLayout::bytes(c->P, true, kPipeConsumers / 32);
        EG_CUDA(c, cudaFuncSetAttribute(k_fused_pipe_momentum<kPipeTile, kMomStages, kPipeConsumers, true>,
                                        cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        EG_CUDA(c, cudaFuncSetAttribute(k_fused_pipe_momentum<kPipeTile, kMomStages, kPipeConsumers, false>,
                                        cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        EG_CUDA(c, cudaFuncSetAttribute(k_fused_pipe_general<kPipeTile, kMomStages, kPipeConsumers, true, false, true>,
                                        cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        EG_CUDA(c, cudaFuncSetAttribute(k_fused_pipe_general<kPipeTile, kMomStages, kPipeConsumers, false, false, true>,
                                        cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        EG_CUDA(c, cudaFuncSetAttribute(k_fused_pipe_general<kPipeTile, kMomStages, kPipeConsumers, false, true, true>,
                                        cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        EG_CUDA(c, cudaDeviceSynchronize());
        c->vel = v;
    }
    c->momentum = true;
    c->mu = mu;
    c->carried_valid = false;
    return EG_OK;
}

eg_status eg_read_velocity(eg_ctx* c, float* velocity_host) {
    if (!c || !velocity_host) return EG_ERR_INVALID;
    if (!c->vel) return EG_ERR_STATE;
    DeviceGuard guard(c->device);
    eg_status s = sync_and_check(c);
    if (s != EG_OK) return s;
    EG_CUDA(c, cudaMemcpy(velocity_host, c->vel, (size_t)c->P * c->stride * sizeof(float),
                          cudaMemcpyDeviceToHost));
    return EG_OK;
}

eg_status eg_write_velocity(eg_ctx* c, const float* velocity_host) {
    if (!c || !velocity_host) return EG_ERR_INVALID;
    if (!c->vel) return EG_ERR_STATE;
    DeviceGuard guard(c->device);
    EG_CUDA(c, cudaStreamSynchronize(c->last_stream));
    EG_CUDA(c, cudaMemcpy(c->vel, velocity_host, (size_t)c->P * c->stride * sizeof(float),
                          cudaMemcpyHostToDevice));
    return EG_OK;
}

eg_status eg_reset(eg_ctx* c) {
    if (!c) return EG_ERR_INVALID;
    DeviceGuard guard(c->device);
    EG_CUDA(c, cudaStreamSynchronize(c->last_stream));
    eg_status s = init_state(c);
    if (s != EG_OK) return s;
    EG_CUDA(c, cudaDeviceSynchronize());
    return EG_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------
// averaged model and consensus distance
// ---------------------------------------------------------------------------------------
namespace eg {

// CTAs loop over the fused tile table (1024 elements: one float4 per thread).
// avg[e] = (1/P) sum_i x_i[e] with the sum and the mean in fp64; cons[cta] = sum over the CTA's
// tiles and all replicas of (x_i[e] - mean)^2.  The first kAvgCache replicas stay in registers
// for the second sweep; further ones are read again.
constexpr int kAvgCache = 16;
__global__ void __launch_bounds__(kThreads)
k_average_model(const float* __restrict__ x, float* __restrict__ avg, TileTable tt, int P,
                long long stride, double* __restrict__ cons) {
    static_assert(kFusedTile == kThreads * 4, "one float4 per thread and tile");
    __shared__ double s_warp[kWarps];
    double acc = 0.0;
    const double dP = (double)P;
    for (int tile = blockIdx.x; tile < tt.n_tiles; tile += gridDim.x) {
        const int local = threadIdx.x * 4;
        const int nel = min(4, tt.length[tile] - local);      // live elements of this thread's float4
        if (nel <= 0) continue;
        const float* col = x + tt.offset[tile] + local;        // padding inside a tensor's slot may be read
        float4 v[kAvgCache];
        double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
        // all loads first and without a branch on P (a row index past the last replica is
        // clamped and its value not used), so that they are in flight together
#pragma unroll
        for (int i = 0; i < kAvgCache; ++i) v[i] = ld_stream(col + (long long)min(i, P - 1) * stride);
#pragma unroll
        for (int i = 0; i < kAvgCache; ++i) {
            if (i < P) {
                s0 = __dadd_rn(s0, (double)v[i].x); s1 = __dadd_rn(s1, (double)v[i].y);
                s2 = __dadd_rn(s2, (double)v[i].z); s3 = __dadd_rn(s3, (double)v[i].w);
            }
        }
        for (int i = kAvgCache; i < P; ++i) {
            const float4 a = ld_stream(col + (long long)i * stride);
            s0 = __dadd_rn(s0, (double)a.x); s1 = __dadd_rn(s1, (double)a.y);
            s2 = __dadd_rn(s2, (double)a.z); s3 = __dadd_rn(s3, (double)a.w);
        }
        const double m0 = __ddiv_rn(s0, dP), m1 = __ddiv_rn(s1, dP), m2 = __ddiv_rn(s2, dP), m3 = __ddiv_rn(s3, dP);
        float* out = avg + tt.offset[tile] + local;
        if (nel == 4) {
            *reinterpret_cast<float4*>(out) = make_float4(__double2float_rn(m0), __double2float_rn(m1),
                                                          __double2float_rn(m2), __double2float_rn(m3));
        } else {                                               // padding is never written
            out[0] = __double2float_rn(m0);
            if (nel > 1) out[1] = __double2float_rn(m1);
            if (nel > 2) out[2] = __double2float_rn(m2);
        }
        if (cons) {
            auto add = [&](float4 a) {
                const double d0 = __dsub_rn((double)a.x, m0), d1 = __dsub_rn((double)a.y, m1);
                const double d2 = __dsub_rn((double)a.z, m2), d3 = __dsub_rn((double)a.w, m3);
                acc = __fma_rn(d0, d0, acc);
                if (nel > 1) acc = __fma_rn(d1, d1, acc);
                if (nel > 2) acc = __fma_rn(d2, d2, acc);
                if (nel > 3) acc = __fma_rn(d3, d3, acc);
            };
#pragma unroll
            for (int i = 0; i < kAvgCache; ++i)
                if (i < P) add(v[i]);
            for (int i = kAvgCache; i < P; ++i) add(ld_stream(col + (long long)i * stride));
        }
    }
    if (cons) {
        const double total = block_sum(acc, s_warp);
        if (threadIdx.x == 0) cons[blockIdx.x] = total;
    }
}

__global__ void __launch_bounds__(kThreads)
k_sum_partials(const double* __restrict__ in, int n, double* __restrict__ out) {
    __shared__ double s_warp[kWarps];
    double acc = 0.0;
    for (int q = threadIdx.x; q < n; q += kThreads) acc = __dadd_rn(acc, in[q]);
    const double total = block_sum(acc, s_warp);
    if (threadIdx.x == 0) *out = total;
}

}  // namespace eg

extern "C" {

eg_status eg_average_model(eg_ctx* c, const float* params, float* avg_dev, double* consensus_host,
                           void* stream_v) {
    if (!c || !params || !avg_dev) return EG_ERR_INVALID;
    DeviceGuard guard(c->device);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const TileTable tf = c->tiles_fused.view(c->err);
    const int grid = std::min(tf.n_tiles, c->sms * 8);
    k_average_model<<<grid, kThreads, 0, stream>>>(params, avg_dev, tf, c->P, c->stride,
                                                   consensus_host ? c->cons_partials : nullptr);
    if (consensus_host) {
        k_sum_partials<<<1, kThreads, 0, stream>>>(c->cons_partials, grid, c->cons_partials + grid);
        EG_CUDA(c, cudaMemcpyAsync(consensus_host, c->cons_partials + grid, sizeof(double),
                                   cudaMemcpyDeviceToHost, stream));
        EG_CUDA(c, cudaStreamSynchronize(stream));
    }
    EG_CUDA(c, cudaGetLastError());
    return EG_OK;
}

// ---------------------------------------------------------------------------------------
// checkpoint
// ---------------------------------------------------------------------------------------
// Everything a context needs to continue a run: the header names the context the state belongs
// to (an import into a context created or configured differently is refused), then the
// iteration counter and counters, the trigger state, the mailboxes, and -- when the context
// has them -- the delivery state (received copies, messages in flight) and the velocities.
struct StateHeader {
    uint64_t magic;
    int64_t P, T, H, stride, n_total, topk, k_num, k_den, variant;
    int64_t step;
    uint64_t messages, bytes, events;
    int64_t hops, mode, force_first, delivery, velocity;
    double horizon, delta_init, delta_fixed, cap_alpha, cap_beta, mu;
    uint64_t arrivals;
    int64_t quant_bits;
};

static size_t state_bytes(const eg_ctx* c) {
    const size_t S = (size_t)c->P * c->T, n = (size_t)c->P * c->stride * sizeof(float);
    size_t b = sizeof(StateHeader) + S * (2 * sizeof(double) + sizeof(long long) + sizeof(int) + 1 +
                                          sizeof(unsigned long long)) +
               S * c->H * sizeof(double) + n;
    if (c->async) b += n + 2 * S;
    if (c->vel) b += n;
    return b;
}

static StateHeader state_header(const eg_ctx* c) {
    StateHeader h{};
    h.magic = kStateMagic; h.P = c->P; h.T = c->T; h.H = c->H; h.stride = c->stride;
    h.n_total = c->n_total; h.topk = c->topk.enabled; h.k_num = c->topk.k_num; h.k_den = c->topk.k_den;
    h.variant = c->variant; h.hops = c->hops; h.mode = c->thr.mode; h.force_first = c->thr.force_first_event;
    h.delivery = c->async ? 1 : 0; h.velocity = c->vel ? 1 : 0;
    h.horizon = c->thr.horizon; h.delta_init = c->thr.delta_init; h.delta_fixed = c->thr.delta_fixed;
    h.cap_alpha = c->cap_alpha; h.cap_beta = c->cap_beta; h.mu = c->momentum ? c->mu : 0.0;
    h.quant_bits = c->quant_bits;
    return h;
}

eg_status eg_export_state(eg_ctx* c, void* host_buf, size_t* bytes) {
    if (!c || !bytes) return EG_ERR_INVALID;
    const size_t need = state_bytes(c);
    if (!host_buf) { *bytes = need; return EG_OK; }
    if (*bytes < need) { *bytes = need; return EG_ERR_INVALID; }
    DeviceGuard guard(c->device);
    eg_status s = sync_and_check(c);
    if (s != EG_OK) return s;
    const size_t S = (size_t)c->P * c->T, n = (size_t)c->P * c->stride * sizeof(float);
    StateHeader h = state_header(c);
    Counters ctr{};
    long long k = 0;
    EG_CUDA(c, cudaMemcpy(&ctr, c->ctr, sizeof(ctr), cudaMemcpyDeviceToHost));
    EG_CUDA(c, cudaMemcpy(&k, c->step_k, sizeof(k), cudaMemcpyDeviceToHost));
    h.step = k; h.messages = ctr.messages; h.bytes = ctr.bytes; h.events = ctr.events;
    if (c->async) {
        unsigned long long a = 0;
        EG_CUDA(c, cudaMemcpy(&a, c->arrivals, sizeof(a), cudaMemcpyDeviceToHost));
        h.arrivals = a;
    }
    char* p = static_cast<char*>(host_buf);
    memcpy(p, &h, sizeof(h)); p += sizeof(h);
#define EG_PULL(ptr, nbytes)                                                     \
    EG_CUDA(c, cudaMemcpy(p, (ptr), (nbytes), cudaMemcpyDeviceToHost)); p += (nbytes)
    EG_PULL(c->st.delta, S * sizeof(double));
    EG_PULL(c->st.khat, S * sizeof(long long));
    EG_PULL(c->st.hist_len, S * sizeof(int));
    EG_PULL(c->st.valid, S);
    EG_PULL(c->st.events, S * sizeof(unsigned long long));
    EG_PULL(c->st.hist, S * c->H * sizeof(double));
    EG_PULL(c->st.sent_norm, S * sizeof(double));
    EG_PULL(c->xhat, n);
    if (c->async) {
        EG_PULL(c->mailbox, n);
        EG_PULL(c->pending, S);
        EG_PULL(c->recv_valid, S);
    }
    if (c->vel) { EG_PULL(c->vel, n); }
#undef EG_PULL
    *bytes = need;
    return EG_OK;
}

eg_status eg_import_state(eg_ctx* c, const void* host_buf, size_t bytes) {
    if (!c || !host_buf || bytes < state_bytes(c)) return EG_ERR_INVALID;
    StateHeader h;
    memcpy(&h, host_buf, sizeof(h));
    const StateHeader w = state_header(c);
    // doubles are compared by their bits: a checkpoint belongs to exactly the rules it was made under
    auto same = [](double a, double b) { return memcmp(&a, &b, sizeof(double)) == 0; };
    if (h.magic != w.magic || h.P != w.P || h.T != w.T || h.H != w.H || h.stride != w.stride ||
        h.n_total != w.n_total || h.topk != w.topk || h.variant != w.variant ||
        (h.topk && (h.k_num != w.k_num || h.k_den != w.k_den)) || h.hops != w.hops || h.mode != w.mode ||
        h.force_first != w.force_first || h.delivery != w.delivery || h.velocity != w.velocity ||
        !same(h.horizon, w.horizon) || !same(h.delta_init, w.delta_init) || !same(h.delta_fixed, w.delta_fixed) ||
        !same(h.cap_alpha, w.cap_alpha) || !same(h.cap_beta, w.cap_beta) || !same(h.mu, w.mu) ||
        h.quant_bits != w.quant_bits || h.step < 0)
        return EG_ERR_INVALID;
    DeviceGuard guard(c->device);
    EG_CUDA(c, cudaStreamSynchronize(c->last_stream));
    eg_status s = init_state(c);
    if (s != EG_OK) return s;
    const size_t S = (size_t)c->P * c->T, n = (size_t)c->P * c->stride * sizeof(float);
    Counters ctr{h.messages, h.bytes, h.events, 0};
    long long k = h.step;
    EG_CUDA(c, cudaMemcpy(c->ctr, &ctr, sizeof(ctr), cudaMemcpyHostToDevice));
    EG_CUDA(c, cudaMemcpy(c->step_k, &k, sizeof(k), cudaMemcpyHostToDevice));
    const char* p = static_cast<const char*>(host_buf) + sizeof(h);
#define EG_PUSH(ptr, nbytes)                                                     \
    EG_CUDA(c, cudaMemcpy((ptr), p, (nbytes), cudaMemcpyHostToDevice)); p += (nbytes)
    EG_PUSH(c->st.delta, S * sizeof(double));
    EG_PUSH(c->st.khat, S * sizeof(long long));
    EG_PUSH(c->st.hist_len, S * sizeof(int));
    EG_PUSH(c->st.valid, S);
    EG_PUSH(c->st.events, S * sizeof(unsigned long long));
    EG_PUSH(c->st.hist, S * c->H * sizeof(double));
    EG_PUSH(c->st.sent_norm, S * sizeof(double));
    EG_PUSH(c->xhat, n);
    if (c->async) {
        EG_PUSH(c->mailbox, n);
        EG_PUSH(c->pending, S);
        EG_PUSH(c->recv_valid, S);
        const unsigned long long a = h.arrivals;
        EG_CUDA(c, cudaMemcpy(c->arrivals, &a, sizeof(a), cudaMemcpyHostToDevice));
    }
    if (c->vel) { EG_PUSH(c->vel, n); }
#undef EG_PUSH
    EG_CUDA(c, cudaDeviceSynchronize());
    c->carried_valid = false;
    c->stepped = h.step > 0;
    return upload_cap(c, h.step);
}

}  // extern "C"
