// Segmented change-norm and the device-side trigger decision.
//
// k_norm_partial: || x - x_hat ||^2 of every (replica, tensor), as one fp64 partial sum per
//                 tile (trigger condition of Section 4: the tested quantity).
// k_decide:       sums the partials of a segment in a fixed order, takes the square root,
//                 tests it against the threshold and, on an event, recomputes the threshold
//                 from the slope history (Eq. (thres); history: Section 7) — all on device.
#pragma once
#include "eg_common.cuh"

namespace eg {

__device__ __forceinline__ double sq_diff4(float4 a, float4 b, int nel, double acc) {
    // fp32 difference, exact fp64 square, fp64 accumulation (a product of two fp32 values
    // is exact in fp64, so the fused multiply-add rounds exactly like multiply-then-add)
    const float d0 = __fsub_rn(a.x, b.x), d1 = __fsub_rn(a.y, b.y);
    const float d2 = __fsub_rn(a.z, b.z), d3 = __fsub_rn(a.w, b.w);
    if (nel > 0) acc = __fma_rn((double)d0, (double)d0, acc);
    if (nel > 1) acc = __fma_rn((double)d1, (double)d1, acc);
    if (nel > 2) acc = __fma_rn((double)d2, (double)d2, acc);
    if (nel > 3) acc = __fma_rn((double)d3, (double)d3, acc);
    return acc;
}

// grid (n_tiles, P).  partials[i * n_tiles + tile].
__global__ void __launch_bounds__(kThreads)
k_norm_partial(const float* __restrict__ x, const float* __restrict__ xhat, TileTable tt,
               long long stride, double* __restrict__ partials, int variant) {
    __shared__ double s_warp[kWarps];
    const int tile = blockIdx.x, i = blockIdx.y;
    if (!tile_ok(tt, tile, 0x7fffffff, stride, kNormTile)) return;   // bounds-checked build only
    const int len = tt.length[tile];
    const long long base = (long long)i * stride + tt.offset[tile];
    constexpr int kIter = kNormTile / (kThreads * 4);
    float4 a[kIter], b[kIter];
    int nel[kIter];
#pragma unroll
    for (int q = 0; q < kIter; ++q) {
        const int local = (q * kThreads + threadIdx.x) * 4;
        nel[q] = min(4, max(0, len - local));
        if (nel[q] > 0) {
            a[q] = ld_stream(x + base + local);
            // change-of-norm variant: sum of x^2 (x - 0 is exact), x_hat is not read
            b[q] = (variant & kChangeOfNorm) ? make_float4(0.f, 0.f, 0.f, 0.f)
                                             : ld_stream(xhat + base + local);
        } else {
            a[q] = b[q] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
    }
    double acc = 0.0;
#pragma unroll
    for (int q = 0; q < kIter; ++q) acc = sq_diff4(a[q], b[q], nel[q], acc);
    const double total = block_sum(acc, s_warp);
    if (threadIdx.x == 0) partials[(long long)i * tt.n_tiles + tile] = total;
}

struct DecideParams {
    int P, T, H;
    int mode;                 // 0 adaptive, 1 fixed
    double horizon;
    int force_first;
    int topk;                 // Top-K messages enabled
    int degree;               // distinct ring neighbours of every replica
    int variant;              // kChangeOfNorm: d = | sqrt(sum) - sent_norm |
    // Bound sqrt(g(k)) on the threshold of a step (Assumption 1 with the geometric sequence
    // g(k) = alpha * beta^k of Corollary 2).  The sequence lives on the device and advances
    // with the iteration counter: iteration k reads cap_g[k & 1], the thread that opens the
    // iteration's decisions writes beta * cap_g[k & 1] into the other slot.  nullptr: no bound.
    double* cap_g;
    double cap_beta;
    int t0, tn;               // tensors [t0, t0 + tn) are decided by this launch
    unsigned int* err;        // the context's error word (bounds-checked build)
    int* ticket;              // tile counter of the walking fused kernel that follows: set to zero (nullptr: none)
    int quant_bits;           // bits per code of a quantised message (0: messages in full precision)
};

// Intermittent delivery: which outstanding messages arrive in this step.
struct DeliveryState {
    const uint8_t* deliver;   // [P*T] host-supplied mask for this step (nullptr: everything arrives)
    uint8_t* pending;         // [P*T] something sent has not arrived yet
    uint8_t* recv_valid;      // [P*T] neighbours have received this tensor at least once
    uint8_t* arrive;          // [P*T] out: arrives in this step
    unsigned long long* arrivals;
    int enabled;
};

// Sum of the partials [q0, q1) of one segment by one warp, lane-strided and in a fixed order;
// the total is valid in lane 0.
__device__ __forceinline__ double segment_sum(const double* __restrict__ p, int q0, int q1, int lane) {
    double acc = 0.0;
    // same order of additions as a plain strided loop, but eight loads are in flight at a time
    int q = q0 + lane;
    for (; q + 7 * 32 < q1; q += 8 * 32) {
        double v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = p[q + u * 32];
#pragma unroll
        for (int u = 0; u < 8; ++u) acc = __dadd_rn(acc, v[u]);
    }
    for (; q < q1; q += 32) acc = __dadd_rn(acc, p[q]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc = __dadd_rn(acc, __shfl_down_sync(0xffffffffu, acc, o));
    return acc;
}

// Bound on the thresholds of iteration k (+inf: none).
__device__ __forceinline__ double iteration_cap(const DecideParams& dp, long long k) {
    return dp.cap_g ? __dsqrt_rn(dp.cap_g[k & 1]) : __longlong_as_double(0x7ff0000000000000ll);
}

// The decision of segment s = (replica, tensor t) in iteration k from `acc`, the sum of its
// partials: test, threshold update, message accounting, flags (one thread).
__device__ __forceinline__ void
decide_segment(double acc, long long s, int t, long long k, double cap, const DecideParams& dp, const SegState& st,
               const long long* __restrict__ numel, const long long* __restrict__ topk_count,
               int* __restrict__ outbox_count, Counters* ctr, const DeliveryState& dl) {
    const double root = __dsqrt_rn(acc);
    const double d = (dp.variant & kChangeOfNorm) ? fabs(__dsub_rn(root, st.sent_norm[s])) : root;
    const double thr = fmin(st.delta[s], cap);
    st.norm[s] = d;
    st.thr_used[s] = thr;
    const bool fire = (dp.force_first && k == 0) || (d >= thr);
    const bool was_valid = st.valid[s] != 0;
    uint8_t snap = 0, sparse = 0, quant = 0;
    int out_count = 0;
    if (fire) {
        if (dp.mode == 0 && was_valid) {
            // slope between this event and the previous one, pushed into the history
            const double slope = __ddiv_rn(d, (double)(k - st.khat[s]));
            double* h = st.hist + s * dp.H;
            int n = st.hist_len[s];
            if (!EG_INDEX_OK(dp.err, n, dp.H + 1)) n = dp.H;
            if (n == dp.H) {
                for (int q = 1; q < dp.H; ++q) h[q - 1] = h[q];
                n = dp.H - 1;
            }
            h[n++] = slope;
            st.hist_len[s] = n;
            double sum = 0.0;
            for (int q = 0; q < n; ++q) sum = __dadd_rn(sum, h[q]);
            st.delta[s] = __dmul_rn(dp.horizon, __ddiv_rn(sum, (double)n));
        }
        unsigned long long payload;
        if (dp.quant_bits && was_valid && !dp.topk) {
            // b-bit codes of the change since the last message and the exponent of their scale
            quant = 1;
            payload = 4ull + ((unsigned long long)numel[t] * (unsigned long long)dp.quant_bits + 7ull) / 8ull;
        } else if (!dp.topk || !was_valid) {   // the first message of a tensor is always dense
            snap = 1;
            payload = 4ull * (unsigned long long)numel[t];
        } else {
            sparse = 1;
            if (st.sparse_steps) atomicAdd(&st.sparse_steps[k & 1], 1u);   // tells the Top-K launch there is work
            out_count = (int)topk_count[t];
            payload = 8ull * (unsigned long long)topk_count[t];
            if (dp.quant_bits) {   // the K_t values as codes: exponent, indices, codes
                quant = 1;
                payload = 4ull + 4ull * (unsigned long long)topk_count[t] +
                          ((unsigned long long)topk_count[t] * (unsigned long long)dp.quant_bits + 7ull) / 8ull;
            }
        }
        if (dp.variant & kChangeOfNorm) st.sent_norm[s] = root;
        st.khat[s] = k;
        st.valid[s] = 1;
        st.events[s] += 1ull;
        atomicAdd(&ctr->events, 1ull);
        if (dp.degree > 0) {
            atomicAdd(&ctr->messages, (unsigned long long)dp.degree);
            atomicAdd(&ctr->bytes, (unsigned long long)dp.degree * payload);
        }
    }
    if (dl.enabled) {
        const bool pend = fire || dl.pending[s] != 0;
        const bool arr = pend && (dl.deliver == nullptr || dl.deliver[s] != 0);
        dl.pending[s] = (pend && !arr) ? 1 : 0;
        dl.arrive[s] = arr ? 1 : 0;
        if (arr) {
            dl.recv_valid[s] = 1;
            atomicAdd(dl.arrivals, 1ull);
        }
    }
    st.flag[s] = fire ? 1 : 0;
    st.snap[s] = snap;
    st.sparse[s] = sparse;
    if (st.quant) st.quant[s] = quant;
    if (outbox_count) outbox_count[s] = out_count;
}

// One warp per (replica, tensor).  grid ceil(P*T / kWarps).
__global__ void __launch_bounds__(kThreads)
k_decide(const double* __restrict__ partials, const int* __restrict__ seg_begin, int n_tiles,
         DecideParams dp, SegState st, const long long* __restrict__ numel,
         const long long* __restrict__ topk_count, int* __restrict__ outbox_count,
         Counters* ctr, const long long* __restrict__ step_k, DeliveryState dl) {
    pdl_release();      // the kernel after this one may set itself up meanwhile
    pdl_wait();         // the partial sums come from the kernel before this one
    const int lane = threadIdx.x & 31;
    // work item: (replica, tensor of the launch's range)
    const long long w = (long long)blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (w >= (long long)dp.P * dp.tn) return;
    const int i = (int)(w / dp.tn), t = dp.t0 + (int)(w % dp.tn);
    const long long s = (long long)i * dp.T + t;
    if (!EG_INDEX_OK(dp.err, t, dp.T) || !EG_INDEX_OK(dp.err, seg_begin[t + 1] - 1, n_tiles) ||
        !EG_INDEX_OK(dp.err, seg_begin[t], seg_begin[t + 1]))
        return;                                               // bounds-checked build only
    const double acc = segment_sum(partials + (long long)i * n_tiles, seg_begin[t], seg_begin[t + 1], lane);
    if (lane != 0) return;
    const long long k = *step_k;
    if (w == 0 && st.sparse_steps) st.sparse_steps[(k + 1) & 1] = 0;   // the next iteration's count starts at zero
    if (w == 0 && dp.ticket) *dp.ticket = 0;
    const double cap = iteration_cap(dp, k);
    // next term of the sequence, once per iteration (the launch that holds tensor 0)
    if (w == 0 && dp.t0 == 0 && dp.cap_g) dp.cap_g[(k + 1) & 1] = __dmul_rn(dp.cap_g[k & 1], dp.cap_beta);
    decide_segment(acc, s, t, k, cap, dp, st, numel, topk_count, outbox_count, ctr, dl);
}

}  // namespace eg
