// The whole iteration of Algorithm B in ONE launch, for problems of a few hundred tiles.
//
// With a parameter set that small the iteration is bound by launch latency and by chains of
// dependent memory round trips, not by bandwidth: the decision kernel and the pipelined
// average/update kernel each cost several microseconds of latency for a few microseconds'
// worth of data.  Here a CTA owns one 1024-element tile of one tensor for ALL replicas and
//   1. starts the bulk copies of every replica's (x, x_hat) tile at once (2 P copies on one
//      mbarrier) and loads its own column of every replica's gradient into registers, so the
//      data costs one round trip whatever P is;
//   2. meanwhile takes, for its own use, the P trigger decisions of its tensor from the norm
//      partial sums and the trigger state -- every CTA of a tensor arrives at the same P
//      decisions because they are a pure function of what the previous launch left;
//   3. averages, updates and snapshots from shared memory (same arithmetic and the same order
//      of operations as the pipelined kernel), and emits the next iteration's norm partials;
//   4. the CTA of a tensor that finishes reading the state LAST (a counter per tensor) commits
//      the decisions: thresholds, histories, flags, message counters.  Nobody waits for
//      anybody: no CTA reads the trigger state after it has taken its ticket, and only the last
//      ticket holder writes it.
// The iteration counter is bumped by the CTA that finishes last of all.  The carried partial
// sums alternate between two buffers picked by the parity of the iteration counter, which is
// read on the device, so a captured launch can be replayed.
#pragma once
#include "eg_common.cuh"
#include "eg_fused.cuh"
#include "eg_fused_pipe.cuh"
#include "eg_norm.cuh"

namespace eg {

constexpr int kSmallMaxP = 16;            // 2 * P tiles of 4 KB in shared memory, P gradient columns in registers
constexpr int kSmallTile = kPipeTile;     // the fused tile table is shared with the other kernels

struct SmallArgs {
    const double* norm_partials;   // partials of a norm pass that ran before this launch, or nullptr:
                                   //   take the ones carried by the previous launch
    int norm_n_tiles;
    double* carried[2];            // [P][n_tiles] each; iteration k reads [k & 1], writes [(k + 1) & 1]
    int write_carried;             // emit the partials for the next iteration
    const int2* range_fused;       // [n_tiles] partials [x, y) of the tile's tensor in the carried buffers
    const int2* range_norm;        // [n_tiles] the same in the norm pass's buffer
    int* arrived;                  // [T] CTAs of tensor t that have read the trigger state (self-resetting)
    int* done;                     // CTAs that have finished (self-resetting)
};

__host__ __device__ inline size_t small_smem_bytes(int P) {
    return (size_t)P * 2 * kSmallTile * sizeof(float) + 64 /* barrier, flags, modes */ +
           (size_t)P * kWarps * sizeof(double);
}

// PMAX: compile-time bound on P (the gradient columns live in a register array).
template <int PMAX>
__global__ void __launch_bounds__(kThreads, PMAX <= 8 ? 3 : 1)
k_step_small(float* __restrict__ x, const float* __restrict__ g, float* __restrict__ xhat, TileTable tt,
             int P, long long stride, float lr, SmallArgs sa, DecideParams dp, SegState st,
             const long long* __restrict__ numel, Counters* ctr, long long* step_k,
             unsigned int* __restrict__ err) {
    extern __shared__ __align__(128) unsigned char smem[];
    float* tiles = reinterpret_cast<float*>(smem);                       // [P][2][tile]: x, x_hat
    unsigned char* tail = smem + (size_t)P * 2 * kSmallTile * sizeof(float);
    uint64_t* bar = reinterpret_cast<uint64_t*>(tail);
    volatile int* s_abort = reinterpret_cast<volatile int*>(tail + 8);
    volatile int* s_last = reinterpret_cast<volatile int*>(tail + 12);
    uint8_t* s_mode = tail + 16;                                         // bit 0: dense message, bit 1: valid
    double* s_red = reinterpret_cast<double*>(tail + 64);                // [P][kWarps]

    const int tile = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (!tile_ok(tt, tile, dp.T, stride, kSmallTile) || !EG_INDEX_OK(err, P - 1, PMAX)) return;   // bounds-checked build only
    const int t = tt.tensor[tile];
    const int len = tt.length[tile];
    const long long off = tt.offset[tile];
    const uint32_t copy_bytes = (uint32_t)(((len + 3) & ~3) * 4);
    const long long k = *step_k;
    const double cap = iteration_cap(dp, k);

    if (tid == 0) {
        mbar_init(bar, 1);
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_expect_tx(bar, 2u * (uint32_t)P * copy_bytes);
        for (int j = 0; j < P; ++j) {
            float* dst = tiles + (size_t)j * 2 * kSmallTile;
            const long long src = (long long)j * stride + off;
            bulk_g2s(dst, x + src, copy_bytes, bar);
            bulk_g2s(dst + kSmallTile, xhat + src, copy_bytes, bar);
        }
    }
    // this thread's column of every replica's gradient (a tensor's slot is padded to 128 bytes,
    // so the float4 at a ragged end stays inside it)
    const int c = tid * 4;
    const int nel = min(4, max(0, len - c));
    float4 gq[PMAX];
#pragma unroll
    for (int j = 0; j < PMAX; ++j)
        gq[j] = (j < P && nel > 0) ? ld_stream(g + (long long)j * stride + off + c) : make_float4(0.f, 0.f, 0.f, 0.f);

    // the P decisions of this tensor, while the copies are under way
    // (the ranges are stored per tile so that they arrive with the tile's own record instead of
    // one dependent load later)
    const int2 r_fused = sa.range_fused[tile];
    const double* p_in;
    int q0, q1, p_stride;
    if (sa.norm_partials) {
        const int2 r_norm = sa.range_norm[tile];
        p_in = sa.norm_partials; p_stride = sa.norm_n_tiles;
        q0 = r_norm.x; q1 = r_norm.y;
    } else {
        p_in = (k & 1) ? sa.carried[1] : sa.carried[0]; p_stride = tt.n_tiles;
        q0 = r_fused.x; q1 = r_fused.y;
    }
    if (!EG_INDEX_OK(err, q0, p_stride) || !EG_INDEX_OK(err, q1 - 1, p_stride)) return;   // ranges of partial sums
    double mine[(kSmallMaxP + kWarps - 1) / kWarps];     // lane 0: the sums this warp took
#pragma unroll
    for (int r = 0; r < (kSmallMaxP + kWarps - 1) / kWarps; ++r) {
        const int j = warp + r * kWarps;
        mine[r] = 0.0;
        if (j < P) {
            const long long s = (long long)j * dp.T + t;
            const double delta = st.delta[s];           // in flight together with the partials
            const uint8_t was_valid = st.valid[s];
            const double acc = segment_sum(p_in + (long long)j * p_stride, q0, q1, lane);
            mine[r] = acc;
            if (lane == 0) {
                const bool fire = (dp.force_first && k == 0) || (__dsqrt_rn(acc) >= fmin(delta, cap));
                s_mode[j] = (uint8_t)((fire ? 1 : 0) | ((fire || was_valid != 0) ? 2 : 0));
            }
        }
    }
    __syncthreads();
    if (tid == 0) {
        // every read of the trigger state by this CTA is behind us: take the tensor's ticket
        __threadfence();
        const int n_t = r_fused.y - r_fused.x;
        *s_last = (atomicAdd(&sa.arrived[t], 1) == n_t - 1) ? 1 : 0;
    }

    // the same answer in every lane of a warp (the warp sums below use the full mask)
    const bool ok = __all_sync(0xffffffffu, mbar_wait_bounded(bar, 0, s_abort, err));
    // threads beyond the end of a short tile run along (their stores and squares are masked
    // by nel == 0) so that whole warps take part in the warp sums
    if (ok) {
        const double neg_lr = -(double)lr;
        const double w_one = 1.0, w_half = 0.5, w_third = __ddiv_rn(1.0, 3.0);
        const bool has_left = P >= 2, has_right = P >= 3;
        auto contribution = [&](int j) {     // what replica j's neighbours average with
            const float* base = tiles + (size_t)j * 2 * kSmallTile;
            return *reinterpret_cast<const float4*>(((s_mode[j] & 1) ? base : base + kSmallTile) + c);
        };
        float4 hcf = contribution(0);
        const float4 hlf = contribution(P - 1);
        double hp[4] = {(double)hlf.x, (double)hlf.y, (double)hlf.z, (double)hlf.w};
        double hc[4] = {(double)hcf.x, (double)hcf.y, (double)hcf.z, (double)hcf.w};
        unsigned mode_prev = s_mode[P - 1], mode_cur = s_mode[0];
#pragma unroll
        for (int j = 0; j < PMAX; ++j) {
            if (j >= P) break;
            const int jn = (j + 1 < P) ? j + 1 : 0;
            const unsigned mode_next = s_mode[jn];
            const float4 hnf = contribution(jn);
            const float* base = tiles + (size_t)j * 2 * kSmallTile;
            const float4 gf = gq[j];
            const double hn[4] = {(double)hnf.x, (double)hnf.y, (double)hnf.z, (double)hnf.w};
            const double gd[4] = {(double)gf.x, (double)gf.y, (double)gf.z, (double)gf.w};
            const bool sn = (mode_cur & 1) != 0;
            double xd[4];
            if (sn) {           // a dense message: the contribution IS this replica's x
#pragma unroll
                for (int q = 0; q < 4; ++q) xd[q] = hc[q];
            } else {
                const float4 xf = *reinterpret_cast<const float4*>(base + c);
                xd[0] = (double)xf.x; xd[1] = (double)xf.y; xd[2] = (double)xf.z; xd[3] = (double)xf.w;
            }
            const bool ul = has_left && (mode_prev & 2) != 0;
            const bool ur = has_right && (mode_next & 2) != 0;
            const double w = (ul && ur) ? w_third : ((ul || ur) ? w_half : w_one);
            float xn[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                double sum = xd[q];
                if (ul) sum = __dadd_rn(sum, hp[q]);
                if (ur) sum = __dadd_rn(sum, hn[q]);
                xn[q] = __double2float_rn(__fma_rn(neg_lr, gd[q], __dmul_rn(sum, w)));
            }
            const float4 xn4 = make_float4(xn[0], xn[1], xn[2], xn[3]);
            const long long dst = (long long)j * stride + off + c;
            store_masked(x + dst, xn4, nel);
            if (sn) store_masked(xhat + dst, hcf, nel);       // x_hat <- the x that was tested
            if (sa.write_carried) {
                double acc = sq_diff4(xn4, hcf, nel, 0.0);    // hcf is x_hat after this iteration
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) acc = __dadd_rn(acc, __shfl_down_sync(0xffffffffu, acc, o));
                if (lane == 0) s_red[j * kWarps + warp] = acc;
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) { hp[q] = hc[q]; hc[q] = hn[q]; }
            hcf = hnf;
            mode_prev = mode_cur; mode_cur = mode_next;
        }
    }
    if (*s_abort) {
        // failure path only: give copies in flight time to land before the CTA retires
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) {}
    }
    __syncthreads();
    if (sa.write_carried && ok) {
        double* p_out = (k & 1) ? sa.carried[0] : sa.carried[1];
        for (int j = tid; j < P; j += kThreads) {
            double r = 0.0;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) r = __dadd_rn(r, s_red[j * kWarps + w]);
            p_out[(long long)j * tt.n_tiles + tile] = r;
        }
    }
    if (*s_last) {
        // last reader of this tensor's trigger state: commit its P decisions
        if (lane == 0) {
#pragma unroll
            for (int r = 0; r < (kSmallMaxP + kWarps - 1) / kWarps; ++r) {
                const int j = warp + r * kWarps;
                if (j < P)
                    decide_segment(mine[r], (long long)j * dp.T + t, t, k, cap, dp, st, numel, nullptr, nullptr, ctr,
                                   DeliveryState{nullptr, nullptr, nullptr, nullptr, nullptr, 0});
            }
        }
        if (tid == 0) sa.arrived[t] = 0;
    }
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        if (atomicAdd(sa.done, 1) == (int)gridDim.x - 1) {   // last CTA of the launch
            if (dp.cap_g) dp.cap_g[(k + 1) & 1] = __dmul_rn(dp.cap_g[k & 1], dp.cap_beta);
            *step_k = k + 1;
            *sa.done = 0;
        }
    }
}

}  // namespace eg
