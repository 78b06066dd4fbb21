// Fused dense snapshot / consensus average / SGD update, bulk-copy pipelined version.
//
// Same arithmetic and the same element-axis tiling as k_fused (eg_fused.cuh); what differs is
// how the operands reach the SM.  One producer thread streams the (x, g, x_hat) tiles of the
// replicas, in ring order, into a ring of shared-memory stages with 1-D bulk asynchronous
// copies (cp.async.bulk, completion on an mbarrier, no multicast), so the bytes in flight
// are bounded by shared memory instead of registers; 8 consumer warps read their float4
// column of three adjacent stages (replica j-1, j, j+1) and write the results straight to
// global memory.  Every thread always owns the same column, so the two wrap-around operands
// (replica P-1 for replica 0, replica 0 for replica P-1) live in two extra shared buffers
// that are private per column.
//
// Every mbarrier wait is bounded: when the limit is hit the CTA raises an abort flag, sets a
// bit in the context's error word, lets its copies land and returns.
#pragma once
#include "eg_common.cuh"
#include "eg_fused.cuh"

namespace eg {

constexpr int kPipeTile = 1024;                 // elements per CTA (one float4 per consumer)
constexpr int kPipeStages = 5;
constexpr int kPipeThreads = kThreads + 32;     // 8 consumer warps + 1 producer warp
constexpr long long kWaitLimitCycles = 2000000000ll;   // about one second
constexpr unsigned kErrPipeTimeout = 8u;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// 1-D bulk copy global -> this CTA's shared memory; src, dst 16-byte aligned, bytes % 16 == 0.
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst)),
                 "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, volatile int* s_abort,
                                                  unsigned int* err) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (*s_abort) return false;
        if (clock64() - t0 > kWaitLimitCycles) {
            *s_abort = 1;
            atomicOr(err, kErrPipeTimeout);
            return false;
        }
    }
    return true;
}

struct PipeSmem {   // offsets into dynamic shared memory, all multiples of 16
    static constexpr int kTileBytes = kPipeTile * 4;
    static constexpr int kStageBytes = 3 * kTileBytes;
    static constexpr int kWrapL = kPipeStages * kStageBytes;
    static constexpr int kWrapR = kWrapL + kTileBytes;
    static constexpr int kBars = kWrapR + kTileBytes;              // full[S], empty[S], wrap
    static constexpr int kFlags = kBars + 8 * (2 * kPipeStages + 1) + 8;
    __host__ __device__ static size_t bytes(int P, bool carry) {
        size_t b = kFlags + 16 + ((2 * (size_t)P + 15) & ~(size_t)15);
        if (carry) b += (size_t)P * kWarps * sizeof(double);
        return b;
    }
};

// grid n_tiles (tile table with kPipeTile elements per tile), kPipeThreads threads.
template <bool CARRY>
__global__ void __launch_bounds__(kPipeThreads)
k_fused_pipe(float* __restrict__ x, const float* __restrict__ g, float* __restrict__ xhat,
             const uint8_t* __restrict__ snap, const uint8_t* __restrict__ valid, TileTable tt,
             int P, int T, long long stride, float lr, double* __restrict__ partials,
             long long* step_k, unsigned int* __restrict__ err) {
    extern __shared__ __align__(128) unsigned char smem[];
    float* stages = reinterpret_cast<float*>(smem);
    float* wrap_l = reinterpret_cast<float*>(smem + PipeSmem::kWrapL);   // contribution of replica P-1
    float* wrap_r = reinterpret_cast<float*>(smem + PipeSmem::kWrapR);   // contribution of replica 0
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + PipeSmem::kBars);
    uint64_t* empty = full + kPipeStages;
    uint64_t* wrap_bar = empty + kPipeStages;
    volatile int* s_abort = reinterpret_cast<volatile int*>(smem + PipeSmem::kFlags);
    uint8_t* s_snap = smem + PipeSmem::kFlags + 16;
    uint8_t* s_valid = s_snap + P;
    double* s_red = reinterpret_cast<double*>(s_snap + ((2 * P + 15) & ~15));

    const int tile = blockIdx.x, tid = threadIdx.x;
    const int t = tt.tensor[tile];
    const int len = tt.length[tile];
    const long long off = tt.offset[tile];
    const uint32_t copy_bytes = (uint32_t)(((len + 3) & ~3) * 4);

    for (int j = tid; j < P; j += kPipeThreads) {
        s_snap[j] = snap[(long long)j * T + t];
        s_valid[j] = valid[(long long)j * T + t];
    }
    if (tid == 0) {
        for (int s = 0; s < kPipeStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], kWarps);
        }
        mbar_init(wrap_bar, 1);
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (blockIdx.x == 0) *step_k += 1;   // nothing in this launch reads it
    }
    __syncthreads();

    const bool snap_last = s_snap[P - 1] != 0;
    // Replica P-1 contributes wrap_l; its own stage then only needs what wrap_l does not hold.
    const bool last_opt = P >= 2;

    if (tid >= kThreads) {
        // ------------------------------------------------------------------ producer
        if (tid == kThreads) {
            const long long lb = (long long)(P - 1) * stride + off;
            mbar_expect_tx(wrap_bar, copy_bytes);
            bulk_g2s(wrap_l, (snap_last ? x : xhat) + lb, copy_bytes, wrap_bar);
            for (int j = 0; j < P; ++j) {
                const int s = j % kPipeStages;
                if (j >= kPipeStages &&
                    !mbar_wait_bounded(&empty[s], (uint32_t)((j / kPipeStages - 1) & 1), s_abort, err))
                    break;
                float* st = stages + (size_t)s * 3 * kPipeTile;
                const long long rb = (long long)j * stride + off;
                const bool sn = s_snap[j] != 0;
                const bool is_last = last_opt && (j == P - 1);
                const bool need_x = !(is_last && sn);
                const bool need_h = !sn && !is_last;
                mbar_expect_tx(&full[s], copy_bytes * (1u + (need_x ? 1u : 0u) + (need_h ? 1u : 0u)));
                bulk_g2s(st + kPipeTile, g + rb, copy_bytes, &full[s]);
                if (need_x) bulk_g2s(st, x + rb, copy_bytes, &full[s]);
                if (need_h) bulk_g2s(st + 2 * kPipeTile, xhat + rb, copy_bytes, &full[s]);
            }
        }
    } else {
        // ------------------------------------------------------------------ consumers
        const int c = tid * 4;
        const int nel = min(4, max(0, len - c));
        const int lane = tid & 31, warp = tid >> 5;
        const double neg_lr = -(double)lr;
        const bool has_left = P >= 2, has_right = P >= 3;
        bool ok = mbar_wait_bounded(wrap_bar, 0, s_abort, err) &&
                  mbar_wait_bounded(&full[0], 0, s_abort, err);
        for (int j = 0; ok && j < P; ++j) {
            const int s = j % kPipeStages;
            if (j + 1 < P) {
                ok = mbar_wait_bounded(&full[(j + 1) % kPipeStages],
                                       (uint32_t)(((j + 1) / kPipeStages) & 1), s_abort, err);
                if (!ok) break;
            }
            const float* st = stages + (size_t)s * 3 * kPipeTile;
            const bool sn = s_snap[j] != 0;
            const bool is_last = last_opt && (j == P - 1);
            // where the operands of replica j sit
            const float* xs = (is_last && sn) ? wrap_l : st;
            const float* hs = is_last ? wrap_l : (sn ? st : st + 2 * kPipeTile);
            const float* hl_s;
            const float* hr_s;
            if (j == 0) {
                hl_s = wrap_l;
            } else {
                const float* sp = stages + (size_t)((j - 1) % kPipeStages) * 3 * kPipeTile;
                hl_s = (s_snap[j - 1] != 0) ? sp : sp + 2 * kPipeTile;
            }
            if (j + 1 == P) {
                hr_s = wrap_r;
            } else if (last_opt && j + 1 == P - 1) {
                hr_s = wrap_l;
            } else {
                const float* sq = stages + (size_t)((j + 1) % kPipeStages) * 3 * kPipeTile;
                hr_s = (s_snap[j + 1] != 0) ? sq : sq + 2 * kPipeTile;
            }
            const int jl = (j == 0) ? P - 1 : j - 1, jr = (j + 1 == P) ? 0 : j + 1;
            const bool ul = has_left && s_valid[jl] != 0;
            const bool ur = has_right && s_valid[jr] != 0;
            const double w = __ddiv_rn(1.0, (double)(1 + (ul ? 1 : 0) + (ur ? 1 : 0)));
            double acc = 0.0;
            if (nel > 0) {
                const float4 xc = *reinterpret_cast<const float4*>(xs + c);
                const float4 gc = *reinterpret_cast<const float4*>(st + kPipeTile + c);
                const float4 hc = *reinterpret_cast<const float4*>(hs + c);
                const float4 hl = *reinterpret_cast<const float4*>(hl_s + c);
                const float4 hr = *reinterpret_cast<const float4*>(hr_s + c);
                if (j == 0) *reinterpret_cast<float4*>(wrap_r + c) = hc;   // private to this thread
                const long long rb = (long long)j * stride + off + c;
                const float4 xn = upd4(xc, gc, hl, hr, ul, ur, w, neg_lr);
                store_masked(x + rb, xn, nel);
                if (sn) store_masked(xhat + rb, xc, nel);
                if (CARRY) acc = sq_diff4(xn, hc, nel, acc);
            }
            if (CARRY) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1)
                    acc = __dadd_rn(acc, __shfl_down_sync(0xffffffffu, acc, o));
                if (lane == 0) s_red[j * kWarps + warp] = acc;
            }
            // replica j-1 is not needed any more
            __syncwarp();
            if (lane == 0 && j >= 1) mbar_arrive(&empty[(j - 1) % kPipeStages]);
        }
    }
    if (*s_abort) {
        // failure path only: give copies in flight time to land before the CTA retires
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) {}
    }
    if (CARRY) {
        __syncthreads();
        for (int j = tid; j < P; j += kPipeThreads) {
            double r = 0.0;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) r = __dadd_rn(r, s_red[j * kWarps + w]);
            partials[(long long)j * tt.n_tiles + tile] = r;
        }
    }
}

}  // namespace eg
