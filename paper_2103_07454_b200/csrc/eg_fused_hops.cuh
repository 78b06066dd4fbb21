// Fused dense snapshot / consensus average / SGD update for a ring in which every replica
// averages with the `hops` nearest replicas on EACH side (Section 7: more neighbours per PE
// let information flow sooner; W_ij = 1/(N_i + 1) as in Section 3).  hops == 1 is served by
// the specialised kernels (eg_fused_pipe.cuh, eg_fused.cuh); this one is the general form.
//
// Same element-axis tiling: a thread owns one float4 column and walks the replicas in order.
// No rolling state is needed: the value replica r contributes is x_hat_r once the thread has
// processed r (a dense message has been written into x_hat_r by then), and x_r (dense message
// this step) or x_hat_r before.  Neighbour values are re-read from L1/L2.
#pragma once
#include "eg_common.cuh"
#include "eg_fused.cuh"

namespace eg {

constexpr int kMaxHops = 8;

// grid n_tiles (1024-element tiles), kThreads threads; dynamic shared memory:
//   P bytes of per-replica mode, rounded up to 16, then P*kWarps doubles when CARRY.
template <bool CARRY>
__global__ void __launch_bounds__(kThreads)
k_fused_hops(float* x, const float* __restrict__ g, float* xhat,
             const uint8_t* __restrict__ snap, const uint8_t* __restrict__ valid, TileTable tt,
             int P, int T, long long stride, float lr, double* __restrict__ partials,
             long long* step_k, int variant, int hops, float* mailbox = nullptr,
             const uint8_t* __restrict__ arrive = nullptr, float* vel = nullptr, double mu = 0.0) {
    // Intermittent delivery (arrive != nullptr): x_hat is the SENT copy, `mailbox` the RECEIVED
    // one, `valid` means "received at least once"; otherwise both copies are x_hat.
    // Heavy-ball momentum (vel != nullptr): v <- fp32(mu * v + g) per replica, used in place of g.
    extern __shared__ __align__(128) unsigned char smem[];
    uint8_t* s_mode = smem;   // bit 0: dense message, bit 1: valid, bit 2: contributes own x, bit 3: arrives
    double* s_red = reinterpret_cast<double*>(smem + ((P + 15) & ~15));
    __shared__ int s_off[2 * kMaxHops];                           // distinct neighbour offsets, in order
    __shared__ int s_noff;
    __shared__ double s_w[2 * kMaxHops + 1];                      // 1 / (1 + number heard from)

    const int tile = blockIdx.x, tid = threadIdx.x;
    if (!tile_ok(tt, tile, T, stride, kThreads * 4)) return;     // bounds-checked build only
    const int t = tt.tensor[tile];
    const int len = tt.length[tile];
    const long long off = tt.offset[tile];
    const bool async = arrive != nullptr;
    for (int j = tid; j < P; j += kThreads) {
        const bool sn = snap[(long long)j * T + t] != 0;
        const bool ar = async ? (arrive[(long long)j * T + t] != 0) : sn;
        s_mode[j] = (uint8_t)((sn ? 1 : 0) | (valid[(long long)j * T + t] ? 2 : 0) |
                              ((sn && ar) ? 4 : 0) | (ar ? 8 : 0));
    }
    if (tid == 0) {
        // offsets -1, +1, -2, +2, ... reduced mod P; one entry per distinct neighbour
        int n = 0;
        for (int d = 1; d <= hops; ++d) {
            const int cand[2] = {((-d) % P + P) % P, d % P};
            for (int side = 0; side < 2; ++side) {
                bool seen = cand[side] == 0;
                for (int q = 0; q < n && !seen; ++q) seen = s_off[q] == cand[side];
                if (!seen) s_off[n++] = cand[side];
            }
        }
        s_noff = n;
        for (int q = 0; q <= 2 * kMaxHops; ++q) s_w[q] = __ddiv_rn(1.0, (double)(1 + q));
        if (blockIdx.x == 0) *step_k += 1;   // nothing in this launch reads it
    }
    __syncthreads();

    const int c = tid * 4;
    const int nel = min(4, max(0, len - c));
    const double neg_lr = -(double)lr;
    const int noff = s_noff;
    const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
    float* xc = x + off + c;
    const float* gc = g + off + c;
    float* hc = xhat + off + c;                         // sent copies
    float* mc = (async ? mailbox : xhat) + off + c;     // received copies

    for (int j = 0; j < P; ++j) {
        const bool sn = (s_mode[j] & 1) != 0;
        double acc = 0.0;
        if (nel > 0) {
            const long long rb = (long long)j * stride;
            const float4 xj = *reinterpret_cast<const float4*>(xc + rb);
            float4 gj = ld_stream(gc + rb);
            if (vel) {
                float* vc = vel + off + c + rb;
                const float4 vj = *reinterpret_cast<const float4*>(vc);
                gj = make_float4(__double2float_rn(__fma_rn(mu, (double)vj.x, (double)gj.x)),
                                 __double2float_rn(__fma_rn(mu, (double)vj.y, (double)gj.y)),
                                 __double2float_rn(__fma_rn(mu, (double)vj.z, (double)gj.z)),
                                 __double2float_rn(__fma_rn(mu, (double)vj.w, (double)gj.w)));
                store_masked(vc, gj, nel);
            }
            const unsigned mj = s_mode[j];
            // what this replica contributes to its neighbours in this step
            const float4 hj = (mj & 4) ? xj
                                       : *reinterpret_cast<const float4*>(((mj & 8) ? hc : mc) + rb);
            const float4 own = (variant & kOwnLastSent) ? hj : xj;
            double s0 = (double)own.x, s1 = (double)own.y, s2 = (double)own.z, s3 = (double)own.w;
            int cnt = 0;
            for (int q = 0; q < noff; ++q) {
                int r = j + s_off[q];
                if (r >= P) r -= P;
                const unsigned mode = s_mode[r];
                if (!(mode & 2)) continue;                         // never heard from
                // processed replicas (r < j) have whatever arrived in their mailbox already
                const float* src = (r > j) ? ((mode & 4) ? xc : ((mode & 8) ? hc : mc)) : mc;
                const float4 v = *reinterpret_cast<const float4*>(src + (long long)r * stride);
                s0 = __dadd_rn(s0, (double)v.x); s1 = __dadd_rn(s1, (double)v.y);
                s2 = __dadd_rn(s2, (double)v.z); s3 = __dadd_rn(s3, (double)v.w);
                ++cnt;
            }
            const double w = s_w[cnt];
            float4 xn;
            xn.x = __double2float_rn(__fma_rn(neg_lr, (double)gj.x, __dmul_rn(s0, w)));
            xn.y = __double2float_rn(__fma_rn(neg_lr, (double)gj.y, __dmul_rn(s1, w)));
            xn.z = __double2float_rn(__fma_rn(neg_lr, (double)gj.z, __dmul_rn(s2, w)));
            xn.w = __double2float_rn(__fma_rn(neg_lr, (double)gj.w, __dmul_rn(s3, w)));
            // the message first (later replicas read it), then the parameters
            if (sn) store_masked(hc + rb, xj, nel);
            if (async && (mj & 8)) store_masked(mc + rb, hj, nel);
            store_masked(xc + rb, xn, nel);
            if (CARRY) {
                // the next trigger test compares with what this replica has SENT: its x of this
                // step after a dense message, else the sent copy -- which is what it contributes
                // unless its neighbours still hold an older copy (a message in flight)
                float4 ref = hj;
                if (async && !sn && !(mj & 8)) ref = *reinterpret_cast<const float4*>(hc + rb);
                if (async && sn) ref = xj;
                acc = sq_diff4(xn, (variant & kChangeOfNorm) ? zero4 : ref, nel, acc);
            }
        }
        if (CARRY) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc = __dadd_rn(acc, __shfl_down_sync(0xffffffffu, acc, o));
            if ((tid & 31) == 0) s_red[j * kWarps + (tid >> 5)] = acc;
        }
    }
    if (CARRY) {
        __syncthreads();
        for (int j = tid; j < P; j += kThreads) {
            double r = 0.0;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) r = __dadd_rn(r, s_red[j * kWarps + w]);
            partials[(long long)j * tt.n_tiles + tile] = r;
        }
    }
}

// ---------------------------------------------------------------------------------------
// The same step with every row staged through shared memory by per-thread asynchronous copies.
//
// What replica r contributes to its neighbours in a step is ONE value per element whatever
// the moment it is read: x_r if r sends a dense message that arrives now, else its sent copy
// if an earlier message arrives now, else what its neighbours already hold.  A thread therefore
// copies that row once (16 bytes of its own column, cp.async) into a ring of 2 M + D + 1
// contribution slots, D rows ahead of the replica it is updating, and reads the 2 M
// neighbours of replica j from the ring instead of from L2.  x_j and g_j arrive through two
// more rings D rows ahead.  The contributions of the first and last M replicas, which the other
// end of the ring needs after (before) they were (are) in the ring, have slots of their own.
// Nothing is shared between threads, so there is no barrier: a thread waits for its own copy
// groups only (cp.async.wait_group), which cannot block on anything but memory.
// Needs P >= 2 M + 1 (all 2 M neighbours distinct); smaller rings use k_fused_hops.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
    const uint32_t d = static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst));
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <int M, int D>
struct HopsStaged {
    static constexpr int kRowSlots = D + 1;            // x and g rings
    static constexpr int kContribSlots = 2 * M + D + 1;
    static constexpr int kSlotBytes = kThreads * 16;
    static size_t bytes(int P, bool carry) {
        return (size_t)(2 * kRowSlots + kContribSlots + 2 * M) * kSlotBytes + ((P + 15) & ~15) +
               (carry ? (size_t)P * kWarps * sizeof(double) : 0);
    }
};

template <bool CARRY, int M, int D>
__global__ void __launch_bounds__(kThreads)
k_fused_hops_staged(float* x, const float* __restrict__ g, float* xhat,
                    const uint8_t* __restrict__ snap, const uint8_t* __restrict__ valid, TileTable tt,
                    int P, int T, long long stride, float lr, double* __restrict__ partials,
                    long long* step_k, int variant, float* mailbox = nullptr,
                    const uint8_t* __restrict__ arrive = nullptr) {
    using L = HopsStaged<M, D>;
    constexpr int RX = L::kRowSlots, RC = L::kContribSlots;
    extern __shared__ __align__(128) unsigned char smem[];
    float4* sx = reinterpret_cast<float4*>(smem);
    float4* sg = sx + RX * kThreads;
    float4* sc = sg + RX * kThreads;          // contribution ring: row r in slot r % RC
    float4* s_head = sc + RC * kThreads;      // contributions of replicas 0 .. M-1
    float4* s_tail = s_head + M * kThreads;   // contributions of replicas P-M .. P-1
    uint8_t* s_mode = reinterpret_cast<uint8_t*>(s_tail + M * kThreads);
    double* s_red = reinterpret_cast<double*>(s_mode + ((P + 15) & ~15));
    __shared__ double s_w[2 * M + 1];         // 1 / (1 + number heard from)

    const int tile = blockIdx.x, tid = threadIdx.x;
    if (!tile_ok(tt, tile, T, stride, kThreads * 4)) return;     // bounds-checked build only
    const int t = tt.tensor[tile];
    const int len = tt.length[tile];
    const long long off = tt.offset[tile];
    const bool async = arrive != nullptr;
    for (int j = tid; j < P; j += kThreads) {
        const bool sn = snap[(long long)j * T + t] != 0;
        const bool ar = async ? (arrive[(long long)j * T + t] != 0) : sn;
        s_mode[j] = (uint8_t)((sn ? 1 : 0) | (valid[(long long)j * T + t] ? 2 : 0) |
                              ((sn && ar) ? 4 : 0) | (ar ? 8 : 0));
    }
    if (tid <= 2 * M) s_w[tid] = __ddiv_rn(1.0, (double)(1 + tid));
    if (tid == 0 && blockIdx.x == 0) *step_k += 1;   // nothing in this launch reads it
    __syncthreads();

    const int c = tid * 4;
    const int nel = min(4, max(0, len - c));
    const bool live = nel > 0;
    const double neg_lr = -(double)lr;
    const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
    float* xc = x + off + c;
    const float* gc = g + off + c;
    float* hc = xhat + off + c;                         // sent copies
    float* mc = (async ? mailbox : xhat) + off + c;     // received copies
    auto contribution = [&](int r) -> const float* {
        const unsigned mode = s_mode[r];
        return ((mode & 4) ? xc : ((mode & 8) ? hc : mc)) + (long long)r * stride;
    };

    // The copies are issued as one group per replica step, D steps ahead; the first D groups
    // are issued here, and the very first also brings what replica 0 needs besides its own row.
    // "All but the last D groups have landed" then means the same thing in every step.
#pragma unroll
    for (int v = 0; v < D; ++v) {
        if (live) {
            if (v == 0) {
#pragma unroll
                for (int k = 0; k < M; ++k) {
                    cp_async16(s_tail + k * kThreads + tid, contribution(P - M + k));
                    cp_async16(s_head + k * kThreads + tid, contribution(k));
                    cp_async16(sc + k * kThreads + tid, contribution(k));
                }
            }
            if (v < P) {
                cp_async16(sx + v * kThreads + tid, xc + (long long)v * stride);
                cp_async16(sg + v * kThreads + tid, gc + (long long)v * stride);
            }
            if (v + M < P) cp_async16(sc + ((v + M) % RC) * kThreads + tid, contribution(v + M));
        }
        cp_async_commit();
    }

    int slot_x = 0;            // j % RX
    int slot_c = 0;            // j % RC
    int ahead_x = D % RX;      // (j + D) % RX
    int ahead_c = (M + D) % RC;   // (j + M + D) % RC
    for (int j = 0; j < P; ++j) {
        if (live) {
            if (j + D < P) {
                cp_async16(sx + ahead_x * kThreads + tid, xc + (long long)(j + D) * stride);
                cp_async16(sg + ahead_x * kThreads + tid, gc + (long long)(j + D) * stride);
            }
            if (j + M + D < P) cp_async16(sc + ahead_c * kThreads + tid, contribution(j + M + D));
        }
        cp_async_commit();
        cp_async_wait<D>();     // all but the last D groups: the rows of replica j are here
        double acc = 0.0;
        if (live) {
            const bool sn = (s_mode[j] & 1) != 0;
            const unsigned mj = s_mode[j];
            const float4 xj = sx[slot_x * kThreads + tid];
            const float4 gj = sg[slot_x * kThreads + tid];
            const float4 hj = sc[slot_c * kThreads + tid];
            const float4 own = (variant & kOwnLastSent) ? hj : xj;
            double s0 = (double)own.x, s1 = (double)own.y, s2 = (double)own.z, s3 = (double)own.w;
            int cnt = 0;
#pragma unroll
            for (int d = 1; d <= M; ++d) {
#pragma unroll
                for (int side = 0; side < 2; ++side) {           // left first, then right
                    const int r = side ? j + d : j - d;
                    const int rr = r < 0 ? r + P : (r >= P ? r - P : r);
                    if (!(s_mode[rr] & 2)) continue;              // never heard from
                    float4 v;
                    if (r < 0) {
                        v = s_tail[(r + M) * kThreads + tid];
                    } else if (r >= P) {
                        v = s_head[(r - P) * kThreads + tid];
                    } else {
                        int sl = side ? slot_c + d : slot_c - d;
                        sl = sl < 0 ? sl + RC : (sl >= RC ? sl - RC : sl);
                        v = sc[sl * kThreads + tid];
                    }
                    s0 = __dadd_rn(s0, (double)v.x); s1 = __dadd_rn(s1, (double)v.y);
                    s2 = __dadd_rn(s2, (double)v.z); s3 = __dadd_rn(s3, (double)v.w);
                    ++cnt;
                }
            }
            const double w = s_w[cnt];
            float4 xn;
            xn.x = __double2float_rn(__fma_rn(neg_lr, (double)gj.x, __dmul_rn(s0, w)));
            xn.y = __double2float_rn(__fma_rn(neg_lr, (double)gj.y, __dmul_rn(s1, w)));
            xn.z = __double2float_rn(__fma_rn(neg_lr, (double)gj.z, __dmul_rn(s2, w)));
            xn.w = __double2float_rn(__fma_rn(neg_lr, (double)gj.w, __dmul_rn(s3, w)));
            const long long rb = (long long)j * stride;
            if (sn) store_masked(hc + rb, xj, nel);
            if (async && (mj & 8)) store_masked(mc + rb, hj, nel);
            store_masked(xc + rb, xn, nel);
            if (CARRY) acc = sq_diff4(xn, (variant & kChangeOfNorm) ? zero4 : hj, nel, acc);
        }
        if (CARRY) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc = __dadd_rn(acc, __shfl_down_sync(0xffffffffu, acc, o));
            if ((tid & 31) == 0) s_red[j * kWarps + (tid >> 5)] = acc;
        }
        if (++slot_x == RX) slot_x = 0;
        if (++slot_c == RC) slot_c = 0;
        if (++ahead_x == RX) ahead_x = 0;
        if (++ahead_c == RC) ahead_c = 0;
    }
    cp_async_wait<0>();
    if (CARRY) {
        __syncthreads();
        for (int j = tid; j < P; j += kThreads) {
            double r = 0.0;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) r = __dadd_rn(r, s_red[j * kWarps + w]);
            partials[(long long)j * tt.n_tiles + tile] = r;
        }
    }
}

}  // namespace eg
