// Fused dense snapshot / consensus average / SGD update (Eq. (dist_sgd_event) with
// W_ij = 1/(N_i + 1) on the ring of Section 3; the snapshot is the one-sided put of
// Section 6 into the mailbox x_hat).
//
// Work is tiled over the ELEMENT axis; every thread owns a few float4 columns and walks the
// ring of replicas in registers.  All coupling of the update is between replicas at the same
// element index, so the in-place update of x needs no second buffer and no ordering between
// CTAs: a thread has loaded everything that depends on x_j before it overwrites x_j.
// The value a neighbour contributes is x_j itself when replica j sends a dense message in
// this step (x_hat_j is then only written, never read) and the stored x_hat_j otherwise.
#pragma once
#include "eg_common.cuh"
#include "eg_norm.cuh"

namespace eg {

__device__ __forceinline__ float upd1(float x, float g, float hl, float hr, bool ul, bool ur,
                                      double w, double neg_lr) {
    double s = (double)x;
    if (ul) s = __dadd_rn(s, (double)hl);
    if (ur) s = __dadd_rn(s, (double)hr);
    return __double2float_rn(__fma_rn(neg_lr, (double)g, __dmul_rn(s, w)));
}

__device__ __forceinline__ float4 upd4(float4 x, float4 g, float4 hl, float4 hr, bool ul,
                                       bool ur, double w, double neg_lr) {
    float4 r;
    r.x = upd1(x.x, g.x, hl.x, hr.x, ul, ur, w, neg_lr);
    r.y = upd1(x.y, g.y, hl.y, hr.y, ul, ur, w, neg_lr);
    r.z = upd1(x.z, g.z, hl.z, hr.z, ul, ur, w, neg_lr);
    r.w = upd1(x.w, g.w, hl.w, hr.w, ul, ur, w, neg_lr);
    return r;
}

__device__ __forceinline__ void store_masked(float* p, float4 v, int nel) {
    if (nel == 4) {
        st_stream(p, v);
    } else {  // ragged end of a tensor: never write the padding
        if (nel > 0) p[0] = v.x;
        if (nel > 1) p[1] = v.y;
        if (nel > 2) p[2] = v.z;
    }
}

// grid n_tiles (tiles of kThreads*4*VPT elements), dynamic shared memory:
//   2*P bytes (snap, valid) rounded up to 16, then P*kWarps doubles when CARRY.
// CARRY: also emit, per (replica, tile), the partial sum of (x_new - x_hat)^2 that the next
// step's trigger test needs.
template <int VPT, bool CARRY>
__global__ void __launch_bounds__(kThreads)
k_fused(float* __restrict__ x, const float* __restrict__ g, float* __restrict__ xhat,
        const uint8_t* __restrict__ snap, const uint8_t* __restrict__ valid, TileTable tt,
        int P, int T, long long stride, float lr, double* __restrict__ partials,
        long long* step_k, int variant, float* vel = nullptr, double mu = 0.0) {
    extern __shared__ __align__(128) unsigned char smem[];
    uint8_t* s_snap = smem;
    uint8_t* s_valid = smem + P;
    double* s_red = reinterpret_cast<double*>(smem + ((2 * P + 15) & ~15));

    const int tile = blockIdx.x, tid = threadIdx.x;
    if (!tile_ok(tt, tile, T, stride, kThreads * 4 * VPT)) return;   // bounds-checked build only
    const int t = tt.tensor[tile];
    const int len = tt.length[tile];
    const long long off = tt.offset[tile];
    for (int j = tid; j < P; j += kThreads) {
        s_snap[j] = snap[(long long)j * T + t];
        s_valid[j] = valid[(long long)j * T + t];
    }
    if (blockIdx.x == 0 && tid == 0) *step_k += 1;  // nothing in this launch reads it
    __syncthreads();

    int nel[VPT];
    long long e[VPT];
#pragma unroll
    for (int v = 0; v < VPT; ++v) {
        const int local = (v * kThreads + tid) * 4;
        nel[v] = min(4, max(0, len - local));
        e[v] = off + local;
    }
    const double neg_lr = -(double)lr;
    const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
    const bool has_left = P >= 2, has_right = P >= 3;  // P == 2: one distinct neighbour

    // h_* hold the value replica j contributes to its neighbours for this thread's columns
    float4 h_last[VPT], h_prev[VPT], h_cur[VPT], h_first[VPT], x_cur[VPT], g_cur[VPT];
    const bool snap_last = s_snap[P - 1] != 0;
    {
        const long long rb = (long long)(P - 1) * stride;
        const bool s0 = s_snap[0] != 0;
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            h_last[v] = x_cur[v] = g_cur[v] = h_cur[v] = zero4;
            if (nel[v] > 0) {
                h_last[v] = ld_stream((snap_last ? x : xhat) + rb + e[v]);
                x_cur[v] = ld_stream(x + e[v]);
                g_cur[v] = ld_stream(g + e[v]);
                h_cur[v] = s0 ? x_cur[v] : ld_stream(xhat + e[v]);
            }
            h_prev[v] = h_last[v];
            h_first[v] = h_cur[v];
        }
    }

    for (int j = 0; j < P; ++j) {
        const long long rb = (long long)j * stride;
        float4 x_nxt[VPT], g_nxt[VPT], h_nxt[VPT];
        if (j + 1 < P) {
            const long long nb = rb + stride;
            const bool sn = s_snap[j + 1] != 0;
            const bool is_last = (j + 1 == P - 1);
#pragma unroll
            for (int v = 0; v < VPT; ++v) {
                x_nxt[v] = g_nxt[v] = h_nxt[v] = zero4;
                if (nel[v] > 0) {
                    // replica P-1 was fetched before the loop; do not read it twice
                    x_nxt[v] = (is_last && snap_last) ? h_last[v] : ld_stream(x + nb + e[v]);
                    g_nxt[v] = ld_stream(g + nb + e[v]);
                    h_nxt[v] = is_last ? h_last[v]
                                       : (sn ? x_nxt[v] : ld_stream(xhat + nb + e[v]));
                }
            }
        } else {
#pragma unroll
            for (int v = 0; v < VPT; ++v) { x_nxt[v] = g_nxt[v] = zero4; h_nxt[v] = h_first[v]; }
        }
        const int jl = (j == 0) ? P - 1 : j - 1, jr = (j + 1 == P) ? 0 : j + 1;
        if (!EG_INDEX_OK(tt.err, jl, P) || !EG_INDEX_OK(tt.err, jr, P)) break;
        const bool ul = has_left && s_valid[jl] != 0;
        const bool ur = has_right && s_valid[jr] != 0;
        const double w = __ddiv_rn(1.0, (double)(1 + (ul ? 1 : 0) + (ur ? 1 : 0)));
        const bool sn = s_snap[j] != 0;
        double acc = 0.0;
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            if (nel[v] > 0) {
                if (vel) {   // heavy-ball momentum: v <- fp32(mu * v + g), used in place of g
                    float* vc = vel + rb + e[v];
                    const float4 vj = *reinterpret_cast<const float4*>(vc);
                    const float4 gj = g_cur[v];
                    g_cur[v] = make_float4(__double2float_rn(__fma_rn(mu, (double)vj.x, (double)gj.x)),
                                           __double2float_rn(__fma_rn(mu, (double)vj.y, (double)gj.y)),
                                           __double2float_rn(__fma_rn(mu, (double)vj.z, (double)gj.z)),
                                           __double2float_rn(__fma_rn(mu, (double)vj.w, (double)gj.w)));
                    store_masked(vc, g_cur[v], nel[v]);
                }
                const float4 own = (variant & kOwnLastSent) ? h_cur[v] : x_cur[v];
                const float4 xn = upd4(own, g_cur[v], h_prev[v], h_nxt[v], ul, ur, w, neg_lr);
                store_masked(x + rb + e[v], xn, nel[v]);
                if (sn) store_masked(xhat + rb + e[v], x_cur[v], nel[v]);
                if (CARRY) acc = sq_diff4(xn, (variant & kChangeOfNorm) ? zero4 : h_cur[v], nel[v], acc);
            }
        }
        if (CARRY) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1)
                acc = __dadd_rn(acc, __shfl_down_sync(0xffffffffu, acc, o));
            if ((tid & 31) == 0) s_red[j * kWarps + (tid >> 5)] = acc;
        }
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            h_prev[v] = h_cur[v];
            h_cur[v] = h_nxt[v];
            x_cur[v] = x_nxt[v];
            g_cur[v] = g_nxt[v];
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

}  // namespace eg
