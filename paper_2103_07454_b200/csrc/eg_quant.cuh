// Quantised messages: a second compression on top of the events (Section 7 names quantization as
// something that can be applied on top of event-triggered communication; it gives no scheme, the
// one built here is stated in include/eventgrad.h at eg_set_quantisation).
//
// On an event of a tensor that has been sent before, the message carries b-bit codes of the change
// since the last message, d[e] = x[e] - x_hat[e] (fp32), on a power-of-two grid:
//   L = 2^(b-1) - 1,  E = the smallest integer with L 2^E >= max|d|,
//   q[e] = d[e] / 2^E rounded to the nearest integer (ties to even),
//   x_hat[e] <- fp32(fp64(x_hat[e]) + q[e] 2^E)     (sender and receivers alike).
// The decision kernel marks such events (SegState::quant) instead of asking the averaging kernel
// for a dense snapshot; three short kernels then deliver the message into x_hat before the
// averaging kernel runs, which finds the sender's x_hat already updated -- the way a Top-K message
// is delivered -- so every form of the averaging kernel works with quantised messages unchanged:
//   k_quant_max    per tile of a marked segment: max|d| (infinite when a change is not finite)
//   k_quant_scale  per marked segment: E from the largest change; a change that is not finite
//                  turns the message into a full-precision one (and corrects the byte counter)
//   k_quant_apply  per tile of a marked segment: the update of x_hat above (or x_hat <- x)
// The kernels walk all (replica, tile) pairs with a fixed grid: the threads of a CTA first look,
// each at a pair of its own, for the marked ones (one round of loads for 256 pairs), then the CTA
// works through those it found.  An iteration without quantised messages costs three launches of
// a few microseconds.
#pragma once
#include "eg_common.cuh"
#include "eg_norm.cuh"

namespace eg {

constexpr uint8_t kQuantCodes = 1;       // SegState::quant: the message is E and the codes
constexpr uint8_t kQuantFull = 2;        // ... a change was not finite: the message is x itself

struct QuantArgs {
    const float* x;
    float* xhat;
    TileTable tt;              // the norm tiles (kNormTile elements)
    int P, T;
    long long stride;
    uint8_t* quant;            // [P*T] SegState::quant
    float* tile_max;           // [P][n_tiles]
    int* qexp;                 // [P*T] E of the segment's message
    const long long* numel;    // [T]
    const uint8_t* sparse;     // [P*T] SegState::sparse: the message is a Top-K message; its values are
                               //       quantised by the Top-K packing kernel (which needs E from here)
    const long long* topk_count;   // [T] K_t (nullptr without Top-K)
    int bits;
    int degree;                // distinct ring neighbours of a replica
    Counters* ctr;
};

// The marked pairs among the kThreads pairs `first + (j * gridDim.x + blockIdx.x)`, j = 0 ..
// kThreads - 1, into `list` (any order); returns how many.  All threads of the CTA call it.
__device__ __forceinline__ int quant_marked_pairs(const QuantArgs& a, long long first, long long pairs, int* list,
                                                  int* count) {
    if (threadIdx.x == 0) *count = 0;
    __syncthreads();
    const long long w = first + (long long)threadIdx.x * gridDim.x + blockIdx.x;
    if (w < pairs) {
        const int i = (int)(w / a.tt.n_tiles), tile = (int)(w % a.tt.n_tiles);
        if (a.quant[(long long)i * a.T + a.tt.tensor[tile]] != 0) list[atomicAdd(count, 1)] = (int)(w - first);
    }
    __syncthreads();
    return *count;
}

// grid: any; CTA b takes the (replica, tile) pairs b, b + grid, ...
__global__ void __launch_bounds__(kThreads) k_quant_max(QuantArgs a) {
    __shared__ float s_warp[kWarps];
    __shared__ int s_list[kThreads], s_count;
    const long long pairs = (long long)a.P * a.tt.n_tiles;
    for (long long first = 0; first < pairs; first += (long long)gridDim.x * kThreads) {
      const int found = quant_marked_pairs(a, first, pairs, s_list, &s_count);
      for (int f = 0; f < found; ++f) {
        const long long w = first + s_list[f];
        const int i = (int)(w / a.tt.n_tiles), tile = (int)(w % a.tt.n_tiles);
        if (!tile_ok(a.tt, tile, a.T, a.stride, kNormTile)) continue;  // bounds-checked build only
        const int len = a.tt.length[tile];
        const long long base = (long long)i * a.stride + a.tt.offset[tile];
        float m = 0.f;
        bool bad = false;
        for (int local = threadIdx.x * 4; local < len; local += kThreads * 4) {
            const float4 xv = ld_stream(a.x + base + local), hv = *reinterpret_cast<const float4*>(a.xhat + base + local);
            const float d[4] = {fabsf(__fsub_rn(xv.x, hv.x)), fabsf(__fsub_rn(xv.y, hv.y)),
                                fabsf(__fsub_rn(xv.z, hv.z)), fabsf(__fsub_rn(xv.w, hv.w))};
            const int nel = min(4, len - local);
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (c < nel) {
                    bad = bad || !(d[c] <= 3.402823466e+38f);
                    m = fmaxf(m, d[c]);          // (a NaN is dropped here and caught by `bad`)
                }
        }
        if (bad) m = __uint_as_float(0x7f800000u);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        __syncthreads();                                   // the previous pair's values have been read
        if ((threadIdx.x & 31) == 0) s_warp[threadIdx.x >> 5] = m;
        __syncthreads();
        if (threadIdx.x == 0) {
            float all = s_warp[0];
#pragma unroll
            for (int q = 1; q < kWarps; ++q) all = fmaxf(all, s_warp[q]);
            a.tile_max[w] = all;
        }
      }
    }
}

// One warp per (replica, tensor).  grid ceil(P*T / kWarps).
__global__ void __launch_bounds__(kThreads) k_quant_scale(QuantArgs a) {
    const int lane = threadIdx.x & 31;
    const long long s = (long long)blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (s >= (long long)a.P * a.T) return;
    if (a.quant[s] == 0) return;
    const int i = (int)(s / a.T), t = (int)(s % a.T);
    const float* tm = a.tile_max + (long long)i * a.tt.n_tiles;
    float m = 0.f;
    for (int q = a.tt.seg_begin[t] + lane; q < a.tt.seg_begin[t + 1]; q += 32) m = fmaxf(m, tm[q]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane != 0) return;
    if (!(m <= 3.402823466e+38f)) {
        // a change that is not finite: the message is the tensor itself
        a.quant[s] = kQuantFull;
        a.qexp[s] = 0;
        const unsigned long long n = (unsigned long long)a.numel[t];
        unsigned long long coded = 4ull + (n * (unsigned long long)a.bits + 7ull) / 8ull, full = 4ull * n;
        if (a.sparse && a.sparse[s]) {      // a Top-K message: 8 K_t bytes in full, E + indices + codes otherwise
            const unsigned long long K = (unsigned long long)a.topk_count[t];
            coded = 4ull + 4ull * K + (K * (unsigned long long)a.bits + 7ull) / 8ull;
            full = 8ull * K;
        }
        if (a.degree > 0) {
            // (unsigned arithmetic: the two updates together add degree * (full - coded))
            atomicAdd(&a.ctr->bytes, (unsigned long long)a.degree * full);
            atomicAdd(&a.ctr->bytes, 0ull - (unsigned long long)a.degree * coded);
        }
        return;
    }
    int E = 0;
    if (m > 0.f) {
        // m = f 2^p with 0.5 <= f < 1, so 2^(p-1) <= m < 2^p; with E0 = p - (b - 1) the grid of
        // E0 - 1 ends below 2^(p-1) and that of E0 + 1 above 2^p: E is E0 or E0 + 1
        int p;
        (void)frexpf(m, &p);
        const double L = (double)((1 << (a.bits - 1)) - 1);
        const int E0 = p - (a.bits - 1);
        E = (__dmul_rn(L, pow2_double(E0)) >= (double)m) ? E0 : E0 + 1;
    }
    a.qexp[s] = E;
}

// grid: any; CTA b takes the (replica, tile) pairs b, b + grid, ...
__global__ void __launch_bounds__(kThreads) k_quant_apply(QuantArgs a) {
    __shared__ int s_list[kThreads], s_count;
    const long long pairs = (long long)a.P * a.tt.n_tiles;
    const double L = (double)((1 << (a.bits - 1)) - 1);
    for (long long first = 0; first < pairs; first += (long long)gridDim.x * kThreads) {
      const int found = quant_marked_pairs(a, first, pairs, s_list, &s_count);
      for (int f = 0; f < found; ++f) {
        const long long w = first + s_list[f];
        const int i = (int)(w / a.tt.n_tiles), tile = (int)(w % a.tt.n_tiles);
        if (!tile_ok(a.tt, tile, a.T, a.stride, kNormTile)) continue;  // bounds-checked build only
        const int t = a.tt.tensor[tile];
        const long long s = (long long)i * a.T + t;
        const uint8_t kind = a.quant[s];
        if (a.sparse && a.sparse[s]) continue;      // a Top-K message: delivered by the Top-K packing kernel
        const int len = a.tt.length[tile];
        const long long base = (long long)i * a.stride + a.tt.offset[tile];
        const int E = a.qexp[s];
        const double up = pow2_double(E), down = pow2_double(-E);
        constexpr int kIter = kNormTile / (kThreads * 4);
        float4 xq[kIter], hq[kIter];
#pragma unroll
        for (int q = 0; q < kIter; ++q) {       // all eight loads of the tile before the first use
            const int local = (q * kThreads + threadIdx.x) * 4;
            if (local < len) {
                xq[q] = ld_stream(a.x + base + local);
                hq[q] = *reinterpret_cast<const float4*>(a.xhat + base + local);
            } else {
                xq[q] = hq[q] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
#pragma unroll
        for (int q = 0; q < kIter; ++q) {
            const int local = (q * kThreads + threadIdx.x) * 4;
            if (local >= len) continue;
            const float4 xv = xq[q];
            float4 hv = hq[q];
            const int nel = min(4, len - local);
            if (kind == kQuantFull) {
                hv = xv;
            } else {
                const float xs[4] = {xv.x, xv.y, xv.z, xv.w};
                float hs[4] = {hv.x, hv.y, hv.z, hv.w};
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const float d = __fsub_rn(xs[c], hs[c]);
                    double q = rint(__dmul_rn((double)d, down));         // exact scaling, ties to even
                    q = fmin(fmax(q, -L), L);
                    hs[c] = __double2float_rn(__dadd_rn((double)hs[c], __dmul_rn(q, up)));
                }
                hv = make_float4(hs[0], hs[1], hs[2], hs[3]);
            }
            float* out = a.xhat + base + local;
            if (nel == 4) {
                *reinterpret_cast<float4*>(out) = hv;
            } else {
                if (nel > 0) out[0] = hv.x;
                if (nel > 1) out[1] = hv.y;
                if (nel > 2) out[2] = hv.z;
            }
        }
      }
    }
}

}  // namespace eg
