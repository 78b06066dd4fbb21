// Top-K messages (Top-K paragraph of Section 7): for every segment whose event sends a
// sparse message, find exactly the K_t entries with the largest |x - x_hat| (ties to the lower
// index), pack them as (index, value) in ascending index order into the replica's outbox,
// and scatter them into the mailbox x_hat "on receipt".
//
// The rank key is the bit pattern of |x - x_hat| (fp32), which orders like the magnitude.
// Radix select over three digits (11 + 10 + 10 bits) gives the K_t-th largest key tau and
// the number of entries equal to tau that still belong to the message; an ordered
// compaction (per-tile counts -> exclusive scan -> write) then emits the message.
// Every kernel tests the per-segment `sparse` flag on the device and returns at once for
// segments without a sparse message, so the host never looks at a decision.
#pragma once
#include "eg_common.cuh"

namespace eg {

struct TopkState {
    unsigned int* hist;        // [P*T][kMaxBins]
    unsigned int* prefix;      // [P*T] key bits resolved so far (after the last digit: tau)
    unsigned int* remaining;   // [P*T] rank still to resolve (after the last digit: number of
                               //       entries equal to tau that are part of the message)
    uint2* tile_count;         // [P][n_tiles] (greater, equal) per tile, then their prefixes
    int2* outbox;              // [P][sum K_t] (index, value bits)
    const long long* out_off;  // [T] start of tensor t inside one replica's outbox
    const long long* count;    // [T] K_t
    long long out_stride;      // sum K_t
};

__device__ __forceinline__ unsigned int rank_key(float a, float b) {
    return __float_as_uint(__fsub_rn(a, b)) & 0x7fffffffu;
}

// digit 0: bits 30..20, digit 1: bits 19..10, digit 2: bits 9..0
__device__ __forceinline__ int digit_shift(int digit) { return digit == 0 ? 20 : (digit == 1 ? 10 : 0); }
__device__ __forceinline__ int digit_bits(int digit) { return digit == 0 ? kDigitBits0 : kDigitBits1; }

// grid (n_tiles, P): histogram of one digit over the keys that match the resolved prefix.
__global__ void __launch_bounds__(kThreads)
k_topk_hist(const float* __restrict__ x, const float* __restrict__ xhat, TileTable tt, int T,
            long long stride, const uint8_t* __restrict__ sparse, TopkState tk, int digit) {
    const int tile = blockIdx.x, i = blockIdx.y;
    const int t = tt.tensor[tile];
    const long long s = (long long)i * T + t;
    if (!sparse[s]) return;
    __shared__ unsigned int s_hist[kMaxBins];
    const int nbins = 1 << digit_bits(digit);
    for (int b = threadIdx.x; b < nbins; b += kThreads) s_hist[b] = 0;
    __syncthreads();
    const int len = tt.length[tile];
    const long long base = (long long)i * stride + tt.offset[tile];
    const int shift = digit_shift(digit);
    const int hi_shift = shift + digit_bits(digit);       // bits above this digit
    const unsigned int want = (digit == 0) ? 0u : tk.prefix[s];
    for (int local = threadIdx.x * 4; local < len; local += kThreads * 4) {
        const float4 a = ld_stream(x + base + local), b = ld_stream(xhat + base + local);
        const unsigned int k[4] = {rank_key(a.x, b.x), rank_key(a.y, b.y), rank_key(a.z, b.z),
                                   rank_key(a.w, b.w)};
        const int nel = min(4, len - local);
#pragma unroll
        for (int c = 0; c < 4; ++c)
            if (c < nel && (digit == 0 || (k[c] >> hi_shift) == want))
                atomicAdd(&s_hist[(k[c] >> shift) & (nbins - 1)], 1u);
    }
    __syncthreads();
    unsigned int* gh = tk.hist + s * kMaxBins;
    for (int b = threadIdx.x; b < nbins; b += kThreads)
        if (s_hist[b]) atomicAdd(&gh[b], s_hist[b]);
}

// grid P*T, one CTA per segment: pick the bin that holds the wanted rank, counting from the
// largest key downwards; clear the histogram for the next digit.
__global__ void __launch_bounds__(kThreads)
k_topk_pick(int T, const uint8_t* __restrict__ sparse, TopkState tk, int digit) {
    const long long s = blockIdx.x;
    if (!sparse[s]) return;
    const int t = (int)(s % T);
    __shared__ unsigned int s_sum[kThreads];
    __shared__ unsigned int s_above[kThreads];
    const int nbins = 1 << digit_bits(digit);
    const int per = nbins / kThreads;                      // 8 or 4 bins per thread
    unsigned int* gh = tk.hist + s * kMaxBins;
    // thread 0 owns the highest bins
    const int top = nbins - 1 - threadIdx.x * per;
    unsigned int c[8];
    unsigned int mine = 0;
    for (int q = 0; q < per; ++q) { c[q] = gh[top - q]; mine += c[q]; }
    s_sum[threadIdx.x] = mine;
    __syncthreads();
    if (threadIdx.x == 0) {                                // 256 adds: exclusive scan from the top
        unsigned int run = 0;
        for (int q = 0; q < kThreads; ++q) { s_above[q] = run; run += s_sum[q]; }
    }
    __syncthreads();
    const unsigned int rem = (digit == 0) ? (unsigned int)tk.count[t] : tk.remaining[s];
    unsigned int above = s_above[threadIdx.x];
    if (above < rem && rem <= above + mine) {
        for (int q = 0; q < per; ++q) {
            if (rem <= above + c[q]) {
                const unsigned int old = (digit == 0) ? 0u : tk.prefix[s];
                tk.prefix[s] = (old << digit_bits(digit)) | (unsigned int)(top - q);
                tk.remaining[s] = rem - above;
                break;
            }
            above += c[q];
        }
    }
    for (int q = 0; q < per; ++q) gh[top - q] = 0;
}

// grid (n_tiles, P): per tile, how many keys are greater than / equal to tau.
__global__ void __launch_bounds__(kThreads)
k_topk_count(const float* __restrict__ x, const float* __restrict__ xhat, TileTable tt, int T,
             long long stride, const uint8_t* __restrict__ sparse, TopkState tk) {
    const int tile = blockIdx.x, i = blockIdx.y;
    const int t = tt.tensor[tile];
    const long long s = (long long)i * T + t;
    if (!sparse[s]) return;
    const unsigned int tau = tk.prefix[s];
    const int len = tt.length[tile];
    const long long base = (long long)i * stride + tt.offset[tile];
    unsigned int gt = 0, eq = 0;
    for (int local = threadIdx.x * 4; local < len; local += kThreads * 4) {
        const float4 a = ld_stream(x + base + local), b = ld_stream(xhat + base + local);
        const unsigned int k[4] = {rank_key(a.x, b.x), rank_key(a.y, b.y), rank_key(a.z, b.z),
                                   rank_key(a.w, b.w)};
        const int nel = min(4, len - local);
#pragma unroll
        for (int c = 0; c < 4; ++c)
            if (c < nel) { gt += (k[c] > tau); eq += (k[c] == tau); }
    }
    __shared__ unsigned int s_gt[kWarps], s_eq[kWarps];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        gt += __shfl_down_sync(0xffffffffu, gt, o);
        eq += __shfl_down_sync(0xffffffffu, eq, o);
    }
    if ((threadIdx.x & 31) == 0) { s_gt[threadIdx.x >> 5] = gt; s_eq[threadIdx.x >> 5] = eq; }
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned int a = 0, b = 0;
        for (int w = 0; w < kWarps; ++w) { a += s_gt[w]; b += s_eq[w]; }
        tk.tile_count[(long long)i * tt.n_tiles + tile] = make_uint2(a, b);
    }
}

// grid P*T, one CTA per segment: exclusive prefix of the tile counts, in tile order.
__global__ void __launch_bounds__(kThreads)
k_topk_scan(TileTable tt, int T, const uint8_t* __restrict__ sparse, TopkState tk) {
    const long long s = blockIdx.x;
    if (!sparse[s]) return;
    const int i = (int)(s / T), t = (int)(s % T);
    const int q0 = tt.seg_begin[t], q1 = tt.seg_begin[t + 1];
    uint2* tc = tk.tile_count + (long long)i * tt.n_tiles;
    __shared__ unsigned int s_gt[kThreads], s_eq[kThreads];
    __shared__ unsigned int s_run[2];
    if (threadIdx.x == 0) s_run[0] = s_run[1] = 0;
    __syncthreads();
    for (int c0 = q0; c0 < q1; c0 += kThreads) {
        const int q = c0 + threadIdx.x;
        uint2 v = make_uint2(0, 0);
        if (q < q1) v = tc[q];
        s_gt[threadIdx.x] = v.x;
        s_eq[threadIdx.x] = v.y;
        __syncthreads();
        if (threadIdx.x == 0) {
            unsigned int a = s_run[0], b = s_run[1];
            for (int z = 0; z < kThreads; ++z) {
                const unsigned int ga = s_gt[z], gb = s_eq[z];
                s_gt[z] = a; s_eq[z] = b;
                a += ga; b += gb;
            }
            s_run[0] = a; s_run[1] = b;
        }
        __syncthreads();
        if (q < q1) tc[q] = make_uint2(s_gt[threadIdx.x], s_eq[threadIdx.x]);
        __syncthreads();
    }
}

// grid (n_tiles, P): ordered compaction of the selected entries of one tile into the outbox.
// An entry is selected if key > tau, or key == tau and fewer than `remaining` equal keys
// precede it in the tensor.  Its slot is (#greater before it) + min(#equal before it, remaining).
__global__ void __launch_bounds__(kThreads)
k_topk_write(const float* __restrict__ x, const float* __restrict__ xhat, TileTable tt, int T,
             long long stride, const uint8_t* __restrict__ sparse, TopkState tk,
             unsigned int* __restrict__ err) {
    const int tile = blockIdx.x, i = blockIdx.y;
    const int t = tt.tensor[tile];
    const long long s = (long long)i * T + t;
    if (!sparse[s]) return;
    const unsigned int tau = tk.prefix[s], take = tk.remaining[s];
    const int len = tt.length[tile];
    const long long base = (long long)i * stride + tt.offset[tile];
    const int first = (int)(tt.offset[tile] - tt.offset[tt.seg_begin[t]]);  // index of the tile's first element
    const uint2 before = tk.tile_count[(long long)i * tt.n_tiles + tile];
    const long long K = tk.count[t];
    int2* out = tk.outbox + (long long)i * tk.out_stride + tk.out_off[t];
    __shared__ unsigned int s_gt[kWarps], s_eq[kWarps];
    unsigned int run_gt = before.x, run_eq = before.y;       // entries before this chunk
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int c0 = 0; c0 < len; c0 += kThreads * 4) {
        const int local = c0 + threadIdx.x * 4;
        unsigned int k[4] = {0, 0, 0, 0};
        float xv[4] = {0.f, 0.f, 0.f, 0.f};
        int nel = 0;
        if (local < len) {
            const float4 a = ld_stream(x + base + local), b = ld_stream(xhat + base + local);
            k[0] = rank_key(a.x, b.x); k[1] = rank_key(a.y, b.y);
            k[2] = rank_key(a.z, b.z); k[3] = rank_key(a.w, b.w);
            xv[0] = a.x; xv[1] = a.y; xv[2] = a.z; xv[3] = a.w;
            nel = min(4, len - local);
        }
        unsigned int gt = 0, eq = 0;
#pragma unroll
        for (int c = 0; c < 4; ++c)
            if (c < nel) { gt += (k[c] > tau); eq += (k[c] == tau); }
        // exclusive scan over the CTA in thread order (= index order)
        unsigned int sgt = gt, seq = eq;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned int a = __shfl_up_sync(0xffffffffu, sgt, o);
            const unsigned int b = __shfl_up_sync(0xffffffffu, seq, o);
            if (lane >= o) { sgt += a; seq += b; }
        }
        if (lane == 31) { s_gt[warp] = sgt; s_eq[warp] = seq; }
        __syncthreads();
        unsigned int wgt = 0, weq = 0, tot_gt = 0, tot_eq = 0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            if (w < warp) { wgt += s_gt[w]; weq += s_eq[w]; }
            tot_gt += s_gt[w]; tot_eq += s_eq[w];
        }
        unsigned int my_gt = run_gt + wgt + sgt - gt;         // greater keys before my first entry
        unsigned int my_eq = run_eq + weq + seq - eq;         // equal keys before my first entry
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            if (c < nel) {
                const bool is_gt = k[c] > tau, is_eq = k[c] == tau;
                if (is_gt || (is_eq && my_eq < take)) {
                    const long long slot = (long long)my_gt + (long long)min(my_eq, take);
                    if (slot < K) out[slot] = make_int2(first + local + c, __float_as_int(xv[c]));
                    else atomicOr(err, 2u);
                }
                my_gt += is_gt; my_eq += is_eq;
            }
        }
        run_gt += tot_gt; run_eq += tot_eq;
        __syncthreads();
    }
}

// grid (n_tiles, P): the receiver's side — write the received values into the mailbox.
// CTA `tile` of a tensor handles outbox entries [rank*kNormTile, (rank+1)*kNormTile) where
// rank is the tile's position inside its tensor (K_t <= n_t, so the tiles cover the outbox).
__global__ void __launch_bounds__(kThreads)
k_topk_scatter(float* __restrict__ xhat, TileTable tt, int T, long long stride,
               const uint8_t* __restrict__ sparse, TopkState tk, const long long* __restrict__ numel,
               unsigned int* __restrict__ err) {
    const int tile = blockIdx.x, i = blockIdx.y;
    const int t = tt.tensor[tile];
    const long long s = (long long)i * T + t;
    if (!sparse[s]) return;
    const long long K = tk.count[t];
    const long long lo = (long long)(tile - tt.seg_begin[t]) * kNormTile;
    if (lo >= K) return;
    const long long hi = min(K, lo + kNormTile);
    const int2* in = tk.outbox + (long long)i * tk.out_stride + tk.out_off[t];
    float* dst = xhat + (long long)i * stride + tt.offset[tt.seg_begin[t]];
    const long long n = numel[t];
    for (long long q = lo + threadIdx.x; q < hi; q += kThreads) {
        const int2 m = in[q];
        if (m.x >= 0 && m.x < n) dst[m.x] = __int_as_float(m.y);
        else atomicOr(err, 4u);
    }
}

}  // namespace eg
