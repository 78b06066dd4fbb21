// Top-K messages (Top-K paragraph of Section 7): for every segment whose event sends a
// sparse message, find exactly the K_t entries with the largest |x - x_hat| (ties to the lower
// index), pack them as (index, value) in ascending index order into the replica's outbox,
// and scatter them into the mailbox x_hat "on receipt".
//
// The rank key is the bit pattern of |x - x_hat| (fp32), which orders like the magnitude.
// The K_t-th largest key tau is found by radix select over three digits (11 + 10 + 10 bits):
//   pass A  (reads x, x_hat)  histogram of the top digit                     -> bin b0
//   pass B  (reads x, x_hat)  keys whose top digit is b0 ("candidates") are copied, tile by
//                             tile, into a candidate buffer; keys above b0 are counted per tile
//   digits 1 and 2            histograms over the candidates only (a few percent of the data)
//   per-tile counts           from the candidates only
//   pass C  (reads x, x_hat)  ordered compaction into the outbox
// so a sparse message costs three passes over its tensor.  The host knows nothing about the
// decisions: a one-CTA planning kernel turns the device-side `sparse` flags into a compact list
// of work tiles, and every other kernel runs a fixed-size grid over that list (an empty list
// costs a few microseconds per launch).
#pragma once
#include "eg_common.cuh"

namespace eg {

constexpr int kTopkGrid = 148 * 8;      // CTAs of the tile kernels (they loop over the work list)
constexpr int kTopkSegGrid = 148 * 4;   // CTAs of the per-segment kernels
constexpr int kPlanThreads = 1024;

struct TopkPlan {
    int n_sparse;       // segments that send a sparse message in this step
    int total_tiles;    // their tiles
};

struct TopkState {
    TopkPlan* plan;
    int* sp_seg;               // [P*T] segment id of the q-th sparse segment
    int* sp_begin;             // [P*T+1] first work tile of the q-th sparse segment
    unsigned int* hist;        // [P*T][kMaxBins]
    unsigned int* prefix;      // [P*T] key bits resolved so far (after the last digit: tau)
    unsigned int* remaining;   // [P*T] rank still to resolve (after the last digit: number of
                               //       entries equal to tau that are part of the message)
    unsigned int* cand;        // [P][stride] candidate keys of a tile, at the tile's own offset
    int* tile_cand;            // [P][n_tiles] candidates stored for the tile
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

// One CTA: compact list of the sparse segments and of their tiles, in segment order.
__global__ void __launch_bounds__(kPlanThreads)
k_topk_plan(int S, int T, const uint8_t* __restrict__ sparse, const int* __restrict__ seg_begin,
            TopkState tk) {
    __shared__ int s_cnt[kPlanThreads], s_tiles[kPlanThreads];
    const int per = (S + kPlanThreads - 1) / kPlanThreads;
    const int lo = threadIdx.x * per, hi = min(S, lo + per);
    int cnt = 0, tiles = 0;
    for (int s = lo; s < hi; ++s)
        if (sparse[s]) { const int t = s % T; ++cnt; tiles += seg_begin[t + 1] - seg_begin[t]; }
    s_cnt[threadIdx.x] = cnt;
    s_tiles[threadIdx.x] = tiles;
    __syncthreads();
    // inclusive scan (Hillis-Steele) over the 1024 per-thread totals
    for (int o = 1; o < kPlanThreads; o <<= 1) {
        int a = 0, b = 0;
        if (threadIdx.x >= o) { a = s_cnt[threadIdx.x - o]; b = s_tiles[threadIdx.x - o]; }
        __syncthreads();
        s_cnt[threadIdx.x] += a;
        s_tiles[threadIdx.x] += b;
        __syncthreads();
    }
    int q = s_cnt[threadIdx.x] - cnt, w = s_tiles[threadIdx.x] - tiles;
    for (int s = lo; s < hi; ++s)
        if (sparse[s]) {
            const int t = s % T;
            tk.sp_seg[q] = s;
            tk.sp_begin[q] = w;
            ++q;
            w += seg_begin[t + 1] - seg_begin[t];
        }
    if (threadIdx.x == kPlanThreads - 1) {
        tk.plan->n_sparse = s_cnt[threadIdx.x];
        tk.plan->total_tiles = s_tiles[threadIdx.x];
        tk.sp_begin[s_cnt[threadIdx.x]] = s_tiles[threadIdx.x];
    }
}

// Contiguous share of the work-tile list for this CTA and the sparse slot of its first tile.
struct WorkRange {
    int w0, w1, q;
};
__device__ __forceinline__ WorkRange work_range(const TopkState& tk) {
    const int total = tk.plan->total_tiles, nq = tk.plan->n_sparse;
    const int chunk = (total + (int)gridDim.x - 1) / (int)gridDim.x;
    WorkRange r;
    r.w0 = min(total, (int)blockIdx.x * chunk);
    r.w1 = min(total, r.w0 + chunk);
    int lo = 0, hi = max(nq - 1, 0);            // last q with sp_begin[q] <= w0
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (tk.sp_begin[mid] <= r.w0) lo = mid; else hi = mid - 1;
    }
    r.q = lo;
    return r;
}

// Pass A and the two candidate passes: histogram of one digit.
// CANDIDATES == false: over the keys of the tile (digit 0).
// CANDIDATES == true : over the candidate keys of the tile that match the resolved prefix.
template <bool CANDIDATES>
__global__ void __launch_bounds__(kThreads)
k_topk_hist(const float* __restrict__ x, const float* __restrict__ xhat, TileTable tt, int T,
            long long stride, TopkState tk, int digit) {
    __shared__ unsigned int s_hist[kMaxBins];
    WorkRange r = work_range(tk);
    if (r.w0 >= r.w1) return;
    const int nbins = 1 << digit_bits(digit);
    const int shift = digit_shift(digit);
    const int hi_shift = shift + digit_bits(digit);
    for (int b = threadIdx.x; b < nbins; b += kThreads) s_hist[b] = 0;
    __syncthreads();
    int q = r.q;
    for (int w = r.w0; w < r.w1; ++w) {
        while (w >= tk.sp_begin[q + 1]) ++q;
        const int s = tk.sp_seg[q];
        const int i = s / T, t = s - i * T;
        const int tile = tt.seg_begin[t] + (w - tk.sp_begin[q]);
        if (!CANDIDATES) {
            const int len = tt.length[tile];
            const long long base = (long long)i * stride + tt.offset[tile];
            for (int local = threadIdx.x * 4; local < len; local += kThreads * 4) {
                const float4 a = ld_stream(x + base + local), b = ld_stream(xhat + base + local);
                const unsigned int k[4] = {rank_key(a.x, b.x), rank_key(a.y, b.y), rank_key(a.z, b.z),
                                           rank_key(a.w, b.w)};
                const int nel = min(4, len - local);
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (c < nel) atomicAdd(&s_hist[(k[c] >> shift) & (nbins - 1)], 1u);
            }
        } else {
            const unsigned int want = tk.prefix[s];
            const unsigned int* cd = tk.cand + (long long)i * stride + tt.offset[tile];
            const int n = tk.tile_cand[(long long)i * tt.n_tiles + tile];
            for (int e = threadIdx.x; e < n; e += kThreads) {
                const unsigned int k = cd[e];
                if ((k >> hi_shift) == want) atomicAdd(&s_hist[(k >> shift) & (nbins - 1)], 1u);
            }
        }
        // flush when the next tile belongs to another segment (or this was the last one)
        if (w + 1 == r.w1 || w + 1 >= tk.sp_begin[q + 1]) {
            __syncthreads();
            unsigned int* gh = tk.hist + (long long)s * kMaxBins;
            for (int b = threadIdx.x; b < nbins; b += kThreads) {
                const unsigned int v = s_hist[b];
                if (v) { atomicAdd(&gh[b], v); s_hist[b] = 0; }
            }
            __syncthreads();
        }
    }
}

// One CTA per sparse segment: pick the bin that holds the wanted rank, counting from the
// largest key downwards; clear the histogram for the next digit.
__global__ void __launch_bounds__(kThreads)
k_topk_pick(int T, TopkState tk, int digit) {
    __shared__ unsigned int s_sum[kThreads];
    __shared__ unsigned int s_above[kThreads];
    const int nq = tk.plan->n_sparse;
    const int nbins = 1 << digit_bits(digit);
    const int per = nbins / kThreads;                      // 8 or 4 bins per thread
    for (int q = blockIdx.x; q < nq; q += gridDim.x) {
        const int s = tk.sp_seg[q];
        const int t = s % T;
        unsigned int* gh = tk.hist + (long long)s * kMaxBins;
        const int top = nbins - 1 - threadIdx.x * per;     // thread 0 owns the highest bins
        unsigned int c[8];
        unsigned int mine = 0;
        for (int z = 0; z < per; ++z) { c[z] = gh[top - z]; mine += c[z]; gh[top - z] = 0; }
        s_sum[threadIdx.x] = mine;
        __syncthreads();
        if (threadIdx.x == 0) {                            // exclusive scan from the top
            unsigned int run = 0;
            for (int z = 0; z < kThreads; ++z) { s_above[z] = run; run += s_sum[z]; }
        }
        __syncthreads();
        const unsigned int rem = (digit == 0) ? (unsigned int)tk.count[t] : tk.remaining[s];
        unsigned int above = s_above[threadIdx.x];
        if (above < rem && rem <= above + mine) {
            for (int z = 0; z < per; ++z) {
                if (rem <= above + c[z]) {
                    const unsigned int old = (digit == 0) ? 0u : tk.prefix[s];
                    tk.prefix[s] = (old << digit_bits(digit)) | (unsigned int)(top - z);
                    tk.remaining[s] = rem - above;
                    break;
                }
                above += c[z];
            }
        }
        __syncthreads();
    }
}

// Pass B: per tile, copy the keys whose top digit equals the chosen bin into the tile's slice
// of the candidate buffer (order inside the tile is irrelevant for selecting tau) and count the
// keys whose top digit is larger.
__global__ void __launch_bounds__(kThreads)
k_topk_collect(const float* __restrict__ x, const float* __restrict__ xhat, TileTable tt, int T,
               long long stride, TopkState tk) {
    __shared__ unsigned int s_n, s_gt;
    WorkRange r = work_range(tk);
    int q = r.q;
    for (int w = r.w0; w < r.w1; ++w) {
        while (w >= tk.sp_begin[q + 1]) ++q;
        const int s = tk.sp_seg[q];
        const int i = s / T, t = s - i * T;
        const int tile = tt.seg_begin[t] + (w - tk.sp_begin[q]);
        const unsigned int b0 = tk.prefix[s];
        const int len = tt.length[tile];
        const long long base = (long long)i * stride + tt.offset[tile];
        unsigned int* cd = tk.cand + base;
        if (threadIdx.x == 0) { s_n = 0; s_gt = 0; }
        __syncthreads();
        unsigned int gt = 0;
        for (int local = threadIdx.x * 4; local < len; local += kThreads * 4) {
            const float4 a = ld_stream(x + base + local), b = ld_stream(xhat + base + local);
            const unsigned int k[4] = {rank_key(a.x, b.x), rank_key(a.y, b.y), rank_key(a.z, b.z),
                                       rank_key(a.w, b.w)};
            const int nel = min(4, len - local);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                if (c < nel) {
                    const unsigned int d0 = k[c] >> 20;
                    gt += (d0 > b0);
                    if (d0 == b0) cd[atomicAdd(&s_n, 1u)] = k[c];
                }
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) gt += __shfl_down_sync(0xffffffffu, gt, o);
        if ((threadIdx.x & 31) == 0 && gt) atomicAdd(&s_gt, gt);
        __syncthreads();
        if (threadIdx.x == 0) {
            tk.tile_cand[(long long)i * tt.n_tiles + tile] = (int)s_n;
            tk.tile_count[(long long)i * tt.n_tiles + tile] = make_uint2(s_gt, 0u);
        }
        __syncthreads();
    }
}

// Per tile, from its candidates only: keys greater than / equal to tau.
__global__ void __launch_bounds__(kThreads)
k_topk_count(TileTable tt, int T, long long stride, TopkState tk) {
    __shared__ unsigned int s_gt, s_eq;
    WorkRange r = work_range(tk);
    int q = r.q;
    for (int w = r.w0; w < r.w1; ++w) {
        while (w >= tk.sp_begin[q + 1]) ++q;
        const int s = tk.sp_seg[q];
        const int i = s / T, t = s - i * T;
        const int tile = tt.seg_begin[t] + (w - tk.sp_begin[q]);
        const unsigned int tau = tk.prefix[s];
        const unsigned int* cd = tk.cand + (long long)i * stride + tt.offset[tile];
        const int n = tk.tile_cand[(long long)i * tt.n_tiles + tile];
        if (threadIdx.x == 0) { s_gt = 0; s_eq = 0; }
        __syncthreads();
        unsigned int gt = 0, eq = 0;
        for (int e = threadIdx.x; e < n; e += kThreads) {
            const unsigned int k = cd[e];
            gt += (k > tau);
            eq += (k == tau);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            gt += __shfl_down_sync(0xffffffffu, gt, o);
            eq += __shfl_down_sync(0xffffffffu, eq, o);
        }
        if ((threadIdx.x & 31) == 0) {
            if (gt) atomicAdd(&s_gt, gt);
            if (eq) atomicAdd(&s_eq, eq);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            uint2* tc = tk.tile_count + (long long)i * tt.n_tiles + tile;
            *tc = make_uint2(tc->x + s_gt, s_eq);
        }
        __syncthreads();
    }
}

// One CTA per sparse segment: exclusive prefix of the tile counts, in tile order.
__global__ void __launch_bounds__(kThreads)
k_topk_scan(TileTable tt, int T, TopkState tk) {
    __shared__ unsigned int s_gt[kThreads], s_eq[kThreads];
    __shared__ unsigned int s_run[2];
    const int nq = tk.plan->n_sparse;
    for (int q = blockIdx.x; q < nq; q += gridDim.x) {
        const int s = tk.sp_seg[q];
        const int i = s / T, t = s - i * T;
        const int q0 = tt.seg_begin[t], q1 = tt.seg_begin[t + 1];
        uint2* tc = tk.tile_count + (long long)i * tt.n_tiles;
        if (threadIdx.x == 0) s_run[0] = s_run[1] = 0;
        __syncthreads();
        for (int c0 = q0; c0 < q1; c0 += kThreads) {
            const int z = c0 + threadIdx.x;
            uint2 v = make_uint2(0, 0);
            if (z < q1) v = tc[z];
            // inclusive scan over the chunk, in tile order
            unsigned int a = v.x, b = v.y;
            const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned int pa = __shfl_up_sync(0xffffffffu, a, o);
                const unsigned int pb = __shfl_up_sync(0xffffffffu, b, o);
                if (lane >= o) { a += pa; b += pb; }
            }
            if (lane == 31) { s_gt[warp] = a; s_eq[warp] = b; }
            __syncthreads();
            unsigned int wa = 0, wb = 0, ta = 0, tb = 0;
#pragma unroll
            for (int u = 0; u < kWarps; ++u) {
                if (u < warp) { wa += s_gt[u]; wb += s_eq[u]; }
                ta += s_gt[u]; tb += s_eq[u];
            }
            if (z < q1) tc[z] = make_uint2(s_run[0] + wa + a - v.x, s_run[1] + wb + b - v.y);
            __syncthreads();
            if (threadIdx.x == 0) { s_run[0] += ta; s_run[1] += tb; }
            __syncthreads();
        }
    }
}

// Pass C: ordered compaction of the selected entries of one tile into the outbox.
// An entry is selected if key > tau, or key == tau and fewer than `remaining` equal keys
// precede it in the tensor.  Its slot is (#greater before it) + min(#equal before it, remaining).
__global__ void __launch_bounds__(kThreads)
k_topk_write(const float* __restrict__ x, const float* __restrict__ xhat, TileTable tt, int T,
             long long stride, TopkState tk, unsigned int* __restrict__ err) {
    __shared__ unsigned int s_gt[kWarps], s_eq[kWarps];
    WorkRange r = work_range(tk);
    int q = r.q;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int w = r.w0; w < r.w1; ++w) {
        while (w >= tk.sp_begin[q + 1]) ++q;
        const int s = tk.sp_seg[q];
        const int i = s / T, t = s - i * T;
        const int tile = tt.seg_begin[t] + (w - tk.sp_begin[q]);
        const unsigned int tau = tk.prefix[s], take = tk.remaining[s];
        const int len = tt.length[tile];
        const long long base = (long long)i * stride + tt.offset[tile];
        const int first = (int)(tt.offset[tile] - tt.offset[tt.seg_begin[t]]);  // index of the tile's first element
        const uint2 before = tk.tile_count[(long long)i * tt.n_tiles + tile];
        const long long K = tk.count[t];
        int2* out = tk.outbox + (long long)i * tk.out_stride + tk.out_off[t];
        unsigned int run_gt = before.x, run_eq = before.y;       // entries before this chunk
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
            for (int u = 0; u < kWarps; ++u) {
                if (u < warp) { wgt += s_gt[u]; weq += s_eq[u]; }
                tot_gt += s_gt[u]; tot_eq += s_eq[u];
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
}

// The receiver's side: write the received values into the mailbox.  Work tile number r of a
// tensor handles outbox entries [r*kNormTile, (r+1)*kNormTile) (K_t <= n_t, so the tensor's
// tiles cover its outbox).
__global__ void __launch_bounds__(kThreads)
k_topk_scatter(float* __restrict__ xhat, TileTable tt, int T, long long stride, TopkState tk,
               const long long* __restrict__ numel, unsigned int* __restrict__ err) {
    WorkRange r = work_range(tk);
    int q = r.q;
    for (int w = r.w0; w < r.w1; ++w) {
        while (w >= tk.sp_begin[q + 1]) ++q;
        const int s = tk.sp_seg[q];
        const int i = s / T, t = s - i * T;
        const long long K = tk.count[t];
        const long long lo = (long long)(w - tk.sp_begin[q]) * kNormTile;
        if (lo >= K) continue;
        const long long hi = min(K, lo + kNormTile);
        const int2* in = tk.outbox + (long long)i * tk.out_stride + tk.out_off[t];
        float* dst = xhat + (long long)i * stride + tt.offset[tt.seg_begin[t]];
        const long long n = numel[t];
        for (long long e = lo + threadIdx.x; e < hi; e += kThreads) {
            const int2 m = in[e];
            if (m.x >= 0 && m.x < n) dst[m.x] = __int_as_float(m.y);
            else atomicOr(err, 4u);
        }
    }
}

}  // namespace eg
