// Top-K messages (Top-K paragraph of Section 7): for every segment whose event sends a
// sparse message, find exactly the K_t entries with the largest |x - x_hat| (ties to the lower
// index), pack them as (index, value) in ascending index order into the replica's outbox,
// and deliver them into the mailbox x_hat.
//
// The rank key is the bit pattern of |x - x_hat| (fp32), which orders like the magnitude.
// The K_t-th largest key tau is found by radix select over three digits (11 + 10 + 10 bits):
//   pass A  (reads x, x_hat)  histogram of the top digit                     -> bin b0
//   pass B  (reads x, x_hat)  keys whose top digit is b0 ("candidates") are copied, tile by
//                             tile, into a candidate buffer; keys above b0 are counted per tile;
//                             digit 1 of the candidates is histogrammed on the way
//   digit 2, per-tile counts  from the candidates only (a few percent of the data)
//   pass C  (reads x, x_hat)  ordered compaction into the outbox and delivery into x_hat
// so a sparse message costs three passes over its tensor.  The host knows nothing about the
// decisions: a planning phase turns the device-side `sparse` flags into a compact list of work
// tiles and every other phase runs a fixed-size grid over that list.  All phases run in one
// cooperative launch (k_topk_all, bottom of this file).
#pragma once
#include <cooperative_groups.h>

#include "eg_common.cuh"

namespace eg {

constexpr int kTopkGrid = 148 * 8;      // CTAs of the tile kernels (they loop over the work list)
constexpr int kTopkSegGrid = 148 * 4;   // CTAs of the per-segment kernels

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
    int* tile_cand;            // [P][n_tiles][8] candidates stored by each warp for the tile
    unsigned int* tile_gt;     // [P][n_tiles][8] keys above the chosen bin seen by each warp
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
__device__ __forceinline__ int digit_bits(int digit) { return digit == 0 ? kDigitBits0 : kDigitBits1; }

// One CTA (of kThreads threads): compact list of the sparse segments and of their tiles, in
// segment order.
__device__ __forceinline__ void topk_plan(int S, int T, const uint8_t* __restrict__ sparse,
                                          const int* __restrict__ seg_begin, const TopkState& tk) {
    __shared__ int s_cnt[kThreads], s_tiles[kThreads];
    const int per = (S + kThreads - 1) / kThreads;
    const int lo = threadIdx.x * per, hi = min(S, lo + per);
    int cnt = 0, tiles = 0;
    for (int s = lo; s < hi; ++s)
        if (sparse[s]) { const int t = s % T; ++cnt; tiles += seg_begin[t + 1] - seg_begin[t]; }
    s_cnt[threadIdx.x] = cnt;
    s_tiles[threadIdx.x] = tiles;
    __syncthreads();
    // inclusive scan (Hillis-Steele) over the per-thread totals
    for (int o = 1; o < kThreads; o <<= 1) {
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
    if (threadIdx.x == kThreads - 1) {
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

// Walks a CTA's share of the work list.  Segment-level values are re-read only when the
// segment changes, so consecutive tiles of one tensor cost two dependent loads, not six.
struct WorkCursor {
    int q, end, s, i, t, first_tile, begin;
    __device__ __forceinline__ void init(const TopkState& tk, const TileTable& tt, int T, int q0) {
        q = q0 - 1;
        end = -1;
        (void)tk; (void)tt; (void)T;
    }
    // returns the tile id of work item w; `changed` tells whether a new segment started
    __device__ __forceinline__ int advance(const TopkState& tk, const TileTable& tt, int T, int w,
                                           bool& changed) {
        changed = false;
        while (w >= end) {
            ++q;
            begin = tk.sp_begin[q];
            end = tk.sp_begin[q + 1];
            changed = true;
        }
        if (changed) {
            s = tk.sp_seg[q];
            i = s / T;
            t = s - i * T;
            first_tile = tt.seg_begin[t];
        }
        return first_tile + (w - begin);
    }
};

// Pass A: histogram of the top digit of every key of the work tiles.
__device__ __forceinline__ void
topk_hist(const float* __restrict__ x, const float* __restrict__ xhat, TileTable tt, int T,
            long long stride, TopkState tk) {
    __shared__ unsigned int s_hist[kMaxBins];
    WorkRange r = work_range(tk);
    if (r.w0 >= r.w1) return;
    for (int b = threadIdx.x; b < kMaxBins; b += kThreads) s_hist[b] = 0;
    __syncthreads();
    WorkCursor cur;
    cur.init(tk, tt, T, r.q);
    for (int w = r.w0; w < r.w1; ++w) {
        bool changed;
        const int tile = cur.advance(tk, tt, T, w, changed);
        const int len = tt.length[tile];
        const long long base = (long long)cur.i * stride + tt.offset[tile];
        for (int local = threadIdx.x * 4; local < len; local += kThreads * 4) {
            const float4 a = ld_stream(x + base + local), b = ld_stream(xhat + base + local);
            const unsigned int k[4] = {rank_key(a.x, b.x), rank_key(a.y, b.y), rank_key(a.z, b.z),
                                       rank_key(a.w, b.w)};
            const int nel = min(4, len - local);
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (c < nel) atomicAdd(&s_hist[k[c] >> 20], 1u);
        }
        // flush when the next tile belongs to another segment (or this was the last one)
        if (w + 1 == r.w1 || w + 1 >= cur.end) {
            __syncthreads();
            unsigned int* gh = tk.hist + (long long)cur.s * kMaxBins;
            for (int b = threadIdx.x; b < kMaxBins; b += kThreads) {
                const unsigned int v = s_hist[b];
                if (v) { atomicAdd(&gh[b], v); s_hist[b] = 0; }
            }
            __syncthreads();
        }
    }
}

// One CTA per sparse segment: pick the bin that holds the wanted rank, counting from the
// largest key downwards; clear the histogram for the next digit.
__device__ __forceinline__ void
topk_pick(int T, TopkState tk, int digit) {
    __shared__ unsigned int s_warp[kWarps];
    const int nq = tk.plan->n_sparse;
    const int nbins = 1 << digit_bits(digit);
    const int per = nbins / kThreads;                      // 8 or 4 bins per thread
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int q = blockIdx.x; q < nq; q += gridDim.x) {
        const int s = tk.sp_seg[q];
        const int t = s % T;
        unsigned int* gh = tk.hist + (long long)s * kMaxBins;
        const int top = nbins - 1 - threadIdx.x * per;     // thread 0 owns the highest bins
        unsigned int c[8];
        unsigned int mine = 0;
        for (int z = 0; z < per; ++z) { c[z] = gh[top - z]; mine += c[z]; gh[top - z] = 0; }
        // exclusive scan of `mine` over the CTA, from the highest bins down
        unsigned int inc = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned int v = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += v;
        }
        if (lane == 31) s_warp[warp] = inc;
        __syncthreads();
        unsigned int above = inc - mine;
#pragma unroll
        for (int u = 0; u < kWarps; ++u)
            if (u < warp) above += s_warp[u];
        const unsigned int rem = (digit == 0) ? (unsigned int)tk.count[t] : tk.remaining[s];
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

constexpr int kSubSlices = kWarps;                       // candidate sub-slices per tile: one per warp

// Warp w of a CTA owns, in every 1024-element chunk of a tile, the 128 elements starting at
// 128*w.  Its candidate sub-slice starts after the elements owned by the warps before it, so
// the eight sub-slices exactly fill the tile's own slice whatever the tile's length.
__device__ __forceinline__ int sub_offset(int len, int w) {
    int o = 0;
#pragma unroll
    for (int v = 0; v < kNormTile / (kThreads * 4); ++v)
        o += min(max(len - v * kThreads * 4, 0), w * 128);
    return o;
}

// Pass B: per tile, copy the keys whose top digit equals the chosen bin into the candidate
// buffer (order is irrelevant for selecting tau), count the keys whose top digit is larger, and
// histogram digit 1 of the candidates.  Every warp owns 512 elements of the tile and a private
// sub-slice of the tile's candidate slice, so no counter is shared: a thread marks its
// candidates in a 16-bit mask, a warp scan of the counts gives its first slot, and the keys
// are fetched back from shared memory (written and read by the same thread).
__device__ __forceinline__ void
topk_collect(const float* __restrict__ x, const float* __restrict__ xhat, TileTable tt, int T,
               long long stride, TopkState tk) {
    constexpr int kBins1 = 1 << kDigitBits1;
    constexpr int kChunks = kNormTile / (kThreads * 4);
    __shared__ unsigned int s_hist[kBins1];
    __shared__ uint4 s_key[kNormTile / 4];
    WorkRange r = work_range(tk);
    if (r.w0 >= r.w1) return;
    for (int b = threadIdx.x; b < kBins1; b += kThreads) s_hist[b] = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    WorkCursor cur;
    cur.init(tk, tt, T, r.q);
    unsigned int b0 = 0;
    for (int w = r.w0; w < r.w1; ++w) {
        bool changed;
        const int tile = cur.advance(tk, tt, T, w, changed);
        if (changed) b0 = tk.prefix[cur.s];
        const int i = cur.i;
        const int len = tt.length[tile];
        const long long base = (long long)i * stride + tt.offset[tile];
        unsigned int mask = 0, gt = 0;
#pragma unroll
        for (int v = 0; v < kChunks; ++v) {
            const int local = (v * kThreads + threadIdx.x) * 4;
            if (local < len) {
                const float4 a = ld_stream(x + base + local), b = ld_stream(xhat + base + local);
                const uint4 k = make_uint4(rank_key(a.x, b.x), rank_key(a.y, b.y), rank_key(a.z, b.z),
                                           rank_key(a.w, b.w));
                s_key[v * kThreads + threadIdx.x] = k;
                const int nel = len - local;      // >= 1; 4 or more for all but the ragged end
                const unsigned int d[4] = {k.x >> 20, k.y >> 20, k.z >> 20, k.w >> 20};
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const bool live = c < nel;
                    gt += (live && d[c] > b0);
                    mask |= (live && d[c] == b0) ? (1u << (4 * v + c)) : 0u;
                }
            }
        }
        // first slot of this thread inside its warp's sub-slice
        const unsigned int cnt = __popc(mask);
        unsigned int inc = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned int u = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += u;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) gt += __shfl_down_sync(0xffffffffu, gt, o);
        unsigned int* cd = tk.cand + base + sub_offset(len, warp);
        unsigned int pos = inc - cnt;
        const unsigned int* my_keys = reinterpret_cast<const unsigned int*>(s_key);
        while (mask) {
            const int bit = __ffs(mask) - 1;
            mask &= mask - 1;
            const unsigned int key = my_keys[((bit >> 2) * kThreads + threadIdx.x) * 4 + (bit & 3)];
            cd[pos++] = key;
            atomicAdd(&s_hist[(key >> 10) & (kBins1 - 1)], 1u);
        }
        const long long slot = ((long long)i * tt.n_tiles + tile) * kSubSlices + warp;
        if (lane == 31) tk.tile_cand[slot] = (int)inc;          // candidates of this warp
        if (lane == 0) tk.tile_gt[slot] = gt;                   // keys above the bin, this warp
        if (w + 1 == r.w1 || w + 1 >= cur.end) {   // last tile of this segment here
            __syncthreads();
            unsigned int* gh = tk.hist + (long long)cur.s * kMaxBins;
            for (int b = threadIdx.x; b < kBins1; b += kThreads) {
                const unsigned int v = s_hist[b];
                if (v) { atomicAdd(&gh[b], v); s_hist[b] = 0; }
            }
            __syncthreads();
        }
    }
}

// Work tile number w of this step (used by the one-warp-per-tile kernels).
struct WarpTile {
    int s, i, t, tile;
};
__device__ __forceinline__ WarpTile warp_tile(const TopkState& tk, const TileTable& tt, int T, int w) {
    int lo = 0, hi = tk.plan->n_sparse - 1;      // last q with sp_begin[q] <= w
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (tk.sp_begin[mid] <= w) lo = mid; else hi = mid - 1;
    }
    WarpTile r;
    r.s = tk.sp_seg[lo];
    r.i = r.s / T;
    r.t = r.s - r.i * T;
    r.tile = tt.seg_begin[r.t] + (w - tk.sp_begin[lo]);
    return r;
}

// Digit 2 over the candidates: one warp per tile, global histogram updated directly (only the
// candidates that match the 21 resolved bits take part: about one in a thousand).
__device__ __forceinline__ void
topk_hist_cand(TileTable tt, int T, long long stride, TopkState tk) {
    const int total = tk.plan->total_tiles;
    const int lane = threadIdx.x & 31;
    const int nwarps = gridDim.x * kWarps;
    for (int w = blockIdx.x * kWarps + (threadIdx.x >> 5); w < total; w += nwarps) {
        const WarpTile z = warp_tile(tk, tt, T, w);
        const unsigned int want = tk.prefix[z.s];
        const unsigned int* cd = tk.cand + (long long)z.i * stride + tt.offset[z.tile];
        const int* n_sub = tk.tile_cand + ((long long)z.i * tt.n_tiles + z.tile) * kSubSlices;
        const int len = tt.length[z.tile];
        unsigned int* gh = tk.hist + (long long)z.s * kMaxBins;
        for (int sub = 0; sub < kSubSlices; ++sub) {
            const int n = n_sub[sub];
            const unsigned int* cs = cd + sub_offset(len, sub);
            for (int e = lane; e < n; e += 32) {
                const unsigned int k = cs[e];
                if ((k >> 10) == want) atomicAdd(&gh[k & ((1 << kDigitBits2) - 1)], 1u);
            }
        }
    }
}

// Per tile: keys greater than / equal to tau, from the per-warp counts of pass B and the
// tile's candidates.  One warp per tile.
__device__ __forceinline__ void
topk_count(TileTable tt, int T, long long stride, TopkState tk) {
    const int total = tk.plan->total_tiles;
    const int lane = threadIdx.x & 31;
    const int nwarps = gridDim.x * kWarps;
    for (int w = blockIdx.x * kWarps + (threadIdx.x >> 5); w < total; w += nwarps) {
        const WarpTile z = warp_tile(tk, tt, T, w);
        const unsigned int tau = tk.prefix[z.s];
        const unsigned int* cd = tk.cand + (long long)z.i * stride + tt.offset[z.tile];
        const long long slot = ((long long)z.i * tt.n_tiles + z.tile) * kSubSlices;
        const int len = tt.length[z.tile];
        unsigned int gt = (lane < kSubSlices) ? tk.tile_gt[slot + lane] : 0u, eq = 0;
        for (int sub = 0; sub < kSubSlices; ++sub) {
            const int n = tk.tile_cand[slot + sub];
            const unsigned int* cs = cd + sub_offset(len, sub);
            for (int e = lane; e < n; e += 32) {
                const unsigned int k = cs[e];
                gt += (k > tau);
                eq += (k == tau);
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            gt += __shfl_down_sync(0xffffffffu, gt, o);
            eq += __shfl_down_sync(0xffffffffu, eq, o);
        }
        if (lane == 0) tk.tile_count[(long long)z.i * tt.n_tiles + z.tile] = make_uint2(gt, eq);
    }
}

// One CTA per sparse segment: exclusive prefix of the tile counts, in tile order.
__device__ __forceinline__ void
topk_scan(TileTable tt, int T, TopkState tk) {
    __shared__ unsigned int s_gt[kWarps], s_eq[kWarps];
    __shared__ unsigned int s_run[2];
    const int nq = tk.plan->n_sparse;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
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
            unsigned int a = v.x, b = v.y;     // inclusive scan over the chunk, in tile order
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

// Pass C: ordered compaction of the selected entries of one tile into the outbox, and delivery:
// the same (index, value) pairs are written into the mailbox x_hat, which is what the receivers
// hold once the message has arrived.
// An entry is selected if key > tau, or key == tau and fewer than `remaining` equal keys
// precede it in the tensor.  Its slot is (#greater before it) + min(#equal before it, remaining).
// A tile is read as four coalesced chunks of 1024 elements (thread t owns elements 4t..4t+3 of
// every chunk).  A thread records which of its 16 elements are greater / equal in two 16-bit
// masks and parks the x values in shared memory (read back by the same thread); the four
// per-chunk counts travel through ONE scan, packed 16 bits each into a 64-bit word (a chunk
// holds at most 1024 entries, so the fields cannot overflow); then only the marked elements
// are visited.  A thread has read the x_hat entries it owns before it overwrites any of them,
// and no thread touches another thread's entries.
__device__ __forceinline__ void
topk_write(const float* __restrict__ x, float* xhat, TileTable tt, int T, long long stride,
             TopkState tk, unsigned int* __restrict__ err) {
    constexpr int kChunks = kNormTile / (kThreads * 4);   // 4
    static_assert(kChunks == 4, "the packed scan holds four 16-bit fields");
    __shared__ unsigned long long s_pg[kWarps], s_pe[kWarps];
    __shared__ float4 s_val[kNormTile / 4];
    WorkRange r = work_range(tk);
    WorkCursor cur;
    cur.init(tk, tt, T, r.q);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned int tau = 0, take = 0, K = 0;
    int2* out = nullptr;
    for (int w = r.w0; w < r.w1; ++w) {
        bool changed;
        const int tile = cur.advance(tk, tt, T, w, changed);
        if (changed) {
            tau = tk.prefix[cur.s];
            take = tk.remaining[cur.s];
            K = (unsigned int)tk.count[cur.t];
            out = tk.outbox + (long long)cur.i * tk.out_stride + tk.out_off[cur.t];
        }
        const int i = cur.i;
        const int len = tt.length[tile];
        const long long base = (long long)i * stride + tt.offset[tile];
        const int first = (tile - cur.first_tile) * kNormTile;   // index of the tile's first element
        const uint2 before = tk.tile_count[(long long)i * tt.n_tiles + tile];
        unsigned int gmask = 0, emask = 0;
        unsigned long long pg = 0, pe = 0;
#pragma unroll
        for (int v = 0; v < kChunks; ++v) {
            const int local = (v * kThreads + threadIdx.x) * 4;
            if (local < len) {
                const float4 a = ld_stream(x + base + local), b = ld_stream(xhat + base + local);
                s_val[v * kThreads + threadIdx.x] = a;
                const unsigned int k[4] = {rank_key(a.x, b.x), rank_key(a.y, b.y), rank_key(a.z, b.z),
                                           rank_key(a.w, b.w)};
                const int nel = len - local;
                unsigned int g = 0, e = 0;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const bool live = c < nel;
                    g |= (live && k[c] > tau) ? (1u << c) : 0u;
                    e |= (live && k[c] == tau) ? (1u << c) : 0u;
                }
                gmask |= g << (4 * v);
                emask |= e << (4 * v);
                pg |= (unsigned long long)__popc(g) << (16 * v);
                pe |= (unsigned long long)__popc(e) << (16 * v);
            }
        }
        // inclusive scan over the CTA in thread order, all four chunks at once
        unsigned long long sg = pg, se = pe;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long a = __shfl_up_sync(0xffffffffu, sg, o);
            const unsigned long long b = __shfl_up_sync(0xffffffffu, se, o);
            if (lane >= o) { sg += a; se += b; }
        }
        if (lane == 31) { s_pg[warp] = sg; s_pe[warp] = se; }
        __syncthreads();
        unsigned long long wg = 0, we = 0, tg = 0, te = 0;
#pragma unroll
        for (int u = 0; u < kWarps; ++u) {
            if (u < warp) { wg += s_pg[u]; we += s_pe[u]; }
            tg += s_pg[u]; te += s_pe[u];
        }
        const unsigned long long xg = wg + sg - pg, xe = we + se - pe;   // exclusive, per chunk
        unsigned int run_gt = before.x, run_eq = before.y;               // entries before chunk v
        const float* my_val = reinterpret_cast<const float*>(s_val);
#pragma unroll
        for (int v = 0; v < kChunks; ++v) {
            unsigned int m = ((gmask | emask) >> (4 * v)) & 0xfu;
            if (m) {
                const int local = (v * kThreads + threadIdx.x) * 4;
                unsigned int my_gt = run_gt + (unsigned int)((xg >> (16 * v)) & 0xffffu);
                unsigned int my_eq = run_eq + (unsigned int)((xe >> (16 * v)) & 0xffffu);
                const unsigned int en = (emask >> (4 * v)) & 0xfu;
                while (m) {
                    const int c = __ffs(m) - 1;
                    m &= m - 1;
                    const bool is_eq = (en >> c) & 1u;
                    if (!is_eq || my_eq < take) {
                        const unsigned int slot = my_gt + min(my_eq, take);
                        const float val = my_val[local + c];
                        if (slot < K) {
                            out[slot] = make_int2(first + local + c, __float_as_int(val));
                            xhat[base + local + c] = val;
                        } else {
                            atomicOr(err, 2u);
                        }
                    }
                    my_gt += is_eq ? 0u : 1u;
                    my_eq += is_eq ? 1u : 0u;
                }
            }
            run_gt += (unsigned int)((tg >> (16 * v)) & 0xffffu);
            run_eq += (unsigned int)((te >> (16 * v)) & 0xffffu);
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------------
// Launch forms.  k_topk_all runs the whole sequence in ONE cooperative launch with grid-wide
// barriers between the phases, and every CTA leaves after the first barrier when no segment
// sends a sparse message in this step -- a quiet step then costs one launch instead of ten.
// The single-phase kernels below are the fallback where a cooperative launch is not available.
// ---------------------------------------------------------------------------------------
struct TopkArgs {
    const float* x;
    float* xhat;
    TileTable tt;
    int S, T;
    long long stride;
    const uint8_t* sparse;
    TopkState tk;
    unsigned int* err;
};

__global__ void __launch_bounds__(kThreads, 4) k_topk_all(TopkArgs a) {
    cooperative_groups::grid_group grid = cooperative_groups::this_grid();
    if (blockIdx.x == 0) topk_plan(a.S, a.T, a.sparse, a.tt.seg_begin, a.tk);
    grid.sync();
    if (a.tk.plan->n_sparse == 0) return;          // the same for every CTA
    topk_hist(a.x, a.xhat, a.tt, a.T, a.stride, a.tk);
    grid.sync();
    topk_pick(a.T, a.tk, 0);
    grid.sync();
    topk_collect(a.x, a.xhat, a.tt, a.T, a.stride, a.tk);
    grid.sync();
    topk_pick(a.T, a.tk, 1);
    grid.sync();
    topk_hist_cand(a.tt, a.T, a.stride, a.tk);
    grid.sync();
    topk_pick(a.T, a.tk, 2);
    grid.sync();
    topk_count(a.tt, a.T, a.stride, a.tk);
    grid.sync();
    topk_scan(a.tt, a.T, a.tk);
    grid.sync();
    topk_write(a.x, a.xhat, a.tt, a.T, a.stride, a.tk, a.err);
}

__global__ void __launch_bounds__(kThreads) k_topk_plan(TopkArgs a) {
    topk_plan(a.S, a.T, a.sparse, a.tt.seg_begin, a.tk);
}
__global__ void __launch_bounds__(kThreads) k_topk_hist(TopkArgs a) {
    topk_hist(a.x, a.xhat, a.tt, a.T, a.stride, a.tk);
}
__global__ void __launch_bounds__(kThreads) k_topk_pick(TopkArgs a, int digit) { topk_pick(a.T, a.tk, digit); }
__global__ void __launch_bounds__(kThreads, 4) k_topk_collect(TopkArgs a) {
    topk_collect(a.x, a.xhat, a.tt, a.T, a.stride, a.tk);
}
__global__ void __launch_bounds__(kThreads) k_topk_hist_cand(TopkArgs a) {
    topk_hist_cand(a.tt, a.T, a.stride, a.tk);
}
__global__ void __launch_bounds__(kThreads) k_topk_count(TopkArgs a) { topk_count(a.tt, a.T, a.stride, a.tk); }
__global__ void __launch_bounds__(kThreads) k_topk_scan(TopkArgs a) { topk_scan(a.tt, a.T, a.tk); }
__global__ void __launch_bounds__(kThreads, 4) k_topk_write(TopkArgs a) {
    topk_write(a.x, a.xhat, a.tt, a.T, a.stride, a.tk, a.err);
}

}  // namespace eg
