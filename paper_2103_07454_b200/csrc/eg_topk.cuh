// Top-K messages (Top-K paragraph of Section 7): for every segment whose event sends a
// sparse message, find exactly the K_t entries with the largest |x - x_hat| (ties to the lower
// index), pack them as (index, value) in ascending index order into the replica's outbox,
// and deliver them into the mailbox x_hat.
//
// The rank key is the bit pattern of |x - x_hat| (fp32), which orders like the magnitude.
// The K_t-th largest key tau is found by radix select over three digits (11 + 10 + 10 bits):
//   pass A  (reads x, x_hat)  histogram of the top digit                     -> bin b0
//   pass B  (reads x, x_hat)  every element whose top digit is >= b0 is copied, tile by tile and
//                             in index order, into an entry buffer as (20 low key bits, position,
//                             value of x); digit 1 of the undecided ones (top digit == b0) is
//                             histogrammed on the way
//   digit 2, per-tile counts, ordered compaction into the outbox and delivery into x_hat:
//                             from the entries only (K_t plus the population of one bin: a few
//                             percent of the tensor)
// so a sparse message costs two passes over its tensor.  The host knows nothing about the
// decisions: a planning phase turns the device-side `sparse` flags into a compact list of work
// tiles and every other phase runs a fixed-size grid over that list.  All phases can run in one
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
    int chunk;          // work tiles per planned share (kTopkGrid shares, or one per CTA of the single launch)
};

struct TopkState {
    TopkPlan* plan;
    int* sp_seg;               // [P*T] segment id of the q-th sparse segment
    int* sp_begin;             // [P*T+1] first work tile of the q-th sparse segment
    int* cta_q;                // [kTopkGrid] sparse slot that holds the first work tile of CTA c's share
    unsigned int* hist;        // [P*T][kMaxBins]
    unsigned int* prefix;      // [P*T] key bits resolved so far (after the last digit: tau)
    unsigned int* remaining;   // [P*T] rank still to resolve (after the last digit: number of
                               //       entries equal to tau that are part of the message)
    uint2* ent;                // [P][stride] entries (meta, value bits) of a tile, at the tile's own offset
    int* tile_cand;            // [P][n_tiles][8] entries stored by each warp for the tile
    unsigned int* tile_sub;    // [P][n_tiles][8] of those, (greater than tau) | (equal to tau) << 16
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
                                          const int* __restrict__ seg_begin, const TopkState& tk,
                                          int n_cta) {
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
    // the tile phases give CTA c the work tiles [c * chunk, (c + 1) * chunk): note for every c
    // the sparse slot its first tile falls into, so that no phase has to search for it
    const int chunk = (s_tiles[kThreads - 1] + n_cta - 1) / n_cta;
    if (threadIdx.x == 0) tk.plan->chunk = chunk;
    int q = s_cnt[threadIdx.x] - cnt, w = s_tiles[threadIdx.x] - tiles;
    for (int s = lo; s < hi; ++s)
        if (sparse[s]) {
            const int t = s % T;
            const int w_end = w + seg_begin[t + 1] - seg_begin[t];
            tk.sp_seg[q] = s;
            tk.sp_begin[q] = w;
            for (int c = (w + chunk - 1) / chunk; c < n_cta && c * chunk < w_end; ++c) tk.cta_q[c] = q;
            ++q;
            w = w_end;
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
// `shares`: planned shares per CTA (a phase may run with a grid `shares` times smaller than planned).
__device__ __forceinline__ WorkRange work_range(const TopkState& tk, int shares = 1) {
    const int total = tk.plan->total_tiles;
    const int chunk = tk.plan->chunk;
    WorkRange r;
    r.w0 = min(total, (int)blockIdx.x * shares * chunk);
    r.w1 = min(total, r.w0 + shares * chunk);
    r.q = (r.w0 < r.w1) ? tk.cta_q[blockIdx.x * shares] : 0;
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

// One warp per sparse segment: pick the bin that holds the wanted rank, counting from the
// largest key downwards; clear the histogram for the next digit.  The histogram is walked in
// blocks of 1024 bins from the top; a lane owns 32 consecutive bins of a block (eight 16-byte
// loads, all in flight together), one warp scan places the rank in a lane, which then walks
// its own bins.
__device__ __forceinline__ void
topk_pick(int T, TopkState tk, int digit) {
    constexpr int kBlock = 1024, kPer = kBlock / 32;
    const int nq = tk.plan->n_sparse;
    const int nbins = 1 << digit_bits(digit);
    const int lane = threadIdx.x & 31;
    const int nwarps = gridDim.x * kWarps;
    for (int q = blockIdx.x * kWarps + (threadIdx.x >> 5); q < nq; q += nwarps) {
        const int s = tk.sp_seg[q];
        const int t = s % T;
        unsigned int* gh = tk.hist + (long long)s * kMaxBins;
        const unsigned int rem = (digit == 0) ? (unsigned int)tk.count[t] : tk.remaining[s];
        unsigned int above_blocks = 0;      // keys in the blocks already walked
        bool found = false;                 // the same in every lane
        for (int blk = nbins / kBlock - 1; blk >= 0; --blk) {
            uint4* g4 = reinterpret_cast<uint4*>(gh + blk * kBlock + lane * kPer);
            if (found) {                    // only the clearing is left
#pragma unroll
                for (int j = 0; j < kPer / 4; ++j) g4[j] = make_uint4(0u, 0u, 0u, 0u);
                continue;
            }
            unsigned int c[kPer];
#pragma unroll
            for (int j = 0; j < kPer / 4; ++j) {
                const uint4 v = g4[j];
                c[4 * j] = v.x; c[4 * j + 1] = v.y; c[4 * j + 2] = v.z; c[4 * j + 3] = v.w;
            }
#pragma unroll
            for (int j = 0; j < kPer / 4; ++j) g4[j] = make_uint4(0u, 0u, 0u, 0u);
            unsigned int mine = 0;
#pragma unroll
            for (int z = 0; z < kPer; ++z) mine += c[z];
            unsigned int inc = mine;        // inclusive sum over this and the higher lanes
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned int v = __shfl_down_sync(0xffffffffu, inc, o);
                if (lane + o < 32) inc += v;
            }
            unsigned int above = above_blocks + inc - mine;
            const bool here = above < rem && rem <= above + mine;
            if (here) {
                bool done = false;
#pragma unroll
                for (int z = kPer - 1; z >= 0; --z) {
                    if (!done && rem <= above + c[z]) {
                        const unsigned int old = (digit == 0) ? 0u : tk.prefix[s];
                        tk.prefix[s] = (old << digit_bits(digit)) | (unsigned int)(blk * kBlock + lane * kPer + z);
                        tk.remaining[s] = rem - above;
                        done = true;
                    }
                    above += c[z];
                }
            }
            found = __any_sync(0xffffffffu, here);
            above_blocks += __shfl_sync(0xffffffffu, inc, 0);
        }
    }
}

constexpr int kSubSlices = kWarps;                       // entry sub-slices per tile: one per warp
constexpr int kWarpSpan = kNormTile / kWarps;            // 512 consecutive elements of a tile per warp
constexpr int kSubChunks = kWarpSpan / 128;              // read as 4 chunks of 128 (one float4 per lane)
static_assert(kWarpSpan == 512 && kSubChunks == 4, "entry words hold a 9-bit position and four 8-bit counts");

// An entry describes one element whose top digit is at least the chosen bin b0:
//   meta = sure << 29 | (key & 0xfffff) << 9 | position inside the warp's 512 elements
//   val  = bits of x at that element
// `sure` marks a top digit above b0 (the element is part of the message whatever the lower
// digits say); otherwise the top digit equals b0 and the 20 low key bits decide.
constexpr unsigned int kEntSure = 1u << 29;
__device__ __forceinline__ unsigned int ent_low20(unsigned int meta) { return (meta >> 9) & 0xfffffu; }
__device__ __forceinline__ bool ent_sure(unsigned int meta) { return (meta & kEntSure) != 0u; }

// Warp w of a CTA owns elements [512 w, 512 w + 512) of a tile; its entries start at the same
// place in the tile's slice of the entry buffer, so the slices can never overlap.
__device__ __forceinline__ int sub_offset(int len, int w) { return min(len, w * kWarpSpan); }

// Pass B: per tile, every element whose top digit is at least b0 is copied as an entry into the
// tile's slice of the entry buffer, IN ASCENDING INDEX ORDER inside each warp's sub-slice (the
// later phases rely on that order: concatenating the sub-slices of a tensor's tiles lists its
// entries by index).  Digit 1 of the undecided entries is histogrammed on the way.  Nothing is
// shared between warps except that histogram: a lane marks its elements in four 4-bit masks,
// one warp scan of the four packed 8-bit counts (a chunk holds 128 elements, so a field cannot
// overflow) gives every lane its first slot in each chunk.
__device__ __forceinline__ void
topk_collect(const float* __restrict__ x, const float* __restrict__ xhat, TileTable tt, int T,
               long long stride, TopkState tk) {
    constexpr int kBins1 = 1 << kDigitBits1;
    __shared__ unsigned int s_hist[kBins1];
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
        unsigned int key[4 * kSubChunks];
        float val[4 * kSubChunks];
        unsigned int mask = 0, packed = 0;      // bit 4j+c: element c of chunk j is an entry
#pragma unroll
        for (int j = 0; j < kSubChunks; ++j) {
            const int local = warp * kWarpSpan + j * 128 + lane * 4;
            float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
            if (local < len) { a = ld_stream(x + base + local); b = ld_stream(xhat + base + local); }
            key[4 * j + 0] = rank_key(a.x, b.x); key[4 * j + 1] = rank_key(a.y, b.y);
            key[4 * j + 2] = rank_key(a.z, b.z); key[4 * j + 3] = rank_key(a.w, b.w);
            val[4 * j + 0] = a.x; val[4 * j + 1] = a.y; val[4 * j + 2] = a.z; val[4 * j + 3] = a.w;
            const int nel = len - local;          // live elements of this float4 (<= 0: none)
            unsigned int m = 0;
#pragma unroll
            for (int c = 0; c < 4; ++c) m |= (c < nel && (key[4 * j + c] >> 20) >= b0) ? (1u << c) : 0u;
            mask |= m << (4 * j);
            packed |= (unsigned int)__popc(m) << (8 * j);
        }
        unsigned int inc = packed;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned int u = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += u;
        }
        const unsigned int tot = __shfl_sync(0xffffffffu, inc, 31);
        const unsigned int excl = inc - packed;
        uint2* ent = tk.ent + base + sub_offset(len, warp);
        unsigned int chunk_first = 0;
#pragma unroll
        for (int j = 0; j < kSubChunks; ++j) {
            unsigned int pos = chunk_first + ((excl >> (8 * j)) & 0xffu);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                if (mask & (1u << (4 * j + c))) {
                    const unsigned int k = key[4 * j + c];
                    const bool sure = (k >> 20) > b0;
                    ent[pos++] = make_uint2((sure ? kEntSure : 0u) | ((k & 0xfffffu) << 9) |
                                                (unsigned int)(j * 128 + lane * 4 + c),
                                            __float_as_uint(val[4 * j + c]));
                    if (!sure) atomicAdd(&s_hist[(k >> 10) & (kBins1 - 1)], 1u);
                }
            }
            chunk_first += (tot >> (8 * j)) & 0xffu;
        }
        if (lane == 0) tk.tile_cand[((long long)i * tt.n_tiles + tile) * kSubSlices + warp] = (int)chunk_first;
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

// The one-warp-per-tile phases: a CTA takes a contiguous share of the work list (one search
// per CTA), its warps take the tiles of that share in turn, each walking forward with its own
// cursor.
struct WarpTile {
    int s, i, t, tile;
};
struct WarpWalk {
    WorkRange r;
    WorkCursor cur;
    int w;
    __device__ __forceinline__ void init(const TopkState& tk, const TileTable& tt, int T, int shares = 1) {
        r = work_range(tk, shares);
        cur.init(tk, tt, T, r.q);
        w = r.w0 + (int)(threadIdx.x >> 5);
    }
    __device__ __forceinline__ bool next(const TopkState& tk, const TileTable& tt, int T, WarpTile& z) {
        if (w >= r.w1) return false;
        bool changed;
        z.tile = cur.advance(tk, tt, T, w, changed);
        z.s = cur.s; z.i = cur.i; z.t = cur.t;
        w += kWarps;
        return true;
    }
};

// The entries of one tile: sub-slice u (the elements [512 u, 512 u + 512) of the tile, in index
// order) holds n[u] entries starting at place min(len, 512 u) of the tile's slice.  The phases
// below walk four sub-slices side by side -- round r touches entries 32 r + lane of each of
// them, four independent loads per lane -- because a tile rarely holds more than a few
// dozen entries per sub-slice and a walk one after the other would wait for memory eight times
// instead of twice.
constexpr int kSubGroup = 4;        // sub-slices walked side by side
struct TileEntries {
    int n[kSubSlices];
    const uint2* slice;
    int len;
    long long slot;                 // first of the tile's eight per-sub-slice records
    // `mine`: lane u < 8 brings the entry count of sub-slice u (see TileFeed)
    __device__ __forceinline__ void init(const TopkState& tk, const TileTable& tt, long long stride,
                                         const WarpTile& z, int mine) {
        slot = ((long long)z.i * tt.n_tiles + z.tile) * kSubSlices;
#pragma unroll
        for (int u = 0; u < kSubSlices; ++u) n[u] = __shfl_sync(0xffffffffu, mine, u);
        slice = tk.ent + (long long)z.i * stride + tt.offset[z.tile];
        len = tt.length[z.tile];
    }
    __device__ __forceinline__ const uint2* sub(int u) const { return slice + min(len, u * kWarpSpan); }
    // largest entry count among the sub-slices u0 .. u0 + kSubGroup - 1
    __device__ __forceinline__ int most_of(int u0) const {
        int m = 0;
#pragma unroll
        for (int v = 0; v < kSubGroup; ++v) m = max(m, n[u0 + v]);
        return m;
    }
};

// A warp's tiles, one ahead: while a tile is worked on, the entry counts of the warp's next
// tile are already on their way, so a tile costs one wait less.
struct TileFeed {
    WarpWalk walk;
    WarpTile ahead;
    int ahead_mine;
    bool have;
    __device__ __forceinline__ int fetch(const TopkState& tk, const TileTable& tt) const {
        const int lane = threadIdx.x & 31;
        return (lane < kSubSlices)
                   ? tk.tile_cand[((long long)ahead.i * tt.n_tiles + ahead.tile) * kSubSlices + lane] : 0;
    }
    __device__ __forceinline__ void init(const TopkState& tk, const TileTable& tt, int T, int shares) {
        walk.init(tk, tt, T, shares);
        have = walk.next(tk, tt, T, ahead);
        ahead_mine = have ? fetch(tk, tt) : 0;
    }
    __device__ __forceinline__ bool next(const TopkState& tk, const TileTable& tt, int T, WarpTile& z, int& mine) {
        if (!have) return false;
        z = ahead;
        mine = ahead_mine;
        have = walk.next(tk, tt, T, ahead);
        ahead_mine = have ? fetch(tk, tt) : 0;
        return true;
    }
};

// Digit 2 over the entries: one warp per tile, global histogram updated directly (only the
// undecided entries that match the 21 resolved bits take part: about one in a thousand).
__device__ __forceinline__ void
topk_hist_cand(TileTable tt, int T, long long stride, TopkState tk, int shares = 1) {
    const int lane = threadIdx.x & 31;
    TileFeed feed;
    feed.init(tk, tt, T, shares);
    WarpTile z;
    int mine_n;
    int s_now = -1;
    unsigned int want = 0;
    while (feed.next(tk, tt, T, z, mine_n)) {
        if (z.s != s_now) { s_now = z.s; want = tk.prefix[z.s] & ((1u << kDigitBits1) - 1); }   // digit 1 of tau
        unsigned int* gh = tk.hist + (long long)z.s * kMaxBins;
        TileEntries te;
        te.init(tk, tt, stride, z, mine_n);
#pragma unroll
        for (int u0 = 0; u0 < kSubSlices; u0 += kSubGroup) {
            for (int f = lane; f - lane < te.most_of(u0); f += 32) {
                unsigned int meta[kSubGroup];
#pragma unroll
                for (int v = 0; v < kSubGroup; ++v) meta[v] = (f < te.n[u0 + v]) ? te.sub(u0 + v)[f].x : kEntSure;
#pragma unroll
                for (int v = 0; v < kSubGroup; ++v) {
                    const unsigned int low = ent_low20(meta[v]);
                    if (!ent_sure(meta[v]) && (low >> kDigitBits2) == want)
                        atomicAdd(&gh[low & ((1u << kDigitBits2) - 1)], 1u);
                }
            }
        }
    }
}

// Per tile and per sub-slice: keys greater than / equal to tau, from the entries.  One warp per
// tile.  tile_sub gets the eight (greater | equal << 16) pairs, tile_count the tile's totals.
__device__ __forceinline__ void
topk_count(TileTable tt, int T, long long stride, TopkState tk, int shares = 1) {
    const int lane = threadIdx.x & 31;
    TileFeed feed;
    feed.init(tk, tt, T, shares);
    WarpTile z;
    int mine_n;
    int s_now = -1;
    unsigned int tau20 = 0;
    while (feed.next(tk, tt, T, z, mine_n)) {
        if (z.s != s_now) { s_now = z.s; tau20 = tk.prefix[z.s] & 0xfffffu; }
        TileEntries te;
        te.init(tk, tt, stride, z, mine_n);
        unsigned int mine = 0, all_gt = 0, all_eq = 0;
#pragma unroll
        for (int u0 = 0; u0 < kSubSlices; u0 += kSubGroup) {
            unsigned int gt[kSubGroup], eq[kSubGroup];        // the same in every lane
#pragma unroll
            for (int v = 0; v < kSubGroup; ++v) gt[v] = eq[v] = 0;
            for (int f = lane; f - lane < te.most_of(u0); f += 32) {
                unsigned int meta[kSubGroup];
#pragma unroll
                for (int v = 0; v < kSubGroup; ++v) meta[v] = (f < te.n[u0 + v]) ? te.sub(u0 + v)[f].x : 0u;
#pragma unroll
                for (int v = 0; v < kSubGroup; ++v) {
                    const bool live = f < te.n[u0 + v];
                    const unsigned int low = ent_low20(meta[v]);
                    gt[v] += __popc(__ballot_sync(0xffffffffu, live && (ent_sure(meta[v]) || low > tau20)));
                    eq[v] += __popc(__ballot_sync(0xffffffffu, live && !ent_sure(meta[v]) && low == tau20));
                }
            }
#pragma unroll
            for (int v = 0; v < kSubGroup; ++v) {
                if (lane == u0 + v) mine = gt[v] | (eq[v] << 16);
                all_gt += gt[v];
                all_eq += eq[v];
            }
        }
        if (lane < kSubSlices) tk.tile_sub[te.slot + lane] = mine;
        if (lane == 0) tk.tile_count[(long long)z.i * tt.n_tiles + z.tile] = make_uint2(all_gt, all_eq);
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

// Pass C: ordered compaction of the selected entries into the outbox, and delivery: the same
// (index, value) pairs are written into the mailbox x_hat, which is what the receivers hold
// once the message has arrived.  Works from the entries alone (a few percent of the tensor);
// x and x_hat are not read again.
// An entry is selected if key > tau, or key == tau and fewer than `remaining` equal keys
// precede it in the tensor.  Its slot is (#greater before it) + min(#equal before it, remaining).
// One warp per tile walks the tile's entries in index order, 32 at a time; ballots give every
// lane the number of greater / equal entries before its own.
__device__ __forceinline__ void
topk_write(float* xhat, TileTable tt, int T, long long stride, TopkState tk, unsigned int* __restrict__ err,
           int shares = 1) {
    const int lane = threadIdx.x & 31;
    const unsigned int below = (1u << lane) - 1u;
    TileFeed feed;
    feed.init(tk, tt, T, shares);
    WarpTile z;
    int mine_n;
    int s_now = -1;
    unsigned int tau20 = 0, take = 0, K = 0;
    int2* out = nullptr;
    while (feed.next(tk, tt, T, z, mine_n)) {
        if (z.s != s_now) {
            s_now = z.s;
            tau20 = tk.prefix[z.s] & 0xfffffu;
            take = tk.remaining[z.s];
            K = (unsigned int)tk.count[z.t];
            out = tk.outbox + (long long)z.i * tk.out_stride + tk.out_off[z.t];
        }
        TileEntries te;
        te.init(tk, tt, stride, z, mine_n);
        const uint2 before = tk.tile_count[(long long)z.i * tt.n_tiles + z.tile];
        const unsigned int sub_mine = (lane < kSubSlices) ? tk.tile_sub[te.slot + lane] : 0u;
        const long long base = (long long)z.i * stride + tt.offset[z.tile];
        const int first = (z.tile - tt.seg_begin[z.t]) * kNormTile;   // index of the tile's first element
        unsigned int gt_before = before.x, eq_before = before.y;   // entries before sub-slice u0, whole tensor
#pragma unroll
        for (int u0 = 0; u0 < kSubSlices; u0 += kSubGroup) {
            unsigned int run_gt[kSubGroup], run_eq[kSubGroup];     // the same in every lane
#pragma unroll
            for (int v = 0; v < kSubGroup; ++v) {
                const unsigned int packed = __shfl_sync(0xffffffffu, sub_mine, u0 + v);
                run_gt[v] = gt_before;
                run_eq[v] = eq_before;
                gt_before += packed & 0xffffu;
                eq_before += packed >> 16;
            }
            for (int f = lane; f - lane < te.most_of(u0); f += 32) {
                uint2 e[kSubGroup];
#pragma unroll
                for (int v = 0; v < kSubGroup; ++v)
                    e[v] = (f < te.n[u0 + v]) ? te.sub(u0 + v)[f] : make_uint2(0u, 0u);
#pragma unroll
                for (int v = 0; v < kSubGroup; ++v) {
                    const bool live = f < te.n[u0 + v];
                    const unsigned int low = ent_low20(e[v].x);
                    const bool g = live && (ent_sure(e[v].x) || low > tau20);
                    const bool q = live && !ent_sure(e[v].x) && low == tau20;
                    const unsigned int bg = __ballot_sync(0xffffffffu, g), bq = __ballot_sync(0xffffffffu, q);
                    const unsigned int my_gt = run_gt[v] + __popc(bg & below), my_eq = run_eq[v] + __popc(bq & below);
                    if (g || (q && my_eq < take)) {
                        const unsigned int slot = my_gt + min(my_eq, take);
                        const int local = (u0 + v) * kWarpSpan + (int)(e[v].x & 0x1ffu);
                        if (slot < K && local < te.len) {
                            out[slot] = make_int2(first + local, (int)e[v].y);
                            xhat[base + local] = __uint_as_float(e[v].y);
                        } else {
                            atomicOr(err, 2u);
                        }
                    }
                    run_gt[v] += __popc(bg);
                    run_eq[v] += __popc(bq);
                }
            }
        }
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
    const unsigned int* sparse_steps;   // [2] sparse messages decided in the iteration of this parity
    const long long* step_k;
};

__global__ void __launch_bounds__(kThreads, 4) k_topk_all(TopkArgs a) {
    cooperative_groups::grid_group grid = cooperative_groups::this_grid();
    // a quiet iteration (the decision kernel counted no sparse message) ends here, before any
    // grid-wide barrier: the same answer in every CTA
    if (a.sparse_steps[*a.step_k & 1] == 0) return;
    if (blockIdx.x == 0) topk_plan(a.S, a.T, a.sparse, a.tt.seg_begin, a.tk, (int)gridDim.x);
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
    topk_write(a.xhat, a.tt, a.T, a.stride, a.tk, a.err);
}

__global__ void __launch_bounds__(kThreads) k_topk_plan(TopkArgs a) {
    topk_plan(a.S, a.T, a.sparse, a.tt.seg_begin, a.tk, kTopkGrid);   // every tile phase runs kTopkGrid CTAs
}
__global__ void __launch_bounds__(kThreads) k_topk_hist(TopkArgs a) {
    topk_hist(a.x, a.xhat, a.tt, a.T, a.stride, a.tk);
}
__global__ void __launch_bounds__(kThreads) k_topk_pick(TopkArgs a, int digit) { topk_pick(a.T, a.tk, digit); }
#ifndef EG_COLLECT_MINB
#define EG_COLLECT_MINB 4
#endif
__global__ void __launch_bounds__(kThreads, EG_COLLECT_MINB) k_topk_collect(TopkArgs a) {
    topk_collect(a.x, a.xhat, a.tt, a.T, a.stride, a.tk);
}
// The phases that work from the entries keep more registers than the streaming passes: they
// run half the planned CTAs, each taking two planned shares.
constexpr int kEntryShares = 2;
__global__ void __launch_bounds__(kThreads, 4) k_topk_hist_cand(TopkArgs a) {
    topk_hist_cand(a.tt, a.T, a.stride, a.tk, kEntryShares);
}
__global__ void __launch_bounds__(kThreads, 4) k_topk_count(TopkArgs a) {
    topk_count(a.tt, a.T, a.stride, a.tk, kEntryShares);
}
__global__ void __launch_bounds__(kThreads) k_topk_scan(TopkArgs a) { topk_scan(a.tt, a.T, a.tk); }
__global__ void __launch_bounds__(kThreads, 4) k_topk_write(TopkArgs a) {
    topk_write(a.xhat, a.tt, a.T, a.stride, a.tk, a.err, kEntryShares);
}

}  // namespace eg
