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
//   digit 2 together with per-tile counts, then ordered compaction into the outbox and delivery
//   into x_hat:               two walks over the entries only (K_t plus the population of one
//                             bin: a few percent of the tensor)
// so a sparse message costs two passes over its tensor.  The host knows nothing about the
// decisions: a planning phase turns the device-side `sparse` flags into a compact list of work
// tiles and every other phase runs a fixed-size grid over that list.  All phases can run in one
// cooperative launch (k_topk_all, bottom of this file).
#pragma once
#include <cooperative_groups.h>

#include "eg_common.cuh"

namespace eg {

constexpr int kTopkCtasPerSm = 8;      // CTAs per multiprocessor of the tile kernels (they loop over the work list)
constexpr int kTopkSegCtasPerSm = 4;   // ... of the per-segment kernels

struct TopkPlan {
    int n_sparse;       // segments that send a sparse message in this step
    int total_tiles;    // their tiles
    int chunk;          // work tiles per planned share (one share per CTA of the tile phases)
};

struct TopkState {
    TopkPlan* plan;
    int* sp_seg;               // [P*T] segment id of the q-th sparse segment
    int* sp_begin;             // [P*T+1] first work tile of the q-th sparse segment
    int* cta_q;                // [CTAs of the tile phases] sparse slot that holds the first work tile of CTA c's share
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
            if (!EG_INDEX_OK(tt.err, q, tk.plan->n_sparse)) { changed = true; break; }   // (the loop would not end)
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
// shared between warps except that histogram.  Entries are few (a few percent of the elements),
// so the pass is split: first every lane only MARKS its sixteen elements in a bit mask (a chunk
// holds 128 elements, so one warp scan of the four packed 8-bit counts gives every lane its
// first slot in each chunk); then a lane walks the set bits of its mask -- usually none, one or
// two -- and builds each entry from the element itself, which it reads again (the line has just
// been fetched by this warp, so the second read is served by the caches).
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
    const int mine = warp * kWarpSpan + lane * 4;      // this lane's first element of the tile
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
        float4 a[kSubChunks], b[kSubChunks];
#pragma unroll
        for (int j = 0; j < kSubChunks; ++j) {
            const int local = mine + j * 128;
            a[j] = b[j] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (local < len) { a[j] = ld_stream(x + base + local); b[j] = ld_stream(xhat + base + local); }
        }
        unsigned int mask = 0, packed = 0;      // bit 4j+c: element c of chunk j is an entry
#pragma unroll
        for (int j = 0; j < kSubChunks; ++j) {
            const int nel = len - (mine + j * 128);   // live elements of this float4 (<= 0: none)
            unsigned int m = 0;
            m |= (0 < nel && (rank_key(a[j].x, b[j].x) >> 20) >= b0) ? 1u : 0u;
            m |= (1 < nel && (rank_key(a[j].y, b[j].y) >> 20) >= b0) ? 2u : 0u;
            m |= (2 < nel && (rank_key(a[j].z, b[j].z) >> 20) >= b0) ? 4u : 0u;
            m |= (3 < nel && (rank_key(a[j].w, b[j].w) >> 20) >= b0) ? 8u : 0u;
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
        // first slot of this lane in each chunk, 10 bits each (a sub-slice holds at most 512 entries)
        unsigned long long first = 0;
        unsigned int chunk_first = 0;
#pragma unroll
        for (int j = 0; j < kSubChunks; ++j) {
            first |= (unsigned long long)(chunk_first + ((excl >> (8 * j)) & 0xffu)) << (10 * j);
            chunk_first += (tot >> (8 * j)) & 0xffu;
        }
        uint2* ent = tk.ent + base + sub_offset(len, warp);
        const float* xs = x + base + mine;
        const float* hs = xhat + base + mine;
        unsigned int todo = mask;
        while (todo) {
            const int bit = __ffs(todo) - 1;
            todo &= todo - 1u;
            const int j = bit >> 2, e = j * 128 + (bit & 3);       // element mine + e of the tile
            const float xv = xs[e];
            const unsigned int k = rank_key(xv, hs[e]);
            const bool sure = (k >> 20) > b0;
            // slot: the lane's first slot in the chunk plus its own earlier entries of that chunk
            const unsigned int pos = (unsigned int)((first >> (10 * j)) & 0x3ffu) +
                                     __popc(mask & ((1u << bit) - 1u) & (0xfu << (4 * j)));
            if (!EG_INDEX_OK(tt.err, pos, kWarpSpan) || !EG_INDEX_OK(tt.err, sub_offset(len, warp) + pos, len)) continue;
            ent[pos] = make_uint2((sure ? kEntSure : 0u) | ((k & 0xfffffu) << 9) | (unsigned int)(lane * 4 + e),
                                  __float_as_uint(xv));
            if (!sure) atomicAdd(&s_hist[(k >> 10) & (kBins1 - 1)], 1u);
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
// order) holds n_u entries starting at place min(len, 512 u) of the tile's slice.  A tile
// rarely holds more than a dozen entries per sub-slice, so the phases below read all eight
// sub-slices at once: lane 4 u + r takes the entries r, r + 4, r + 8, ... of sub-slice u, four
// of them (kRounds) per trip to memory, and every lane has its loads in flight together.
constexpr int kRounds = 4;          // entries per lane and trip
constexpr int kGroupLanes = 4;      // lanes per sub-slice
static_assert(kSubSlices * kGroupLanes == 32, "one warp covers the eight sub-slices of a tile");

// A warp's tiles, one ahead: while a tile is worked on, the entry counts of the warp's next
// tile are already on their way, so a tile costs one wait less.  Every lane gets the count of
// its own sub-slice.
struct TileFeed {
    WarpWalk walk;
    WarpTile ahead;
    int ahead_mine;
    bool have;
    __device__ __forceinline__ int fetch(const TopkState& tk, const TileTable& tt) const {
        const int u = (threadIdx.x & 31) / kGroupLanes;
        return tk.tile_cand[((long long)ahead.i * tt.n_tiles + ahead.tile) * kSubSlices + u];
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

// (greater, equal) counts of a tile's eight sub-slices from per-lane counts: sums over the four
// lanes of every sub-slice, stores the eight packed pairs and the tile's totals.
__device__ __forceinline__ void
store_tile_counts(const TopkState& tk, long long slot, long long tile_index, unsigned int gt, unsigned int eq) {
    const int lane = threadIdx.x & 31;
    unsigned int both = gt | (eq << 16);            // a sub-slice holds at most 512 entries
    both += __shfl_xor_sync(0xffffffffu, both, 1);
    both += __shfl_xor_sync(0xffffffffu, both, 2);
    if ((lane & (kGroupLanes - 1)) == 0) tk.tile_sub[slot + lane / kGroupLanes] = both;
    unsigned int all_gt = both & 0xffffu, all_eq = both >> 16;     // a tile holds at most 4096
    all_gt += __shfl_xor_sync(0xffffffffu, all_gt, 4); all_eq += __shfl_xor_sync(0xffffffffu, all_eq, 4);
    all_gt += __shfl_xor_sync(0xffffffffu, all_gt, 8); all_eq += __shfl_xor_sync(0xffffffffu, all_eq, 8);
    all_gt += __shfl_xor_sync(0xffffffffu, all_gt, 16); all_eq += __shfl_xor_sync(0xffffffffu, all_eq, 16);
    if (lane == 0) tk.tile_count[tile_index] = make_uint2(all_gt, all_eq);
}

// Digit 2 over the entries, and the counts the compaction needs.  One warp per tile.  With the 21
// key bits resolved so far an entry is greater than tau for sure (a larger top digit, or the
// same top digit and a larger digit 1), smaller for sure, or OPEN (both digits equal: digit 2
// decides).  Open entries -- about one in a thousand -- go into the digit-2 histogram.  Per
// sub-slice and per tile the kernel stores (greater for sure, open); for a tile without open
// entries these are already its final (greater than tau, equal to tau) counts, the few tiles
// that have some are counted again once tau is complete (topk_scan).
__device__ __forceinline__ void
topk_digit2(TileTable tt, int T, long long stride, TopkState tk, int shares = 1) {
    const int lane = threadIdx.x & 31, u = lane / kGroupLanes, r = lane % kGroupLanes;
    TileFeed feed;
    feed.init(tk, tt, T, shares);
    WarpTile z;
    int n;                               // entries of this lane's sub-slice
    int s_now = -1;
    unsigned int want = 0;
    unsigned int* gh = nullptr;
    while (feed.next(tk, tt, T, z, n)) {
        if (z.s != s_now) {
            s_now = z.s;
            want = tk.prefix[z.s] & ((1u << kDigitBits1) - 1);      // digit 1 of tau
            gh = tk.hist + (long long)z.s * kMaxBins;
        }
        const int len = tt.length[z.tile];
        const uint2* sub = tk.ent + (long long)z.i * stride + tt.offset[z.tile] + min(len, u * kWarpSpan);
        unsigned int gt = 0, open = 0;
        for (int f0 = r; __any_sync(0xffffffffu, f0 - r < n); f0 += kRounds * kGroupLanes) {
            unsigned int meta[kRounds];
#pragma unroll
            for (int q = 0; q < kRounds; ++q) {
                const int f = f0 + q * kGroupLanes;
                meta[q] = (f < n) ? sub[f].x : 0u;
            }
#pragma unroll
            for (int q = 0; q < kRounds; ++q) {
                const bool live = f0 + q * kGroupLanes < n;
                const unsigned int low = ent_low20(meta[q]), d1 = low >> kDigitBits2;
                if (live && (ent_sure(meta[q]) || d1 > want)) ++gt;
                if (live && !ent_sure(meta[q]) && d1 == want) {
                    ++open;
                    atomicAdd(&gh[low & ((1u << kDigitBits2) - 1)], 1u);
                }
            }
        }
        store_tile_counts(tk, ((long long)z.i * tt.n_tiles + z.tile) * kSubSlices,
                          (long long)z.i * tt.n_tiles + z.tile, gt, open);
    }
}

// (greater than tau, equal to tau) per sub-slice and per tile, counted from the entries of one tile
// by one warp with all 31 bits of tau known.
__device__ __forceinline__ void
count_tile_exact(const TileTable& tt, long long stride, const TopkState& tk, int i, int tile, unsigned int tau20) {
    const int lane = threadIdx.x & 31, u = lane / kGroupLanes, r = lane % kGroupLanes;
    const long long index = (long long)i * tt.n_tiles + tile;
    const int n = tk.tile_cand[index * kSubSlices + u];
    const int len = tt.length[tile];
    const uint2* sub = tk.ent + (long long)i * stride + tt.offset[tile] + min(len, u * kWarpSpan);
    unsigned int gt = 0, eq = 0;
    for (int f = r; f < n; f += kGroupLanes) {
        const unsigned int meta = sub[f].x, low = ent_low20(meta);
        if (ent_sure(meta) || low > tau20) ++gt;
        else if (low == tau20) ++eq;
    }
    store_tile_counts(tk, index * kSubSlices, index, gt, eq);
}

// One CTA per sparse segment.  First the tiles that held open entries are counted again, now
// that tau is complete (a handful per tensor, unless many keys tie); then the exclusive prefix
// of the tile counts, in tile order.
__device__ __forceinline__ void
topk_scan(TileTable tt, int T, long long stride, TopkState tk) {
    __shared__ unsigned int s_gt[kWarps], s_eq[kWarps];
    __shared__ unsigned int s_run[2];
    const int nq = tk.plan->n_sparse;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int q = blockIdx.x; q < nq; q += gridDim.x) {
        const int s = tk.sp_seg[q];
        const int i = s / T, t = s - i * T;
        const int q0 = tt.seg_begin[t], q1 = tt.seg_begin[t + 1];
        uint2* tc = tk.tile_count + (long long)i * tt.n_tiles;
        const unsigned int tau20 = tk.prefix[s] & 0xfffffu;
        for (int c0 = q0; c0 < q1; c0 += 32 * kWarps) {
            // a lane looks at one tile; the warp then counts the marked ones together, one by one
            const int z = c0 + warp * 32 + lane;
            unsigned int marked = __ballot_sync(0xffffffffu, z < q1 && tc[z].y != 0u);
            while (marked) {
                const int l = __ffs(marked) - 1;
                marked &= marked - 1u;
                count_tile_exact(tt, stride, tk, i, c0 + warp * 32 + l, tau20);
            }
        }
        if (threadIdx.x == 0) s_run[0] = s_run[1] = 0;
        __syncthreads();            // the recounted pairs are visible to the whole CTA
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

// Ordered compaction of the selected entries into the outbox, and delivery: the same
// (index, value) pairs are written into the mailbox x_hat, which is what the receivers hold
// once the message has arrived.  Works from the entries alone (a few percent of the tensor);
// x and x_hat are not read again.
// An entry is selected if key > tau, or key == tau and fewer than `remaining` equal keys
// precede it in the tensor.  Its slot is (#greater before it) + min(#equal before it, remaining).
// One warp per tile; within a sub-slice the entries are taken in index order, four at a time by
// the four lanes of the sub-slice, and ballots give every lane the number of greater / equal
// entries before its own.
__device__ __forceinline__ void
topk_write(float* xhat, TileTable tt, int T, long long stride, TopkState tk, unsigned int* __restrict__ err,
           int shares = 1) {
    const int lane = threadIdx.x & 31, u = lane / kGroupLanes, r = lane % kGroupLanes;
    const unsigned int group = (unsigned int)((1u << kGroupLanes) - 1u) << (u * kGroupLanes);   // lanes of this sub-slice
    const unsigned int lower = ((1u << r) - 1u) << (u * kGroupLanes);                            // ... before this lane
    TileFeed feed;
    feed.init(tk, tt, T, shares);
    WarpTile z;
    int n;
    int s_now = -1;
    unsigned int tau20 = 0, take = 0, K = 0;
    int2* out = nullptr;
    while (feed.next(tk, tt, T, z, n)) {
        if (z.s != s_now) {
            s_now = z.s;
            tau20 = tk.prefix[z.s] & 0xfffffu;
            take = tk.remaining[z.s];
            K = (unsigned int)tk.count[z.t];
            out = tk.outbox + (long long)z.i * tk.out_stride + tk.out_off[z.t];
        }
        const long long index = (long long)z.i * tt.n_tiles + z.tile;
        const uint2 before = tk.tile_count[index];
        const unsigned int sub_mine = tk.tile_sub[index * kSubSlices + u];
        const int len = tt.length[z.tile];
        const long long base = (long long)z.i * stride + tt.offset[z.tile];
        const uint2* sub = tk.ent + base + min(len, u * kWarpSpan);
        const int first = (z.tile - tt.seg_begin[z.t]) * kNormTile;   // index of the tile's first element
        // selected entries of the whole tensor before this sub-slice: the tile's prefix plus the
        // sub-slices before it (all four lanes of a sub-slice hold the same pair)
        unsigned int inc = sub_mine;
#pragma unroll
        for (int o = kGroupLanes; o < 32; o <<= 1) {
            const unsigned int v = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += v;
        }
        unsigned int run_gt = before.x + ((inc - sub_mine) & 0xffffu);
        unsigned int run_eq = before.y + ((inc - sub_mine) >> 16);
        for (int f0 = r; __any_sync(0xffffffffu, f0 - r < n); f0 += kRounds * kGroupLanes) {
            uint2 e[kRounds];
#pragma unroll
            for (int q = 0; q < kRounds; ++q) {
                const int f = f0 + q * kGroupLanes;
                e[q] = (f < n) ? sub[f] : make_uint2(0u, 0u);
            }
#pragma unroll
            for (int q = 0; q < kRounds; ++q) {
                const bool live = f0 + q * kGroupLanes < n;
                const unsigned int low = ent_low20(e[q].x);
                const bool g = live && (ent_sure(e[q].x) || low > tau20);
                const bool same = live && !ent_sure(e[q].x) && low == tau20;
                const unsigned int bg = __ballot_sync(0xffffffffu, g), bq = __ballot_sync(0xffffffffu, same);
                const unsigned int my_gt = run_gt + __popc(bg & lower), my_eq = run_eq + __popc(bq & lower);
                if (g || (same && my_eq < take)) {
                    const unsigned int slot = my_gt + min(my_eq, take);
                    const int local = u * kWarpSpan + (int)(e[q].x & 0x1ffu);
                    if (slot < K && local < len) {
                        out[slot] = make_int2(first + local, (int)e[q].y);
                        xhat[base + local] = __uint_as_float(e[q].y);
                    } else {
                        atomicOr(err, kErrTopkSlot);
                    }
                }
                run_gt += __popc(bg & group);
                run_eq += __popc(bq & group);
            }
        }
    }
}

// ---------------------------------------------------------------------------------------
// Launch forms.  k_topk_all runs the whole sequence in ONE cooperative launch with grid-wide
// barriers between the phases, and every CTA leaves after the first barrier when no segment
// sends a sparse message in this step -- a quiet step then costs one launch instead of ten.
// The single-phase kernels below are used for large problems and where a cooperative launch is
// not available.
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
    int plan_ctas;                      // CTAs of the tile phases when they are launched one by one
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
    topk_digit2(a.tt, a.T, a.stride, a.tk);
    grid.sync();
    topk_pick(a.T, a.tk, 2);
    grid.sync();
    topk_scan(a.tt, a.T, a.stride, a.tk);
    grid.sync();
    topk_write(a.xhat, a.tt, a.T, a.stride, a.tk, a.err);
}

// Every single-phase kernel may be launched while the kernel before it drains (programmatic
// dependent launch): it lets its own successor do the same and then waits for its predecessor
// before it reads anything.
__global__ void __launch_bounds__(kThreads) k_topk_plan(TopkArgs a) {
    pdl_release(); pdl_wait();
    topk_plan(a.S, a.T, a.sparse, a.tt.seg_begin, a.tk, a.plan_ctas);
}
__global__ void __launch_bounds__(kThreads) k_topk_hist(TopkArgs a) {
    pdl_release(); pdl_wait();
    topk_hist(a.x, a.xhat, a.tt, a.T, a.stride, a.tk);
}
__global__ void __launch_bounds__(kThreads) k_topk_pick(TopkArgs a, int digit) {
    pdl_release(); pdl_wait();
    topk_pick(a.T, a.tk, digit);
}
#ifndef EG_COLLECT_MINB
#define EG_COLLECT_MINB 4
#endif
__global__ void __launch_bounds__(kThreads, EG_COLLECT_MINB) k_topk_collect(TopkArgs a) {
    pdl_release(); pdl_wait();
    topk_collect(a.x, a.xhat, a.tt, a.T, a.stride, a.tk);
}
// The phases that work from the entries run half the planned CTAs, each taking two planned shares.
constexpr int kEntryShares = 2;
__global__ void __launch_bounds__(kThreads, 4) k_topk_digit2(TopkArgs a) {
    pdl_release(); pdl_wait();
    topk_digit2(a.tt, a.T, a.stride, a.tk, kEntryShares);
}
__global__ void __launch_bounds__(kThreads) k_topk_scan(TopkArgs a) {
    pdl_release(); pdl_wait();
    topk_scan(a.tt, a.T, a.stride, a.tk);
}
__global__ void __launch_bounds__(kThreads, 4) k_topk_write(TopkArgs a) {
    pdl_release(); pdl_wait();
    topk_write(a.xhat, a.tt, a.T, a.stride, a.tk, a.err, kEntryShares);
}

}  // namespace eg
