// Top-K messages (Top-K paragraph of Section 7): for every segment whose event sends a
// sparse message, find exactly the K_t entries with the largest |x - x_hat| (ties to the lower
// index), pack them as (index, value) in ascending index order into the replica's outbox,
// and deliver them into the mailbox x_hat.
//
// The rank key is the bit pattern of |x - x_hat| (fp32), which orders like the magnitude; its
// top digit is bits 30..20 (11 bits), digit 1 bits 19..10, digit 2 bits 9..0.  The K_t-th
// largest key tau is found exactly, in ONE pass over the tensor plus work on a few percent of it:
//   guess    a histogram of the top digit over a pseudo-random SAMPLE of the tensor's tiles
//            (one in 2 ... 16 for large tensors, all of them for small ones) gives a bin
//            b' that lies, with a safety margin, at or below the bin of tau;
//   collect  (reads x, x_hat once) every element whose top digit is >= b' is copied, tile by
//            tile and in index order, into an entry buffer as (top digit - b', 20 low key
//            bits, position, value of x); the entries are counted per top digit, and digit 1 of
//            the entries in the two lowest bins is histogrammed on the way;
//   resolve  the exact counts of the collected bins give the bin of tau (no sampling involved
//            any more: every element at or above b' is an entry) and the rank inside it; then
//            digit 1 from its histogram;
//   digit 2 together with per-tile counts, then ordered compaction into the outbox and delivery
//            into x_hat: two walks over the entries only.
// Where the guess fails -- fewer than K_t elements at or above b', or tau more than one bin
// above b' -- the segment is selected again the plain way: full histogram of the top digit,
// exact bin, collect.  With all tiles sampled the guess IS the exact bin, so small tensors and
// the repeat path are the two-pass radix select without any guessing.
// The host knows nothing about the decisions: a planning phase turns the device-side `sparse`
// flags into a compact list of work tiles and every other phase runs a fixed-size grid over that
// list.  All phases can run in one cooperative launch (k_topk_all, bottom of this file).
#pragma once
#include <cooperative_groups.h>

#include "eg_common.cuh"
#include "eg_fused_pipe.cuh"

namespace eg {

constexpr int kTopkCtasPerSm = 8;      // CTAs per multiprocessor of the tile kernels (they loop over the work list)
constexpr int kTopkSegCtasPerSm = 4;   // ... of the per-segment kernels

// The work tiles of a list are cut into chunks of equal size, kFine of them for every CTA of the
// tile phases: a phase whose tiles all cost the same gives a CTA kFine consecutive chunks, in the
// sampling phase (whose tiles do not) a CTA takes the next chunk whenever it has finished one.
constexpr int kFine = 16;
struct TopkPlan {
    int n_sparse;       // segments on the list
    int total_tiles;    // their tiles
    int chunk;          // work tiles per chunk
    int n_chunks;       // chunks planned
    int ticket;         // next chunk to hand out in the sampling phase
};

// A list of segments to select from and of their tiles.  List 0: the segments that send a sparse
// message in this iteration; list 1: those of them that are selected again without guessing.
struct WorkList {
    TopkPlan* plan;
    int* sp_seg;               // [P*T] segment id of the q-th listed segment
    int* sp_begin;             // [P*T+1] first work tile of the q-th listed segment
    int* cta_q;                // [chunks] list slot that holds the first work tile of chunk c
};

constexpr int kOffBins = 8;                // top digits b' .. b'+6 are told apart, anything above counts as b'+7
constexpr int kOffHist = 2;                // digit 1 is histogrammed for top digits b' and b'+1

struct TopkState {
    WorkList list[2];
    unsigned int* hist;        // [P*T][kMaxBins]
    unsigned int* prefix;      // [P*T] b' after the guess; key bits resolved so far afterwards (at the end: tau)
    unsigned int* remaining;   // [P*T] rank still to resolve (at the end: number of
                               //       entries equal to tau that are part of the message)
    unsigned int* offcnt;      // [P*T][kOffBins] entries per top digit, relative to b'
    uint8_t* offsel;           // [P*T] top digit of tau, relative to b'
    uint8_t* redo;             // [P*T] the guess failed: select again without guessing
    unsigned int* redo_count;  // number of such segments in this iteration
    unsigned long long* redo_total;   // ... since the context was created or reset
    uint2* ent;                // [P][stride] entries (meta, value bits) of a tile, at the tile's own offset
    int* tile_cand;            // [P][n_tiles][8] entries stored by each warp for the tile
    unsigned int* tile_sub;    // [P][n_tiles][8] of those, (greater than tau) | (equal to tau) << 16
    uint2* tile_count;         // [P][n_tiles] (greater, equal) per tile, then their prefixes
    int2* outbox;              // [P][sum K_t] (index, value bits)
    const long long* out_off;  // [T] start of tensor t inside one replica's outbox
    const long long* count;    // [T] K_t
    const long long* numel;    // [T] n_t
    long long out_stride;      // sum K_t
    float guess_margin;        // safety margin of the guess, in standard deviations of the sampled count
    // quantised Top-K messages (eg_set_quantisation in a Top-K context): which segments' values go
    // out as codes (SegState::quant == 1) and the exponent of their scale (found by the quantising
    // kernels before the select runs); nullptr: values in full precision
    const uint8_t* quant;      // [P*T]
    const int* qexp;           // [P*T]
    int quant_bits;
};

__device__ __forceinline__ unsigned int rank_key(float a, float b) {
    return __float_as_uint(__fsub_rn(a, b)) & 0x7fffffffu;
}

// digit 0: bits 30..20, digit 1: bits 19..10, digit 2: bits 9..0
__device__ __forceinline__ int digit_bits(int digit) { return digit == 0 ? kDigitBits0 : kDigitBits1; }

// One CTA (of up to kPlanThreads threads; the more, the shorter each thread's run of segments):
// compact list of the flagged segments and of their tiles, in segment order.  `main_list`: also
// forget the previous iteration's repeat requests.
constexpr int kPlanThreads = 1024;
__device__ __forceinline__ void topk_plan(int S, int T, const uint8_t* __restrict__ flagged,
                                          const int* __restrict__ seg_begin, const TopkState& tk,
                                          const WorkList& wl, int n_cta, bool main_list) {
    __shared__ int s_cnt[kPlanThreads], s_tiles[kPlanThreads];
    const int nt = (int)blockDim.x;
    const int per = (S + nt - 1) / nt;
    const int lo = threadIdx.x * per, hi = min(S, lo + per);
    int cnt = 0, tiles = 0;
    for (int s = lo; s < hi; ++s) {
        if (flagged[s]) { const int t = s % T; ++cnt; tiles += seg_begin[t + 1] - seg_begin[t]; }
        if (main_list) tk.redo[s] = 0;
    }
    if (main_list && threadIdx.x == 0) *tk.redo_count = 0u;
    s_cnt[threadIdx.x] = cnt;
    s_tiles[threadIdx.x] = tiles;
    __syncthreads();
    // inclusive scan (Hillis-Steele) over the per-thread totals
    for (int o = 1; o < nt; o <<= 1) {
        int a = 0, b = 0;
        if (threadIdx.x >= o) { a = s_cnt[threadIdx.x - o]; b = s_tiles[threadIdx.x - o]; }
        __syncthreads();
        s_cnt[threadIdx.x] += a;
        s_tiles[threadIdx.x] += b;
        __syncthreads();
    }
    // chunk c holds the work tiles [c * chunk, (c + 1) * chunk): note for every c the list slot
    // its first tile falls into, so that no phase has to search for it
    n_cta *= kFine;
    const int chunk = max(1, (s_tiles[nt - 1] + n_cta - 1) / n_cta);
    if (threadIdx.x == 0) { wl.plan->chunk = chunk; wl.plan->n_chunks = n_cta; wl.plan->ticket = 0; }
    int q = s_cnt[threadIdx.x] - cnt, w = s_tiles[threadIdx.x] - tiles;
    for (int s = lo; s < hi; ++s)
        if (flagged[s]) {
            const int t = s % T;
            const int w_end = w + seg_begin[t + 1] - seg_begin[t];
            wl.sp_seg[q] = s;
            wl.sp_begin[q] = w;
            for (int c = (w + chunk - 1) / chunk; c < n_cta && c * chunk < w_end; ++c) wl.cta_q[c] = q;
            ++q;
            w = w_end;
        }
    if (threadIdx.x == nt - 1) {
        wl.plan->n_sparse = s_cnt[threadIdx.x];
        wl.plan->total_tiles = s_tiles[threadIdx.x];
        wl.sp_begin[s_cnt[threadIdx.x]] = s_tiles[threadIdx.x];
    }
    __syncthreads();      // the shared arrays may be used again by a second call
}

// A run of work tiles and the list slot of its first tile.
struct WorkRange {
    int w0, w1, q;
};
// The chunks [first, first + count) of the list.
__device__ __forceinline__ WorkRange chunk_range(const WorkList& wl, int first, int count) {
    const int total = wl.plan->total_tiles;
    const int chunk = wl.plan->chunk;
    WorkRange r;
    r.w0 = (int)min((long long)total, (long long)first * chunk);
    r.w1 = (int)min((long long)total, (long long)r.w0 + (long long)count * chunk);
    r.q = (r.w0 < r.w1) ? wl.cta_q[first] : 0;
    return r;
}
// Contiguous share of this CTA.  `shares`: planned shares per CTA (a phase may run with a grid
// `shares` times smaller than planned).
__device__ __forceinline__ WorkRange work_range(const WorkList& wl, int shares = 1) {
    return chunk_range(wl, (int)blockIdx.x * shares * kFine, shares * kFine);
}

// Walks a CTA's share of the work list.  Segment-level values are re-read only when the
// segment changes, so consecutive tiles of one tensor cost two dependent loads, not six.
struct WorkCursor {
    int q, end, s, i, t, first_tile, begin;
    __device__ __forceinline__ void init(int q0) {
        q = q0 - 1;
        end = -1;
    }
    // returns the tile id of work item w; `changed` tells whether a new segment started
    __device__ __forceinline__ int advance(const WorkList& wl, const TileTable& tt, int T, int w,
                                           bool& changed) {
        changed = false;
        while (w >= end) {
            ++q;
            if (!EG_INDEX_OK(tt.err, q, wl.plan->n_sparse)) { changed = true; break; }   // (the loop would not end)
            begin = wl.sp_begin[q];
            end = wl.sp_begin[q + 1];
            changed = true;
        }
        if (changed) {
            s = wl.sp_seg[q];
            i = s / T;
            t = s - i * T;
            first_tile = tt.seg_begin[t];
        }
        return first_tile + (w - begin);
    }
};

// ---------------------------------------------------------------------------------------
// The sample.  Of a tensor with K_t wanted entries one tile (4096 consecutive elements) in
// 2^shift is looked at, chosen by a hash of the tile's number (the first tile always), so that
// about 600 of the wanted entries fall into the sample whatever the size of the tensor (the
// relative error of a count of 600 is 4 %).  Whole tiles, because a tile that is skipped costs
// nothing, while a tile of which only some lines are read costs as much time as a whole one.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ int sample_shift(long long k_t) {
    int sh = 0;
    while (sh < 4 && (k_t >> (sh + 1)) >= 600) ++sh;
    return sh;
}
__device__ __forceinline__ bool tile_sampled(unsigned int tile_in_tensor, unsigned int salt, int shift) {
    unsigned int h = (tile_in_tensor + salt * 0x9E3779B1u) * 0x85EBCA77u;
    h ^= h >> 15;
    h *= 0xC2B2AE3Du;
    h ^= h >> 13;
    return tile_in_tensor == 0u || (h & ((1u << shift) - 1u)) == 0u;
}

// Histogram of the top digit of the keys of the work tiles: of the sampled tiles only (`sampled`),
// or of every element.
__device__ __forceinline__ void
topk_hist(const float* __restrict__ x, const float* __restrict__ xhat, TileTable tt, int T,
          long long stride, const TopkState& tk, const WorkList& wl, bool sampled) {
    __shared__ unsigned int s_hist[kMaxBins];
    for (int b = threadIdx.x; b < kMaxBins; b += kThreads) s_hist[b] = 0;
    __syncthreads();
    // every tile costs the same when all are read: one contiguous share; sampled: chunk after
    // chunk as handed out by a counter, because the fraction that is read differs from tensor to
    // tensor
    __shared__ int s_ticket;
    const int n_chunks = wl.plan->n_chunks;
    for (int first = (int)blockIdx.x * kFine;;) {
        if (sampled) {
            __syncthreads();                  // everybody has read the previous ticket
            if (threadIdx.x == 0) s_ticket = atomicAdd(&wl.plan->ticket, 1);
            __syncthreads();
            first = s_ticket;
        }
        if (first >= n_chunks) break;
        const WorkRange r = chunk_range(wl, first, sampled ? 1 : kFine);
        if (r.w0 >= r.w1) break;
        WorkCursor cur;
        cur.init(r.q);
        int shift = 0;
        bool any = false;                     // something of the current segment sits in s_hist
        for (int w = r.w0; w < r.w1; ++w) {
            bool changed;
            const int tile = cur.advance(wl, tt, T, w, changed);
            if (changed) shift = sampled ? sample_shift(tk.count[cur.t]) : 0;
            if (shift == 0 || tile_sampled((unsigned int)(tile - cur.first_tile), (unsigned int)cur.s, shift)) {
                any = true;
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
            }
            // flush when the next tile belongs to another segment (or this was the last one)
            if ((w + 1 == r.w1 || w + 1 >= cur.end) && any) {
                __syncthreads();
                unsigned int* gh = tk.hist + (long long)cur.s * kMaxBins;
                for (int b = threadIdx.x; b < kMaxBins; b += kThreads) {
                    const unsigned int v = s_hist[b];
                    if (v) { atomicAdd(&gh[b], v); s_hist[b] = 0; }
                }
                __syncthreads();
                any = false;
            }
        }
        if (!sampled) break;
    }
}

// One warp: the bin of a histogram of `nbins` bins (a multiple of 1024) that holds rank `rem`,
// counting from the highest bin downwards; the histogram is cleared on the way.  It is walked in
// blocks of 1024 bins from the top; a lane owns 32 consecutive bins of a block (eight 16-byte
// loads, all in flight together), one warp scan places the rank in a lane, which then walks
// its own bins.  Returns false when the histogram holds fewer than `rem` keys.  `bin` and
// `above_out` (keys in the bins above the chosen one) are valid in every lane.
__device__ __forceinline__ bool
pick_bin(unsigned int* gh, int nbins, unsigned int rem, unsigned int& bin, unsigned int& above_out) {
    constexpr int kBlock = 1024, kPer = kBlock / 32;
    const int lane = threadIdx.x & 31;
    unsigned int above_blocks = 0;      // keys in the blocks already walked
    bool found = false;                 // the same in every lane
    unsigned int my_bin = 0, my_above = 0;
    int owner = 0;
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
                    my_bin = (unsigned int)(blk * kBlock + lane * kPer + z);
                    my_above = above;
                    done = true;
                }
                above += c[z];
            }
        }
        const unsigned int where = __ballot_sync(0xffffffffu, here);
        if (where) { found = true; owner = __ffs(where) - 1; }
        above_blocks += __shfl_sync(0xffffffffu, inc, 0);
    }
    bin = __shfl_sync(0xffffffffu, my_bin, owner);
    above_out = __shfl_sync(0xffffffffu, my_above, owner);
    return found;
}

// One warp per listed segment: digit `digit` (0 or 2) of tau from the segment's histogram.
// Digit 0 is only taken this way from a histogram over ALL elements of the tensor.
__device__ __forceinline__ void
topk_pick(int T, const TopkState& tk, const WorkList& wl, int digit) {
    const int nq = wl.plan->n_sparse;
    const int nbins = 1 << digit_bits(digit);
    const int lane = threadIdx.x & 31;
    const int nwarps = gridDim.x * kWarps;
    for (int q = blockIdx.x * kWarps + (threadIdx.x >> 5); q < nq; q += nwarps) {
        const int s = wl.sp_seg[q];
        const int t = s % T;
        const unsigned int rem = (digit == 0) ? (unsigned int)tk.count[t] : tk.remaining[s];
        unsigned int bin, above;
        const bool found = pick_bin(tk.hist + (long long)s * kMaxBins, nbins, rem, bin, above);
        if (lane == 0 && found) {
            const unsigned int old = (digit == 0) ? 0u : tk.prefix[s];
            tk.prefix[s] = (old << digit_bits(digit)) | bin;
            tk.remaining[s] = rem - above;
        }
    }
}

// One warp per sparse segment: from the histogram of the sampled tiles, a bin b' that is at or
// below the bin of the K_t-th largest key unless the sample is off by more than the margin.
// With m of the tensor's n elements in the sample, the number of sampled elements among the
// K_t largest has mean K_t m / n and variance about K_t (m / n)(1 - m / n); b' is the bin that
// holds the sample's rank mean + margin * deviation + 1.  A sample that holds every element
// (m == n) makes b' the exact bin.  A rank beyond the sample gives b' = 0: everything is collected.
__device__ __forceinline__ void
topk_guess(int T, const TopkState& tk, const WorkList& wl) {
    const int nq = wl.plan->n_sparse;
    const int lane = threadIdx.x & 31;
    const int nwarps = gridDim.x * kWarps;
    for (int q = blockIdx.x * kWarps + (threadIdx.x >> 5); q < nq; q += nwarps) {
        const int s = wl.sp_seg[q];
        const int t = s % T;
        unsigned int* gh = tk.hist + (long long)s * kMaxBins;
        const long long K = tk.count[t], n = tk.numel[t];
        unsigned int rank = (unsigned int)K;
        if (sample_shift(K) != 0) {
            // size of the sample: the tiles are chosen by a hash, so their number varies
            unsigned int m = 0;
            const uint4* g4 = reinterpret_cast<const uint4*>(gh);
            for (int j = lane; j < kMaxBins / 4; j += 32) { const uint4 v = g4[j]; m += v.x + v.y + v.z + v.w; }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) m += __shfl_xor_sync(0xffffffffu, m, o);
            if ((long long)m < n) {
                const float frac = (float)m / (float)n;
                const float mean = (float)K * frac;
                const float dev = sqrtf(fmaxf(mean * (1.f - frac), 0.f));
                const float want = ceilf(mean + tk.guess_margin * dev) + 1.f;
                rank = (unsigned int)fminf(fmaxf(want, 1.f), 4.0e9f);
            }
        }
        unsigned int bin, above;
        const bool found = pick_bin(gh, kMaxBins, rank, bin, above);
        if (lane == 0) tk.prefix[s] = found ? bin : 0u;
    }
}

constexpr int kSubSlices = kWarps;                       // entry sub-slices per tile: one per warp
constexpr int kWarpSpan = kNormTile / kWarps;            // 512 consecutive elements of a tile per warp
constexpr int kSubChunks = kWarpSpan / 128;              // read as 4 chunks of 128 (one float4 per lane)
static_assert(kWarpSpan == 512 && kSubChunks == 4, "entry words hold a 9-bit position and four 8-bit counts");

// An entry describes one element whose top digit is at least b':
//   meta = min(top digit - b', 7) << 29 | (key & 0xfffff) << 9 | position inside the warp's 512 elements
//   val  = bits of x at that element
// Once the bin of tau is known (offsel, relative to b'), an entry with a larger top digit is part
// of the message whatever its lower digits say, one with a smaller top digit is not, and for the
// others the 20 low key bits decide.
__device__ __forceinline__ unsigned int ent_low20(unsigned int meta) { return (meta >> 9) & 0xfffffu; }
__device__ __forceinline__ unsigned int ent_off(unsigned int meta) { return meta >> 29; }

// Warp w of a CTA owns elements [512 w, 512 w + 512) of a tile; its entries start at the same
// place in the tile's slice of the entry buffer, so the slices can never overlap.
__device__ __forceinline__ int sub_offset(int len, int w) { return min(len, w * kWarpSpan); }

// The collecting pass: per tile, every element whose top digit is at least b' is copied as an
// entry into the tile's slice of the entry buffer, IN ASCENDING INDEX ORDER inside each warp's
// sub-slice (the later phases rely on that order: concatenating the sub-slices of a tensor's
// tiles lists its entries by index).  The entries are counted per top digit and digit 1 of those
// in the two lowest bins is histogrammed on the way.  Nothing is shared between warps except
// these counters.  Entries are few, so the work is split: every lane MARKS its sixteen elements
// in four 4-bit masks (one floating-point comparison per element: non-negative floats order
// like their bit patterns, so |x - x_hat| >= the float whose bits are b' << 20 says the same as
// the comparison of the top digits); one warp scan of the four packed 8-bit counts (a chunk
// holds 128 elements, so a field cannot overflow) gives every lane its first slot in each chunk;
// the marked elements go to a small per-warp staging area in slot order, and the warp then
// turns them into entries side by side, one per lane, with coalesced stores.
constexpr int kStage = 128;     // staged elements per warp and tile; fuller sub-slices are written directly
__device__ __forceinline__ void
topk_collect(const float* __restrict__ x, const float* __restrict__ xhat, TileTable tt, int T,
             long long stride, const TopkState& tk, const WorkList& wl) {
    constexpr int kBins1 = 1 << kDigitBits1;
    static_assert(kOffHist * kBins1 == kMaxBins, "the digit-1 histograms of two bins share the segment's histogram");
    __shared__ unsigned int s_hist[kOffHist * kBins1];
    __shared__ unsigned int s_off[kOffBins];
    __shared__ float2 s_pair[kWarps][kStage];             // (x, x_hat) of a marked element
    __shared__ unsigned short s_where[kWarps][kStage];    // its position inside the warp's 512 elements
    WorkRange r = work_range(wl);
    if (r.w0 >= r.w1) return;
    for (int b = threadIdx.x; b < kOffHist * kBins1; b += kThreads) s_hist[b] = 0;
    if (threadIdx.x < kOffBins) s_off[threadIdx.x] = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int mine = warp * kWarpSpan + lane * 4;      // this lane's first element of the tile
    WorkCursor cur;
    cur.init(r.q);
    unsigned int b0 = 0;
    float thr = 0.f;
    // one entry from an element: counted, digit 1 histogrammed, stored at slot `pos`
    auto emit = [&](uint2* ent, int room, float xv, float hv, unsigned int pos, unsigned int where) {
        const unsigned int k = rank_key(xv, hv);
        const unsigned int off = min((k >> 20) - b0, (unsigned int)(kOffBins - 1));
        if (!EG_INDEX_OK(tt.err, pos, room)) return;
        ent[pos] = make_uint2((off << 29) | ((k & 0xfffffu) << 9) | where, __float_as_uint(xv));
        atomicAdd(&s_off[off], 1u);
        if (off < (unsigned int)kOffHist) atomicAdd(&s_hist[off * kBins1 + ((k >> 10) & (kBins1 - 1))], 1u);
    };
    for (int w = r.w0; w < r.w1; ++w) {
        bool changed;
        const int tile = cur.advance(wl, tt, T, w, changed);
        if (changed) { b0 = tk.prefix[cur.s]; thr = __uint_as_float(b0 << 20); }
        const int i = cur.i;
        const int len = tt.length[tile];
        const long long base = (long long)i * stride + tt.offset[tile];
        float4 a[kSubChunks], b[kSubChunks];
        unsigned int mask = 0, packed = 0;      // bit 4j+c: element c of chunk j is an entry
        if (len == kNormTile) {                 // a whole tile: no element needs a length test
#pragma unroll
            for (int j = 0; j < kSubChunks; ++j) {
                a[j] = ld_stream(x + base + mine + j * 128);
                b[j] = ld_stream(xhat + base + mine + j * 128);
            }
#pragma unroll
            for (int j = 0; j < kSubChunks; ++j) {
                unsigned int m = 0;
                m |= !(fabsf(__fsub_rn(a[j].x, b[j].x)) < thr) ? 1u : 0u;
                m |= !(fabsf(__fsub_rn(a[j].y, b[j].y)) < thr) ? 2u : 0u;
                m |= !(fabsf(__fsub_rn(a[j].z, b[j].z)) < thr) ? 4u : 0u;
                m |= !(fabsf(__fsub_rn(a[j].w, b[j].w)) < thr) ? 8u : 0u;
                mask |= m << (4 * j);
                packed |= (unsigned int)__popc(m) << (8 * j);
            }
        } else {
#pragma unroll
            for (int j = 0; j < kSubChunks; ++j) {
                const int local = mine + j * 128;
                a[j] = b[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (local < len) { a[j] = ld_stream(x + base + local); b[j] = ld_stream(xhat + base + local); }
            }
#pragma unroll
            for (int j = 0; j < kSubChunks; ++j) {
                const int nel = len - (mine + j * 128);   // live elements of this float4 (<= 0: none)
                unsigned int m = 0;
                m |= (0 < nel && !(fabsf(__fsub_rn(a[j].x, b[j].x)) < thr)) ? 1u : 0u;
                m |= (1 < nel && !(fabsf(__fsub_rn(a[j].y, b[j].y)) < thr)) ? 2u : 0u;
                m |= (2 < nel && !(fabsf(__fsub_rn(a[j].z, b[j].z)) < thr)) ? 4u : 0u;
                m |= (3 < nel && !(fabsf(__fsub_rn(a[j].w, b[j].w)) < thr)) ? 8u : 0u;
                mask |= m << (4 * j);
                packed |= (unsigned int)__popc(m) << (8 * j);
            }
        }
        unsigned int inc = packed;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned int u = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += u;
        }
        const unsigned int tot = __shfl_sync(0xffffffffu, inc, 31);
        const unsigned int excl = inc - packed;
        const unsigned int total = (tot & 0xffu) + ((tot >> 8) & 0xffu) + ((tot >> 16) & 0xffu) + (tot >> 24);
        uint2* ent = tk.ent + base + sub_offset(len, warp);
        const int room = len - sub_offset(len, warp);      // slots of this sub-slice (bounds-checked build)
        if (total <= (unsigned int)kStage) {
            unsigned int chunk_first = 0;
#pragma unroll
            for (int j = 0; j < kSubChunks; ++j) {
                const unsigned int m = (mask >> (4 * j)) & 0xfu;
                if (m) {                                         // few lanes hold an entry in a given chunk
                    unsigned int pos = chunk_first + ((excl >> (8 * j)) & 0xffu);
                    const unsigned short where = (unsigned short)(j * 128 + lane * 4);
                    if (m & 1u) { s_pair[warp][pos] = make_float2(a[j].x, b[j].x); s_where[warp][pos++] = where; }
                    if (m & 2u) { s_pair[warp][pos] = make_float2(a[j].y, b[j].y); s_where[warp][pos++] = where + 1; }
                    if (m & 4u) { s_pair[warp][pos] = make_float2(a[j].z, b[j].z); s_where[warp][pos++] = where + 2; }
                    if (m & 8u) { s_pair[warp][pos] = make_float2(a[j].w, b[j].w); s_where[warp][pos++] = where + 3; }
                }
                chunk_first += (tot >> (8 * j)) & 0xffu;
            }
            __syncwarp();
            for (unsigned int e = lane; e < total; e += 32) {
                const float2 v = s_pair[warp][e];
                emit(ent, room, v.x, v.y, e, s_where[warp][e]);
            }
            __syncwarp();
        } else {
            unsigned int chunk_first = 0;
#pragma unroll
            for (int j = 0; j < kSubChunks; ++j) {
                const unsigned int m = (mask >> (4 * j)) & 0xfu;
                if (m) {
                    unsigned int pos = chunk_first + ((excl >> (8 * j)) & 0xffu);
                    const unsigned int where = (unsigned int)(j * 128 + lane * 4);
                    if (m & 1u) emit(ent, room, a[j].x, b[j].x, pos++, where);
                    if (m & 2u) emit(ent, room, a[j].y, b[j].y, pos++, where + 1);
                    if (m & 4u) emit(ent, room, a[j].z, b[j].z, pos++, where + 2);
                    if (m & 8u) emit(ent, room, a[j].w, b[j].w, pos++, where + 3);
                }
                chunk_first += (tot >> (8 * j)) & 0xffu;
            }
        }
        if (lane == 0) tk.tile_cand[((long long)i * tt.n_tiles + tile) * kSubSlices + warp] = (int)total;
        if (w + 1 == r.w1 || w + 1 >= cur.end) {   // last tile of this segment here
            __syncthreads();
            unsigned int* gh = tk.hist + (long long)cur.s * kMaxBins;
            for (int b = threadIdx.x; b < kOffHist * kBins1; b += kThreads) {
                const unsigned int v = s_hist[b];
                if (v) { atomicAdd(&gh[b], v); s_hist[b] = 0; }
            }
            if (threadIdx.x < kOffBins) {
                const unsigned int v = s_off[threadIdx.x];
                if (v) { atomicAdd(&tk.offcnt[(long long)cur.s * kOffBins + threadIdx.x], v); s_off[threadIdx.x] = 0; }
            }
            __syncthreads();
        }
    }
}

// The collecting pass with the tiles staged through shared memory (the form the single-phase
// launch uses; needs eg_fused_pipe.cuh's barrier and bulk-copy wrappers).  Same entries, counts
// and histograms as topk_collect.  One producer warp walks the CTA's share of the work list and
// brings tile after tile -- 16 KB of x and 16 KB of x_hat, two bulk asynchronous copies -- into a
// ring of kCollectStages stages together with a small header (segment, bin, length, where the
// entries go), so that the bytes in flight do not depend on what the eight consumer warps are
// doing; the consumers read their 512 elements from shared memory, mark them, and since the
// tile stays where it is they build the entries from it by position afterwards.
constexpr int kCollectStages = 3;
constexpr int kCollectThreads = kThreads + 32;
struct CollectHeader {
    int len, i, tile, s;        // elements of the tile, replica, tile id, segment id
    unsigned int b0;            // the bin b' of the segment
    int last_of_segment;        // flush the counters after this tile
    int pad[2];
};
struct CollectSmem {
    static constexpr int kStageBytes = 2 * kNormTile * 4;                       // x, x_hat
    static constexpr int kHeaders = kCollectStages * kStageBytes;
    static constexpr int kBars = kHeaders + kCollectStages * (int)sizeof(CollectHeader);
    static constexpr int kHist = kBars + 8 * 2 * kCollectStages + 16;             // full[S], empty[S], abort flag
    static constexpr int kOff = kHist + kMaxBins * 4;
    static constexpr int kWhere = kOff + kOffBins * 4 + 32;
    static constexpr int kBytes = kWhere + kWarps * kWarpSpan * 2;                // a position per possible entry
};

__device__ __forceinline__ void
topk_collect_staged(const float* __restrict__ x, const float* __restrict__ xhat, TileTable tt, int T,
                    long long stride, const TopkState& tk, const WorkList& wl, unsigned int* __restrict__ err,
                    int shares) {
    constexpr int kBins1 = 1 << kDigitBits1;
    extern __shared__ __align__(128) unsigned char smem[];
    CollectHeader* headers = reinterpret_cast<CollectHeader*>(smem + CollectSmem::kHeaders);
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + CollectSmem::kBars);
    uint64_t* empty = full + kCollectStages;
    volatile int* s_abort = reinterpret_cast<volatile int*>(empty + kCollectStages);
    unsigned int* s_hist = reinterpret_cast<unsigned int*>(smem + CollectSmem::kHist);
    unsigned int* s_off = reinterpret_cast<unsigned int*>(smem + CollectSmem::kOff);
    unsigned short* s_where = reinterpret_cast<unsigned short*>(smem + CollectSmem::kWhere);
    const WorkRange r = work_range(wl, shares);
    if (r.w0 >= r.w1) return;                   // the same in every thread
    const int tid = threadIdx.x;
    for (int b = tid; b < kMaxBins; b += kCollectThreads) s_hist[b] = 0;
    if (tid < kOffBins) s_off[tid] = 0;
    if (tid == 0) {
        for (int s = 0; s < kCollectStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], kWarps); }
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (tid >= kThreads) {
        // ------------------------------------------------------------------ producer (one lane)
        if (tid == kThreads) {
            WorkCursor cur;
            cur.init(r.q);
            unsigned int b0 = 0;
            int s = 0;
            for (int w = r.w0, n = 0; w < r.w1; ++w, ++n) {
                bool changed;
                const int tile = cur.advance(wl, tt, T, w, changed);
                if (changed) b0 = tk.prefix[cur.s];
                const int len = tt.length[tile];
                const long long base = (long long)cur.i * stride + tt.offset[tile];
                if (n >= kCollectStages &&
                    !mbar_wait_bounded(&empty[s], (uint32_t)((n / kCollectStages - 1) & 1), s_abort, err))
                    break;
                CollectHeader h;
                h.len = len; h.i = cur.i; h.tile = tile; h.s = cur.s; h.b0 = b0;
                h.last_of_segment = (w + 1 == r.w1 || w + 1 >= cur.end) ? 1 : 0;
                h.pad[0] = h.pad[1] = 0;
                headers[s] = h;
                const uint32_t bytes = (uint32_t)(((len + 3) & ~3) * 4);
                float* st = reinterpret_cast<float*>(smem + s * CollectSmem::kStageBytes);
                mbar_expect_tx(&full[s], 2u * bytes);      // (a release: the header is visible with the data)
                bulk_g2s(st, x + base, bytes, &full[s]);
                bulk_g2s(st + kNormTile, xhat + base, bytes, &full[s]);
                if (++s == kCollectStages) s = 0;
            }
        }
    } else {
        // ------------------------------------------------------------------ consumers
        const int lane = tid & 31, warp = tid >> 5;
        const int mine = warp * kWarpSpan + lane * 4;      // this lane's first element of the tile
        unsigned short* my_where = s_where + warp * kWarpSpan;
        int s = 0;
        for (int w = r.w0, n = 0; w < r.w1; ++w, ++n) {
            if (!mbar_wait_bounded(&full[s], (uint32_t)((n / kCollectStages) & 1), s_abort, err)) break;
            const CollectHeader h = headers[s];
            const float* sx = reinterpret_cast<const float*>(smem + s * CollectSmem::kStageBytes);
            const float* sh = sx + kNormTile;
            const unsigned int b0 = h.b0;
            const float thr = __uint_as_float(b0 << 20);
            const int len = h.len;
            unsigned int mask = 0, packed = 0;      // bit 4j+c: element c of chunk j is an entry
#pragma unroll
            for (int j = 0; j < kSubChunks; ++j) {
                const int local = mine + j * 128;
                const int nel = len - local;          // live elements of this float4 (<= 0: none)
                unsigned int m = 0;
                if (nel > 0) {
                    const float4 a = *reinterpret_cast<const float4*>(sx + local);
                    const float4 b = *reinterpret_cast<const float4*>(sh + local);
                    m |= !(fabsf(__fsub_rn(a.x, b.x)) < thr) ? 1u : 0u;
                    m |= (1 < nel && !(fabsf(__fsub_rn(a.y, b.y)) < thr)) ? 2u : 0u;
                    m |= (2 < nel && !(fabsf(__fsub_rn(a.z, b.z)) < thr)) ? 4u : 0u;
                    m |= (3 < nel && !(fabsf(__fsub_rn(a.w, b.w)) < thr)) ? 8u : 0u;
                }
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
            const unsigned int total = (tot & 0xffu) + ((tot >> 8) & 0xffu) + ((tot >> 16) & 0xffu) + (tot >> 24);
            // positions of the marked elements, in slot order
            unsigned int chunk_first = 0;
#pragma unroll
            for (int j = 0; j < kSubChunks; ++j) {
                const unsigned int m = (mask >> (4 * j)) & 0xfu;
                if (m) {                                         // few lanes hold an entry in a given chunk
                    unsigned int pos = chunk_first + ((excl >> (8 * j)) & 0xffu);
                    const unsigned short where = (unsigned short)(j * 128 + lane * 4);
                    if (m & 1u) my_where[pos++] = where;
                    if (m & 2u) my_where[pos++] = where + 1;
                    if (m & 4u) my_where[pos++] = where + 2;
                    if (m & 8u) my_where[pos++] = where + 3;
                }
                chunk_first += (tot >> (8 * j)) & 0xffu;
            }
            __syncwarp();
            // the entries, one per lane, from the tile in shared memory
            const long long base = (long long)h.i * stride + tt.offset[h.tile];
            uint2* ent = tk.ent + base + sub_offset(len, warp);
            const int room = len - sub_offset(len, warp);      // slots of this sub-slice (bounds-checked build)
            for (unsigned int e = lane; e < total; e += 32) {
                const unsigned int where = my_where[e];
                const float xv = sx[warp * kWarpSpan + where];
                const unsigned int k = rank_key(xv, sh[warp * kWarpSpan + where]);
                const unsigned int off = min((k >> 20) - b0, (unsigned int)(kOffBins - 1));
                if (!EG_INDEX_OK(tt.err, e, room)) continue;
                ent[e] = make_uint2((off << 29) | ((k & 0xfffffu) << 9) | where, __float_as_uint(xv));
                atomicAdd(&s_off[off], 1u);
                if (off < (unsigned int)kOffHist) atomicAdd(&s_hist[off * kBins1 + ((k >> 10) & (kBins1 - 1))], 1u);
            }
            if (lane == 0) tk.tile_cand[((long long)h.i * tt.n_tiles + h.tile) * kSubSlices + warp] = (int)total;
            // everything this warp needs from the stage has been read
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[s]);
            if (h.last_of_segment) {
                // the eight consumer warps meet (the producer does not take part)
                asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory");
                unsigned int* gh = tk.hist + (long long)h.s * kMaxBins;
                for (int b = tid; b < kMaxBins; b += kThreads) {
                    const unsigned int v = s_hist[b];
                    if (v) { atomicAdd(&gh[b], v); s_hist[b] = 0; }
                }
                if (tid < kOffBins) {
                    const unsigned int v = s_off[tid];
                    if (v) { atomicAdd(&tk.offcnt[(long long)h.s * kOffBins + tid], v); s_off[tid] = 0; }
                }
                asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory");
            }
            if (++s == kCollectStages) s = 0;
        }
    }
    if (*s_abort) {
        // failure path only: give copies in flight time to land before the CTA retires
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) {}
    }
}

// One warp per listed segment, after the collecting pass: the exact counts of the collected bins
// place tau's top digit (counting K_t entries down from the highest bin) and the rank left
// inside that bin; digit 1 then comes from the bin's digit-1 histogram.  A segment whose guess
// did not work out -- fewer than K_t entries, tau in the catch-all bin, or in a bin without a
// digit-1 histogram -- is marked for the exact repeat instead.  Both histograms and the
// counters are left cleared.
__device__ __forceinline__ void
topk_resolve(int T, const TopkState& tk, const WorkList& wl, bool is_repeat, unsigned int* __restrict__ err) {
    constexpr int kBins1 = 1 << kDigitBits1;
    const int nq = wl.plan->n_sparse;
    const int lane = threadIdx.x & 31;
    const int nwarps = gridDim.x * kWarps;
    for (int q = blockIdx.x * kWarps + (threadIdx.x >> 5); q < nq; q += nwarps) {
        const int s = wl.sp_seg[q];
        const int t = s % T;
        unsigned int* oc = tk.offcnt + (long long)s * kOffBins;
        const unsigned int mine = (lane < kOffBins) ? oc[lane] : 0u;
        if (lane < kOffBins) oc[lane] = 0u;
        const unsigned int K = (unsigned int)tk.count[t];
        unsigned int above = 0;
        int sel = -1;
#pragma unroll
        for (int o = kOffBins - 1; o >= 0; --o) {
            const unsigned int c = __shfl_sync(0xffffffffu, mine, o);
            if (sel < 0) {
                if (K <= above + c) sel = o; else above += c;
            }
        }
        unsigned int* gh = tk.hist + (long long)s * kMaxBins;
        const bool ok = sel >= 0 && sel < kOffHist;
        bool found = false;
        if (ok) {
            unsigned int bin, above1;
            const unsigned int rem = K - above;
            found = pick_bin(gh + sel * kBins1, kBins1, rem, bin, above1);
            if (lane == 0 && found) {
                tk.prefix[s] = ((tk.prefix[s] + (unsigned int)sel) << kDigitBits1) | bin;
                tk.remaining[s] = rem - above1;
                tk.offsel[s] = (uint8_t)sel;
            }
        }
        // clear what pick_bin has not walked
        for (int h = 0; h < kOffHist; ++h) {
            if (ok && h == sel) continue;
            uint4* g4 = reinterpret_cast<uint4*>(gh + h * kBins1);
            for (int j = lane; j < kBins1 / 4; j += 32) g4[j] = make_uint4(0u, 0u, 0u, 0u);
        }
        if (lane == 0 && !(ok && found)) {
            if (is_repeat) {
                atomicOr(err, kErrTopkSlot);      // an exact bin always resolves
            } else {
                tk.redo[s] = 1;
                atomicAdd(tk.redo_count, 1u);
                atomicAdd(tk.redo_total, 1ull);
            }
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
    __device__ __forceinline__ void init(const WorkList& wl, int shares = 1) {
        r = work_range(wl, shares);
        cur.init(r.q);
        w = r.w0 + (int)(threadIdx.x >> 5);
    }
    __device__ __forceinline__ bool next(const WorkList& wl, const TileTable& tt, int T, WarpTile& z) {
        if (w >= r.w1) return false;
        bool changed;
        z.tile = cur.advance(wl, tt, T, w, changed);
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
    __device__ __forceinline__ void init(const TopkState& tk, const WorkList& wl, const TileTable& tt, int T,
                                         int shares) {
        walk.init(wl, shares);
        have = walk.next(wl, tt, T, ahead);
        ahead_mine = have ? fetch(tk, tt) : 0;
    }
    __device__ __forceinline__ bool next(const TopkState& tk, const WorkList& wl, const TileTable& tt, int T,
                                         WarpTile& z, int& mine) {
        if (!have) return false;
        z = ahead;
        mine = ahead_mine;
        have = walk.next(wl, tt, T, ahead);
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
// that have some are counted again once tau is complete (topk_recount).
__device__ __forceinline__ void
topk_digit2(TileTable tt, int T, long long stride, const TopkState& tk, const WorkList& wl, int shares = 1) {
    const int lane = threadIdx.x & 31, u = lane / kGroupLanes, r = lane % kGroupLanes;
    TileFeed feed;
    feed.init(tk, wl, tt, T, shares);
    WarpTile z;
    int n;                               // entries of this lane's sub-slice
    int s_now = -1;
    unsigned int want = 0, sel = 0;
    unsigned int* gh = nullptr;
    while (feed.next(tk, wl, tt, T, z, n)) {
        if (z.s != s_now) {
            s_now = z.s;
            want = tk.prefix[z.s] & ((1u << kDigitBits1) - 1);      // digit 1 of tau
            sel = tk.offsel[z.s];
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
                const unsigned int off = ent_off(meta[q]), low = ent_low20(meta[q]), d1 = low >> kDigitBits2;
                if (live && (off > sel || (off == sel && d1 > want))) ++gt;
                if (live && off == sel && d1 == want) {
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
count_tile_exact(const TileTable& tt, long long stride, const TopkState& tk, int i, int tile, unsigned int sel,
                 unsigned int tau20) {
    const int lane = threadIdx.x & 31, u = lane / kGroupLanes, r = lane % kGroupLanes;
    const long long index = (long long)i * tt.n_tiles + tile;
    const int n = tk.tile_cand[index * kSubSlices + u];
    const int len = tt.length[tile];
    const uint2* sub = tk.ent + (long long)i * stride + tt.offset[tile] + min(len, u * kWarpSpan);
    unsigned int gt = 0, eq = 0;
    for (int f = r; f < n; f += kGroupLanes) {
        const unsigned int meta = sub[f].x, off = ent_off(meta), low = ent_low20(meta);
        if (off > sel || (off == sel && low > tau20)) ++gt;
        else if (off == sel && low == tau20) ++eq;
    }
    store_tile_counts(tk, index * kSubSlices, index, gt, eq);
}

// Once tau is complete: the tiles that held open entries are counted again (a handful per tensor
// unless many keys tie).  One warp per tile of the work list; a tile without open entries costs
// one 8-byte read.
__device__ __forceinline__ void
topk_recount(TileTable tt, int T, long long stride, const TopkState& tk, const WorkList& wl, int shares = 1) {
    WarpWalk walk;
    walk.init(wl, shares);
    WarpTile z;
    int s_now = -1;
    unsigned int tau20 = 0, sel = 0;
    while (walk.next(wl, tt, T, z)) {
        if (tk.tile_count[(long long)z.i * tt.n_tiles + z.tile].y == 0u) continue;     // the same in every lane
        if (z.s != s_now) { s_now = z.s; tau20 = tk.prefix[z.s] & 0xfffffu; sel = tk.offsel[z.s]; }
        count_tile_exact(tt, stride, tk, z.i, z.tile, sel, tau20);
    }
}

// One CTA per sparse segment: the exclusive prefix of the tile counts, in tile order.
__device__ __forceinline__ void
topk_scan(TileTable tt, int T, long long stride, const TopkState& tk, const WorkList& wl) {
    __shared__ unsigned int s_gt[kWarps], s_eq[kWarps];
    __shared__ unsigned int s_run[2];
    const int nq = wl.plan->n_sparse;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int q = blockIdx.x; q < nq; q += gridDim.x) {
        const int s = wl.sp_seg[q];
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

// Ordered compaction of the selected entries into the outbox, and delivery: the same
// (index, value) pairs are written into the mailbox x_hat, which is what the receivers hold
// once the message has arrived.  Works from the entries alone (a few percent of the tensor);
// x and x_hat are not read again.
// (Delivering from the averaging kernel that runs next -- it reads x and x_hat anyway and can
// tell the entries greater than tau by one comparison -- was built and measured: the scattered
// words here cost as much as the comparisons there, and the quiet iterations paid for the
// larger kernel, so the delivery stayed here.)
// An entry is selected if key > tau, or key == tau and fewer than `remaining` equal keys
// precede it in the tensor.  Its slot is (#greater before it) + min(#equal before it, remaining).
// One warp per tile; within a sub-slice the entries are taken in index order, four at a time by
// the four lanes of the sub-slice, and ballots give every lane the number of greater / equal
// entries before its own.
__device__ __forceinline__ void
topk_write(float* xhat, TileTable tt, int T, long long stride, const TopkState& tk, const WorkList& wl,
           unsigned int* __restrict__ err, int shares = 1) {
    const int lane = threadIdx.x & 31, u = lane / kGroupLanes, r = lane % kGroupLanes;
    const unsigned int group = (unsigned int)((1u << kGroupLanes) - 1u) << (u * kGroupLanes);   // lanes of this sub-slice
    const unsigned int lower = ((1u << r) - 1u) << (u * kGroupLanes);                            // ... before this lane
    TileFeed feed;
    feed.init(tk, wl, tt, T, shares);
    WarpTile z;
    int n;
    int s_now = -1;
    unsigned int tau20 = 0, take = 0, K = 0, sel = 0;
    int2* out = nullptr;
    bool coded = false;            // the segment's values go out as codes of the change
    double up = 1.0, down = 1.0, qmax = 0.0;
    while (feed.next(tk, wl, tt, T, z, n)) {
        if (z.s != s_now) {
            s_now = z.s;
            tau20 = tk.prefix[z.s] & 0xfffffu;
            sel = tk.offsel[z.s];
            take = tk.remaining[z.s];
            K = (unsigned int)tk.count[z.t];
            out = tk.outbox + (long long)z.i * tk.out_stride + tk.out_off[z.t];
            coded = tk.quant != nullptr && tk.quant[z.s] == 1;
            if (coded) {
                const int E = tk.qexp[z.s];
                up = pow2_double(E); down = pow2_double(-E);
                qmax = (double)((1 << (tk.quant_bits - 1)) - 1);
            }
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
                const unsigned int off = ent_off(e[q].x), low = ent_low20(e[q].x);
                const bool g = live && (off > sel || (off == sel && low > tau20));
                const bool same = live && off == sel && low == tau20;
                const unsigned int bg = __ballot_sync(0xffffffffu, g), bq = __ballot_sync(0xffffffffu, same);
                const unsigned int my_gt = run_gt + __popc(bg & lower), my_eq = run_eq + __popc(bq & lower);
                if (g || (same && my_eq < take)) {
                    const unsigned int slot = my_gt + min(my_eq, take);
                    const int local = u * kWarpSpan + (int)(e[q].x & 0x1ffu);
                    if (slot < K && local < len) {
                        unsigned int bits = e[q].y;          // x at the entry: what a plain message delivers
                        if (coded) {
                            // the change as a code on the segment's grid; what arrives is x_hat + code * 2^E
                            const float had = xhat[base + local];
                            const float d = __fsub_rn(__uint_as_float(bits), had);
                            double code = rint(__dmul_rn((double)d, down));
                            code = fmin(fmax(code, -qmax), qmax);
                            bits = __float_as_uint(__double2float_rn(__dadd_rn((double)had, __dmul_rn(code, up))));
                        }
                        out[slot] = make_int2(first + local, (int)bits);
                        xhat[base + local] = __uint_as_float(bits);
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
// sends a sparse message in this step -- a quiet step then costs one launch.
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
    const WorkList& all = a.tk.list[0];
    const WorkList& again = a.tk.list[1];
    if (blockIdx.x == 0) topk_plan(a.S, a.T, a.sparse, a.tt.seg_begin, a.tk, all, (int)gridDim.x, true);
    grid.sync();
    if (all.plan->n_sparse == 0) return;          // the same for every CTA
    topk_hist(a.x, a.xhat, a.tt, a.T, a.stride, a.tk, all, true);
    grid.sync();
    topk_guess(a.T, a.tk, all);
    grid.sync();
    topk_collect(a.x, a.xhat, a.tt, a.T, a.stride, a.tk, all);
    grid.sync();
    topk_resolve(a.T, a.tk, all, false, a.err);
    grid.sync();
    if (*a.tk.redo_count != 0u) {                  // the same for every CTA
        if (blockIdx.x == 0) topk_plan(a.S, a.T, a.tk.redo, a.tt.seg_begin, a.tk, again, (int)gridDim.x, false);
        grid.sync();
        topk_hist(a.x, a.xhat, a.tt, a.T, a.stride, a.tk, again, false);
        grid.sync();
        topk_pick(a.T, a.tk, again, 0);
        grid.sync();
        topk_collect(a.x, a.xhat, a.tt, a.T, a.stride, a.tk, again);
        grid.sync();
        topk_resolve(a.T, a.tk, again, true, a.err);
        grid.sync();
    }
    topk_digit2(a.tt, a.T, a.stride, a.tk, all);
    grid.sync();
    topk_pick(a.T, a.tk, all, 2);
    grid.sync();
    topk_recount(a.tt, a.T, a.stride, a.tk, all);
    grid.sync();
    topk_scan(a.tt, a.T, a.stride, a.tk, all);
    grid.sync();
    topk_write(a.xhat, a.tt, a.T, a.stride, a.tk, all, a.err);
}

// Every single-phase kernel can be launched as a dependent launch: it waits for its predecessor
// before it reads anything.  None of them lets its successor in before it ends: a successor let
// in at the start of a kernel that goes on for a millisecond made that kernel much slower.  `which` names the work list: 0 for this iteration's sparse
// segments, 1 for the exact repeat; the kernels of the repeat leave at once when no segment
// asked for it.
__device__ __forceinline__ bool topk_enter(const TopkArgs& a, int which) {
    pdl_wait();
    return which == 0 || *a.tk.redo_count != 0u;
}
__global__ void __launch_bounds__(kPlanThreads) k_topk_plan(TopkArgs a, int which) {
    if (!topk_enter(a, which)) return;
    topk_plan(a.S, a.T, which ? a.tk.redo : a.sparse, a.tt.seg_begin, a.tk, a.tk.list[which], a.plan_ctas, which == 0);
}
__global__ void __launch_bounds__(kThreads) k_topk_hist(TopkArgs a, int which) {
    if (!topk_enter(a, which)) return;
    topk_hist(a.x, a.xhat, a.tt, a.T, a.stride, a.tk, a.tk.list[which], which == 0);
}
__global__ void __launch_bounds__(kThreads) k_topk_guess(TopkArgs a) {
    if (!topk_enter(a, 0)) return;
    topk_guess(a.T, a.tk, a.tk.list[0]);
}
__global__ void __launch_bounds__(kThreads) k_topk_pick(TopkArgs a, int which, int digit) {
    if (!topk_enter(a, which)) return;
    topk_pick(a.T, a.tk, a.tk.list[which], digit);
}
// The collecting pass runs kCollectShares planned shares per CTA (two CTAs of 288 threads and
// 107 KB of shared memory fit a multiprocessor).
constexpr int kCollectShares = 4;
__global__ void __launch_bounds__(kCollectThreads, 2) k_topk_collect(TopkArgs a, int which) {
    if (!topk_enter(a, which)) return;
    topk_collect_staged(a.x, a.xhat, a.tt, a.T, a.stride, a.tk, a.tk.list[which], a.err, kCollectShares);
}
__global__ void __launch_bounds__(kThreads) k_topk_resolve(TopkArgs a, int which) {
    if (!topk_enter(a, which)) return;
    topk_resolve(a.T, a.tk, a.tk.list[which], which != 0, a.err);
}
// The phases that work from the entries: planned shares per CTA and CTAs per multiprocessor.
#ifndef EG_ENTRY_SHARES
#define EG_ENTRY_SHARES 2
#endif
#ifndef EG_ENTRY_MINB
#define EG_ENTRY_MINB 4
#endif
constexpr int kEntryShares = EG_ENTRY_SHARES;
__global__ void __launch_bounds__(kThreads, EG_ENTRY_MINB) k_topk_digit2(TopkArgs a) {
    if (!topk_enter(a, 0)) return;
    topk_digit2(a.tt, a.T, a.stride, a.tk, a.tk.list[0], kEntryShares);
}
__global__ void __launch_bounds__(kThreads, EG_ENTRY_MINB) k_topk_recount(TopkArgs a) {
    if (!topk_enter(a, 0)) return;
    topk_recount(a.tt, a.T, a.stride, a.tk, a.tk.list[0], kEntryShares);
}
__global__ void __launch_bounds__(kThreads) k_topk_scan(TopkArgs a) {
    if (!topk_enter(a, 0)) return;
    topk_scan(a.tt, a.T, a.stride, a.tk, a.tk.list[0]);
}
__global__ void __launch_bounds__(kThreads, EG_ENTRY_MINB) k_topk_write(TopkArgs a) {
    if (!topk_enter(a, 0)) return;
    topk_write(a.xhat, a.tt, a.T, a.stride, a.tk, a.tk.list[0], a.err, kEntryShares);
}

}  // namespace eg
