// Fused dense snapshot / consensus average / SGD update, bulk-copy pipelined version.
//
// Same arithmetic and the same element-axis tiling as k_fused (eg_fused.cuh); what differs is
// how the operands reach the SM.  One producer thread streams the (x, g, x_hat) tiles of the
// replicas, in ring order, into a ring of shared-memory stages with 1-D bulk asynchronous
// copies (cp.async.bulk, completion on an mbarrier, no multicast), so the bytes in flight
// are bounded by shared memory instead of registers; 4 consumer warps read their float4
// columns (two per thread) of two adjacent stages (replica j and the contribution of replica j+1; that of
// replica j-1 is carried in registers) and write the results straight to global memory.  Every thread always owns the same column, so the two wrap-around operands
// (replica P-1 for replica 0, replica 0 for replica P-1) live in two extra shared buffers
// that are private per column.
//
// A CTA works through several tiles, one after the other, and keeps the ring full across them.
//
// Every mbarrier wait is bounded: when the limit is hit the CTA raises an abort flag, sets a
// bit in the context's error word, lets its copies land and returns.
#pragma once
#include "eg_common.cuh"
#include "eg_fused.cuh"

namespace eg {

#ifndef EG_PIPE_CONSUMERS
#define EG_PIPE_CONSUMERS 128   // two float4 columns per consumer thread: the per-replica control
                                // flow is paid once per eight elements (256 measured 0-3 % slower)
#endif
#ifndef EG_PIPE_STAGES
#define EG_PIPE_STAGES 5
#endif
constexpr int kPipeTile = 1024;                   // elements per CTA and stage
constexpr int kPipeStages = EG_PIPE_STAGES;
constexpr int kPipeConsumers = EG_PIPE_CONSUMERS; // consumer threads (+ one producer warp)
constexpr int kPipeThreads = kPipeConsumers + 32;
constexpr long long kWaitLimitCycles = 2000000000ll;   // about one second

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
#ifndef EG_WAIT_HINT_NS
#define EG_WAIT_HINT_NS 1000
#endif
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
#if EG_WAIT_HINT_NS > 0
    // the hint lets the hardware keep the warp suspended (no issue slots used) until the phase
    // completes or the time runs out
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"((uint32_t)EG_WAIT_HINT_NS)
        : "memory");
#else
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
#endif
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
                                                  unsigned int* err,
                                                  long long limit_cycles = kWaitLimitCycles) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    unsigned int spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 63u) != 0) continue;       // look at the clock every 64 polls only
        if (*s_abort) return false;
        if (clock64() - t0 > limit_cycles) {
            *s_abort = 1;
            atomicOr(err, kErrWaitTimeout);
            return false;
        }
    }
    return true;
}

struct PipeCfg {
    int tile;        // elements per CTA and stage
    int stages;
    int consumers;   // consumer threads; each owns tile / (4 * consumers) float4 columns
};

// Shared-memory layout (dynamic), all offsets multiples of 16.
// RUNS: a CTA may take several tiles (two wrap-around buffers, two mode tables).
template <int TILE, int STAGES, int ARRAYS = 3, bool RUNS = true>
struct PipeSmem {
    static constexpr int kTileBytes = TILE * 4;
    static constexpr int kStageBytes = ARRAYS * kTileBytes;       // x, g, x_hat (, velocity)
    static constexpr int kWrapL = STAGES * kStageBytes;           // two buffers: consecutive tiles alternate
    static constexpr int kWrapR = kWrapL + (RUNS ? 2 : 1) * kTileBytes;
    static constexpr int kBars = kWrapR + kTileBytes;             // full[S], empty[S], wrap[2]
    static constexpr int kFlags = kBars + 8 * (2 * STAGES + 2);
    static constexpr int kModes = kFlags + 16 + 2 * 32;           // after the flags: two tile headers of 32 bytes
    // then 16 bytes of flags, two tile headers, two tables of per-replica modes (consecutive tiles alternate) and,
    // for the carried norm, per stage one slot of 8 doubles per consumer warp (see the consumers'
    // end of a replica and the producer warp's reduce_slot)
    __host__ __device__ static size_t mode_bytes(int P) { return ((size_t)P + 15) & ~(size_t)15; }
    __host__ __device__ static size_t bytes(int P, bool carry, int consumer_warps) {
        size_t b = kModes + (RUNS ? 2 : 1) * mode_bytes(P);
        if (carry) b += (size_t)STAGES * consumer_warps * 8 * sizeof(double);
        return b;
    }
};

// Body of the kernels below.  The launch covers `n_launch` tiles of the tile table (TILE elements
// per tile).  CTA b begins with tile b; launched with fewer CTAs than tiles and a `ticket`
// counter (zeroed by the decision kernel before it), a CTA goes on with tile gridDim.x + the
// counter's next value, and so on until the tiles are used up.  The CTAs running at any moment
// then work on neighbouring tiles, as they would with one tile per CTA, however far they drift
// apart (runs of consecutive tiles per CTA measured 5-10 % slower at 16 and 64 replicas, the
// fixed stride b, b + gridDim.x, ... 2-10 % slower from 16 replicas on).  A walking CTA keeps
// its ring of stages full across tiles: the producer warp starts on the replicas of the next
// tile while the consumers still work on the current one, so that a CTA pays for filling and
// draining the ring once, not once per tile (with few replicas that was a large part of a
// CTA's life).  The producer knows its tiles three ahead (number, then record, then flags, each
// fetched a tile before it is needed) and tells the consumers about each through a header in
// shared memory.  What belongs to a tile and not to a stage -- the header, the per-replica
// modes and the wrap-around contribution of replica P-1 -- exists twice and consecutive tiles
// alternate; this is safe when P >= STAGES (the producer is then never more than one tile
// ahead of the consumers), which the host guarantees by launching one CTA per tile otherwise.
// CONSUMERS + 32 threads; COLS = TILE / (4 * CONSUMERS) float4 columns per consumer thread.
//
// ASYNC (intermittent delivery): x_hat is what a replica has SENT, `mailbox` what its
// neighbours have RECEIVED, `arrive` says whose outstanding messages arrive in this step and
// `valid` is then "received at least once".  A replica contributes its own x (dense message
// that arrives now), its sent copy (older message arriving now; copied into the mailbox on
// the way) or its mailbox (nothing arrives).  Without ASYNC the two copies are one buffer and
// every message arrives at once, which is the code path of the synchronous method.
// PLAIN: the default readings only (the `variant` argument is ignored), so that the common
// path carries no variant tests.
// MOM (heavy-ball momentum, an extension to another training algorithm): every replica owns a
// velocity `vel` laid out like x; a stage carries a fourth tile (v), the consumers form
// v <- fp32(mu * v + g) in fp64, write it back and use it in place of the gradient.
// RUNS = false (the momentum kernel, whose four tiles per stage leave no room for the second
// wrap-around buffer at three CTAs per multiprocessor): one tile per CTA.
template <int TILE, int STAGES, int CONSUMERS, bool CARRY, bool ASYNC, bool PLAIN, bool MOM = false,
          bool RUNS = !MOM>
__device__ __forceinline__ void
fused_pipe_body(float* __restrict__ x, const float* __restrict__ g, float* __restrict__ xhat,
                const uint8_t* __restrict__ snap, const uint8_t* __restrict__ valid, const TileTable& tt,
                int P, int T, long long stride, float lr, double* __restrict__ partials,
                long long* step_k, unsigned int* __restrict__ err, int variant_arg,
                float* mailbox, const uint8_t* __restrict__ arrive, int n_launch, int* ticket,
                float* __restrict__ vel = nullptr, double mu = 0.0) {
    constexpr int kArr = MOM ? 4 : 3;              // tiles per stage
    static_assert(!(ASYNC && CARRY), "the carried norm is not produced under intermittent delivery");
    const int variant = PLAIN ? 0 : variant_arg;
    // mode bit that says "contributes its own x": the dense-message bit itself unless ASYNC
    constexpr unsigned kCx = ASYNC ? 4u : 1u;
    using L = PipeSmem<TILE, STAGES, kArr, RUNS>;
    constexpr int COLS = TILE / (4 * CONSUMERS);
    constexpr int CWARPS = CONSUMERS / 32;
    static_assert(COLS * 4 * CONSUMERS == TILE, "tile must be covered exactly");
    extern __shared__ __align__(128) unsigned char smem[];
    float* stages = reinterpret_cast<float*>(smem);
    float* wrap_l2 = reinterpret_cast<float*>(smem + L::kWrapL);  // [2][TILE] contribution of replica P-1
    float* wrap_r = reinterpret_cast<float*>(smem + L::kWrapR);   // contribution of replica 0
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::kBars);
    uint64_t* empty = full + STAGES;
    uint64_t* wrap_bar2 = empty + STAGES;                          // [2]
    volatile int* s_abort = reinterpret_cast<volatile int*>(smem + L::kFlags);
    // bit 0: dense message, bit 1: valid, bit 2: contributes its own x, bit 3: arrives now
    // what the producer tells the consumers about a tile: which one, its length and place, and
    // whether this CTA has another tile after it
    struct TileHeader { int tile, len; long long off; int has_next; int pad[3]; };
    static_assert(sizeof(TileHeader) == 32, "two headers sit between the flags and the mode tables");
    TileHeader* s_hdr = reinterpret_cast<TileHeader*>(smem + L::kFlags + 16);   // [2]
    uint8_t* s_mode2 = smem + L::kModes;                           // [2][mode_bytes(P)]
    const int mode_stride = (int)L::mode_bytes(P);
    double* s_part = reinterpret_cast<double*>(s_mode2 + (RUNS ? 2 : 1) * mode_stride);   // [STAGES][CWARPS * 8]

    const int tid = threadIdx.x;
    // Tiles of this CTA: the first is its own number; with RUNS further ones follow -- first + hop,
    // first + 2 hop, ... below last, or (`ticket` given) whatever a counter shared by the CTAs
    // hands out next, so that tiles are begun in order however unevenly the CTAs advance.
    const int first = (int)blockIdx.x, hop = (int)gridDim.x;
    const int last = RUNS ? n_launch : min(n_launch, first + 1);
    if (first >= last) return;                   // the same in every thread

    // up to here nothing that a kernel writes has been read.  The kernel after this one is let
    // in when every CTA has begun its LAST tile (below): released at the start of a kernel that
    // goes on for long, it made this kernel up to 45 % slower (measured).
    pdl_wait();
    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], CWARPS);
        }
        mbar_init(&wrap_bar2[0], 1);
        mbar_init(&wrap_bar2[1], 1);
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (blockIdx.x == 0 && step_k) *step_k += 1;   // nothing in this launch reads it
    }
    __syncthreads();
    const bool last_opt = P >= 2;   // replica P-1 contributes wrap_l; its own stage then only needs what wrap_l does not hold

    if (tid >= CONSUMERS) {
        // ------------------------------------------------------------------ producer warp
        // All 32 lanes walk the loop: they fill in the per-replica modes of a tile together, lane 0
        // issues the copies, and with CARRY the warp also finishes the sums of squares that the
        // consumers leave behind (8 values per consumer warp and replica, in the slot of the
        // replica's stage): once a stage has been released, its slot is complete.
        const int pl = tid - CONSUMERS;
        auto reduce_slot = [&](int slot, int tile, int j) {
            static_assert(CWARPS == 8 || CWARPS == 4 || CWARPS == 2, "a slot holds 64, 32 or 16 values");
            const double* sp = s_part + slot * (CWARPS * 8);
            double r = (CWARPS == 8) ? __dadd_rn(sp[pl], sp[32 + pl])
                                     : ((CWARPS == 4 || pl < 16) ? sp[pl & (CWARPS * 8 - 1)] : 0.0);
            if (CWARPS == 2 && pl >= 16) r = 0.0;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) r = __dadd_rn(r, __shfl_xor_sync(0xffffffffu, r, o));
            if (pl == 0 && EG_INDEX_OK(err, j, P) && EG_INDEX_OK(err, slot, STAGES))
                partials[(long long)j * tt.n_tiles + tile] = r;
        };
        // Items are (tile, replica) pairs in the order they go through the ring; item m uses
        // stage m % STAGES in its (m / STAGES)-th filling.  retire(m): wait until the consumers
        // have released item m, then (CARRY) finish its sum of squares.
        int retired = 0, r_buf = 0, r_j = 0;          // next item to retire: replica r_j of the tile of header r_buf
        auto retire = [&]() -> bool {
            const int sm = retired % STAGES;
            bool alive = mbar_wait_bounded(&empty[sm], (uint32_t)((retired / STAGES) & 1), s_abort, err);
            alive = __all_sync(0xffffffffu, alive);
            if (!alive) return false;
            if (CARRY) reduce_slot(sm, s_hdr[r_buf].tile, r_j);
            ++retired;
            if (++r_j == P) { r_j = 0; r_buf = RUNS ? (r_buf ^ 1) : 0; }
            return true;
        };
        // the record of a tile: lane-uniform
        struct Rec { int t, len; long long off; };
        auto load_rec = [&](int tile) {
            Rec r;
            r.t = tt.tensor[tile]; r.len = tt.length[tile]; r.off = tt.offset[tile];
            return r;
        };
        // the per-replica flags of a tile: read one tile ahead, two replicas per lane, and kept
        // as they come (the first use of a loaded value would make the warp wait for it) --
        // rings of up to 64 replicas; larger ones read their flags when the tile begins
        constexpr int kPre = 2;
        const bool prefetch = P <= 32 * kPre;
        uint8_t pre_sn[kPre], pre_va[kPre], pre_ar[kPre];
        auto mode_of = [&](uint8_t sn_b, uint8_t va_b, uint8_t ar_b) -> uint8_t {
            const bool sn = sn_b != 0;
            const bool ar = ASYNC ? (ar_b != 0) : sn;
            return (uint8_t)((sn ? 1u : 0u) | (va_b ? 2u : 0u) | ((sn && ar) ? 4u : 0u) | (ar ? 8u : 0u));
        };
        auto fetch_flags = [&](int t) {
#pragma unroll
            for (int q = 0; q < kPre; ++q) {
                const long long at = (long long)min(pl + 32 * q, P - 1) * T + t;
                pre_sn[q] = snap[at];
                pre_va[q] = valid[at];
                pre_ar[q] = ASYNC ? arrive[at] : (uint8_t)0;
            }
        };
        // The tiles to come, known three ahead: the number of tile it + 3 is asked for when tile it
        // begins (lane 0 holds the counter's answer; it is passed round one tile later, when it has
        // long arrived), the record of tile it + 2 is read then, and the flags of tile it + 1.
        int seq = first;                              // fixed stride: the last number formed
        auto ask = [&]() -> int {
            if (ticket) return (pl == 0) ? hop + atomicAdd(ticket, 1) : 0;
            seq += hop;
            return seq;
        };
        auto told = [&](int raw) -> int {             // the answer, in every lane; none left: last
            const int id = ticket ? __shfl_sync(0xffffffffu, raw, 0) : raw;
            return (id >= 0 && id < last) ? id : last;
        };
        int issued = 0, s = 0;
        bool alive = true;
        const int raw1 = RUNS ? ask() : last, raw2 = RUNS ? ask() : last;
        int raw3 = RUNS ? ask() : last;               // three requests on their way together
        int id0 = first, id1 = RUNS ? told(raw1) : last, id2 = RUNS ? told(raw2) : last;
        Rec rec = load_rec(id0);
        Rec rec1 = (id1 < last) ? load_rec(id1) : rec;
        Rec rec2 = (id2 < last) ? load_rec(id2) : rec;
        if (prefetch) fetch_flags(rec.t);
        for (int it = 0; id0 < last && alive; ++it) {
            const int tile = id0;
            if (!tile_ok(tt, tile, T, stride, TILE)) break;      // bounds-checked build only (the consumers leave too)
            if (id1 >= last) pdl_release();
            const int buf = RUNS ? (it & 1) : 0;
            uint8_t* sm = s_mode2 + buf * mode_stride;
            // modes of this tile (its flags were read one tile ago), then the flags of the next
            if (prefetch) {
#pragma unroll
                for (int q = 0; q < kPre; ++q)
                    if (pl + 32 * q < P) sm[pl + 32 * q] = mode_of(pre_sn[q], pre_va[q], pre_ar[q]);
            } else {
                for (int j = pl; j < P; j += 32) {
                    const long long at = (long long)j * T + rec.t;
                    sm[j] = mode_of(snap[at], valid[at], ASYNC ? arrive[at] : (uint8_t)0);
                }
            }
            const Rec cur = rec;
            if (pl == 0) {
                TileHeader h;
                h.tile = tile; h.len = cur.len; h.off = cur.off; h.has_next = id1 < last ? 1 : 0;
                h.pad[0] = h.pad[1] = h.pad[2] = 0;
                s_hdr[buf] = h;
            }
            __syncwarp();
            // move on by one tile: numbers, records, flags
            id0 = id1; id1 = id2; id2 = RUNS ? told(raw3) : last;
            rec = rec1; rec1 = rec2;
            if (RUNS) raw3 = ask();
            if (id2 < last) rec2 = load_rec(id2);
            if (prefetch && id0 < last) fetch_flags(rec.t);
            const uint32_t copy_bytes = (uint32_t)(((cur.len + 3) & ~3) * 4);
            const float* xp = x + cur.off;
            const float* gp = g + cur.off;
            const float* hp = xhat + cur.off;
            const float* mp = ASYNC ? mailbox + cur.off : hp;
            const float* vp = MOM ? vel + cur.off : nullptr;
            if (pl == 0) {
                const bool cx_last = (sm[P - 1] & kCx) != 0;
                mbar_expect_tx(&wrap_bar2[buf], copy_bytes);
                bulk_g2s(wrap_l2 + buf * TILE,
                         (cx_last ? xp : ((sm[P - 1] & 8) ? hp : mp)) + (long long)(P - 1) * stride,
                         copy_bytes, &wrap_bar2[buf]);
            }
            for (int j = 0; j < P; ++j) {
                if (issued >= STAGES && !retire()) { alive = false; break; }   // before the stage is filled again
                if (pl == 0 && EG_INDEX_OK(err, s, STAGES)) {
                    float* st = stages + s * (kArr * TILE);
                    const bool cx = (sm[j] & kCx) != 0;
                    const bool is_last = last_opt && (j == P - 1);
                    const bool need_x = !(is_last && cx);
                    const bool need_h = !cx && !is_last;
                    mbar_expect_tx(&full[s],
                                   copy_bytes * ((MOM ? 2u : 1u) + (need_x ? 1u : 0u) + (need_h ? 1u : 0u)));
                    bulk_g2s(st + TILE, gp, copy_bytes, &full[s]);
                    if (MOM) { bulk_g2s(st + 3 * TILE, vp, copy_bytes, &full[s]); vp += stride; }
                    if (need_x) bulk_g2s(st, xp, copy_bytes, &full[s]);
                    if (need_h) bulk_g2s(st + 2 * TILE, (sm[j] & 8) ? hp : mp, copy_bytes, &full[s]);
                    xp += stride; gp += stride; hp += stride; mp += stride;
                }
                ++issued;
                if (++s == STAGES) s = 0;
            }
        }
        if (CARRY) {
            // the items whose stages are not filled again
            while (alive && retired < issued) alive = retire();
        }
    } else {
        // ------------------------------------------------------------------ consumers
        const int lane = tid & 31, warp = tid >> 5;
        const int c0 = tid * 4;                      // column v starts at c0 + v * 4 * CONSUMERS
        const double neg_lr = -(double)lr;
        const double w_one = 1.0, w_half = 0.5, w_third = __ddiv_rn(1.0, 3.0);
        const bool has_left = P >= 2, has_right = P >= 3;
        // the ring position of the next item: stage s in a filling of parity par_s, and the one after it
        int s = 0, s1 = (STAGES > 1) ? 1 : 0;
        uint32_t par_s = 0u, parity1 = (STAGES > 1) ? 0u : 1u;
        bool ok = true;
        bool more_tiles = true;
        for (int it = 0; more_tiles && ok; ++it) {
            const int buf = RUNS ? (it & 1) : 0;
            const uint8_t* s_mode = s_mode2 + buf * mode_stride;
            const float* wrap_l = wrap_l2 + buf * TILE;
            uint64_t* wrap_bar = &wrap_bar2[buf];
            // contributions of replica j-1 and j to their neighbours, for this thread's columns,
            // kept as doubles so that every value is converted once
            double hp[COLS][4], hc[COLS][4];
            ok = mbar_wait_bounded(wrap_bar, (uint32_t)((it >> (RUNS ? 1 : 0)) & 1), s_abort, err) &&
                 mbar_wait_bounded(&full[s], par_s, s_abort, err);
            if (!ok) break;
            // (the header and the mode table were written before the tile's first copies were started)
            const int tile = s_hdr[buf].tile;
            const int len_now = s_hdr[buf].len;
            const long long off_now = s_hdr[buf].off;
            more_tiles = s_hdr[buf].has_next != 0;
            if (!tile_ok(tt, tile, T, stride, TILE)) break;      // bounds-checked build only (the producer leaves too)
            if (!more_tiles) pdl_release();
            int nel[COLS];
#pragma unroll
            for (int v = 0; v < COLS; ++v) nel[v] = min(4, max(0, len_now - (v * CONSUMERS + tid) * 4));
            unsigned mode_prev = s_mode[P - 1], mode_cur = s_mode[0];
#pragma unroll
            for (int v = 0; v < COLS; ++v) {
                const int c = c0 + v * 4 * CONSUMERS;
                const float* st0 = stages + s * (kArr * TILE);
                const float4 a = *reinterpret_cast<const float4*>(wrap_l + c);
                const float4 b = *reinterpret_cast<const float4*>(((mode_cur & kCx) ? st0 : st0 + 2 * TILE) + c);
                hp[v][0] = a.x; hp[v][1] = a.y; hp[v][2] = a.z; hp[v][3] = a.w;
                hc[v][0] = b.x; hc[v][1] = b.y; hc[v][2] = b.z; hc[v][3] = b.w;
            }
            float* xo = x + off_now + c0;                // output pointers of replica j
            float* ho = xhat + off_now + c0;
            float* mo = ASYNC ? mailbox + off_now + c0 : nullptr;
            float* vo = MOM ? vel + off_now + c0 : nullptr;
            // One replica.  A = contributions of replica j-1, B = of replica j, C receives those of
            // replica j+1.  The three arrays swap roles from one replica to the next (see the loop
            // below), so nothing is copied between them.
            auto one_replica = [&](const int j, double (&hA)[COLS][4], double (&hB)[COLS][4],
                                   double (&hC)[COLS][4]) -> bool {
                const bool more = j + 1 < P;
                if (!EG_INDEX_OK(err, s, STAGES) || !EG_INDEX_OK(err, s1, STAGES) || !EG_INDEX_OK(err, j, P)) return false;
                if (more) {
                    ok = mbar_wait_bounded(&full[s1], parity1, s_abort, err);
                    if (!ok) return false;
                }
                const unsigned mode_next = s_mode[more ? j + 1 : 0];
                const float* st = stages + s * (kArr * TILE);
                const bool sn = (mode_cur & 1) != 0;
                const bool cx = (mode_cur & kCx) != 0;     // == sn unless ASYNC
                const bool is_last = last_opt && !more;
                // fp32 copy of this replica's contribution (its old x when a dense message arrives)
                const float* hs = is_last ? wrap_l : (cx ? st : st + 2 * TILE);
                // contribution of replica j+1
                const float* sq = stages + s1 * (kArr * TILE);
                const float* hn_s = !more ? wrap_r
                                          : ((last_opt && j + 2 == P) ? wrap_l
                                                                      : ((mode_next & kCx) ? sq : sq + 2 * TILE));
                const bool ul = has_left && (mode_prev & 2) != 0;
                const bool ur = has_right && (mode_next & 2) != 0;
                const double w = (ul && ur) ? w_third : ((ul || ur) ? w_half : w_one);
                double acc = 0.0;
    #pragma unroll
                for (int v = 0; v < COLS; ++v) {
                    if (PLAIN && !ASYNC && !MOM && nel[v] == 4 && ul && ur) {
                        // The common case -- a full float4, both neighbours heard from, default
                        // readings -- as straight-line code: the same operations in the same order
                        // as the general form below, without its per-element conditions.
                        const int c = c0 + v * 4 * CONSUMERS;
                        const float4 hcf = *reinterpret_cast<const float4*>(hs + c);
                        const float4 hnf = *reinterpret_cast<const float4*>(hn_s + c);
                        const float4 gf = *reinterpret_cast<const float4*>(st + TILE + c);
                        if (j == 0) *reinterpret_cast<float4*>(wrap_r + c) = hcf;
                        hC[v][0] = (double)hnf.x; hC[v][1] = (double)hnf.y; hC[v][2] = (double)hnf.z; hC[v][3] = (double)hnf.w;
                        double xd[4];
                        if (cx) {
    #pragma unroll
                            for (int q = 0; q < 4; ++q) xd[q] = hB[v][q];
                        } else {
                            const float4 xf = *reinterpret_cast<const float4*>(st + c);
                            xd[0] = (double)xf.x; xd[1] = (double)xf.y; xd[2] = (double)xf.z; xd[3] = (double)xf.w;
                        }
                        float4 xn4;
                        xn4.x = __double2float_rn(__fma_rn(neg_lr, (double)gf.x,
                                    __dmul_rn(__dadd_rn(__dadd_rn(xd[0], hA[v][0]), hC[v][0]), w_third)));
                        xn4.y = __double2float_rn(__fma_rn(neg_lr, (double)gf.y,
                                    __dmul_rn(__dadd_rn(__dadd_rn(xd[1], hA[v][1]), hC[v][1]), w_third)));
                        xn4.z = __double2float_rn(__fma_rn(neg_lr, (double)gf.z,
                                    __dmul_rn(__dadd_rn(__dadd_rn(xd[2], hA[v][2]), hC[v][2]), w_third)));
                        xn4.w = __double2float_rn(__fma_rn(neg_lr, (double)gf.w,
                                    __dmul_rn(__dadd_rn(__dadd_rn(xd[3], hA[v][3]), hC[v][3]), w_third)));
                        st_stream(xo + v * 4 * CONSUMERS, xn4);
                        if (sn) st_stream(ho + v * 4 * CONSUMERS, hcf);
                        if (CARRY) {
                            const float d0 = __fsub_rn(xn4.x, hcf.x), d1 = __fsub_rn(xn4.y, hcf.y);
                            const float d2 = __fsub_rn(xn4.z, hcf.z), d3 = __fsub_rn(xn4.w, hcf.w);
                            acc = __fma_rn((double)d0, (double)d0, acc);
                            acc = __fma_rn((double)d1, (double)d1, acc);
                            acc = __fma_rn((double)d2, (double)d2, acc);
                            acc = __fma_rn((double)d3, (double)d3, acc);
                        }
                    } else if (nel[v] > 0) {
                        const int c = c0 + v * 4 * CONSUMERS;
                        const float4 hcf = *reinterpret_cast<const float4*>(hs + c);
                        const float4 hnf = *reinterpret_cast<const float4*>(hn_s + c);
                        const float4 gf = *reinterpret_cast<const float4*>(st + TILE + c);
                        if (j == 0) *reinterpret_cast<float4*>(wrap_r + c) = hcf;   // private to this thread
                        hC[v][0] = (double)hnf.x; hC[v][1] = (double)hnf.y; hC[v][2] = (double)hnf.z; hC[v][3] = (double)hnf.w;
                        double gd[4] = {(double)gf.x, (double)gf.y, (double)gf.z, (double)gf.w};
                        if (MOM) {      // v <- mu * v + g, kept in fp32; the update then uses gamma * v
                            const float4 vf = *reinterpret_cast<const float4*>(st + 3 * TILE + c);
                            const float vn[4] = {__double2float_rn(__fma_rn(mu, (double)vf.x, gd[0])),
                                                 __double2float_rn(__fma_rn(mu, (double)vf.y, gd[1])),
                                                 __double2float_rn(__fma_rn(mu, (double)vf.z, gd[2])),
                                                 __double2float_rn(__fma_rn(mu, (double)vf.w, gd[3]))};
                            store_masked(vo + v * 4 * CONSUMERS, make_float4(vn[0], vn[1], vn[2], vn[3]), nel[v]);
    #pragma unroll
                            for (int q = 0; q < 4; ++q) gd[q] = (double)vn[q];
                        }
                        double xd[4];
                        float4 x_old = make_float4(0.f, 0.f, 0.f, 0.f);   // only needed under ASYNC
                        if (cx || (variant & kOwnLastSent)) {   // own term = this replica's contribution
    #pragma unroll
                            for (int q = 0; q < 4; ++q) xd[q] = hB[v][q];
                            if (ASYNC) x_old = hcf;
                        } else {
                            const float4 xf = *reinterpret_cast<const float4*>(st + c);
                            xd[0] = (double)xf.x; xd[1] = (double)xf.y; xd[2] = (double)xf.z; xd[3] = (double)xf.w;
                            if (ASYNC) x_old = xf;
                        }
                        float xn[4];
    #pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            double sum = xd[q];
                            if (ul) sum = __dadd_rn(sum, hA[v][q]);
                            if (ur) sum = __dadd_rn(sum, hC[v][q]);
                            xn[q] = __double2float_rn(__fma_rn(neg_lr, gd[q], __dmul_rn(sum, w)));
                        }
                        const float4 xn4 = make_float4(xn[0], xn[1], xn[2], xn[3]);
                        store_masked(xo + v * 4 * CONSUMERS, xn4, nel[v]);
                        // a dense message: the sender's record becomes its old x (== hcf unless ASYNC)
                        if (sn) store_masked(ho + v * 4 * CONSUMERS, ASYNC ? x_old : hcf, nel[v]);
                        if (ASYNC && (mode_cur & 8)) store_masked(mo + v * 4 * CONSUMERS, hcf, nel[v]);
                        if (CARRY)
                            acc = sq_diff4(xn4, (variant & kChangeOfNorm) ? make_float4(0.f, 0.f, 0.f, 0.f) : hcf,
                                           nel[v], acc);
                    }
                }
                if (CARRY) {
                    // two of the five rounds of the warp sum; the producer warp does the rest once
                    // this stage has been released by all consumer warps
                    acc = __dadd_rn(acc, __shfl_xor_sync(0xffffffffu, acc, 16));
                    acc = __dadd_rn(acc, __shfl_xor_sync(0xffffffffu, acc, 8));
                    if (lane < 8) s_part[s * (CWARPS * 8) + warp * 8 + lane] = acc;
                }
                // everything later iterations need from this stage now sits in registers
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[s]);
                xo += stride; ho += stride;
                if (ASYNC) mo += stride;
                if (MOM) vo += stride;
                mode_prev = mode_cur; mode_cur = mode_next;
                s = s1;
                par_s = parity1;
                if (++s1 == STAGES) { s1 = 0; parity1 ^= 1u; }
                return true;
            };
            double hn[COLS][4];
            for (int j = 0; ok && j < P; j += 3) {
                if (!one_replica(j, hp, hc, hn)) { ok = false; break; }
                if (j + 1 < P && !one_replica(j + 1, hc, hn, hp)) { ok = false; break; }
                if (j + 2 < P && !one_replica(j + 2, hn, hp, hc)) { ok = false; break; }
            }
        }
    }
    if (*s_abort) {
        // failure path only: give copies in flight time to land before the CTA retires
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) {}
    }
}

// The method as the paper's formulas state it (default readings, synchronous delivery).  No
// register bound is requested: the body needs 72 registers, which lets 3 CTAs share an SM.
template <int TILE, int STAGES, int CONSUMERS, bool CARRY>
__global__ void __launch_bounds__(CONSUMERS + 32, 3)
k_fused_pipe(float* __restrict__ x, const float* __restrict__ g, float* __restrict__ xhat,
             const uint8_t* __restrict__ snap, const uint8_t* __restrict__ valid, TileTable tt,
             int P, int T, long long stride, float lr, double* __restrict__ partials,
             long long* step_k, unsigned int* __restrict__ err, int n_launch, int* ticket) {
    fused_pipe_body<TILE, STAGES, CONSUMERS, CARRY, false, true>(x, g, xhat, snap, valid, tt, P, T, stride, lr,
                                                                partials, step_k, err, 0, nullptr, nullptr,
                                                                n_launch, ticket);
}

// Heavy-ball momentum on the default readings (eg_set_momentum): four tiles per stage.
template <int TILE, int STAGES, int CONSUMERS, bool CARRY>
__global__ void __launch_bounds__(CONSUMERS + 32)
k_fused_pipe_momentum(float* __restrict__ x, const float* __restrict__ g, float* __restrict__ xhat,
                      const uint8_t* __restrict__ snap, const uint8_t* __restrict__ valid, TileTable tt,
                      int P, int T, long long stride, float lr, double* __restrict__ partials,
                      long long* step_k, unsigned int* __restrict__ err, int n_launch,
                      float* __restrict__ vel, double mu) {
    fused_pipe_body<TILE, STAGES, CONSUMERS, CARRY, false, true, true>(x, g, xhat, snap, valid, tt, P, T, stride,
                                                                      lr, partials, step_k, err, 0, nullptr,
                                                                      nullptr, n_launch, nullptr, vel, mu);
}

// Variants (eg_set_variant) and intermittent delivery; bounded to 72 registers for 3 CTAs per SM.
// MOM: with heavy-ball momentum (four tiles per stage, one tile per CTA).
template <int TILE, int STAGES, int CONSUMERS, bool CARRY, bool ASYNC, bool MOM = false>
__global__ void __launch_bounds__(CONSUMERS + 32, 3)
k_fused_pipe_general(float* __restrict__ x, const float* __restrict__ g, float* __restrict__ xhat,
                     const uint8_t* __restrict__ snap, const uint8_t* __restrict__ valid, TileTable tt,
                     int P, int T, long long stride, float lr, double* __restrict__ partials,
                     long long* step_k, unsigned int* __restrict__ err, int n_launch, int variant,
                     float* mailbox, const uint8_t* __restrict__ arrive, int* ticket,
                     float* __restrict__ vel = nullptr, double mu = 0.0) {
    fused_pipe_body<TILE, STAGES, CONSUMERS, CARRY, ASYNC, false, MOM>(x, g, xhat, snap, valid, tt, P, T, stride,
                                                                      lr, partials, step_k, err, variant, mailbox,
                                                                      arrive, n_launch, ticket, vel, mu);
}

// Self-test of the bounded wait: one warp waits on a barrier that nothing ever completes.  The
// wait gives up after `limit_cycles`, sets the time-out bit in the error word and the kernel
// returns normally, so the context stays usable.
__global__ void __launch_bounds__(32) k_selftest_wait(unsigned int* err, long long limit_cycles,
                                                      int* gave_up) {
    __shared__ uint64_t bar;
    __shared__ int s_abort;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    const bool ok = mbar_wait_bounded(&bar, 0, &s_abort, err, limit_cycles);
    if (threadIdx.x == 0) *gave_up = ok ? 0 : 1;
}

}  // namespace eg
