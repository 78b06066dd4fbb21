// Shared device-side declarations of the EventGraD step library (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace eg {

constexpr int kThreads = 256;          // threads per CTA in every streaming kernel
constexpr int kWarps = kThreads / 32;
constexpr int kNormTile = 4096;        // elements per CTA of the norm / Top-K kernels
constexpr int kMaxReplicas = 1024;     // P limit (shared-memory tables are sized by P)
constexpr int kMaxHistory = 64;

// Top-K radix select: the 31-bit key bits(|x - x_hat|) is resolved in three digits.
constexpr int kDigitBits0 = 11, kDigitBits1 = 10, kDigitBits2 = 10;
constexpr int kMaxBins = 1 << kDigitBits0;

// Tile table: a tile is a run of at most `tile` consecutive elements of one tensor.
struct TileTable {
    const int* tensor;           // [n_tiles] tensor id
    const long long* offset;     // [n_tiles] element offset inside one replica
    const int* length;           // [n_tiles] elements in the tile
    const int* seg_begin;        // [T+1] first tile of every tensor
    int n_tiles;
    unsigned int* err;           // the context's error word (bounds-checked build)
};

// Bits of a context's error word (set by kernels, read by the calls that synchronise).
constexpr unsigned kErrTopkSlot = 2u;      // a Top-K entry pointed outside its message or tile
constexpr unsigned kErrBounds = 4u;        // bounds-checked build: an index left its table
constexpr unsigned kErrWaitTimeout = 8u;   // a bounded wait on a shared-memory barrier ran out

// Bounds-checked build (-DEG_DEBUG): every index a kernel forms into a table -- tile records,
// per-replica modes, pipeline stages, partial sums, entry slots -- is compared with the table's
// size first.  A miss sets kErrBounds in the error word and the access is skipped; nothing traps.
// In the normal build the checks compile to nothing.
#ifdef EG_DEBUG
__device__ __forceinline__ bool index_ok(unsigned int* err, long long idx, long long n) {
    if (idx >= 0 && idx < n) return true;
    if (err) atomicOr(err, kErrBounds);
    return false;
}
#define EG_INDEX_OK(err, idx, n) ::eg::index_ok((err), (long long)(idx), (long long)(n))
#else
#define EG_INDEX_OK(err, idx, n) true
#endif

// The record of tile `tile` lies inside its table and describes elements inside one replica.
__device__ __forceinline__ bool tile_ok(const TileTable& tt, int tile, int T, long long stride, int tile_elems) {
#ifdef EG_DEBUG
    if (!EG_INDEX_OK(tt.err, tile, tt.n_tiles)) return false;
    return EG_INDEX_OK(tt.err, tt.tensor[tile], T) && EG_INDEX_OK(tt.err, tt.length[tile] - 1, tile_elems) &&
           EG_INDEX_OK(tt.err, tt.offset[tile] + tt.length[tile] - 1, stride);
#else
    (void)tt; (void)tile; (void)T; (void)stride; (void)tile_elems;
    return true;
#endif
}

// 2^k as a double, -1022 <= k <= 1023
__device__ __forceinline__ double pow2_double(int k) {
    return __longlong_as_double((long long)(k + 1023) << 52);
}

// Per-(replica, tensor) trigger state and the decisions of the current step, all [P*T].
struct SegState {
    double* delta;               // threshold in force
    long long* khat;             // iteration of the last event
    double* hist;                // [P*T][H] slopes, oldest first
    int* hist_len;
    uint8_t* valid;              // the tensor has been sent at least once
    uint8_t* flag;               // event in this step
    uint8_t* snap;               // event whose message is dense (x_hat <- x in the fused kernel)
    uint8_t* sparse;             // event whose message is a Top-K message
    double* norm;                // d of this step
    double* thr_used;            // delta that d was compared with
    unsigned long long* events;  // events so far
    double* sent_norm;           // ||x|| at the last event (change-of-norm variant)
    unsigned int* sparse_steps;  // [2] Top-K messages decided in the iteration of this parity (nullptr: dense)
    uint8_t* quant;              // event whose message is quantised and delivered into x_hat by the
                                 // quantising kernels before the averaging kernel runs (nullptr: never)
};

// Variants of the method that the paper's text also admits (kernel argument `variant`).
constexpr int kOwnLastSent = 1;    // own term of the average is x_hat_i (Eq. (dist_sgd_event) literally)
constexpr int kChangeOfNorm = 2;   // tested quantity is | ||x|| - ||x at the last event|| |

struct Counters {                // device-resident, 64-bit
    unsigned long long messages, bytes, events, pad;
};

// Programmatic dependent launch.  A kernel launched with the programmatic-serialization
// attribute may start while its predecessor in the stream is still running; pdl_wait() returns
// once that predecessor has completed and its writes are visible (a no-op for an ordinary
// launch), so everything before it must touch only data that no earlier kernel writes.
// pdl_release() lets the next kernel of the stream start its own preamble early.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ float4 ld_stream(const float* p) {
    return __ldcs(reinterpret_cast<const float4*>(p));
}
__device__ __forceinline__ void st_stream(float* p, float4 v) {
    __stcs(reinterpret_cast<float4*>(p), v);
}

// Sum over the CTA in a fixed order (lane tree, then warps in ascending order); the result
// is valid in thread 0.
__device__ __forceinline__ double block_sum(double v, double* s_warp) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = __dadd_rn(v, __shfl_down_sync(0xffffffffu, v, o));
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) s_warp[warp] = v;
    __syncthreads();
    double r = 0.0;
    if (threadIdx.x == 0) {
#pragma unroll
        for (int w = 0; w < kWarps; ++w) r = __dadd_rn(r, s_warp[w]);
    }
    return r;
}

}  // namespace eg
