// eg_change_norms_static: the segmented change norm || x - x_hat || for callers that must
// not allocate.  Same arithmetic, tile size and summation order as the norm pass of eg_step
// (k_norm_partial + the partial sum of k_decide), but
//   * no context: the tensor table travels by value in the kernel arguments, and
//   * the per-tile partial sums live in a fixed array inside the library's device image
//     instead of memory obtained from cudaMalloc.
// Nothing in this file calls cudaMalloc, cudaFree or any routine that allocates.
#include "../../include/eventgrad.h"

#include <mutex>

#include "eg_common.cuh"

namespace {

using namespace eg;

constexpr int kStaticMaxTensors = EG_STATIC_MAX_TENSORS;
constexpr long long kStaticMaxPartials = EG_STATIC_MAX_PARTIALS;   // doubles: 4 MiB
constexpr int kMaxDevices = 64;

// The scratch.  One copy per GPU that loads the library, held until the process exits.
static __device__ __align__(256) double g_static_partials[kStaticMaxPartials];

// acc + sum of the first nel squared fp32 differences, element by element in fp64 (the
// accumulation order of the norm pass of eg_step)
__device__ __forceinline__ double acc_sq_diff(float4 a, float4 b, int nel, double acc) {
    const float d0 = __fsub_rn(a.x, b.x), d1 = __fsub_rn(a.y, b.y);
    const float d2 = __fsub_rn(a.z, b.z), d3 = __fsub_rn(a.w, b.w);
    if (nel > 0) acc = __fma_rn((double)d0, (double)d0, acc);
    if (nel > 1) acc = __fma_rn((double)d1, (double)d1, acc);
    if (nel > 2) acc = __fma_rn((double)d2, (double)d2, acc);
    if (nel > 3) acc = __fma_rn((double)d3, (double)d3, acc);
    return acc;
}

struct StaticTable {                 // passed by value (3.1 KB of kernel arguments)
    long long offset[kStaticMaxTensors];   // first element of tensor t inside one replica
    int numel[kStaticMaxTensors];
    int tile_begin[kStaticMaxTensors + 1]; // first tile of tensor t
    int T;
};

// grid (total tiles, P).  partials[i * n_tiles + tile]
__global__ void __launch_bounds__(kThreads)
k_static_norm_partial(const float* __restrict__ x, const float* __restrict__ xhat,
                      const __grid_constant__ StaticTable tab, long long stride, int n_tiles,
                      double* __restrict__ partials) {
    __shared__ double s_warp[kWarps];
    const int tile = blockIdx.x, i = blockIdx.y;
    int lo = 0, hi = tab.T - 1;          // tensor whose tile range holds `tile`
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (tab.tile_begin[mid] <= tile) lo = mid; else hi = mid - 1;
    }
    const int first = (tile - tab.tile_begin[lo]) * kNormTile;
    const int len = min(kNormTile, tab.numel[lo] - first);
    const long long base = (long long)i * stride + tab.offset[lo] + first;
    double acc = 0.0;
    constexpr int kIter = kNormTile / (kThreads * 4);
#pragma unroll
    for (int q = 0; q < kIter; ++q) {
        const int local = (q * kThreads + threadIdx.x) * 4;
        const int nel = min(4, max(0, len - local));
        if (nel == 4) {
            acc = acc_sq_diff(ld_stream(x + base + local), ld_stream(xhat + base + local), 4, acc);
        } else if (nel > 0) {   // ragged end; the caller's layout need not be padded
            float a[4] = {0.f, 0.f, 0.f, 0.f}, b[4] = {0.f, 0.f, 0.f, 0.f};
            for (int e = 0; e < nel; ++e) { a[e] = x[base + local + e]; b[e] = xhat[base + local + e]; }
            acc = acc_sq_diff(make_float4(a[0], a[1], a[2], a[3]), make_float4(b[0], b[1], b[2], b[3]), nel, acc);
        }
    }
    const double total = block_sum(acc, s_warp);
    if (threadIdx.x == 0) partials[(long long)i * n_tiles + tile] = total;
}

// One warp per (replica, tensor): fixed-order sum of its partials, square root.
__global__ void __launch_bounds__(kThreads)
k_static_norm_final(const double* __restrict__ partials, const __grid_constant__ StaticTable tab,
                    int P, int n_tiles, double* __restrict__ norms) {
    const int lane = threadIdx.x & 31;
    const long long s = (long long)blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (s >= (long long)P * tab.T) return;
    const int i = (int)(s / tab.T), t = (int)(s % tab.T);
    const double* p = partials + (long long)i * n_tiles;
    double acc = 0.0;
    for (int q = tab.tile_begin[t] + lane; q < tab.tile_begin[t + 1]; q += 32) acc = __dadd_rn(acc, p[q]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc = __dadd_rn(acc, __shfl_down_sync(0xffffffffu, acc, o));
    if (lane == 0) norms[s] = __dsqrt_rn(acc);
}

std::mutex g_mu;
double* g_scratch_addr[kMaxDevices] = {nullptr};   // device address of g_static_partials, per device

}  // namespace

extern "C" eg_status eg_change_norms_static(const float* x_dev, const float* xhat_dev, int P,
                                            int64_t replica_stride, const int64_t* tensor_offset_host,
                                            const int64_t* layer_numel_host, int T, double* norms_dev,
                                            void* stream_v) {
    if (!x_dev || !xhat_dev || !tensor_offset_host || !layer_numel_host || !norms_dev) return EG_ERR_INVALID;
    // P is the second grid dimension of the first kernel
    if (P < 1 || P > 65535 || T < 1 || T > kStaticMaxTensors || replica_stride < 1) return EG_ERR_INVALID;
    if (((uintptr_t)x_dev & 15u) || ((uintptr_t)xhat_dev & 15u) || (replica_stride & 3)) return EG_ERR_INVALID;
    StaticTable tab;
    long long tiles = 0;
    for (int t = 0; t < T; ++t) {
        const int64_t n = layer_numel_host[t], o = tensor_offset_host[t];
        if (n < 1 || n > 0x7fffffffll || o < 0 || (o & 3) || o > replica_stride - n) return EG_ERR_INVALID;
        tab.offset[t] = o;
        tab.numel[t] = (int)n;
        tab.tile_begin[t] = (int)tiles;
        tiles += (n + kNormTile - 1) / kNormTile;
        if (tiles * P > kStaticMaxPartials) return EG_ERR_INVALID;   // beyond the fixed scratch
    }
    tab.tile_begin[T] = (int)tiles;
    tab.T = T;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return EG_ERR_CUDA;
    double* scratch = nullptr;
    {
        // The array's name is only a host-side handle; a kernel needs its device address, which
        // differs per GPU.  Looked up once per device, with that device current.
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_scratch_addr[dev]) {
            void* p = nullptr;
            if (cudaGetSymbolAddress(&p, g_static_partials) != cudaSuccess || !p) return EG_ERR_CUDA;
            g_scratch_addr[dev] = static_cast<double*>(p);
        }
        scratch = g_scratch_addr[dev];
    }
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    // The status of each launch is taken from the launch itself, so that an error left behind
    // by an unrelated earlier call is neither reported here nor cleared.
    long long stride_ll = (long long)replica_stride;
    int n_tiles = (int)tiles;
    void* args1[] = {&x_dev, &xhat_dev, &tab, &stride_ll, &n_tiles, &scratch};
    if (cudaLaunchKernel((const void*)k_static_norm_partial, dim3((unsigned)tiles, (unsigned)P), dim3(kThreads),
                         args1, 0, stream) != cudaSuccess)
        return EG_ERR_CUDA;          // the second kernel is not launched on stale partial sums
    const long long S = (long long)P * T;
    const double* scratch_c = scratch;
    void* args2[] = {&scratch_c, &tab, &P, &n_tiles, &norms_dev};
    if (cudaLaunchKernel((const void*)k_static_norm_final, dim3((unsigned)((S + kWarps - 1) / kWarps)),
                         dim3(kThreads), args2, 0, stream) != cudaSuccess)
        return EG_ERR_CUDA;
    return EG_OK;
}
