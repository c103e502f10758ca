// intsgd_sqdiff_noalloc: the squared step length ||x - x_prev||^2 for callers that must not
// allocate device memory.
//
// Every other entry point of this library needs a context, and creating a context calls cudaMalloc
// for its state block and reduction scratch.  Some hosts cannot do that at the point where they need
// the norm: a training loop that has handed all device memory to its framework's caching allocator
// and forbids raw cudaMalloc afterwards, a latency-critical loop where an implicit device
// synchronisation by the allocator is unacceptable, or a plug-in that is only given buffers and a
// stream.  For them the per-block partial sums of the reduction live in a fixed array that is part
// of the library image: it costs kScratchBytes on every GPU that loads the library, for the life of
// the process, and it bounds the vector length to INTSGD_NOALLOC_MAX_D coordinates.
//
// The array is shared by all calls on a device and keeps the previous call's partials; the arrival
// counter is the only word that must start at zero and is cleared on the stream before each launch.
// Two calls that overlap on the GPU (different streams, or threads) race on it.
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "intsgd.h"

namespace {

constexpr int kThreads = 256;
constexpr int kUnitsPerThread = 16;                                    // 4 coordinates each
constexpr int64_t kCoordsPerBlock = (int64_t)kThreads * kUnitsPerThread * 4;   // 16384
constexpr int kMaxBlocks = (int)(INTSGD_NOALLOC_MAX_D / kCoordsPerBlock);      // 16384 partial sums
constexpr int kMaxDevices = 64;
static_assert((int64_t)kMaxBlocks * kCoordsPerBlock == INTSGD_NOALLOC_MAX_D, "block tiling must cover the maximum");

// partial[b] for b < kMaxBlocks, then the arrival counter.  128 KiB + 8 bytes per GPU.
struct Scratch {
    double partial[kMaxBlocks];
    unsigned long long arrived;
};
constexpr size_t kScratchBytes = sizeof(Scratch);

// In host code this name is only a handle for cudaGetSymbolAddress; kernels are given the address
// that call returns.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

__device__ __forceinline__ double tree32(double v) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_down_sync(0xFFFFFFFFu, v, off);
    return v;
}

__device__ double block_sum(double v, double* s_warp) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    v = tree32(v);
    if (lane == 0) s_warp[warp] = v;
    __syncthreads();
    double t = 0.0;
    if (warp == 0) t = tree32(lane < kThreads / 32 ? s_warp[lane] : 0.0);
    __syncthreads();
    return t;   // valid in thread 0
}

// Block b reduces coordinates [b * kCoordsPerBlock, (b + 1) * kCoordsPerBlock) in a fixed order, so
// the result depends on d only, not on the GPU.  The last block to arrive adds the partials.
template <bool ALIGNED>
__global__ void __launch_bounds__(kThreads) sqdiff_noalloc_kernel(const float* __restrict__ x,
                                                                  const float* __restrict__ x_prev, int64_t d,
                                                                  Scratch* scratch, double* out) {
    __shared__ double s_warp[kThreads / 32];
    __shared__ bool s_last;
    const int64_t begin = (int64_t)blockIdx.x * kCoordsPerBlock;
    const int64_t end = (begin + kCoordsPerBlock < d) ? begin + kCoordsPerBlock : d;
    double acc = 0.0;
    if (ALIGNED) {
        const int64_t u0 = begin >> 2, u1 = end >> 2;   // begin is a multiple of 4
        for (int64_t u = u0 + threadIdx.x; u < u1; u += kThreads) {
            const float4 a = ((const float4*)x)[u], b = ((const float4*)x_prev)[u];
            const float d0 = __fsub_rn(a.x, b.x), d1 = __fsub_rn(a.y, b.y);
            const float d2 = __fsub_rn(a.z, b.z), d3 = __fsub_rn(a.w, b.w);
            acc = __fma_rn((double)d0, (double)d0, acc);
            acc = __fma_rn((double)d1, (double)d1, acc);
            acc = __fma_rn((double)d2, (double)d2, acc);
            acc = __fma_rn((double)d3, (double)d3, acc);
        }
        if (threadIdx.x == 0)
            for (int64_t j = u1 << 2; j < end; ++j) {
                const float dj = __fsub_rn(x[j], x_prev[j]);
                acc = __fma_rn((double)dj, (double)dj, acc);
            }
    } else {
        for (int64_t j = begin + threadIdx.x; j < end; j += kThreads) {
            const float dj = __fsub_rn(x[j], x_prev[j]);
            acc = __fma_rn((double)dj, (double)dj, acc);
        }
    }
    const double bsum = block_sum(acc, s_warp);
    if (threadIdx.x == 0) {
        __stcg(&scratch->partial[blockIdx.x], bsum);
        __threadfence();
        s_last = (atomicAdd(&scratch->arrived, 1ull) == (unsigned long long)gridDim.x - 1);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    double v = 0.0;
    for (unsigned b = threadIdx.x; b < gridDim.x; b += kThreads) v += __ldcg(&scratch->partial[b]);
    const double total = block_sum(v, s_warp);
    if (threadIdx.x == 0) {
        *out = total;
        scratch->arrived = 0;
    }
}

// Device address of the scratch array, looked up once per device with that device current.
Scratch* scratch_address(int device, cudaError_t* err) {
    static std::mutex mu;
    static Scratch* table[kMaxDevices] = {};
    std::lock_guard<std::mutex> lock(mu);
    if (!table[device]) {
        void* p = nullptr;
        *err = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (*err != cudaSuccess) return nullptr;
        table[device] = static_cast<Scratch*>(p);
    }
    *err = cudaSuccess;
    return table[device];
}

}  // namespace

extern "C" int intsgd_sqdiff_noalloc(const float* x, const float* x_prev, int64_t d, double* out, void* stream) {
    if (!x || !x_prev || !out) return INTSGD_ERR_INVALID_ARG;
    if (d < 1) return INTSGD_ERR_INVALID_ARG;
    if (d > INTSGD_NOALLOC_MAX_D) return INTSGD_ERR_TOO_LARGE;
    if (reinterpret_cast<uintptr_t>(x) % 4 || reinterpret_cast<uintptr_t>(x_prev) % 4 ||
        reinterpret_cast<uintptr_t>(out) % 8)
        return INTSGD_ERR_ALIGN;
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) return INTSGD_ERR_CUDA;
    if (device < 0 || device >= kMaxDevices) return INTSGD_ERR_UNSUPPORTED;
    cudaError_t e;
    Scratch* scratch = scratch_address(device, &e);
    if (!scratch) return INTSGD_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(&scratch->arrived, 0, sizeof(unsigned long long), s) != cudaSuccess) return INTSGD_ERR_CUDA;
    const unsigned blocks = (unsigned)((d + kCoordsPerBlock - 1) / kCoordsPerBlock);
    const bool aligned = reinterpret_cast<uintptr_t>(x) % 16 == 0 && reinterpret_cast<uintptr_t>(x_prev) % 16 == 0;
    if (aligned) sqdiff_noalloc_kernel<true><<<blocks, kThreads, 0, s>>>(x, x_prev, d, scratch, out);
    else sqdiff_noalloc_kernel<false><<<blocks, kThreads, 0, s>>>(x, x_prev, d, scratch, out);
    return cudaGetLastError() == cudaSuccess ? INTSGD_OK : INTSGD_ERR_CUDA;
}
