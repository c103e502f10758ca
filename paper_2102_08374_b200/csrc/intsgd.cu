// Host side of the IntSGD step library: argument checks, launch shapes, the C ABI of intsgd.h.
// Every step of the path runs in the kernels of intsgd_kernels.cuh; there is no CPU fallback.
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <limits>
#include <new>
#include <vector>

#include "intsgd_tuning.h"
#include "intsgd_diana.cuh"
#include "intsgd_encode_pipe.cuh"
#include "intsgd_kernels.cuh"
#include "intsgd_pipe.cuh"

using namespace intsgd;

struct intsgd_ctx {
    intsgd_config cfg;
    int64_t L;            // clip limit as an integer
    float Lf;             // largest fp32 <= L
    PhiloxKeys keys;
    PhiloxWorkerTable tab;
    int fused_path;       // 0 / 2 = automatic (pipelined kernels when the pointers allow it), 1 = direct kernels
    DevState* d_state;
    double* d_partials;
    int max_grid;
    int sm_count;
    int threads;
    int blocks_per_sm;
    cudaStream_t last_stream;
    int64_t launches;
    // block-wise scales (Algorithm 2); bs.B == 0 means one scalar alpha
    BlockState bs;
    int64_t* d_offsets;
    NormPlan plan[2];     // [0]: covered range of the direct kernels and fp32; [1]: bf16 pipelined (even units)
    void* d_plan_mem[2];
    // device staging for intsgd_step_host (allocated on first use)
    void* stage_grads[INTSGD_MAX_WORKERS];
    float* stage_x;
    int32_t* stage_agg;
    bool follows_scale;         // the next vector launch comes directly behind this step's scale kernel
    cudaStream_t back_stream;   // device->host copies of finished windows (non-blocking stream)
    cudaEvent_t window_done;
    char err[256];
};

namespace {

thread_local char g_create_err[256] = "";

constexpr int kMaxDevices = 64;
constexpr int kDefaultThreads = 256;
constexpr int kDefaultBlocksPerSm = 8;
constexpr int kMaxBlocksPerSm = 32;

int fail(intsgd_ctx* ctx, int code, const char* fmt, const char* detail = "") {
    char* dst = ctx ? ctx->err : g_create_err;
    std::snprintf(dst, 256, fmt, detail);
    return code;
}

#define CUDA_TRY(ctx, expr)                                                                  \
    do {                                                                                     \
        cudaError_t e_ = (expr);                                                             \
        if (e_ != cudaSuccess) return fail((ctx), INTSGD_ERR_CUDA, #expr ": %s", cudaGetErrorString(e_)); \
    } while (0)

// Makes the context's device current for the duration of a call and restores the caller's.
struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    cudaError_t status = cudaSuccess;
    explicit DeviceGuard(int dev) {
        status = cudaGetDevice(&prev);
        if (status == cudaSuccess && prev != dev) {
            status = cudaSetDevice(dev);
            switched = (status == cudaSuccess);
        }
    }
    ~DeviceGuard() {
        if (switched) cudaSetDevice(prev);
    }
};

bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

size_t grad_elem_size(int dt) { return dt == INTSGD_GRAD_BF16 ? 2 : 4; }
size_t payload_elem_size(int dt) { return dt == INTSGD_PAYLOAD_I8 ? 1 : 4; }

// Philox key schedule: round r uses key + r * (Weyl constants), modulo 2^32.
PhiloxKeys make_keys(uint64_t seed) {
    PhiloxKeys k;
    uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
    for (int r = 0; r < 10; ++r) {
        k.k0[r] = k0;
        k.k1[r] = k1;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return k;
}

// Worker-dependent part of Philox rounds 1-2 for counter (unit, 0, worker, step): see
// PhiloxWorkerTable.
PhiloxWorkerTable make_worker_table(const PhiloxKeys& k) {
    PhiloxWorkerTable t;
    for (uint32_t i = 0; i < INTSGD_MAX_WORKERS; ++i) {
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)i;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ k.k0[0];
        const uint64_t q0 = (uint64_t)0xD2511F53u * (uint64_t)n0;
        t.e[i] = make_uint4((uint32_t)p1 ^ k.k0[1], (uint32_t)(q0 >> 32) ^ k.k1[1], (uint32_t)q0, 0u);
    }
    return t;
}

float largest_float_not_above(int64_t L) {
    float f = (float)L;
    if ((double)f > (double)L) f = std::nextafterf(f, 0.0f);
    return f;
}

int grid_for(const intsgd_ctx* ctx, int64_t work_items) {
    int64_t blocks = (work_items + ctx->threads - 1) / ctx->threads;
    const int64_t cap = (int64_t)ctx->sm_count * ctx->blocks_per_sm;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (int)blocks;
}

void base_params(const intsgd_ctx* ctx, VecParams& P) {
    std::memset(&P, 0, sizeof P);
    P.st = ctx->d_state;
    P.partials = ctx->d_partials;
    P.d = ctx->cfg.d;
    P.n = ctx->cfg.n;
    P.alpha_override = std::numeric_limits<float>::quiet_NaN();
    P.Lf = ctx->Lf;
    P.agg_limit = (ctx->cfg.payload_dtype == INTSGD_PAYLOAD_I8) ? 127 : std::numeric_limits<int32_t>::max();
    P.keys = ctx->keys;
    P.tab = ctx->tab;
}

int check_vector(intsgd_ctx* ctx, const void* p, size_t elem, const char* what, bool* all16) {
    if (!p) return fail(ctx, INTSGD_ERR_INVALID_ARG, "%s is NULL", what);
    if (!aligned_to(p, elem)) return fail(ctx, INTSGD_ERR_ALIGN, "%s is not aligned to its element size", what);
    if (!aligned_to(p, 16)) *all16 = false;
    return INTSGD_OK;
}

int after_launch(intsgd_ctx* ctx, const char* what) {
    ctx->launches += 1;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        std::snprintf(ctx->err, 256, "launch of %s failed: %s", what, cudaGetErrorString(e));
        return INTSGD_ERR_CUDA;
    }
    return INTSGD_OK;
}

// ---- launchers -------------------------------------------------------------------------

// Launch as a programmatic dependent of the kernel in front of it on the stream: the grid may become resident
// while that kernel drains (its launch latency leaves the step's path); every kernel launched this way executes
// griddepcontrol.wait before it touches memory the kernel in front writes.
template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t s, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

int launch_scale(intsgd_ctx* ctx, double eta, double dx2_override, cudaStream_t s) {
    if (!(eta > 0.0) || !std::isfinite(eta)) return fail(ctx, INTSGD_ERR_INVALID_ARG, "eta_k must be finite and > 0");
    if (std::isnan(dx2_override) || std::isinf(dx2_override))
        return fail(ctx, INTSGD_ERR_INVALID_ARG, "dx2_override must be finite (negative = use the state)");
    const double dd = (double)ctx->cfg.d, dn = (double)ctx->cfg.n;
    if (ctx->bs.B > 0) {
        if (dx2_override >= 0.0)
            return fail(ctx, INTSGD_ERR_UNSUPPORTED, "dx2_override is not available with block-wise scales");
        const cudaError_t e = launch_dependent(scale_blocks_kernel, dim3(1), dim3(1024), s, ctx->d_state, ctx->bs, dd, 2.0 * dn, dn,
                                               eta, ctx->cfg.beta, ctx->cfg.eps, (int32_t)ctx->cfg.n);
        if (e != cudaSuccess) return fail(ctx, INTSGD_ERR_CUDA, "launch of scale_blocks_kernel failed: %s", cudaGetErrorString(e));
        return after_launch(ctx, "scale_blocks_kernel");
    }
    // The scale kernel may be scheduled while the kernel before it on the stream is still running (it waits
    // for that kernel's completion before it touches the state): its launch latency leaves the step's path.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(1, 1, 1);
    cfg.blockDim = dim3(32, 1, 1);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, scale_kernel, ctx->d_state, std::sqrt(dd), 2.0 * dn, dn, eta, ctx->cfg.beta,
                                             ctx->cfg.eps, dx2_override, (int32_t)ctx->cfg.n);
    if (e != cudaSuccess) {
        std::snprintf(ctx->err, 256, "launch of scale_kernel failed: %s", cudaGetErrorString(e));
        return INTSGD_ERR_CUDA;
    }
    return after_launch(ctx, "scale_kernel");
}

template <int GRAD, int PAY, bool ALIGNED>
void launch_encode_r(const intsgd_ctx* ctx, const VecParams& P, dim3 grid, cudaStream_t s) {
    if (ctx->cfg.rounding == INTSGD_ROUND_NEAREST)
        encode_kernel<GRAD, PAY, ALIGNED, INTSGD_ROUND_NEAREST><<<grid, ctx->threads, 0, s>>>(P);
    else if (ctx->cfg.rounding == INTSGD_ROUND_RANDOM16)
        encode_kernel<GRAD, PAY, ALIGNED, INTSGD_ROUND_RANDOM16><<<grid, ctx->threads, 0, s>>>(P);
    else if (ctx->cfg.rounding == INTSGD_ROUND_RANDOM_COMPARE)
        encode_kernel<GRAD, PAY, ALIGNED, INTSGD_ROUND_RANDOM_COMPARE><<<grid, ctx->threads, 0, s>>>(P);
    else
        encode_kernel<GRAD, PAY, ALIGNED, INTSGD_ROUND_RANDOM><<<grid, ctx->threads, 0, s>>>(P);
}
template <int GRAD, int PAY>
void launch_encode_a(const intsgd_ctx* ctx, const VecParams& P, dim3 grid, bool aligned, cudaStream_t s) {
    if (aligned) launch_encode_r<GRAD, PAY, true>(ctx, P, grid, s);
    else launch_encode_r<GRAD, PAY, false>(ctx, P, grid, s);
}
int launch_encode_pipe(intsgd_ctx* ctx, const VecParams& P, cudaStream_t s);
bool pipe_eligible(const intsgd_ctx* ctx, bool aligned, int64_t d);
void fill_block_params(const intsgd_ctx* ctx, VecParams& P, int64_t covered_end);

template <int GRAD, int PAY, bool ALIGNED>
void launch_encode_blocks_r(const intsgd_ctx* ctx, const VecParams& P, dim3 grid, cudaStream_t s) {
    switch (ctx->cfg.rounding) {
        case INTSGD_ROUND_NEAREST: encode_blocks_kernel<GRAD, PAY, ALIGNED, INTSGD_ROUND_NEAREST><<<grid, ctx->threads, 0, s>>>(P); break;
        case INTSGD_ROUND_RANDOM16: encode_blocks_kernel<GRAD, PAY, ALIGNED, INTSGD_ROUND_RANDOM16><<<grid, ctx->threads, 0, s>>>(P); break;
        case INTSGD_ROUND_RANDOM_COMPARE: encode_blocks_kernel<GRAD, PAY, ALIGNED, INTSGD_ROUND_RANDOM_COMPARE><<<grid, ctx->threads, 0, s>>>(P); break;
        default: encode_blocks_kernel<GRAD, PAY, ALIGNED, INTSGD_ROUND_RANDOM><<<grid, ctx->threads, 0, s>>>(P); break;
    }
}
template <int GRAD, int PAY>
void launch_encode_blocks_a(const intsgd_ctx* ctx, const VecParams& P, dim3 grid, bool aligned, cudaStream_t s) {
    if (aligned) launch_encode_blocks_r<GRAD, PAY, true>(ctx, P, grid, s);
    else launch_encode_blocks_r<GRAD, PAY, false>(ctx, P, grid, s);
}
void launch_encode_blocks(const intsgd_ctx* ctx, const VecParams& P, dim3 grid, bool bf16, bool i8, bool aligned, cudaStream_t s) {
    if (!bf16 && !i8) launch_encode_blocks_a<INTSGD_GRAD_F32, INTSGD_PAYLOAD_I32>(ctx, P, grid, aligned, s);
    else if (!bf16) launch_encode_blocks_a<INTSGD_GRAD_F32, INTSGD_PAYLOAD_I8>(ctx, P, grid, aligned, s);
    else if (!i8) launch_encode_blocks_a<INTSGD_GRAD_BF16, INTSGD_PAYLOAD_I32>(ctx, P, grid, aligned, s);
    else launch_encode_blocks_a<INTSGD_GRAD_BF16, INTSGD_PAYLOAD_I8>(ctx, P, grid, aligned, s);
}

int launch_encode(intsgd_ctx* ctx, const VecParams& P, int workers, bool aligned, cudaStream_t s) {
    // All the workers of a step in one launch: the pipelined kernel (a thread keeps its units across workers).
    if (workers >= 2 && ctx->fused_path != 1 && pipe_eligible(ctx, aligned, P.d)) return launch_encode_pipe(ctx, P, s);
    dim3 grid((unsigned)grid_for(ctx, (ctx->cfg.d + 3) / 4), (unsigned)workers, 1);
    // spread the block budget over the workers handled by one launch
    if (workers > 1) {
        int per = (ctx->sm_count * ctx->blocks_per_sm + workers - 1) / workers;
        if (per < 1) per = 1;
        if ((int)grid.x > per) grid.x = (unsigned)per;
    }
    const bool bf16 = ctx->cfg.grad_dtype == INTSGD_GRAD_BF16, i8 = ctx->cfg.payload_dtype == INTSGD_PAYLOAD_I8;
    if (ctx->bs.B > 0) {
        VecParams Q = P;
        fill_block_params(ctx, Q, (ctx->cfg.d >> 2) << 2);
        launch_encode_blocks(ctx, Q, grid, bf16, i8, aligned, s);
        return after_launch(ctx, "encode_blocks_kernel");
    }
    if (!bf16 && !i8) launch_encode_a<INTSGD_GRAD_F32, INTSGD_PAYLOAD_I32>(ctx, P, grid, aligned, s);
    else if (!bf16 && i8) launch_encode_a<INTSGD_GRAD_F32, INTSGD_PAYLOAD_I8>(ctx, P, grid, aligned, s);
    else if (bf16 && !i8) launch_encode_a<INTSGD_GRAD_BF16, INTSGD_PAYLOAD_I32>(ctx, P, grid, aligned, s);
    else launch_encode_a<INTSGD_GRAD_BF16, INTSGD_PAYLOAD_I8>(ctx, P, grid, aligned, s);
    return after_launch(ctx, "encode_kernel");
}

int launch_block_norm(intsgd_ctx* ctx, int64_t covered_end, bool check_status, bool advance_step, cudaStream_t s);

int launch_aggregate(intsgd_ctx* ctx, const VecParams& P, bool aligned, cudaStream_t s) {
    const bool i8 = ctx->cfg.payload_dtype == INTSGD_PAYLOAD_I8;
    if (ctx->bs.B > 0) {
        VecParams Q = P;
        const int64_t covered = (ctx->cfg.d >> 2) << 2;
        fill_block_params(ctx, Q, covered);
        // the step's scale kernel has cleared the edge partials; clearing them again here keeps a repeated
        // aggregate (without a scale in between) correct as well
        if (cudaMemsetAsync(ctx->bs.edge_sum, 0, sizeof(double) * ctx->bs.B, s) != cudaSuccess)
            return fail(ctx, INTSGD_ERR_CUDA, "cudaMemsetAsync failed");
        const int grid = grid_for(ctx, (ctx->cfg.d + 3) / 4);
        if (!i8 && aligned) aggregate_blocks_kernel<INTSGD_PAYLOAD_I32, true><<<grid, ctx->threads, 0, s>>>(Q);
        else if (!i8) aggregate_blocks_kernel<INTSGD_PAYLOAD_I32, false><<<grid, ctx->threads, 0, s>>>(Q);
        else if (aligned) aggregate_blocks_kernel<INTSGD_PAYLOAD_I8, true><<<grid, ctx->threads, 0, s>>>(Q);
        else aggregate_blocks_kernel<INTSGD_PAYLOAD_I8, false><<<grid, ctx->threads, 0, s>>>(Q);
        const int rc = after_launch(ctx, "aggregate_blocks_kernel");
        if (rc != INTSGD_OK) return rc;
        return launch_block_norm(ctx, covered, true, true, s);
    }
    const int64_t items = (i8 && !aligned) ? ctx->cfg.d : (ctx->cfg.d + 3) / 4;
    const int grid = grid_for(ctx, items);
    if (!i8 && aligned) aggregate_kernel<INTSGD_PAYLOAD_I32, true><<<grid, ctx->threads, 0, s>>>(P);
    else if (!i8) aggregate_kernel<INTSGD_PAYLOAD_I32, false><<<grid, ctx->threads, 0, s>>>(P);
    else if (aligned) aggregate_kernel<INTSGD_PAYLOAD_I8, true><<<grid, ctx->threads, 0, s>>>(P);
    else aggregate_kernel<INTSGD_PAYLOAD_I8, false><<<grid, ctx->threads, 0, s>>>(P);
    return after_launch(ctx, "aggregate_kernel");
}

template <int GRAD, bool ALIGNED>
void launch_fused_r(const intsgd_ctx* ctx, const VecParams& P, int grid, cudaStream_t s) {
    if (ctx->cfg.rounding == INTSGD_ROUND_NEAREST)
        fused_step_kernel<GRAD, ALIGNED, INTSGD_ROUND_NEAREST><<<grid, ctx->threads, 0, s>>>(P);
    else if (ctx->cfg.rounding == INTSGD_ROUND_RANDOM16)
        fused_step_kernel<GRAD, ALIGNED, INTSGD_ROUND_RANDOM16><<<grid, ctx->threads, 0, s>>>(P);
    else if (ctx->cfg.rounding == INTSGD_ROUND_RANDOM_COMPARE)
        fused_step_kernel<GRAD, ALIGNED, INTSGD_ROUND_RANDOM_COMPARE><<<grid, ctx->threads, 0, s>>>(P);
    else
        fused_step_kernel<GRAD, ALIGNED, INTSGD_ROUND_RANDOM><<<grid, ctx->threads, 0, s>>>(P);
}

// Pipelined kernel shape: NC consumer threads (+ one producer warp), UPT units per thread and tile, G worker
// tiles per stage, NS stages; one block per SM, 192 KiB of shared memory.  512 x 2 units with 3 stages of 4 fp32
// (8 bf16) worker tiles is the fastest of the shapes timed on B200 (one or four units per thread, 256 to 992
// consumers, two smaller blocks per SM: all slower).
struct PipeShape { int nc, upt, g, ns; };
template <int GRAD, int ROUND, bool BLOCKS>
cudaError_t launch_pipe_v(const intsgd_ctx* ctx, PipeParams& PP, cudaStream_t s) {
    // bf16 tiles are half as large: a stage holds 8 worker tiles (fewer barrier rounds)
    constexpr PipeShape S = (GRAD == INTSGD_GRAD_BF16) ? PipeShape{512, 2, 8, 3} : PipeShape{512, 2, 4, 3};
    auto kernel = fused_pipe_kernel<GRAD, ROUND, BLOCKS, S.nc, S.upt, S.g, S.ns>;
    const int unit_bytes = (GRAD == INTSGD_GRAD_F32) ? 16 : 8;
    const int smem = S.ns * S.g * S.nc * S.upt * unit_bytes;
    // per instantiation and device: the opt-in to large shared memory (contexts on other threads may race here:
    // setting the attribute twice is harmless, the flag itself is atomic)
    static std::atomic<bool> configured[kMaxDevices] = {};
    const int dev = ctx->cfg.device;
    if (dev < 0 || dev >= kMaxDevices || !configured[dev].load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < kMaxDevices) configured[dev].store(true, std::memory_order_release);
    }
    PP.tiles = (PP.units + S.nc * S.upt - 1) / (S.nc * S.upt);
    int64_t grid = PP.tiles < ctx->sm_count ? PP.tiles : ctx->sm_count;
    // Launched right behind the step's scale kernel, the kernel may start while that one drains: it sets up
    // its barriers and tables, then waits for the scale kernel's results (griddepcontrol.wait).
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(S.nc + 32, 1, 1);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = ctx->follows_scale ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, PP);
}
template <int GRAD, int ROUND>
cudaError_t launch_pipe_t(const intsgd_ctx* ctx, PipeParams& PP, cudaStream_t s) {
    return ctx->bs.B > 0 ? launch_pipe_v<GRAD, ROUND, true>(ctx, PP, s) : launch_pipe_v<GRAD, ROUND, false>(ctx, PP, s);
}
// `d` is the length of the launch (a window of the vector, or all of it).
bool pipe_eligible(const intsgd_ctx* ctx, bool aligned, int64_t d) {
    const int64_t units = d >> 2;
    return aligned && ctx->cfg.d <= ((int64_t)1 << 34) && units >= 2;
}

// Pipelined encode: the default ring shape of the fused kernel (512 consumers, 2 units each, 3 stages of 4 fp32
// or 8 bf16 worker tiles).
template <int GRAD, int PAY, int ROUND, bool BLOCKS>
cudaError_t launch_encode_pipe_b(const intsgd_ctx* ctx, PipeParams& PP, cudaStream_t s) {
    constexpr int NC = 512, UPT = 2, NS = 3, G = (GRAD == INTSGD_GRAD_BF16) ? 8 : 4;
    auto kernel = encode_pipe_kernel<GRAD, PAY, ROUND, BLOCKS, NC, UPT, G, NS>;
    const int smem = NS * G * NC * UPT * ((GRAD == INTSGD_GRAD_F32) ? 16 : 8);
    static std::atomic<bool> configured[kMaxDevices] = {};
    const int dev = ctx->cfg.device;
    if (dev < 0 || dev >= kMaxDevices || !configured[dev].load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < kMaxDevices) configured[dev].store(true, std::memory_order_release);
    }
    PP.tiles = (PP.units + NC * UPT - 1) / (NC * UPT);
    const int64_t grid = PP.tiles < ctx->sm_count ? PP.tiles : ctx->sm_count;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(NC + 32, 1, 1);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = ctx->follows_scale ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, PP);
}
template <int GRAD, int PAY, int ROUND>
cudaError_t launch_encode_pipe_t(const intsgd_ctx* ctx, PipeParams& PP, cudaStream_t s) {
    return ctx->bs.B > 0 ? launch_encode_pipe_b<GRAD, PAY, ROUND, true>(ctx, PP, s) : launch_encode_pipe_b<GRAD, PAY, ROUND, false>(ctx, PP, s);
}
template <int GRAD, int PAY>
cudaError_t launch_encode_pipe_r(const intsgd_ctx* ctx, PipeParams& PP, cudaStream_t s) {
    switch (ctx->cfg.rounding) {
        case INTSGD_ROUND_NEAREST: return launch_encode_pipe_t<GRAD, PAY, INTSGD_ROUND_NEAREST>(ctx, PP, s);
        case INTSGD_ROUND_RANDOM16: return launch_encode_pipe_t<GRAD, PAY, INTSGD_ROUND_RANDOM16>(ctx, PP, s);
        case INTSGD_ROUND_RANDOM_COMPARE: return launch_encode_pipe_t<GRAD, PAY, INTSGD_ROUND_RANDOM_COMPARE>(ctx, PP, s);
        default: return launch_encode_pipe_t<GRAD, PAY, INTSGD_ROUND_RANDOM>(ctx, PP, s);
    }
}
int launch_encode_pipe(intsgd_ctx* ctx, const VecParams& P, cudaStream_t s) {
    PipeParams PP;
    PP.v = P;
    const bool bf16 = ctx->cfg.grad_dtype == INTSGD_GRAD_BF16, i8 = ctx->cfg.payload_dtype == INTSGD_PAYLOAD_I8;
    int64_t units = P.d >> 2;
    if (bf16) units &= ~(int64_t)1;   // bulk copies move multiples of 16 bytes
    PP.units = units;
    PP.tiles = 0;
    PP.fast_limit = ctx->Lf;   // not used: out-of-range values take the counting rule on the spot
    if (ctx->bs.B > 0) fill_block_params(ctx, PP.v, units << 2);
    cudaError_t e;
    if (!bf16 && !i8) e = launch_encode_pipe_r<INTSGD_GRAD_F32, INTSGD_PAYLOAD_I32>(ctx, PP, s);
    else if (!bf16) e = launch_encode_pipe_r<INTSGD_GRAD_F32, INTSGD_PAYLOAD_I8>(ctx, PP, s);
    else if (!i8) e = launch_encode_pipe_r<INTSGD_GRAD_BF16, INTSGD_PAYLOAD_I32>(ctx, PP, s);
    else e = launch_encode_pipe_r<INTSGD_GRAD_BF16, INTSGD_PAYLOAD_I8>(ctx, PP, s);
    if (e != cudaSuccess) {
        std::snprintf(ctx->err, 256, "encode_pipe_kernel launch failed: %s", cudaGetErrorString(e));
        return INTSGD_ERR_CUDA;
    }
    return after_launch(ctx, "encode_pipe_kernel");
}

void fill_block_params(const intsgd_ctx* ctx, VecParams& P, int64_t covered_end) {
    P.bp.offsets = ctx->bs.offsets;
    P.bp.alpha = ctx->bs.alpha;
    P.bp.c = ctx->bs.c;
    P.bp.chunk_sum = ctx->bs.chunk_sum;
    P.bp.chunk_seg = ctx->bs.chunk_seg;
    P.bp.edge_sum = ctx->bs.edge_sum;
    P.bp.tail_sq = ctx->bs.tail_sq;
    P.bp.covered_end = covered_end;
    P.bp.B = ctx->bs.B;
}

// Finishes a block-wise step: per-segment squared step lengths, total, step counter.
int launch_block_norm(intsgd_ctx* ctx, int64_t covered_end, bool check_status, bool advance_step, cudaStream_t s) {
    const NormPlan& plan = (ctx->plan[0].covered_end == covered_end) ? ctx->plan[0] : ctx->plan[1];
    if (plan.covered_end != covered_end) return fail(ctx, INTSGD_ERR_CUDA, "internal: no reduction plan for this launch");
    if (plan.num_slices > 0) {
        const cudaError_t e = launch_dependent(block_norm_slices_kernel, dim3(plan.num_slices), dim3(256), s,
                                               (const DevState*)ctx->d_state, ctx->bs, plan, (int32_t)(check_status ? 1 : 0));
        if (e != cudaSuccess) return fail(ctx, INTSGD_ERR_CUDA, "launch of block_norm_slices_kernel failed: %s", cudaGetErrorString(e));
        const int rc = after_launch(ctx, "block_norm_slices_kernel");
        if (rc != INTSGD_OK) return rc;
    }
    const cudaError_t e = launch_dependent(block_norm_kernel, dim3(ctx->bs.B), dim3(128), s, ctx->d_state, ctx->bs, plan,
                                           (int64_t)ctx->cfg.d, (int32_t)(check_status ? 1 : 0), (int32_t)(advance_step ? 1 : 0));
    if (e != cudaSuccess) return fail(ctx, INTSGD_ERR_CUDA, "launch of block_norm_kernel failed: %s", cudaGetErrorString(e));
    return after_launch(ctx, "block_norm_kernel");
}

int launch_fused_pipe(intsgd_ctx* ctx, const VecParams& P, cudaStream_t s) {
    PipeParams PP;
    PP.v = P;
    const bool bf16 = ctx->cfg.grad_dtype == INTSGD_GRAD_BF16;
    int64_t units = P.d >> 2;
    if (bf16) units &= ~(int64_t)1;   // bulk copies move multiples of 16 bytes
    PP.units = units;
    PP.tiles = 0;   // set by the launcher from the tile shape
    const int64_t covered_end = (P.unit_base << 2) + (units << 2);   // in coordinates of the whole vector
    if (ctx->bs.B > 0) fill_block_params(ctx, PP.v, covered_end);
    // Rounded values are summed as integer-valued floats: exact while n * (T + 1) <= 2^24.
    const float t_max = (float)((1 << 24) / ctx->cfg.n - 2);
    PP.fast_limit = ctx->Lf < t_max ? ctx->Lf : t_max;
    const int rounding = ctx->cfg.rounding;
    cudaError_t e;
    if (!bf16 && rounding == INTSGD_ROUND_RANDOM) e = launch_pipe_t<INTSGD_GRAD_F32, INTSGD_ROUND_RANDOM>(ctx, PP, s);
    else if (!bf16 && rounding == INTSGD_ROUND_RANDOM16) e = launch_pipe_t<INTSGD_GRAD_F32, INTSGD_ROUND_RANDOM16>(ctx, PP, s);
    else if (!bf16 && rounding == INTSGD_ROUND_RANDOM_COMPARE) e = launch_pipe_t<INTSGD_GRAD_F32, INTSGD_ROUND_RANDOM_COMPARE>(ctx, PP, s);
    else if (!bf16) e = launch_pipe_t<INTSGD_GRAD_F32, INTSGD_ROUND_NEAREST>(ctx, PP, s);
    else if (rounding == INTSGD_ROUND_RANDOM) e = launch_pipe_t<INTSGD_GRAD_BF16, INTSGD_ROUND_RANDOM>(ctx, PP, s);
    else if (rounding == INTSGD_ROUND_RANDOM16) e = launch_pipe_t<INTSGD_GRAD_BF16, INTSGD_ROUND_RANDOM16>(ctx, PP, s);
    else if (rounding == INTSGD_ROUND_RANDOM_COMPARE) e = launch_pipe_t<INTSGD_GRAD_BF16, INTSGD_ROUND_RANDOM_COMPARE>(ctx, PP, s);
    else e = launch_pipe_t<INTSGD_GRAD_BF16, INTSGD_ROUND_NEAREST>(ctx, PP, s);
    if (e != cudaSuccess) {
        std::snprintf(ctx->err, 256, "fused_pipe_kernel setup failed: %s", cudaGetErrorString(e));
        return INTSGD_ERR_CUDA;
    }
    const int rc = after_launch(ctx, "fused_pipe_kernel");
    if (rc != INTSGD_OK || ctx->bs.B == 0) return rc;
    if (P.window_flags & kWindowHoldStep) return rc;   // the per-segment norms are finished after the step's last window
    return launch_block_norm(ctx, covered_end, true, true, s);
}

template <int GRAD, bool ALIGNED>
void launch_fused_blocks_r(const intsgd_ctx* ctx, const VecParams& P, int grid, cudaStream_t s) {
    if (ctx->cfg.rounding == INTSGD_ROUND_NEAREST)
        fused_step_blocks_kernel<GRAD, ALIGNED, INTSGD_ROUND_NEAREST><<<grid, ctx->threads, 0, s>>>(P);
    else if (ctx->cfg.rounding == INTSGD_ROUND_RANDOM16)
        fused_step_blocks_kernel<GRAD, ALIGNED, INTSGD_ROUND_RANDOM16><<<grid, ctx->threads, 0, s>>>(P);
    else if (ctx->cfg.rounding == INTSGD_ROUND_RANDOM_COMPARE)
        fused_step_blocks_kernel<GRAD, ALIGNED, INTSGD_ROUND_RANDOM_COMPARE><<<grid, ctx->threads, 0, s>>>(P);
    else
        fused_step_blocks_kernel<GRAD, ALIGNED, INTSGD_ROUND_RANDOM><<<grid, ctx->threads, 0, s>>>(P);
}

int launch_fused(intsgd_ctx* ctx, const VecParams& P, bool aligned, cudaStream_t s) {
    const bool want_pipe = ctx->fused_path != 1 && pipe_eligible(ctx, aligned, P.d);
    if (want_pipe) return launch_fused_pipe(ctx, P, s);
    const int grid = grid_for(ctx, (P.d + 3) / 4);
    const bool bf16 = ctx->cfg.grad_dtype == INTSGD_GRAD_BF16;
    if (ctx->bs.B > 0) {
        VecParams Q = P;
        const int64_t covered = (P.unit_base << 2) + ((P.d >> 2) << 2);
        fill_block_params(ctx, Q, covered);
        if (!bf16 && aligned) launch_fused_blocks_r<INTSGD_GRAD_F32, true>(ctx, Q, grid, s);
        else if (!bf16) launch_fused_blocks_r<INTSGD_GRAD_F32, false>(ctx, Q, grid, s);
        else if (aligned) launch_fused_blocks_r<INTSGD_GRAD_BF16, true>(ctx, Q, grid, s);
        else launch_fused_blocks_r<INTSGD_GRAD_BF16, false>(ctx, Q, grid, s);
        const int rc = after_launch(ctx, "fused_step_blocks_kernel");
        if (rc != INTSGD_OK || (P.window_flags & kWindowHoldStep)) return rc;
        return launch_block_norm(ctx, covered, true, true, s);
    }
    if (!bf16 && aligned) launch_fused_r<INTSGD_GRAD_F32, true>(ctx, P, grid, s);
    else if (!bf16) launch_fused_r<INTSGD_GRAD_F32, false>(ctx, P, grid, s);
    else if (aligned) launch_fused_r<INTSGD_GRAD_BF16, true>(ctx, P, grid, s);
    else launch_fused_r<INTSGD_GRAD_BF16, false>(ctx, P, grid, s);
    return after_launch(ctx, "fused_step_kernel");
}

template <int GRAD, bool ALIGNED>
void launch_diana_r(const intsgd_ctx* ctx, const VecParams& P, int grid, cudaStream_t s) {
    if (ctx->cfg.rounding == INTSGD_ROUND_NEAREST)
        diana_step_kernel<GRAD, ALIGNED, INTSGD_ROUND_NEAREST><<<grid, ctx->threads, 0, s>>>(P);
    else if (ctx->cfg.rounding == INTSGD_ROUND_RANDOM16)
        diana_step_kernel<GRAD, ALIGNED, INTSGD_ROUND_RANDOM16><<<grid, ctx->threads, 0, s>>>(P);
    else if (ctx->cfg.rounding == INTSGD_ROUND_RANDOM_COMPARE)
        diana_step_kernel<GRAD, ALIGNED, INTSGD_ROUND_RANDOM_COMPARE><<<grid, ctx->threads, 0, s>>>(P);
    else
        diana_step_kernel<GRAD, ALIGNED, INTSGD_ROUND_RANDOM><<<grid, ctx->threads, 0, s>>>(P);
}
// Pipelined IntDIANA: 512 consumers, 2 units each, 2 worker slots (gradient tile + shift tile) per stage, 3 stages.
template <int GRAD, int ROUND>
cudaError_t launch_diana_pipe_t(const intsgd_ctx* ctx, PipeParams& PP, cudaStream_t s) {
    constexpr int NC = 512, UPT = 2, G = 2, NS = 3;
    auto kernel = diana_pipe_kernel<GRAD, ROUND, NC, UPT, G, NS>;
    const int smem = NS * G * NC * UPT * (((GRAD == INTSGD_GRAD_F32) ? 16 : 8) + 16);
    static std::atomic<bool> configured[kMaxDevices] = {};
    const int dev = ctx->cfg.device;
    if (dev < 0 || dev >= kMaxDevices || !configured[dev].load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < kMaxDevices) configured[dev].store(true, std::memory_order_release);
    }
    PP.tiles = (PP.units + NC * UPT - 1) / (NC * UPT);
    const int64_t grid = PP.tiles < ctx->sm_count ? PP.tiles : ctx->sm_count;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(NC + 32, 1, 1);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = ctx->follows_scale ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, PP);
}
template <int GRAD>
cudaError_t launch_diana_pipe_r(const intsgd_ctx* ctx, PipeParams& PP, cudaStream_t s) {
    switch (ctx->cfg.rounding) {
        case INTSGD_ROUND_NEAREST: return launch_diana_pipe_t<GRAD, INTSGD_ROUND_NEAREST>(ctx, PP, s);
        case INTSGD_ROUND_RANDOM16: return launch_diana_pipe_t<GRAD, INTSGD_ROUND_RANDOM16>(ctx, PP, s);
        case INTSGD_ROUND_RANDOM_COMPARE: return launch_diana_pipe_t<GRAD, INTSGD_ROUND_RANDOM_COMPARE>(ctx, PP, s);
        default: return launch_diana_pipe_t<GRAD, INTSGD_ROUND_RANDOM>(ctx, PP, s);
    }
}
int launch_diana_pipe(intsgd_ctx* ctx, const VecParams& P, cudaStream_t s) {
    PipeParams PP;
    PP.v = P;
    const bool bf16 = ctx->cfg.grad_dtype == INTSGD_GRAD_BF16;
    int64_t units = P.d >> 2;
    if (bf16) units &= ~(int64_t)1;   // bulk copies move multiples of 16 bytes
    PP.units = units;
    PP.tiles = 0;
    PP.fast_limit = ctx->Lf;   // not used: nothing is deferred in this kernel
    const cudaError_t e = bf16 ? launch_diana_pipe_r<INTSGD_GRAD_BF16>(ctx, PP, s) : launch_diana_pipe_r<INTSGD_GRAD_F32>(ctx, PP, s);
    if (e != cudaSuccess) {
        std::snprintf(ctx->err, 256, "diana_pipe_kernel launch failed: %s", cudaGetErrorString(e));
        return INTSGD_ERR_CUDA;
    }
    return after_launch(ctx, "diana_pipe_kernel");
}

int launch_diana(intsgd_ctx* ctx, const VecParams& P, bool aligned, cudaStream_t s) {
    if (ctx->fused_path != 1 && pipe_eligible(ctx, aligned, P.d)) return launch_diana_pipe(ctx, P, s);
    const int grid = grid_for(ctx, (ctx->cfg.d + 3) / 4);
    const bool bf16 = ctx->cfg.grad_dtype == INTSGD_GRAD_BF16;
    if (!bf16 && aligned) launch_diana_r<INTSGD_GRAD_F32, true>(ctx, P, grid, s);
    else if (!bf16) launch_diana_r<INTSGD_GRAD_F32, false>(ctx, P, grid, s);
    else if (aligned) launch_diana_r<INTSGD_GRAD_BF16, true>(ctx, P, grid, s);
    else launch_diana_r<INTSGD_GRAD_BF16, false>(ctx, P, grid, s);
    return after_launch(ctx, "diana_step_kernel");
}

int launch_exact(intsgd_ctx* ctx, const VecParams& P, bool aligned, cudaStream_t s) {
    const int grid = grid_for(ctx, (P.d + 3) / 4);
    const bool bf16 = ctx->cfg.grad_dtype == INTSGD_GRAD_BF16;
    if (ctx->bs.B > 0) {
        VecParams Q = P;
        const int64_t covered = (P.unit_base << 2) + ((P.d >> 2) << 2);
        fill_block_params(ctx, Q, covered);
        if (!(P.window_flags & kWindowAccumulate) &&   // the first (or only) window of the step opens the edge partials
            cudaMemsetAsync(ctx->bs.edge_sum, 0, sizeof(double) * ctx->bs.B, s) != cudaSuccess)
            return fail(ctx, INTSGD_ERR_CUDA, "cudaMemsetAsync failed");
        if (!bf16 && aligned) exact_step_blocks_kernel<INTSGD_GRAD_F32, true><<<grid, ctx->threads, 0, s>>>(Q);
        else if (!bf16) exact_step_blocks_kernel<INTSGD_GRAD_F32, false><<<grid, ctx->threads, 0, s>>>(Q);
        else if (aligned) exact_step_blocks_kernel<INTSGD_GRAD_BF16, true><<<grid, ctx->threads, 0, s>>>(Q);
        else exact_step_blocks_kernel<INTSGD_GRAD_BF16, false><<<grid, ctx->threads, 0, s>>>(Q);
        const int rc = after_launch(ctx, "exact_step_blocks_kernel");
        if (rc != INTSGD_OK || (P.window_flags & kWindowHoldStep)) return rc;
        return launch_block_norm(ctx, covered, false, true, s);
    }
    if (!bf16 && aligned) exact_step_kernel<INTSGD_GRAD_F32, true><<<grid, ctx->threads, 0, s>>>(P);
    else if (!bf16) exact_step_kernel<INTSGD_GRAD_F32, false><<<grid, ctx->threads, 0, s>>>(P);
    else if (aligned) exact_step_kernel<INTSGD_GRAD_BF16, true><<<grid, ctx->threads, 0, s>>>(P);
    else exact_step_kernel<INTSGD_GRAD_BF16, false><<<grid, ctx->threads, 0, s>>>(P);
    return after_launch(ctx, "exact_step_kernel");
}

int read_state_block(intsgd_ctx* ctx, DevState* host) {
    CUDA_TRY(ctx, cudaStreamSynchronize(ctx->last_stream));
    CUDA_TRY(ctx, cudaMemcpy(host, ctx->d_state, sizeof(DevState), cudaMemcpyDeviceToHost));
    return INTSGD_OK;
}

void free_staging(intsgd_ctx* ctx) {
    for (int i = 0; i < INTSGD_MAX_WORKERS; ++i) {
        if (ctx->stage_grads[i]) cudaFree(ctx->stage_grads[i]);
        ctx->stage_grads[i] = nullptr;
    }
    if (ctx->stage_x) cudaFree(ctx->stage_x);
    if (ctx->stage_agg) cudaFree(ctx->stage_agg);
    if (ctx->back_stream) cudaStreamDestroy(ctx->back_stream);
    if (ctx->window_done) cudaEventDestroy(ctx->window_done);
    ctx->back_stream = nullptr;
    ctx->window_done = nullptr;
    ctx->stage_x = nullptr;
    ctx->stage_agg = nullptr;
}

// Host side of NormPlan: slices of the chunk range of every segment for a given covered range.
cudaError_t build_norm_plan(const int64_t* offsets, int B, int64_t covered_end, NormPlan* plan, void** mem) {
    std::vector<int64_t> k0, k1;
    std::vector<int32_t> seg_slice(B + 1, 0);
    for (int l = 0; l < B; ++l) {
        seg_slice[l] = (int32_t)k0.size();
        const int64_t lo = offsets[l];
        const int64_t hi = offsets[l + 1] < covered_end ? offsets[l + 1] : covered_end;
        if (lo >= hi) continue;
        const int64_t first = (lo + kChunkCoords - 1) / kChunkCoords;
        int64_t last = hi / kChunkCoords;   // chunks first .. last-1 end at or before hi
        // the partial chunk that ends the covered range is interior if it starts inside the segment
        if (hi == covered_end && (covered_end % kChunkCoords) != 0 && last * kChunkCoords >= lo) last += 1;
        for (int64_t k = first; k < last; k += kSliceChunks) {
            k0.push_back(k);
            k1.push_back(k + kSliceChunks < last ? k + kSliceChunks : last);
        }
    }
    seg_slice[B] = (int32_t)k0.size();
    const size_t ns = k0.size();
    const size_t bytes = (2 * ns) * sizeof(int64_t) + ns * sizeof(double) + (size_t)(B + 1) * sizeof(int32_t);
    char* base = nullptr;
    cudaError_t e = cudaMalloc((void**)&base, bytes);
    if (e != cudaSuccess) return e;
    int64_t* d_k0 = reinterpret_cast<int64_t*>(base);
    int64_t* d_k1 = d_k0 + ns;
    double* d_sum = reinterpret_cast<double*>(d_k1 + ns);
    int32_t* d_seg = reinterpret_cast<int32_t*>(d_sum + ns);
    if (ns) e = cudaMemcpy(d_k0, k0.data(), ns * sizeof(int64_t), cudaMemcpyHostToDevice);
    if (e == cudaSuccess && ns) e = cudaMemcpy(d_k1, k1.data(), ns * sizeof(int64_t), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(d_seg, seg_slice.data(), (size_t)(B + 1) * sizeof(int32_t), cudaMemcpyHostToDevice);
    if (e != cudaSuccess) { cudaFree(base); return e; }
    plan->k0 = d_k0;
    plan->k1 = d_k1;
    plan->seg_slice = d_seg;
    plan->slice_sum = d_sum;
    plan->covered_end = covered_end;
    plan->num_slices = (int32_t)ns;
    *mem = base;
    return cudaSuccess;
}

void free_blocks(intsgd_ctx* ctx) {
    for (int i = 0; i < 2; ++i) {
        if (ctx->d_plan_mem[i]) cudaFree(ctx->d_plan_mem[i]);
        ctx->d_plan_mem[i] = nullptr;
        std::memset(&ctx->plan[i], 0, sizeof ctx->plan[i]);
        ctx->plan[i].covered_end = -1;
    }
    if (ctx->d_offsets) cudaFree(ctx->d_offsets);
    if (ctx->bs.r) cudaFree(ctx->bs.r);            // one allocation holds every per-segment array
    if (ctx->bs.chunk_sum) cudaFree(ctx->bs.chunk_sum);
    ctx->d_offsets = nullptr;
    std::memset(&ctx->bs, 0, sizeof ctx->bs);
}

int block_mode_unsupported(intsgd_ctx* ctx, const char* what) {
    return fail(ctx, INTSGD_ERR_UNSUPPORTED, "%s is not available with block-wise scales (use intsgd_step, EXACT or FUSED)", what);
}

}  // namespace

// ======================================================================================
// C ABI
// ======================================================================================
extern "C" {

int intsgd_create(intsgd_ctx** out, const intsgd_config* cfg) {
    g_create_err[0] = 0;
    if (!out || !cfg) return fail(nullptr, INTSGD_ERR_INVALID_ARG, "intsgd_create: NULL argument");
    *out = nullptr;
    if (cfg->n < 1 || cfg->n > INTSGD_MAX_WORKERS) return fail(nullptr, INTSGD_ERR_INVALID_ARG, "n must be in 1..64");
    if (cfg->d < 1 || cfg->d > ((int64_t)1 << 40)) return fail(nullptr, INTSGD_ERR_INVALID_ARG, "d must be in 1..2^40");
    if (cfg->grad_dtype != INTSGD_GRAD_F32 && cfg->grad_dtype != INTSGD_GRAD_BF16)
        return fail(nullptr, INTSGD_ERR_INVALID_ARG, "bad grad_dtype");
    if (cfg->payload_dtype != INTSGD_PAYLOAD_I32 && cfg->payload_dtype != INTSGD_PAYLOAD_I8)
        return fail(nullptr, INTSGD_ERR_INVALID_ARG, "bad payload_dtype");
    if (cfg->rounding != INTSGD_ROUND_RANDOM && cfg->rounding != INTSGD_ROUND_NEAREST &&
        cfg->rounding != INTSGD_ROUND_RANDOM16 && cfg->rounding != INTSGD_ROUND_RANDOM_COMPARE)
        return fail(nullptr, INTSGD_ERR_INVALID_ARG, "bad rounding");
    if (!(cfg->beta >= 0.0 && cfg->beta < 1.0)) return fail(nullptr, INTSGD_ERR_INVALID_ARG, "beta must be in [0, 1)");
    if (!(cfg->eps >= 0.0) || !std::isfinite(cfg->eps)) return fail(nullptr, INTSGD_ERR_INVALID_ARG, "eps must be finite and >= 0");
    if (cfg->reserved != 0) return fail(nullptr, INTSGD_ERR_INVALID_ARG, "reserved must be 0");
    const int64_t int32_max = std::numeric_limits<int32_t>::max();
    int64_t L = cfg->clip_limit;
    if (L == 0) L = (cfg->payload_dtype == INTSGD_PAYLOAD_I8) ? 127 : int32_max / cfg->n;
    if (L < 1) return fail(nullptr, INTSGD_ERR_INVALID_ARG, "clip_limit must be positive (0 = default)");
    if (cfg->payload_dtype == INTSGD_PAYLOAD_I8 && L > 127) return fail(nullptr, INTSGD_ERR_INVALID_ARG, "int8 payload needs clip_limit <= 127");
    if (L > int32_max / cfg->n) return fail(nullptr, INTSGD_ERR_INVALID_ARG, "n * clip_limit must fit int32");

    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) {
        cudaGetLastError();
        return fail(nullptr, INTSGD_ERR_CUDA, "no CUDA device: this library has no CPU path");
    }
    if (cfg->device < 0 || cfg->device >= ndev) return fail(nullptr, INTSGD_ERR_INVALID_ARG, "device ordinal out of range");

    intsgd_ctx* ctx = new (std::nothrow) intsgd_ctx();
    if (!ctx) return fail(nullptr, INTSGD_ERR_CUDA, "out of host memory");
    std::memset(ctx, 0, sizeof *ctx);
    ctx->cfg = *cfg;
    ctx->L = L;
    ctx->Lf = largest_float_not_above(L);
    ctx->keys = make_keys(cfg->seed);
    ctx->tab = make_worker_table(ctx->keys);
    ctx->fused_path = 0;
    ctx->plan[0].covered_end = ctx->plan[1].covered_end = -1;
    ctx->threads = kDefaultThreads;
    ctx->blocks_per_sm = kDefaultBlocksPerSm;

    DeviceGuard guard(cfg->device);
    cudaError_t e = guard.status;
    cudaDeviceProp prop;
    if (e == cudaSuccess) e = cudaGetDeviceProperties(&prop, cfg->device);
    if (e == cudaSuccess) {
        ctx->sm_count = prop.multiProcessorCount;
        ctx->max_grid = ctx->sm_count * kMaxBlocksPerSm;
        e = cudaMalloc(&ctx->d_state, sizeof(DevState));
    }
    if (e == cudaSuccess) e = cudaMalloc(&ctx->d_partials, sizeof(double) * ctx->max_grid);
    if (e == cudaSuccess) e = cudaMemset(ctx->d_state, 0, sizeof(DevState));
    if (e == cudaSuccess) e = cudaMemset(ctx->d_partials, 0, sizeof(double) * ctx->max_grid);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        std::snprintf(g_create_err, 256, "intsgd_create: %s", cudaGetErrorString(e));
        if (ctx->d_state) cudaFree(ctx->d_state);
        if (ctx->d_partials) cudaFree(ctx->d_partials);
        delete ctx;
        return INTSGD_ERR_CUDA;
    }
    *out = ctx;
    return INTSGD_OK;
}

int intsgd_destroy(intsgd_ctx* ctx) {
    if (!ctx) return INTSGD_OK;
    DeviceGuard guard(ctx->cfg.device);
    free_staging(ctx);
    free_blocks(ctx);
    cudaFree(ctx->d_state);
    cudaFree(ctx->d_partials);
    delete ctx;
    return INTSGD_OK;
}

int intsgd_scale(intsgd_ctx* ctx, double eta_k, double dx2_override, void* stream) {
    if (!ctx) return INTSGD_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->cfg.device);
    ctx->last_stream = (cudaStream_t)stream;
    return launch_scale(ctx, eta_k, dx2_override, (cudaStream_t)stream);
}

int intsgd_sqdiff(intsgd_ctx* ctx, const float* x, const float* x_prev, void* stream) {
    if (!ctx) return INTSGD_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->cfg.device);
    bool al = true;
    int rc;
    if ((rc = check_vector(ctx, x, 4, "x", &al)) != INTSGD_OK) return rc;
    if ((rc = check_vector(ctx, x_prev, 4, "x_prev", &al)) != INTSGD_OK) return rc;
    VecParams P;
    base_params(ctx, P);
    P.x = const_cast<float*>(x);
    P.x_prev = x_prev;
    cudaStream_t s = (cudaStream_t)stream;
    ctx->last_stream = s;
    const int grid = grid_for(ctx, (ctx->cfg.d + 3) / 4);
    if (ctx->bs.B > 0) {   // one squared difference per block (Algorithm 2's moving averages are per block)
        const int64_t covered = (ctx->cfg.d >> 2) << 2;
        fill_block_params(ctx, P, covered);
        CUDA_TRY(ctx, cudaMemsetAsync(ctx->bs.edge_sum, 0, sizeof(double) * ctx->bs.B, s));
        if (al) sqdiff_blocks_kernel<true><<<grid, ctx->threads, 0, s>>>(P);
        else sqdiff_blocks_kernel<false><<<grid, ctx->threads, 0, s>>>(P);
        if ((rc = after_launch(ctx, "sqdiff_blocks_kernel")) != INTSGD_OK) return rc;
        return launch_block_norm(ctx, covered, false, false, s);
    }
    if (al) sqdiff_kernel<true><<<grid, ctx->threads, 0, s>>>(P);
    else sqdiff_kernel<false><<<grid, ctx->threads, 0, s>>>(P);
    return after_launch(ctx, "sqdiff_kernel");
}

int intsgd_encode(intsgd_ctx* ctx, int32_t worker, const void* grad, void* payload, float alpha_override,
                  void* stream) {
    if (!ctx) return INTSGD_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->cfg.device);
    if (ctx->bs.B > 0 && alpha_override == alpha_override)
        return fail(ctx, INTSGD_ERR_UNSUPPORTED, "alpha_override is not available with block-wise scales (pass NaN)");
    if (worker < 0 || worker >= ctx->cfg.n) return fail(ctx, INTSGD_ERR_INVALID_ARG, "worker index out of range");
    if (std::isinf(alpha_override) || alpha_override <= 0.0f)
        return fail(ctx, INTSGD_ERR_INVALID_ARG, "alpha_override must be NaN (use state) or finite and > 0");
    bool al = true;
    int rc;
    if ((rc = check_vector(ctx, grad, grad_elem_size(ctx->cfg.grad_dtype), "grad", &al)) != INTSGD_OK) return rc;
    if ((rc = check_vector(ctx, payload, payload_elem_size(ctx->cfg.payload_dtype), "payload", &al)) != INTSGD_OK) return rc;
    VecParams P;
    base_params(ctx, P);
    P.in[0] = grad;
    P.out[0] = payload;
    P.worker_base = worker;
    P.alpha_override = alpha_override;
    ctx->last_stream = (cudaStream_t)stream;
    return launch_encode(ctx, P, 1, al, (cudaStream_t)stream);
}

int intsgd_aggregate(intsgd_ctx* ctx, const void* const* payloads, float* x, int32_t* agg, void* stream) {
    if (!ctx) return INTSGD_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->cfg.device);
    if (!payloads) return fail(ctx, INTSGD_ERR_INVALID_ARG, "payloads is NULL");
    bool al = true;
    int rc;
    VecParams P;
    base_params(ctx, P);
    for (int i = 0; i < ctx->cfg.n; ++i) {
        if ((rc = check_vector(ctx, payloads[i], payload_elem_size(ctx->cfg.payload_dtype), "payloads[i]", &al)) != INTSGD_OK) return rc;
        P.in[i] = payloads[i];
    }
    if ((rc = check_vector(ctx, x, 4, "x", &al)) != INTSGD_OK) return rc;
    if (agg && (rc = check_vector(ctx, agg, 4, "agg", &al)) != INTSGD_OK) return rc;
    P.x = x;
    P.agg = agg;
    ctx->last_stream = (cudaStream_t)stream;
    return launch_aggregate(ctx, P, al, (cudaStream_t)stream);
}

int intsgd_step(intsgd_ctx* ctx, const void* const* grads, void* const* payload_scratch, float* x, int32_t* agg,
                double eta_k, int32_t mode, void* stream) {
    if (!ctx) return INTSGD_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->cfg.device);
    if (mode != INTSGD_MODE_EXACT && mode != INTSGD_MODE_TWO_KERNEL && mode != INTSGD_MODE_FUSED)
        return fail(ctx, INTSGD_ERR_INVALID_ARG, "bad mode");
    if (!grads) return fail(ctx, INTSGD_ERR_INVALID_ARG, "grads is NULL");
    if (mode == INTSGD_MODE_TWO_KERNEL && !payload_scratch)
        return fail(ctx, INTSGD_ERR_INVALID_ARG, "TWO_KERNEL mode needs payload_scratch");
    if (!(eta_k > 0.0) || !std::isfinite(eta_k)) return fail(ctx, INTSGD_ERR_INVALID_ARG, "eta_k must be finite and > 0");
    cudaStream_t s = (cudaStream_t)stream;
    bool al = true;
    int rc;
    VecParams P;
    base_params(ctx, P);
    for (int i = 0; i < ctx->cfg.n; ++i) {
        if ((rc = check_vector(ctx, grads[i], grad_elem_size(ctx->cfg.grad_dtype), "grads[i]", &al)) != INTSGD_OK) return rc;
        P.in[i] = grads[i];
    }
    if ((rc = check_vector(ctx, x, 4, "x", &al)) != INTSGD_OK) return rc;
    if (agg && (rc = check_vector(ctx, agg, 4, "agg", &al)) != INTSGD_OK) return rc;
    P.x = x;
    P.agg = agg;
    ctx->last_stream = s;

    if (mode == INTSGD_MODE_EXACT) {
        P.c_exact = (float)(eta_k / (double)ctx->cfg.n);
        P.agg = nullptr;
        return launch_exact(ctx, P, al, s);
    }
    if (mode == INTSGD_MODE_FUSED) {
        if ((rc = launch_scale(ctx, eta_k, -1.0, s)) != INTSGD_OK) return rc;
        ctx->follows_scale = true;
        rc = launch_fused(ctx, P, al, s);
        ctx->follows_scale = false;
        return rc;
    }
    // TWO_KERNEL: the payload buffers' alignment decides the encode stores and aggregate loads.
    bool al_enc = al, al_agg = true;
    if (!aligned_to(x, 16) || (agg && !aligned_to(agg, 16))) al_agg = false;
    for (int i = 0; i < ctx->cfg.n; ++i) {
        if ((rc = check_vector(ctx, payload_scratch[i], payload_elem_size(ctx->cfg.payload_dtype), "payload_scratch[i]", &al_enc)) != INTSGD_OK) return rc;
        if (!aligned_to(payload_scratch[i], 16)) al_agg = false;
        P.out[i] = payload_scratch[i];
    }
    if ((rc = launch_scale(ctx, eta_k, -1.0, s)) != INTSGD_OK) return rc;
    P.worker_base = 0;
    ctx->follows_scale = true;
    rc = launch_encode(ctx, P, ctx->cfg.n, al_enc, s);
    ctx->follows_scale = false;
    if (rc != INTSGD_OK) return rc;
    VecParams A;
    base_params(ctx, A);
    for (int i = 0; i < ctx->cfg.n; ++i) A.in[i] = payload_scratch[i];
    A.x = x;
    A.agg = agg;
    return launch_aggregate(ctx, A, al_agg, s);
}

int intsgd_diana_step(intsgd_ctx* ctx, const void* const* grads, float* const* h_local, float* h_global, float* x,
                      int32_t* agg, double eta_k, void* stream) {
    if (!ctx) return INTSGD_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->cfg.device);
    if (ctx->bs.B > 0) return block_mode_unsupported(ctx, "intsgd_diana_step");
    if (!grads || !h_local) return fail(ctx, INTSGD_ERR_INVALID_ARG, "grads / h_local is NULL");
    if (!(eta_k > 0.0) || !std::isfinite(eta_k)) return fail(ctx, INTSGD_ERR_INVALID_ARG, "eta_k must be finite and > 0");
    cudaStream_t s = (cudaStream_t)stream;
    bool al = true;
    int rc;
    VecParams P;
    base_params(ctx, P);
    for (int i = 0; i < ctx->cfg.n; ++i) {
        if ((rc = check_vector(ctx, grads[i], grad_elem_size(ctx->cfg.grad_dtype), "grads[i]", &al)) != INTSGD_OK) return rc;
        if ((rc = check_vector(ctx, h_local[i], 4, "h_local[i]", &al)) != INTSGD_OK) return rc;
        P.in[i] = grads[i];
        P.out[i] = h_local[i];
    }
    if ((rc = check_vector(ctx, h_global, 4, "h_global", &al)) != INTSGD_OK) return rc;
    if ((rc = check_vector(ctx, x, 4, "x", &al)) != INTSGD_OK) return rc;
    if (agg && (rc = check_vector(ctx, agg, 4, "agg", &al)) != INTSGD_OK) return rc;
    P.h = h_global;
    P.x = x;
    P.agg = agg;
    ctx->last_stream = s;
    if ((rc = launch_scale(ctx, eta_k, -1.0, s)) != INTSGD_OK) return rc;
    ctx->follows_scale = true;
    rc = launch_diana(ctx, P, al, s);
    ctx->follows_scale = false;
    return rc;
}

int intsgd_heuristic_step(intsgd_ctx* ctx, const void* const* grads, float* x, int32_t* agg, double eta_k,
                          int32_t num_bits, void* stream) {
    if (!ctx) return INTSGD_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->cfg.device);
    if (ctx->bs.B > 0) return block_mode_unsupported(ctx, "intsgd_heuristic_step");
    if (!grads) return fail(ctx, INTSGD_ERR_INVALID_ARG, "grads is NULL");
    if (num_bits < 2 || num_bits > 32) return fail(ctx, INTSGD_ERR_INVALID_ARG, "num_bits must be in 2..32");
    if (!(eta_k > 0.0) || !std::isfinite(eta_k)) return fail(ctx, INTSGD_ERR_INVALID_ARG, "eta_k must be finite and > 0");
    cudaStream_t s = (cudaStream_t)stream;
    bool al = true;
    int rc;
    VecParams P;
    base_params(ctx, P);
    for (int i = 0; i < ctx->cfg.n; ++i) {
        if ((rc = check_vector(ctx, grads[i], grad_elem_size(ctx->cfg.grad_dtype), "grads[i]", &al)) != INTSGD_OK) return rc;
        P.in[i] = grads[i];
    }
    if ((rc = check_vector(ctx, x, 4, "x", &al)) != INTSGD_OK) return rc;
    if (agg && (rc = check_vector(ctx, agg, 4, "agg", &al)) != INTSGD_OK) return rc;
    P.x = x;
    P.agg = agg;
    ctx->last_stream = s;
    // profiling pass over every worker's gradient
    const int n = ctx->cfg.n;
    dim3 grid((unsigned)grid_for(ctx, (ctx->cfg.d + 3) / 4), (unsigned)n, 1);
    int per = (ctx->sm_count * ctx->blocks_per_sm + n - 1) / n;
    if (per < 1) per = 1;
    if ((int)grid.x > per) grid.x = (unsigned)per;
    const bool bf16 = ctx->cfg.grad_dtype == INTSGD_GRAD_BF16;
    if (!bf16 && al) maxabs_kernel<INTSGD_GRAD_F32, true><<<grid, ctx->threads, 0, s>>>(P);
    else if (!bf16) maxabs_kernel<INTSGD_GRAD_F32, false><<<grid, ctx->threads, 0, s>>>(P);
    else if (al) maxabs_kernel<INTSGD_GRAD_BF16, true><<<grid, ctx->threads, 0, s>>>(P);
    else maxabs_kernel<INTSGD_GRAD_BF16, false><<<grid, ctx->threads, 0, s>>>(P);
    if ((rc = after_launch(ctx, "maxabs_kernel")) != INTSGD_OK) return rc;
    heuristic_scale_kernel<<<1, 32, 0, s>>>(ctx->d_state, (double)n, eta_k, std::ldexp(1.0, num_bits) - 1.0, n);
    if ((rc = after_launch(ctx, "heuristic_scale_kernel")) != INTSGD_OK) return rc;
    // The pipelined kernel sums integer-valued floats and is exact only below 2^24 / n per value; this
    // rule fills num_bits on purpose, so wide settings run the direct kernel (int32 accumulation).
    const double top = (std::ldexp(1.0, num_bits) - 1.0) / (double)n;
    const int saved_path = ctx->fused_path;
    if (top > (double)((1 << 24) / n - 2)) ctx->fused_path = 1;
    rc = launch_fused(ctx, P, al, s);
    ctx->fused_path = saved_path;
    return rc;
}

// Host-buffer step over windows of the vector: window w is copied in, stepped and copied back while
// window w + 1 is on its way in (the two directions of the link run at the same time).  The windows of
// one step share the scale, the step index and the counters; the random stream is addressed by the
// coordinate's index in the whole vector, so the integers and the iterate are those of a single launch,
// and the squared step length is the sum of the windows' sums.
constexpr int64_t kHostWindow = (int64_t)1 << 22;   // coordinates; a multiple of 4096 (whole tiles and draw pairs)

static int step_host_windowed(intsgd_ctx* ctx, const void* const* host_grads, float* host_x, int32_t* host_agg,
                              double eta_k, int32_t mode, cudaStream_t s) {
    if (!(eta_k > 0.0) || !std::isfinite(eta_k)) return fail(ctx, INTSGD_ERR_INVALID_ARG, "eta_k must be finite and > 0");
    if (mode != INTSGD_MODE_EXACT && mode != INTSGD_MODE_FUSED) return fail(ctx, INTSGD_ERR_INVALID_ARG, "bad mode");
    if (!ctx->back_stream) {
        CUDA_TRY(ctx, cudaStreamCreateWithFlags(&ctx->back_stream, cudaStreamNonBlocking));
        CUDA_TRY(ctx, cudaEventCreateWithFlags(&ctx->window_done, cudaEventDisableTiming));
    }
    const int n = ctx->cfg.n;
    const int64_t d = ctx->cfg.d;
    const size_t gsz = grad_elem_size(ctx->cfg.grad_dtype);
    const bool want_agg = host_agg && mode != INTSGD_MODE_EXACT;
    ctx->last_stream = s;
    int rc;
    if (mode == INTSGD_MODE_FUSED && (rc = launch_scale(ctx, eta_k, -1.0, s)) != INTSGD_OK) return rc;
    for (int64_t off = 0; off < d; off += kHostWindow) {
        const int64_t len = (d - off < kHostWindow) ? d - off : kHostWindow;
        VecParams P;
        base_params(ctx, P);
        P.d = len;
        P.unit_base = off >> 2;
        P.window_flags = (off > 0 ? kWindowAccumulate : 0) | (off + len < d ? kWindowHoldStep : 0);
        for (int i = 0; i < n; ++i) {
            char* dst = (char*)ctx->stage_grads[i] + (size_t)off * gsz;
            CUDA_TRY(ctx, cudaMemcpyAsync(dst, (const char*)host_grads[i] + (size_t)off * gsz, (size_t)len * gsz,
                                          cudaMemcpyHostToDevice, s));
            P.in[i] = dst;
        }
        CUDA_TRY(ctx, cudaMemcpyAsync(ctx->stage_x + off, host_x + off, (size_t)len * sizeof(float), cudaMemcpyHostToDevice, s));
        P.x = ctx->stage_x + off;
        P.agg = want_agg ? ctx->stage_agg + off : nullptr;
        if (mode == INTSGD_MODE_EXACT) {
            P.c_exact = (float)(eta_k / (double)n);
            rc = launch_exact(ctx, P, true, s);
        } else {
            rc = launch_fused(ctx, P, true, s);
        }
        if (rc != INTSGD_OK) return rc;
        CUDA_TRY(ctx, cudaEventRecord(ctx->window_done, s));
        CUDA_TRY(ctx, cudaStreamWaitEvent(ctx->back_stream, ctx->window_done, 0));
        CUDA_TRY(ctx, cudaMemcpyAsync(host_x + off, ctx->stage_x + off, (size_t)len * sizeof(float), cudaMemcpyDeviceToHost,
                                      ctx->back_stream));
        if (want_agg)
            CUDA_TRY(ctx, cudaMemcpyAsync(host_agg + off, ctx->stage_agg + off, (size_t)len * sizeof(int32_t),
                                          cudaMemcpyDeviceToHost, ctx->back_stream));
    }
    return INTSGD_OK;
}

int intsgd_step_host(intsgd_ctx* ctx, const void* const* host_grads, float* host_x, int32_t* host_agg,
                     double eta_k, int32_t mode, void* stream) {
    if (!ctx) return INTSGD_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->cfg.device);
    if (!host_grads || !host_x) return fail(ctx, INTSGD_ERR_INVALID_ARG, "host_grads / host_x is NULL");
    if (mode == INTSGD_MODE_TWO_KERNEL) return fail(ctx, INTSGD_ERR_UNSUPPORTED, "step_host runs EXACT or FUSED");
    const int n = ctx->cfg.n;
    const size_t d = (size_t)ctx->cfg.d;
    const size_t gbytes = d * grad_elem_size(ctx->cfg.grad_dtype);
    for (int i = 0; i < n; ++i)
        if (!host_grads[i]) return fail(ctx, INTSGD_ERR_INVALID_ARG, "host_grads[i] is NULL");
    if (!ctx->stage_agg) {
        // staging is all or nothing: a failed allocation releases what the attempt had obtained
        cudaError_t e = cudaSuccess;
        for (int i = 0; i < n && e == cudaSuccess; ++i)
            if (!ctx->stage_grads[i]) e = cudaMalloc(&ctx->stage_grads[i], gbytes);
        if (e == cudaSuccess && !ctx->stage_x) e = cudaMalloc((void**)&ctx->stage_x, d * sizeof(float));
        if (e == cudaSuccess) e = cudaMalloc((void**)&ctx->stage_agg, d * sizeof(int32_t));
        if (e != cudaSuccess) {
            free_staging(ctx);
            return fail(ctx, INTSGD_ERR_CUDA, "intsgd_step_host: staging allocation failed: %s", cudaGetErrorString(e));
        }
    }
    cudaStream_t s = (cudaStream_t)stream;
    if (d > (size_t)kHostWindow) {
        const int rc = step_host_windowed(ctx, host_grads, host_x, host_agg, eta_k, mode, s);
        if (rc != INTSGD_OK) return rc;
        CUDA_TRY(ctx, cudaStreamSynchronize(ctx->back_stream));
        CUDA_TRY(ctx, cudaStreamSynchronize(s));
        return INTSGD_OK;
    }
    for (int i = 0; i < n; ++i)
        CUDA_TRY(ctx, cudaMemcpyAsync(ctx->stage_grads[i], host_grads[i], gbytes, cudaMemcpyHostToDevice, s));
    CUDA_TRY(ctx, cudaMemcpyAsync(ctx->stage_x, host_x, d * sizeof(float), cudaMemcpyHostToDevice, s));
    const int rc = intsgd_step(ctx, (const void* const*)ctx->stage_grads, nullptr, ctx->stage_x,
                               host_agg ? ctx->stage_agg : nullptr, eta_k, mode, stream);
    if (rc != INTSGD_OK) return rc;
    CUDA_TRY(ctx, cudaMemcpyAsync(host_x, ctx->stage_x, d * sizeof(float), cudaMemcpyDeviceToHost, s));
    if (host_agg && mode != INTSGD_MODE_EXACT)
        CUDA_TRY(ctx, cudaMemcpyAsync(host_agg, ctx->stage_agg, d * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
    CUDA_TRY(ctx, cudaStreamSynchronize(s));
    return INTSGD_OK;
}

int intsgd_get_stats(intsgd_ctx* ctx, intsgd_stats* out) {
    if (!ctx || !out) return INTSGD_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->cfg.device);
    DevState h;
    const int rc = read_state_block(ctx, &h);
    if (rc != INTSGD_OK) return rc;
    std::memset(out, 0, sizeof *out);
    out->state.r = h.r;
    out->state.dx2 = h.dx2;
    out->state.alpha = h.alpha;
    out->state.c = h.c;
    out->state.step = h.step;
    out->state.status = h.status;
    for (int i = 0; i < INTSGD_MAX_WORKERS; ++i) out->clip_count[i] = h.clip_count[i];
    out->nonfinite = h.nonfinite;
    out->agg_overflow = h.agg_overflow;
    out->max_abs_agg = h.max_abs_agg;
    if (h.fault)
        return fail(ctx, INTSGD_ERR_TIMEOUT, "a bounded wait inside a kernel gave up; the results of that step are invalid");
    if (h.status == INTSGD_ERR_SCALE_NONFINITE)
        return fail(ctx, INTSGD_ERR_SCALE_NONFINITE, "alpha_k is not finite and positive (r = 0 with eps = 0?); step not applied");
    return INTSGD_OK;
}

int intsgd_selftest_wait_expiry(intsgd_ctx* ctx, void* stream) {
    if (!ctx) return INTSGD_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->cfg.device);
    cudaStream_t s = (cudaStream_t)stream;
    ctx->last_stream = s;
    wait_expiry_kernel<<<1, 32, 0, s>>>(ctx->d_state, 64u);
    return after_launch(ctx, "wait_expiry_kernel");
}

int intsgd_selftest_philox_rate(intsgd_ctx* ctx, int64_t blocks_per_thread, int32_t extra_ops_per_block,
                                int64_t* philox_blocks, void* stream) {
    if (!ctx) return INTSGD_ERR_INVALID_ARG;
    if (blocks_per_thread < 2 || blocks_per_thread > ((int64_t)1 << 24))
        return fail(ctx, INTSGD_ERR_INVALID_ARG, "blocks_per_thread must be in 2..2^24");
    if (extra_ops_per_block != 0 && extra_ops_per_block != 16 && extra_ops_per_block != 32)
        return fail(ctx, INTSGD_ERR_INVALID_ARG, "extra_ops_per_block must be 0, 16 or 32");
    DeviceGuard guard(ctx->cfg.device);
    cudaStream_t s = (cudaStream_t)stream;
    ctx->last_stream = s;
    const uint32_t per_chain = (uint32_t)(blocks_per_thread / 2);
    // the sink is the state block's spare word; the kernel's store condition never holds in practice
    uint32_t* sink = &ctx->d_state->pad2;
    if (extra_ops_per_block == 0) philox_rate_kernel<0><<<ctx->sm_count, 512, 0, s>>>(ctx->keys, per_chain, 1e-3f, sink);
    else if (extra_ops_per_block == 16) philox_rate_kernel<16><<<ctx->sm_count, 512, 0, s>>>(ctx->keys, per_chain, 1e-3f, sink);
    else philox_rate_kernel<32><<<ctx->sm_count, 512, 0, s>>>(ctx->keys, per_chain, 1e-3f, sink);
    if (philox_blocks) *philox_blocks = (int64_t)ctx->sm_count * 512 * 2 * per_chain;
    return after_launch(ctx, "philox_rate_kernel");
}

int intsgd_get_state(intsgd_ctx* ctx, intsgd_state* out) {
    if (!ctx || !out) return INTSGD_ERR_INVALID_ARG;
    intsgd_stats s;
    const int rc = intsgd_get_stats(ctx, &s);
    // the state block has been read whenever get_stats got as far as its own status checks
    if (rc == INTSGD_OK || rc == INTSGD_ERR_SCALE_NONFINITE || rc == INTSGD_ERR_TIMEOUT) *out = s.state;
    return rc;
}

int intsgd_set_state(intsgd_ctx* ctx, const intsgd_state* in) {
    if (!ctx || !in) return INTSGD_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->cfg.device);
    DevState h;
    int rc = read_state_block(ctx, &h);
    if (rc != INTSGD_OK) return rc;
    h.r = in->r;
    h.dx2 = in->dx2;
    h.alpha = in->alpha;
    h.c = in->c;
    h.step = in->step;
    h.status = in->status;
    h.ticket = 0;
    h.fault = 0;
    CUDA_TRY(ctx, cudaMemcpy(ctx->d_state, &h, sizeof h, cudaMemcpyHostToDevice));
    return INTSGD_OK;
}

int intsgd_set_blocks(intsgd_ctx* ctx, int32_t num_blocks, const int64_t* offsets) {
    if (!ctx) return INTSGD_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->cfg.device);
    CUDA_TRY(ctx, cudaStreamSynchronize(ctx->last_stream));
    if (num_blocks == 0) {
        free_blocks(ctx);
        return INTSGD_OK;
    }
    if (num_blocks < 0 || num_blocks > INTSGD_MAX_BLOCKS || !offsets)
        return fail(ctx, INTSGD_ERR_INVALID_ARG, "num_blocks must be in 0..INTSGD_MAX_BLOCKS with offsets given");
    if (offsets[0] != 0 || offsets[num_blocks] != ctx->cfg.d)
        return fail(ctx, INTSGD_ERR_INVALID_ARG, "offsets must start at 0 and end at d");
    for (int l = 0; l < num_blocks; ++l)
        if (offsets[l + 1] <= offsets[l]) return fail(ctx, INTSGD_ERR_INVALID_ARG, "offsets must be strictly increasing");
    free_blocks(ctx);
    const size_t B = (size_t)num_blocks;
    const size_t chunks = (size_t)((ctx->cfg.d + kChunkCoords - 1) / kChunkCoords);
    // per-segment arrays in one allocation: r, r_new, dx2, edge_sum (double), tail_sq (8 doubles), alpha, c (float)
    const size_t bytes = (4 * B + kMaxTail) * sizeof(double) + 2 * B * sizeof(float);
    void* base = nullptr;
    CUDA_TRY(ctx, cudaMalloc(&ctx->d_offsets, (B + 1) * sizeof(int64_t)));
    cudaError_t e = cudaMalloc(&base, bytes);
    double* chunk = nullptr;
    // chunk partials (double) followed by the chunk -> segment table (int32)
    if (e == cudaSuccess) e = cudaMalloc((void**)&chunk, chunks * (sizeof(double) + sizeof(int32_t)));
    if (e == cudaSuccess) e = cudaMemset(base, 0, bytes);
    if (e == cudaSuccess) e = cudaMemset(chunk, 0, chunks * sizeof(double));
    if (e == cudaSuccess) e = cudaMemcpy(ctx->d_offsets, offsets, (B + 1) * sizeof(int64_t), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) {
        chunk_table_kernel<<<(unsigned)((chunks + 255) / 256), 256>>>(ctx->d_offsets, num_blocks, ctx->cfg.d,
                                                                      reinterpret_cast<int32_t*>(chunk + chunks), (int64_t)chunks);
        e = cudaGetLastError();
        if (e == cudaSuccess) e = cudaDeviceSynchronize();
    }
    // covered ranges: whole units of 4 (direct kernels, fp32 pipelined) and pairs of units (bf16 pipelined)
    const int64_t cov0 = (ctx->cfg.d >> 2) << 2, cov1 = (ctx->cfg.d >> 3) << 3;
    if (e == cudaSuccess) e = build_norm_plan(offsets, num_blocks, cov0, &ctx->plan[0], &ctx->d_plan_mem[0]);
    if (e == cudaSuccess && cov1 != cov0) e = build_norm_plan(offsets, num_blocks, cov1, &ctx->plan[1], &ctx->d_plan_mem[1]);
    if (e != cudaSuccess) {
        for (int i = 0; i < 2; ++i) {
            if (ctx->d_plan_mem[i]) cudaFree(ctx->d_plan_mem[i]);
            ctx->d_plan_mem[i] = nullptr;
            ctx->plan[i].covered_end = -1;
        }
        if (base) cudaFree(base);
        if (chunk) cudaFree(chunk);
        cudaFree(ctx->d_offsets);
        ctx->d_offsets = nullptr;
        return fail(ctx, INTSGD_ERR_CUDA, "intsgd_set_blocks: %s", cudaGetErrorString(e));
    }
    double* dbl = static_cast<double*>(base);
    ctx->bs.offsets = ctx->d_offsets;
    ctx->bs.r = dbl;
    ctx->bs.r_new = dbl + B;
    ctx->bs.dx2 = dbl + 2 * B;
    ctx->bs.edge_sum = dbl + 3 * B;
    ctx->bs.tail_sq = dbl + 4 * B;
    ctx->bs.alpha = reinterpret_cast<float*>(dbl + 4 * B + kMaxTail);
    ctx->bs.c = ctx->bs.alpha + B;
    ctx->bs.chunk_sum = chunk;
    ctx->bs.chunk_seg = reinterpret_cast<int32_t*>(chunk + chunks);
    ctx->bs.B = num_blocks;
    return INTSGD_OK;
}

int intsgd_get_block_state(intsgd_ctx* ctx, double* r, double* dx2, float* alpha, float* c) {
    if (!ctx) return INTSGD_ERR_INVALID_ARG;
    if (ctx->bs.B == 0) return fail(ctx, INTSGD_ERR_INVALID_ARG, "no block partition is set");
    DeviceGuard guard(ctx->cfg.device);
    CUDA_TRY(ctx, cudaStreamSynchronize(ctx->last_stream));
    const size_t B = (size_t)ctx->bs.B;
    if (r) CUDA_TRY(ctx, cudaMemcpy(r, ctx->bs.r, B * sizeof(double), cudaMemcpyDeviceToHost));
    if (dx2) CUDA_TRY(ctx, cudaMemcpy(dx2, ctx->bs.dx2, B * sizeof(double), cudaMemcpyDeviceToHost));
    if (alpha) CUDA_TRY(ctx, cudaMemcpy(alpha, ctx->bs.alpha, B * sizeof(float), cudaMemcpyDeviceToHost));
    if (c) CUDA_TRY(ctx, cudaMemcpy(c, ctx->bs.c, B * sizeof(float), cudaMemcpyDeviceToHost));
    return INTSGD_OK;
}

int intsgd_set_block_state(intsgd_ctx* ctx, const double* r, const double* dx2) {
    if (!ctx) return INTSGD_ERR_INVALID_ARG;
    if (ctx->bs.B == 0) return fail(ctx, INTSGD_ERR_INVALID_ARG, "no block partition is set");
    DeviceGuard guard(ctx->cfg.device);
    CUDA_TRY(ctx, cudaStreamSynchronize(ctx->last_stream));
    const size_t B = (size_t)ctx->bs.B;
    if (r) CUDA_TRY(ctx, cudaMemcpy(ctx->bs.r, r, B * sizeof(double), cudaMemcpyHostToDevice));
    if (dx2) CUDA_TRY(ctx, cudaMemcpy(ctx->bs.dx2, dx2, B * sizeof(double), cudaMemcpyHostToDevice));
    return INTSGD_OK;
}

int intsgd_set_launch(intsgd_ctx* ctx, int32_t threads_per_block, int32_t blocks_per_sm) {
    if (!ctx) return INTSGD_ERR_INVALID_ARG;
    if (threads_per_block != 0) {
        if (threads_per_block < 32 || threads_per_block > kMaxThreads || (threads_per_block % 32) != 0)
            return fail(ctx, INTSGD_ERR_INVALID_ARG, "threads_per_block must be a multiple of 32 in 32..512");
        ctx->threads = threads_per_block;
    }
    if (blocks_per_sm != 0) {
        if (blocks_per_sm < 1 || blocks_per_sm > kMaxBlocksPerSm)
            return fail(ctx, INTSGD_ERR_INVALID_ARG, "blocks_per_sm must be in 1..32");
        ctx->blocks_per_sm = blocks_per_sm;
    }
    return INTSGD_OK;
}

int intsgd_set_fused_path(intsgd_ctx* ctx, int32_t path) {
    if (!ctx) return INTSGD_ERR_INVALID_ARG;
    if (path < 0 || path > 2)
        return fail(ctx, INTSGD_ERR_INVALID_ARG, "path must be 0 (automatic), 1 (direct kernels) or 2 (same as 0)");
    ctx->fused_path = path;
    return INTSGD_OK;
}

int64_t intsgd_launch_count(const intsgd_ctx* ctx) { return ctx ? ctx->launches : 0; }

const char* intsgd_last_error(const intsgd_ctx* ctx) { return ctx ? ctx->err : g_create_err; }

}  // extern "C"
