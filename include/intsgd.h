/*
 * intsgd.h -- C ABI of the IntSGD step library for NVIDIA B200 (sm_100a).
 *
 * One IntSGD iteration (Mishchenko, Wang, Kovalev, Richtarik, "IntSGD: Adaptive Floatless
 * Compression of Stochastic Gradients", Algorithm 1) for n simulated workers whose gradient
 * vectors of length d sit in the memory of ONE GPU:
 *
 *     r_k     = beta r_{k-1} + (1 - beta) ||x^k - x^{k-1}||^2          (Algorithm 1, moving average)
 *     alpha_k = sqrt(d) / sqrt(2 n r_k / eta_k^2 + eps^2)              (Proposition 2)
 *     q_i     = Int(alpha_k g_i)   Int(t) = floor(t) + Bernoulli(t - floor(t))   (Section 2)
 *     S       = sum_i q_i          exact integer sum                   (Algorithm 1, aggregate)
 *     x^{k+1} = x^k - eta_k S / (n alpha_k)                            (Algorithm 1, estimator + update)
 *
 * Conventions
 *  - Every vector pointer is a DEVICE pointer owned by the caller unless the name says "host".
 *    The library never frees or keeps them.  Pointers must be aligned to their element size;
 *    16-byte aligned pointers take the vector path, others a slower element-wise path.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  All vector work is
 *    enqueued on it and returns without synchronising; only create / destroy / get_stats /
 *    get_state / set_state / step_host synchronise.
 *  - Every call returns an int status: 0 = INTSGD_OK, negative = error.  Nothing throws or
 *    aborts.  intsgd_last_error() gives a message for the last failing call on that context.
 *  - Clipping and integer overflow are not errors: they are counted (intsgd_stats).
 *  - A context is not thread-safe; distinct contexts are independent.  Calls on one context
 *    must be issued on one stream (or be ordered by the caller).
 *  - The random stream is counter-based: Philox4x32-10 (Salmon et al., SC'11) with
 *    key = (seed low, seed high), counter = (b low, b high, worker, step), b = j / 4, and
 *    coordinate j uses output word j mod 4.  u = word * 2^-32 truncated to fp32 (its 24 leading
 *    significant bits; u <= 1 - 2^-24); Int(y) = floor(y + u) evaluated on the unrounded sum, with
 *    y = fl32(alpha * g): up with probability y - floor(y).  Results do not depend on the launch shape.
 *  - fp32 arithmetic of the scale, decode and update steps is unfused (separately rounded multiply
 *    and subtract).
 */
#ifndef INTSGD_H_
#define INTSGD_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define INTSGD_MAX_WORKERS 64
#define INTSGD_MAX_BLOCKS  4096

/* status codes */
#define INTSGD_OK                    0
#define INTSGD_ERR_INVALID_ARG      -1   /* null pointer, n or d out of range, eta <= 0, bad enum */
#define INTSGD_ERR_ALIGN            -2   /* pointer not aligned to its element size */
#define INTSGD_ERR_CUDA             -3   /* a CUDA runtime call failed; see intsgd_last_error */
#define INTSGD_ERR_SCALE_NONFINITE  -4   /* alpha_k or c_k not finite or not positive; step not applied */
#define INTSGD_ERR_UNSUPPORTED      -5   /* valid request that is not implemented */
#define INTSGD_ERR_TIMEOUT          -6   /* a bounded wait inside a kernel gave up; that step's results are
                                            invalid; sticky until intsgd_set_state */
#define INTSGD_ERR_TOO_LARGE        -7   /* intsgd_sqdiff_noalloc: d exceeds INTSGD_NOALLOC_MAX_D */

/* enums (plain ints in the structs) */
#define INTSGD_GRAD_F32      0
#define INTSGD_GRAD_BF16     1
#define INTSGD_PAYLOAD_I32   0
#define INTSGD_PAYLOAD_I8    1
#define INTSGD_ROUND_RANDOM  0   /* Int(t) of Section 2 */
#define INTSGD_ROUND_NEAREST 1   /* "IntSGD (Determ.)" of Section 5.1: nearest, ties to even */
#define INTSGD_ROUND_RANDOM16 2  /* Int(t) with 16-bit draws: one Philox block serves 8 coordinates.
                                    Unit u = j / 4 shares the block of pair index
                                    P = ((u >> 10) << 9) | (u & 511) (counter (P low, P high, worker, step))
                                    with unit u ^ 512, takes words 2h and 2h + 1 (h = bit 9 of u); coordinate
                                    e = j mod 4 uses the low (e even) or high (e odd) 16 bits v of word
                                    2h + e / 2; Int(y) = floor(y + v * 2^-16).  Bias at most
                                    2^-16 per value.  Halves the random-number work: an option, not the default */
#define INTSGD_ROUND_RANDOM_COMPARE 3  /* Int(t) drawn by comparison: u = (word >> 8) * 2^-24 (24 bits), up iff
                                          u < fl32(y - floor(y)).  Same law and same Philox words as
                                          INTSGD_ROUND_RANDOM, different draws; three more instructions per value */
#define INTSGD_MODE_EXACT      0 /* Algorithm 1, Init line: x <- x - eta (1/n) sum_i g_i, uncompressed */
#define INTSGD_MODE_TWO_KERNEL 1 /* encode every worker to a payload buffer, then aggregate */
#define INTSGD_MODE_FUSED      2 /* one pass, payloads never reach memory */

typedef struct intsgd_ctx intsgd_ctx;   /* opaque; owns only a small device state block and
                                           a few KiB of reduction scratch */

typedef struct intsgd_config {
    int32_t  n;              /* workers, 1 .. INTSGD_MAX_WORKERS */
    int32_t  grad_dtype;     /* INTSGD_GRAD_* */
    int64_t  d;              /* coordinates, 1 .. 2^40 */
    int32_t  payload_dtype;  /* INTSGD_PAYLOAD_*: the wire type; the aggregate is always int32 */
    int32_t  rounding;       /* INTSGD_ROUND_* */
    double   beta;           /* moving-average factor in [0, 1); paper default 0.9 */
    double   eps;            /* safeguard >= 0 (enters as eps^2); paper default 1e-8 */
    uint64_t seed;           /* Philox key */
    int64_t  clip_limit;     /* symmetric limit L on each payload value; 0 = default:
                                int8 wire -> 127; int32 wire -> floor((2^31 - 1) / n), so that the
                                aggregate of n payloads fits the wire type (Section 5.1).
                                Must satisfy n * L <= 2^31 - 1. */
    int32_t  device;         /* CUDA device ordinal */
    int32_t  reserved;       /* must be 0 */
} intsgd_config;

/* The resumable scalar state.  With x it is everything needed to continue bit-exactly. */
typedef struct intsgd_state {
    double   r;       /* moving average r_k after the last intsgd_scale */
    double   dx2;     /* ||x^{k+1} - x^k||^2 left by the last step (or intsgd_sqdiff) */
    float    alpha;   /* alpha_k used by the last / next encode */
    float    c;       /* eta_k / (n alpha_k), the decode factor */
    uint32_t step;    /* 0-based index of the NEXT step (the Philox counter word) */
    int32_t  status;  /* INTSGD_OK or INTSGD_ERR_SCALE_NONFINITE from the last intsgd_scale */
} intsgd_state;

/* Counters describe the work enqueued since the last intsgd_scale (one step). */
typedef struct intsgd_stats {
    intsgd_state state;
    uint64_t clip_count[INTSGD_MAX_WORKERS]; /* per worker: coordinates with !(|alpha g| <= L) */
    uint64_t nonfinite;      /* coordinates (all workers) whose alpha * g is NaN or +-Inf */
    uint64_t agg_overflow;   /* int8 wire only: coordinates whose sum is outside [-127, 127] */
    int32_t  max_abs_agg;    /* max_j |S_j| ("max integer in the aggregated vector", Appendix C.5) */
    int32_t  reserved;
} intsgd_stats;

/* Lifetime.  create selects cfg->device, allocates the state block (r = 0, dx2 = 0, step = 0)
 * and validates cfg.  destroy frees it; the caller must have synchronised its streams. */
int intsgd_create(intsgd_ctx** out, const intsgd_config* cfg);
int intsgd_destroy(intsgd_ctx* ctx);

/* Algorithm 1, moving-average and scale lines (Proposition 2).  Enqueues a one-thread kernel:
 * r <- beta r + (1 - beta) dx2;  alpha <- fp32(sqrt(d) / sqrt(2 n r / eta^2 + eps^2));
 * c <- fp32(eta / (n alpha)), all in fp64 with separately rounded operations.
 * dx2_override < 0: use the dx2 left in the state by the previous step; >= 0: use this value.
 * Also clears the per-step counters.  eta_k must be finite and > 0 (else INVALID_ARG).
 * If alpha or c is not finite and positive (r = 0 with eps = 0), the state keeps its old r, status
 * becomes INTSGD_ERR_SCALE_NONFINITE, and the vector kernels of this step do nothing; the
 * condition is reported by intsgd_get_stats / intsgd_get_state (this call is asynchronous). */
int intsgd_scale(intsgd_ctx* ctx, double eta_k, double dx2_override, void* stream);

/* Helper for a caller that holds two iterates: state.dx2 <- ||x - x_prev||^2
 * (fp32 differences, fp64 sum; Algorithm 1, argument of the moving average). */
int intsgd_sqdiff(intsgd_ctx* ctx, const float* x, const float* x_prev, void* stream);

/* Algorithm 1, "scale and round the local gradient", for one worker:
 * payload[j] = clip(Int(alpha g[j])), j in [0, d).  grad: d values of cfg.grad_dtype;
 * payload: d values of cfg.payload_dtype.  alpha_override = NaN: use the state's alpha;
 * otherwise use this value.  Adds to clip_count[worker] and nonfinite. */
int intsgd_encode(intsgd_ctx* ctx, int32_t worker, const void* grad, void* payload,
                  float alpha_override, void* stream);

/* Algorithm 1, aggregate + estimator + update in one pass over memory:
 * S_j = sum_i payloads[i][j];  x_j <- x_j - c S_j;  agg[j] = S_j (agg may be NULL);
 * state.dx2 <- ||x_new - x_old||^2;  state.step += 1.
 * payloads: HOST array of n device pointers (read during the call only). */
int intsgd_aggregate(intsgd_ctx* ctx, const void* const* payloads, float* x, int32_t* agg,
                     void* stream);

/* One whole step k: scale (unless mode is EXACT), then
 *   EXACT      : x <- x - eta (1/n) sum_i g_i in fp32, workers added in order 0..n-1
 *                (Algorithm 1, Init line); r is left unchanged; no payloads, no counters.
 *   TWO_KERNEL : encode all workers into payload_scratch[i] (n device buffers of d payload
 *                values, caller-owned), then aggregate.
 *   FUSED      : encode, sum, decode and update in one kernel; payload_scratch ignored.
 * grads, payload_scratch: HOST arrays of n device pointers.  agg may be NULL.
 * Leaves state.dx2 = ||x^{k+1} - x^k||^2 and advances state.step. */
int intsgd_step(intsgd_ctx* ctx, const void* const* grads, void* const* payload_scratch,
                float* x, int32_t* agg, double eta_k, int32_t mode, void* stream);

/* One IntDIANA step (Algorithm 3: IntSGD on gradient differences, for heterogeneous data):
 *     q_i  = clip(Int(alpha_k (g_i - h_i)))          h_i <- h_i + (1/alpha_k) q_i
 *     g~   = h + (1/(n alpha_k)) sum_i q_i           h <- g~         x <- x - eta_k g~
 * (the shift update uses Q(g_i) = (1/alpha) Int(alpha (g_i - h_i)), as the proof of the IntDIANA
 * theorem defines it).  alpha_k comes from the context's scale rule; Algorithm 3 prints its
 * beta = 0, eps = 0 case.  fp32 steps, each rounded once: v = g - h_i; y = alpha v;
 * h_i += fp32(1/alpha) * float(q); t = fp32(1/(n alpha)) * float(S); g~ = h + t; x -= fp32(eta) * g~.
 * h_local: HOST array of n device pointers to float[d] (read and written); h_global: device float[d]
 * (read and written); both start at zero after the exact first step (intsgd_step, MODE_EXACT).
 * Same counters, dx2 and step bookkeeping as intsgd_step.  Not available with a block partition. */
int intsgd_diana_step(intsgd_ctx* ctx, const void* const* grads, float* const* h_local, float* h_global, float* x,
                      int32_t* agg, double eta_k, void* stream);

/* One step of Heuristic IntSGD (Section 5.2 of the paper: the SwitchML scale the paper compares with,
 * built to show what its profiling pass costs).  A first pass over all n gradients finds max |g|
 * (NaN ignored); alpha = (2^num_bits - 1) / (n 2^max_exp), max_exp the smallest integer with
 * max |g| <= 2^max_exp, so that n |alpha g| <= 2^num_bits - 1; then the fused kernel of intsgd_step
 * runs with that alpha and c = eta_k / (n alpha).  The moving average r is left untouched; dx2,
 * counters and the step index are updated as usual.  If max |g| is zero or infinite the step is not
 * applied (INTSGD_ERR_SCALE_NONFINITE at intsgd_get_stats).  Values beyond the context's clip limit
 * still clip (num_bits = 32 exceeds the default int32 limit by a factor of two). */
int intsgd_heuristic_step(intsgd_ctx* ctx, const void* const* grads, float* x, int32_t* agg, double eta_k,
                          int32_t num_bits, void* stream);

/* The same step for a caller whose buffers are in HOST memory (pinned memory recommended):
 * copies the n gradients and x to device staging buffers owned by the context (allocated on
 * first use: n*d gradient values + d floats + d int32), runs intsgd_step, copies x (and agg if
 * not NULL) back, and synchronises the stream before returning. */
int intsgd_step_host(intsgd_ctx* ctx, const void* const* host_grads, float* host_x,
                     int32_t* host_agg, double eta_k, int32_t mode, void* stream);

/* Synchronise the context's last stream and read the state and counters.  Returns
 * INTSGD_ERR_SCALE_NONFINITE if the last intsgd_scale failed that way (out is still filled). */
int intsgd_get_stats(intsgd_ctx* ctx, intsgd_stats* out);
int intsgd_get_state(intsgd_ctx* ctx, intsgd_state* out);
/* Overwrite the scalar state (checkpoint resume; tests that impose alpha and c). */
int intsgd_set_state(intsgd_ctx* ctx, const intsgd_state* in);

/* Block-wise scales (Algorithm 2, "adaptive block quantization"; Proposition 4): the coordinates are
 * split into num_blocks contiguous blocks [offsets[l], offsets[l+1]) -- for instance one per layer --
 * and each block keeps its own moving average and scale:
 *     r_{k,l}     = beta r_{k-1,l} + (1 - beta) ||(x^k)_l - (x^{k-1})_l||^2
 *     alpha_{k,l} = eta_k sqrt(d_l) / sqrt(2 n r_{k,l} + eta_k^2 (d_l / d) eps^2)
 * offsets: HOST array of num_blocks + 1 values, offsets[0] = 0, strictly increasing, last = d.
 * num_blocks = 0 returns to the single scalar alpha of Algorithm 1.  The call synchronises,
 * allocates the per-block state (r = 0, dx2 = 0) and d/128 doubles of reduction scratch.
 * With a partition set, intsgd_step supports INTSGD_MODE_EXACT and INTSGD_MODE_FUSED (intsgd_scale
 * computes all block scales; dx2_override must be negative); intsgd_sqdiff / encode / aggregate and
 * INTSGD_MODE_TWO_KERNEL return INTSGD_ERR_UNSUPPORTED.  intsgd_state.dx2 is the sum over blocks,
 * .alpha and .c are those of block 0; counters are unchanged. */
int intsgd_set_blocks(intsgd_ctx* ctx, int32_t num_blocks, const int64_t* offsets);
/* Per-block state, HOST arrays of num_blocks values each (any may be NULL); both calls synchronise. */
int intsgd_get_block_state(intsgd_ctx* ctx, double* r, double* dx2, float* alpha, float* c);
int intsgd_set_block_state(intsgd_ctx* ctx, const double* r, const double* dx2);

/* Diagnostic of the failure path.  Every wait inside the pipelined kernels is bounded; when one gives up the
 * kernel sets a sticky flag, lets its copies in flight land and returns, and intsgd_get_stats reports
 * INTSGD_ERR_TIMEOUT until intsgd_set_state clears the flag.  This call enqueues a one-thread kernel that runs
 * the same bounded wait (64 polls) on a barrier that nothing ever completes, so that a caller can check, without
 * any fault on the GPU, that an expired wait surfaces as INTSGD_ERR_TIMEOUT and that the context stays usable.
 * It touches no vector and no other state. */
int intsgd_selftest_wait_expiry(intsgd_ctx* ctx, void* stream);

/* Diagnostic for roofline reports: how fast this GPU gets through the integer arithmetic of the random stream
 * when it does nothing else.  Enqueues one register-only kernel (one block of 512 threads per SM, no vector is
 * touched) in which every thread computes blocks_per_thread (2 .. 2^24, rounded down to even) blocks of rounds
 * 3-10 of Philox4x32-10 -- the per-worker part of a draw in the pipelined kernels, 16 32x32->64-bit products each --
 * as two dependent chains.  extra_ops_per_block (0, 16 or 32) adds that many independent fp32 additions per block:
 * the time they add tells whether other instructions hide behind the wide multiplies or queue up behind them (on
 * B200 they queue up: one issue cycle each).  *philox_blocks (may be NULL) receives the number of blocks the launch
 * computes; the caller times the launch on `stream`.  The step kernels' random rounding cannot run faster than the
 * rate measured with extra_ops_per_block = 0. */
int intsgd_selftest_philox_rate(intsgd_ctx* ctx, int64_t blocks_per_thread, int32_t extra_ops_per_block,
                                int64_t* philox_blocks, void* stream);

/* Number of kernels this library has launched on the context since creation. */
int64_t intsgd_launch_count(const intsgd_ctx* ctx);

/* ||x - x_prev||^2 for callers that must not allocate device memory (the paper has no counterpart:
 * this is an addition for hosts that cannot create a context, because intsgd_create calls cudaMalloc
 * -- e.g. a process whose framework owns all device memory and forbids raw allocations, a loop that
 * cannot afford the allocator's implicit synchronisation, or a plug-in that is handed only buffers and
 * a stream).  Needs no context and calls no cudaMalloc / cudaFree or allocating routine: the reduction
 * scratch is a fixed array inside the library image, 128 KiB + 8 bytes on every GPU that loads the
 * library, held until the process exits.
 *   x, x_prev : device, d floats each, 4-byte aligned (16-byte aligned pointers use vector loads)
 *   out       : device, one double, 8-byte aligned; receives sum_j fl32(x_j - x_prev_j)^2 in fp64
 *   d         : 1 .. INTSGD_NOALLOC_MAX_D; larger -> INTSGD_ERR_TOO_LARGE, nothing is enqueued
 * Works on the current device and enqueues on `stream` without synchronising.  The first call on
 * each device looks up the array's device address (cudaGetSymbolAddress) and keeps it for the life of the
 * process: it assumes that the device's primary context is not destroyed (cudaDeviceReset) while the
 * library is in use.  The entry point has two kernels (both pointers 16-byte aligned / otherwise), and the
 * CUDA runtime may load each on its first launch.  Make the first call on a device, and the first call of
 * each alignment kind that will be used, before any stream capture.  All calls on a device share the
 * array: it keeps the previous call's partial sums, its arrival counter is cleared on `stream` before
 * every launch, and two calls that overlap on the GPU race.  The summation order depends only on d and on
 * whether both x and x_prev are 16-byte aligned (the two kernels split a block's coordinates differently
 * over its threads), never on the GPU or on scheduling. */
#define INTSGD_NOALLOC_MAX_D ((int64_t)1 << 28)
int intsgd_sqdiff_noalloc(const float* x, const float* x_prev, int64_t d, double* out, void* stream);

/* Static, NUL-terminated description of the last failing call ("" if none); never NULL.
 * ctx may be NULL to read the message of a failed intsgd_create on this thread. */
const char* intsgd_last_error(const intsgd_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* INTSGD_H_ */
