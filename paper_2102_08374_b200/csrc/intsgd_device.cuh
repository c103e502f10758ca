// Device-side building blocks of the IntSGD step kernels (sm_100a).
//
// Work unit: 4 consecutive coordinates = one Philox4x32-10 block (coordinate j uses word j mod 4
// of block j / 4), one 16-byte fp32 load per worker.  Every kernel walks units grid-stride, so a
// warp touches 512 contiguous bytes of each stream per iteration.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "intsgd.h"

namespace intsgd {

typedef unsigned long long u64;
// Per-block event counters in shared memory: 32 bits are enough (a block cannot see 2^32 elements of
// one worker within the memory of one GPU) and 32-bit shared-memory atomics are native.
typedef uint32_t cnt_t;

// ----------------------------------------------------------------------------------------
// Device-resident state.  The first 32 bytes have the layout of intsgd_state.
// ----------------------------------------------------------------------------------------
struct DevState {
    double r;
    double dx2;
    float alpha;
    float c;
    uint32_t step;
    int32_t status;
    u64 clip_count[INTSGD_MAX_WORKERS];
    u64 nonfinite;
    u64 agg_overflow;
    int32_t max_abs_agg;
    uint32_t ticket;   // blocks that have published their partial in the running reduction
    int32_t fault;     // sticky: a bounded wait inside a kernel gave up (results of that step are invalid)
    float ainv;        // fp32(1 / alpha)        } factors of the IntDIANA step (Algorithm 3),
    float cn;          // fp32(1 / (n alpha))    } written by the scale kernel with alpha and c
    float eta32;       // fp32(eta)              }
    uint32_t maxabs_bits;   // heuristic scale: bits of max |g| found by the profiling pass (0 between steps)
    uint32_t pad2;
};

// Philox4x32-10 round keys (key schedule done once on the host: the key is the same for every
// thread, so the ten (k0, k1) pairs travel as kernel parameters and are read from the constant
// bank).
struct PhiloxKeys {
    uint32_t k0[10];
    uint32_t k1[10];
};

// Round-1/round-2 Philox values that depend only on (seed, worker) when the high counter word is
// zero (d <= 2^34): computed on the host once per context, copied to shared memory by each block.
// Entry i: x = lo(M1 * i) ^ k0[1];  y = hi(M0 * n0) ^ k1[1] with n0 = hi(M1 * i) ^ k0[0];  z = lo(M0 * n0).
struct PhiloxWorkerTable {
    uint4 e[INTSGD_MAX_WORKERS];
};

// Block-wise scales (Algorithm 2); B == 0 means one scalar alpha (Algorithm 1).  See intsgd_blocks.cuh.
struct BlockParams {
    const int64_t* offsets;   // device, B + 1 entries, offsets[0] = 0, offsets[B] = d
    const float* alpha;       // device, B
    const float* c;           // device, B
    double* chunk_sum;        // device, ceil(d / 128)
    const int32_t* chunk_seg; // device, ceil(d / 128): segment of the chunk's first coordinate; sign bit set
                              // when the chunk's 128 coordinates reach into a later segment
    double* edge_sum;         // device, B (cleared when the step opens)
    double* tail_sq;          // device, 8: squared steps of the coordinates after covered_end
    int64_t covered_end;      // coordinates below this are handled as whole units by the launch
    int32_t B;
};

constexpr int kWindowAccumulate = 1;   // state.dx2 += this launch's sum (not the first window of the step)
constexpr int kWindowHoldStep = 2;     // do not advance the step counter (not the last window of the step)

struct VecParams {
    const void* in[INTSGD_MAX_WORKERS];   // gradients (encode / fused / exact) or payloads (aggregate)
    void* out[INTSGD_MAX_WORKERS];        // payloads (encode)
    float* x;
    int32_t* agg;
    const float* x_prev;                  // sqdiff only
    float* h;                             // IntDIANA: global shift (out[i] holds the local shifts)
    DevState* st;
    double* partials;                     // one slot per block of the grid
    int64_t d;
    int32_t n;
    int32_t worker_base;                  // encode: worker index of blockIdx.y == 0
    float alpha_override;                 // encode: NaN = take alpha from the state
    float Lf;                             // clip limit as the largest fp32 <= L
    float c_exact;                        // exact step: fp32(eta / n)
    int32_t agg_limit;                    // coordinates with |S| above this count as agg_overflow
    // A launch may cover a window of the vector (pointers and d describe the window): unit_base is the
    // index of its first unit in the whole vector (random stream), and the flags chain the windows of
    // one step: every window but the first adds its norm partial to the state, every window but the
    // last leaves the step counter alone.
    int64_t unit_base;
    int32_t window_flags;
    PhiloxKeys keys;
    PhiloxWorkerTable tab;
    BlockParams bp;
};

// ----------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11).  One round: the two 32x32->64 products of
// counter words 0 and 2 with the round multipliers; new counter =
// (hi(p1) ^ c1 ^ k0, lo(p1), hi(p0) ^ c3 ^ k1, lo(p0)).
// ----------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               const PhiloxKeys& K) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ K.k0[r];
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ K.k1[r];
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
    }
    return make_uint4(c0, c1, c2, c3);
}

// Philox4x32-10 for counter (unit, 0, worker, step) with rounds 1-2 folded:
// per tile and thread: p0 = M0 * unit -> n3 = lo, n2 = hi ^ step ^ k1[0]; p1' = M1 * n2 -> H, m1.
// per worker: m0 = H ^ e[i].x, m2 = e[i].y ^ n3, m3 = e[i].z; then rounds 3..10.
struct PhiloxThreadPart {
    uint32_t n3, H, m1;
};
__device__ __forceinline__ PhiloxThreadPart philox_thread_part(uint32_t unit_lo, uint32_t step, const PhiloxKeys& K) {
    const uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)unit_lo;
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ step ^ K.k1[0];
    const uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)n2;
    PhiloxThreadPart t;
    t.n3 = (uint32_t)p0;
    t.H = (uint32_t)(p1 >> 32);
    t.m1 = (uint32_t)p1;
    return t;
}
__device__ __forceinline__ uint4 philox_finish(const PhiloxThreadPart& t, uint4 e, const PhiloxKeys& K) {
    uint32_t c0 = t.H ^ e.x, c1 = t.m1, c2 = e.y ^ t.n3, c3 = e.z;
#pragma unroll
    for (int r = 2; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ K.k0[r];
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ K.k1[r];
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
    }
    return make_uint4(c0, c1, c2, c3);
}

// Random draws of unit `unit` (coordinates 4*unit .. 4*unit+3) of `worker` at `step`, one per
// coordinate.  Default stream: the four words of Philox block `unit`.  INTSGD_ROUND_RANDOM16: 16-bit draws; unit u shares the block of pair index
// P = ((u >> 10) << 9) | (u & 511) with the unit 512 places away, takes words 2h and 2h + 1
// (h = bit 9 of u), and coordinate e gets the low (e even) or high (e odd) half of word 2h + e / 2.
template <int ROUND>
__device__ __forceinline__ uint4 draw_unit(int64_t unit, uint32_t worker, uint32_t step, const PhiloxKeys& K) {
    if (ROUND == INTSGD_ROUND_RANDOM16) {
        const uint64_t u = (uint64_t)unit;
        const uint64_t pair = ((u >> 10) << 9) | (u & 511);
        const uint4 w = philox4x32_10((uint32_t)pair, (uint32_t)(pair >> 32), worker, step, K);
        const bool h = (u >> 9) & 1;
        const uint32_t a = h ? w.z : w.x, b = h ? w.w : w.y;
        return make_uint4(a & 0xFFFFu, a >> 16, b & 0xFFFFu, b >> 16);
    }
    return philox4x32_10((uint32_t)unit, (uint32_t)((uint64_t)unit >> 32), worker, step, K);
}

// The same draws with rounds 1-2 folded, for a kernel that keeps a unit across several workers (or a worker
// across several units): draw_thread_part is the unit's half (2 wide multiplies), `e` the worker's half
// (PhiloxWorkerTable entry), draw_unit_folded the remaining rounds (16 wide multiplies).  The folding needs a
// zero high counter word; beyond 2^32 blocks the full ten rounds run.
template <int ROUND>
__device__ __forceinline__ uint64_t draw_block_index(int64_t unit) {
    const uint64_t u = (uint64_t)unit;
    return (ROUND == INTSGD_ROUND_RANDOM16) ? (((u >> 10) << 9) | (u & 511)) : u;
}
template <int ROUND>
__device__ __forceinline__ PhiloxThreadPart draw_thread_part(int64_t unit, uint32_t step, const PhiloxKeys& K) {
    return philox_thread_part((uint32_t)draw_block_index<ROUND>(unit), step, K);
}
template <int ROUND>
__device__ __forceinline__ uint4 draw_unit_folded(const PhiloxThreadPart& tp, int64_t unit, uint4 e, uint32_t worker,
                                                  uint32_t step, const PhiloxKeys& K) {
    const uint64_t idx = draw_block_index<ROUND>(unit);
    const uint4 w = (idx >> 32) ? philox4x32_10((uint32_t)idx, (uint32_t)(idx >> 32), worker, step, K) : philox_finish(tp, e, K);
    if (ROUND == INTSGD_ROUND_RANDOM16) {
        const bool h = ((uint64_t)unit >> 9) & 1;
        const uint32_t a = h ? w.z : w.x, b = h ? w.w : w.y;
        return make_uint4(a & 0xFFFFu, a >> 16, b & 0xFFFFu, b >> 16);
    }
    return w;
}

// The uniform draw is draw_as_float(w) * draw_scale(): the word times 2^-32 truncated to fp32 (the
// conversion rounds toward zero, so u <= 1 - 2^-24), the 16-bit value times 2^-16, or (compare form)
// the word's top 24 bits times 2^-24.
template <int ROUND>
__device__ __forceinline__ float draw_as_float(uint32_t w) {
    if (ROUND == INTSGD_ROUND_RANDOM16) return __uint2float_rn(w);
    if (ROUND == INTSGD_ROUND_RANDOM_COMPARE) return __uint2float_rn(w >> 8);
    return __uint2float_rz(w);
}
template <int ROUND>
__device__ __forceinline__ float draw_scale() {
    if (ROUND == INTSGD_ROUND_RANDOM16) return 1.52587890625e-05f;
    if (ROUND == INTSGD_ROUND_RANDOM_COMPARE) return 5.9604644775390625e-08f;
    return 2.3283064365386963e-10f;
}

// 1.0f if a < b else 0.0f, in one instruction.
__device__ __forceinline__ float lt_as_float(float a, float b) {
    float d;
    asm("set.lt.f32.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
    return d;
}

// ----------------------------------------------------------------------------------------
// Loads and stores.  ALIGNED: every vector pointer of the launch is 16-byte aligned.
// Gradients and payloads are read once (streaming, evict-first); x is read and rewritten.
// ----------------------------------------------------------------------------------------
__device__ __forceinline__ float bf16_widen(uint32_t h16) { return __uint_as_float(h16 << 16); }

template <int GRAD>
__device__ __forceinline__ float grad_at(const void* base, int64_t j) {
    if (GRAD == INTSGD_GRAD_BF16) return bf16_widen(((const uint16_t*)base)[j]);
    return ((const float*)base)[j];
}

template <int GRAD, bool ALIGNED>
__device__ __forceinline__ float4 load_grad4(const void* base, int64_t unit) {
    if (GRAD == INTSGD_GRAD_F32) {
        if (ALIGNED) return __ldcs((const float4*)base + unit);
        const float* p = (const float*)base + 4 * unit;
        return make_float4(__ldcs(p), __ldcs(p + 1), __ldcs(p + 2), __ldcs(p + 3));
    } else {
        if (ALIGNED) {
            const uint2 v = __ldcs((const uint2*)base + unit);
            return make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xFFFF0000u),
                               __uint_as_float(v.y << 16), __uint_as_float(v.y & 0xFFFF0000u));
        }
        const uint16_t* p = (const uint16_t*)base + 4 * unit;
        return make_float4(bf16_widen(__ldcs(p)), bf16_widen(__ldcs(p + 1)), bf16_widen(__ldcs(p + 2)),
                           bf16_widen(__ldcs(p + 3)));
    }
}

template <bool ALIGNED>
__device__ __forceinline__ float4 load_f4(const float* base, int64_t unit) {
    if (ALIGNED) return *((const float4*)base + unit);
    const float* p = base + 4 * unit;
    return make_float4(p[0], p[1], p[2], p[3]);
}
template <bool ALIGNED>
__device__ __forceinline__ void store_f4(float* base, int64_t unit, float4 v) {
    if (ALIGNED) { *((float4*)base + unit) = v; return; }
    float* p = base + 4 * unit;
    p[0] = v.x; p[1] = v.y; p[2] = v.z; p[3] = v.w;
}
template <bool ALIGNED>
__device__ __forceinline__ void store_i4(int32_t* base, int64_t unit, int4 v) {
    if (ALIGNED) { __stcs((int4*)base + unit, v); return; }
    int32_t* p = base + 4 * unit;
    __stcs(p, v.x); __stcs(p + 1, v.y); __stcs(p + 2, v.z); __stcs(p + 3, v.w);
}
template <bool ALIGNED>
__device__ __forceinline__ int4 load_i4(const int32_t* base, int64_t unit) {
    if (ALIGNED) return __ldcs((const int4*)base + unit);
    const int32_t* p = base + 4 * unit;
    return make_int4(__ldcs(p), __ldcs(p + 1), __ldcs(p + 2), __ldcs(p + 3));
}

// Four payload values of one unit: int32 as one 16-byte store, int8 as the four low bytes packed into one word.
template <int PAY>
__device__ __forceinline__ void store_payload4(void* base, int64_t unit, int4 q, bool aligned) {
    if (PAY == INTSGD_PAYLOAD_I32) {
        if (aligned) { __stcs((int4*)base + unit, q); return; }
        int32_t* p = (int32_t*)base + 4 * unit;
        __stcs(p, q.x); __stcs(p + 1, q.y); __stcs(p + 2, q.z); __stcs(p + 3, q.w);
    } else {
        if (aligned) {
            // low bytes of the four values, in order
            const uint32_t packed = __byte_perm(__byte_perm(q.x, q.y, 0x0040), __byte_perm(q.z, q.w, 0x0040), 0x5410);
            __stcs((uint32_t*)base + unit, packed);
            return;
        }
        int8_t* p = (int8_t*)base + 4 * unit;
        p[0] = (int8_t)q.x; p[1] = (int8_t)q.y; p[2] = (int8_t)q.z; p[3] = (int8_t)q.w;
    }
}

// Adds the four signed bytes of one packed int8 unit to the four sums.
__device__ __forceinline__ void add_bytes(int4& s, uint32_t v) {
    s.x += (int)(int8_t)(v & 0xFF);
    s.y += (int)(int8_t)((v >> 8) & 0xFF);
    s.z += (int)(int8_t)((v >> 16) & 0xFF);
    s.w += (int)(int8_t)(v >> 24);
}

// max(|a|, |b|, |c|), NaN if any input is NaN (three-input max of sm_100).
__device__ __forceinline__ float absmax3_nan(float a, float b, float c) {
    float d;
    asm("max.NaN.abs.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// ----------------------------------------------------------------------------------------
// Rounding.  y = fl32(alpha * g).  Random: q = floor(y + u) on the unrounded sum (Int(t), Section 2
// of the paper: up with probability t - floor(t)).  One fused multiply-add rounded toward minus
// infinity forms RD(y + u): the product draw * scale is exact, and rounding the sum down never crosses
// an integer (every integer of the range is an fp32 value, or y is itself an integer and u < 1), so
// floor(RD(y + u)) = floor(y + u).
// ----------------------------------------------------------------------------------------
template <int ROUND>
__device__ __forceinline__ int round_in_range(float y, uint32_t w) {
    if (ROUND == INTSGD_ROUND_NEAREST) return __float2int_rn(y);
    if (ROUND == INTSGD_ROUND_RANDOM_COMPARE) {
        // compare form: f = floor(y), p = fl32(y - f), up iff u < p; done as (float)(w >> 8) < p * 2^24 (exact scalings)
        const float f = floorf(y);
        const float p = __fsub_rn(y, f);
        return __float2int_rz(f) + (draw_as_float<ROUND>(w) < __fmul_rn(p, 16777216.0f) ? 1 : 0);
    }
    return __float2int_rd(__fmaf_rd(draw_as_float<ROUND>(w), draw_scale<ROUND>(), y));
}

// Full rule with clipping: values outside [-Lf, Lf] saturate, NaN becomes 0, and the event is
// counted (Section 5.1: local values are clipped so that the aggregate fits the wire type).
template <int ROUND>
__device__ __forceinline__ int round_full(float y, uint32_t w, float Lf, uint32_t& clipped, uint32_t& nonfinite) {
    if (fabsf(y) <= Lf) return round_in_range<ROUND>(y, w);
    clipped += 1;
    if (!(fabsf(y) <= 3.402823466e+38f)) nonfinite += 1;   // NaN or +-Inf
    if (y > Lf) return (int)Lf;
    if (y < -Lf) return -(int)Lf;
    return 0;   // NaN
}

template <int ROUND>
__device__ __noinline__ int round_checked(float y, uint32_t w, float Lf, cnt_t* clip_slot, cnt_t* nonfinite_slot) {
    uint32_t clipped = 0, nonfinite = 0;
    const int q = round_full<ROUND>(y, w, Lf, clipped, nonfinite);
    if (clipped) atomicAdd(clip_slot, clipped);
    if (nonfinite) atomicAdd(nonfinite_slot, nonfinite);
    return q;
}

// Four values of one worker with the full rule; the counters get one atomic per unit at most.
template <int ROUND>
__device__ __noinline__ int4 round_unit_checked(float y0, float y1, float y2, float y3, uint4 w, float Lf,
                                                cnt_t* clip_slot, cnt_t* nonfinite_slot) {
    uint32_t clipped = 0, nonfinite = 0;
    int4 q;
    q.x = round_full<ROUND>(y0, w.x, Lf, clipped, nonfinite);
    q.y = round_full<ROUND>(y1, w.y, Lf, clipped, nonfinite);
    q.z = round_full<ROUND>(y2, w.z, Lf, clipped, nonfinite);
    q.w = round_full<ROUND>(y3, w.w, Lf, clipped, nonfinite);
    if (clipped) atomicAdd(clip_slot, clipped);
    if (nonfinite) atomicAdd(nonfinite_slot, nonfinite);
    return q;
}

// Four in-range values at once with packed fp32x2 arithmetic; bit-identical to round_in_range on each.
template <int ROUND>
__device__ __forceinline__ int4 round4_in_range(float2 y01, float2 y23, uint4 w) {
    if (ROUND == INTSGD_ROUND_NEAREST)
        return make_int4(__float2int_rn(y01.x), __float2int_rn(y01.y), __float2int_rn(y23.x), __float2int_rn(y23.y));
    if (ROUND == INTSGD_ROUND_RANDOM_COMPARE)
        return make_int4(round_in_range<ROUND>(y01.x, w.x), round_in_range<ROUND>(y01.y, w.y),
                         round_in_range<ROUND>(y23.x, w.z), round_in_range<ROUND>(y23.y, w.w));
    const float2 scale = make_float2(draw_scale<ROUND>(), draw_scale<ROUND>());
    const float2 z01 = __ffma2_rd(make_float2(draw_as_float<ROUND>(w.x), draw_as_float<ROUND>(w.y)), scale, y01);
    const float2 z23 = __ffma2_rd(make_float2(draw_as_float<ROUND>(w.z), draw_as_float<ROUND>(w.w)), scale, y23);
    return make_int4(__float2int_rd(z01.x), __float2int_rd(z01.y), __float2int_rd(z23.x), __float2int_rd(z23.y));
}

// One unit of one worker: scale, round, clip.  The common case (all four values in range) has no
// clamp and no counter traffic.
template <int ROUND>
__device__ __forceinline__ int4 round_unit(float4 g, float alpha, uint4 w, float Lf, cnt_t* clip_slot,
                                           cnt_t* nonfinite_slot) {
    const float2 alpha2 = make_float2(alpha, alpha);
    const float2 y01 = __fmul2_rn(alpha2, make_float2(g.x, g.y));
    const float2 y23 = __fmul2_rn(alpha2, make_float2(g.z, g.w));
    const float m = absmax3_nan(absmax3_nan(y01.x, y01.y, y23.x), y23.y, y23.y);
    if (m <= Lf) return round4_in_range<ROUND>(y01, y23, w);   // false for NaN
    return round_unit_checked<ROUND>(y01.x, y01.y, y23.x, y23.y, w, Lf, clip_slot, nonfinite_slot);
}

// Decode + update of one coordinate: t = fl32(c * float(S)); x_new = fl32(x - t); the squared
// fp32 step length goes to an fp64 accumulator (Algorithm 1: estimator, update, and the argument
// of the next moving average).
__device__ __forceinline__ float update_coord(float x_old, int S, float c, double& acc) {
    const float t = __fmul_rn(c, __int2float_rn(S));
    const float x_new = __fsub_rn(x_old, t);
    const float dj = __fsub_rn(x_new, x_old);
    acc = __fma_rn((double)dj, (double)dj, acc);   // exact product, one rounding: same as mul then add
    return x_new;
}

struct ThreadAcc {
    double dx2;
    int32_t max_abs;
    uint32_t overflow;
};

__device__ __forceinline__ void note_sum(int S, int32_t agg_limit, ThreadAcc& a) {
    const int m = abs(S);
    a.max_abs = max(a.max_abs, m);
    a.overflow += (m > agg_limit) ? 1u : 0u;
}

// ----------------------------------------------------------------------------------------
// Grid-wide reduction of the per-thread accumulators with a fixed shape: warp shuffle tree,
// per-warp slots in shared memory, one fp64 partial per block in global memory; the block that
// takes the last ticket adds the partials (strided, then the same tree) and writes state.dx2.
// The result depends only on the launch shape, never on scheduling.
// ----------------------------------------------------------------------------------------
__device__ __forceinline__ double warp_tree(double v) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_down_sync(0xFFFFFFFFu, v, off);
    return v;
}

__device__ __forceinline__ double block_tree(double v, double* s_warp) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
    v = warp_tree(v);
    if (lane == 0) s_warp[warp] = v;
    __syncthreads();
    double t = 0.0;
    if (warp == 0) {
        t = (lane < nwarps) ? s_warp[lane] : 0.0;
        t = warp_tree(t);
    }
    __syncthreads();
    return t;   // valid in thread 0
}

// max |S| and the int8 overflow count of the whole grid (order-independent integer atomics).
__device__ __forceinline__ void flush_sum_counters(const ThreadAcc& a, DevState* st) {
    const int mx = __reduce_max_sync(0xFFFFFFFFu, a.max_abs);
    const unsigned ov = __reduce_add_sync(0xFFFFFFFFu, a.overflow);
    if ((threadIdx.x & 31) == 0) {
        if (mx > 0) atomicMax(&st->max_abs_agg, mx);
        if (ov) atomicAdd(&st->agg_overflow, (u64)ov);
    }
}

__device__ __forceinline__ void grid_finalize(const ThreadAcc& a, DevState* st, double* partials,
                                              bool advance_step, int window_flags = 0) {
    __shared__ double s_warp[32];
    __shared__ bool s_last;
    flush_sum_counters(a, st);
    const double block_sum = block_tree(a.dx2, s_warp);
    if (threadIdx.x == 0) {
        __stcg(&partials[blockIdx.x], block_sum);
        __threadfence();
        const unsigned t = atomicAdd(&st->ticket, 1u);
        s_last = (t == gridDim.x - 1);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    double v = 0.0;
    for (unsigned b = threadIdx.x; b < gridDim.x; b += blockDim.x) v += __ldcg(&partials[b]);
    const double total = block_tree(v, s_warp);
    if (threadIdx.x == 0) {
        st->dx2 = (window_flags & kWindowAccumulate) ? st->dx2 + total : total;
        if (advance_step && !(window_flags & kWindowHoldStep)) st->step += 1;
        st->ticket = 0;
    }
}

// Per-block clip / non-finite counters live in shared memory (slot i < n: worker i's clipped
// count, slot INTSGD_MAX_WORKERS: non-finite count) and are flushed once per block.
__device__ __forceinline__ void counters_init(cnt_t* s_cnt) {
    for (int t = threadIdx.x; t <= INTSGD_MAX_WORKERS; t += blockDim.x) s_cnt[t] = 0;
    __syncthreads();
}
__device__ __forceinline__ void counters_flush(const cnt_t* s_cnt, DevState* st) {
    __syncthreads();
    for (int t = threadIdx.x; t <= INTSGD_MAX_WORKERS; t += blockDim.x) {
        const u64 v = s_cnt[t];
        if (v) atomicAdd(t < INTSGD_MAX_WORKERS ? &st->clip_count[t] : &st->nonfinite, v);
    }
}

}  // namespace intsgd
