// The IntSGD step kernels (sm_100a).  See intsgd_device.cuh for the unit/stream conventions.
#pragma once

#include "intsgd_device.cuh"

namespace intsgd {

constexpr int kMaxThreads = 512;

// ----------------------------------------------------------------------------------------
// Scale: Algorithm 1's moving average and Proposition 2's alpha_k, one thread, fp64 with
// separately rounded operations.  Also opens a new step: clears the per-step counters.
// ----------------------------------------------------------------------------------------
__global__ void scale_kernel(DevState* st, double sqrt_d, double two_n, double n_as_double, double eta,
                             double beta, double eps, double dx2_override, int32_t n) {
    // a dependent launch (the step's vector kernel) may begin its set-up now; it waits for this grid's
    // completion before it reads the state
    asm volatile("griddepcontrol.launch_dependents;");
    // this launch may itself have started before the kernel in front of it has finished: wait for its writes
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    const double dx2 = (dx2_override >= 0.0) ? dx2_override : st->dx2;
    const double a = __dmul_rn(beta, st->r);
    const double b = __dmul_rn(__dsub_rn(1.0, beta), dx2);
    const double r = __dadd_rn(a, b);
    const double two_n_r = __dmul_rn(two_n, r);
    const double inner = __dadd_rn(__ddiv_rn(two_n_r, __dmul_rn(eta, eta)), __dmul_rn(eps, eps));
    const double alpha64 = __ddiv_rn(sqrt_d, __dsqrt_rn(inner));
    const float alpha = __double2float_rn(alpha64);
    const float c = __double2float_rn(__ddiv_rn(eta, __dmul_rn(n_as_double, (double)alpha)));
    for (int i = 0; i < n; ++i) st->clip_count[i] = 0;
    st->nonfinite = 0;
    st->agg_overflow = 0;
    st->max_abs_agg = 0;
    st->ticket = 0;
    const bool ok = (alpha > 0.0f) && (alpha <= 3.402823466e+38f) && (c > 0.0f) && (c <= 3.402823466e+38f);
    if (!ok) {
        st->status = INTSGD_ERR_SCALE_NONFINITE;
        return;
    }
    st->r = r;
    st->alpha = alpha;
    st->c = c;
    st->ainv = __double2float_rn(__ddiv_rn(1.0, (double)alpha));
    st->cn = __double2float_rn(__ddiv_rn(1.0, __dmul_rn(n_as_double, (double)alpha)));
    st->eta32 = __double2float_rn(eta);
    st->status = INTSGD_OK;
}

// ----------------------------------------------------------------------------------------
// Encode: payload_i = clip(Int(alpha g_i)).  grid = (blocks, workers).
// ----------------------------------------------------------------------------------------
template <int GRAD, int PAY, bool ALIGNED, int ROUND>
__global__ void __launch_bounds__(kMaxThreads) encode_kernel(const __grid_constant__ VecParams P) {
    __shared__ cnt_t s_cnt[INTSGD_MAX_WORKERS + 1];
    DevState* st = P.st;
    if (st->status != INTSGD_OK) return;
    counters_init(s_cnt);
    const float alpha = (P.alpha_override == P.alpha_override) ? P.alpha_override : st->alpha;
    const uint32_t step = st->step;
    const int slot = blockIdx.y;
    const uint32_t worker = (uint32_t)(P.worker_base + slot);
    const void* g = P.in[slot];
    void* out = P.out[slot];
    cnt_t* clip_slot = &s_cnt[worker];
    cnt_t* nonf_slot = &s_cnt[INTSGD_MAX_WORKERS];
    const uint4 e = P.tab.e[worker];   // the worker's half of Philox rounds 1-2 (fixed for the whole block)

    const int64_t full = P.d >> 2;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    if (PAY == INTSGD_PAYLOAD_I32) {
        // 8 bytes per element: bound by memory, so keep the register count (and occupancy) of the plain loop
        for (int64_t unit = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; unit < full; unit += stride) {
            const float4 gv = load_grad4<GRAD, ALIGNED>(g, unit);
            uint4 w = make_uint4(0, 0, 0, 0);
            if (ROUND != INTSGD_ROUND_NEAREST)
                w = draw_unit_folded<ROUND>(draw_thread_part<ROUND>(unit, step, P.keys), unit, e, worker, step, P.keys);
            store_payload4<PAY>(out, unit, round_unit<ROUND>(gv, alpha, w, P.Lf, clip_slot, nonf_slot), ALIGNED);
        }
    } else if (ROUND == INTSGD_ROUND_RANDOM16) {
        // 16-bit draws: iterate over pair indices; the pair's two units (512 apart) share one Philox block.
        const int64_t pairs = ((full + 1023) >> 10) << 9;
        int64_t pr = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
        int64_t ua = ((pr >> 9) << 10) | (pr & 511);
        float4 ga = make_float4(0.f, 0.f, 0.f, 0.f), gb = ga;
        if (pr < pairs && ua < full) ga = load_grad4<GRAD, ALIGNED>(g, ua);
        if (pr < pairs && ua + 512 < full) gb = load_grad4<GRAD, ALIGNED>(g, ua + 512);
        for (; pr < pairs; pr += stride) {
            const int64_t np = pr + stride, nu = ((np >> 9) << 10) | (np & 511);
            const int64_t ca_unit = ua;
            const float4 ca = ga, cb = gb;
            if (np < pairs && nu < full) ga = load_grad4<GRAD, ALIGNED>(g, nu);
            if (np < pairs && nu + 512 < full) gb = load_grad4<GRAD, ALIGNED>(g, nu + 512);
            ua = nu;
            const uint4 w = ((uint64_t)pr >> 32) ? philox4x32_10((uint32_t)pr, (uint32_t)((uint64_t)pr >> 32), worker, step, P.keys)
                                                 : philox_finish(philox_thread_part((uint32_t)pr, step, P.keys), e, P.keys);
            const uint4 wa = make_uint4(w.x & 0xFFFFu, w.x >> 16, w.y & 0xFFFFu, w.y >> 16);
            const uint4 wb = make_uint4(w.z & 0xFFFFu, w.z >> 16, w.w & 0xFFFFu, w.w >> 16);
            if (ca_unit < full)
                store_payload4<PAY>(out, ca_unit, round_unit<ROUND>(ca, alpha, wa, P.Lf, clip_slot, nonf_slot), ALIGNED);
            if (ca_unit + 512 < full)
                store_payload4<PAY>(out, ca_unit + 512, round_unit<ROUND>(cb, alpha, wb, P.Lf, clip_slot, nonf_slot), ALIGNED);
        }
    } else {
        // 5 (3) bytes per element: bound by arithmetic.  Two units per iteration, and the next pair's
        // loads issued before this pair is rounded, so two Philox chains overlap and cover the latency.
        int64_t unit = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
        float4 ga = make_float4(0.f, 0.f, 0.f, 0.f), gb = ga;
        if (unit < full) ga = load_grad4<GRAD, ALIGNED>(g, unit);
        if (unit + stride < full) gb = load_grad4<GRAD, ALIGNED>(g, unit + stride);
        for (; unit < full; unit += 2 * stride) {
            const int64_t ub = unit + stride, na = unit + 2 * stride, nb = unit + 3 * stride;
            const float4 ca = ga, cb = gb;
            if (na < full) ga = load_grad4<GRAD, ALIGNED>(g, na);
            if (nb < full) gb = load_grad4<GRAD, ALIGNED>(g, nb);
            uint4 wa = make_uint4(0, 0, 0, 0), wb = wa;
            if (ROUND != INTSGD_ROUND_NEAREST) {
                wa = draw_unit_folded<ROUND>(draw_thread_part<ROUND>(unit, step, P.keys), unit, e, worker, step, P.keys);
                wb = draw_unit_folded<ROUND>(draw_thread_part<ROUND>(ub, step, P.keys), ub, e, worker, step, P.keys);
            }
            store_payload4<PAY>(out, unit, round_unit<ROUND>(ca, alpha, wa, P.Lf, clip_slot, nonf_slot), ALIGNED);
            if (ub < full) store_payload4<PAY>(out, ub, round_unit<ROUND>(cb, alpha, wb, P.Lf, clip_slot, nonf_slot), ALIGNED);
        }
    }
    const int tail = (int)(P.d & 3);
    if (tail && blockIdx.x == 0 && threadIdx.x == 0) {
        uint4 w = make_uint4(0, 0, 0, 0);
        if (ROUND != INTSGD_ROUND_NEAREST) w = draw_unit<ROUND>(full, worker, step, P.keys);
        const uint32_t wv[4] = {w.x, w.y, w.z, w.w};
        for (int e = 0; e < tail; ++e) {
            const int64_t j = 4 * full + e;
            const float y = __fmul_rn(alpha, grad_at<GRAD>(g, j));
            const int q = round_checked<ROUND>(y, wv[e], P.Lf, clip_slot, nonf_slot);
            if (PAY == INTSGD_PAYLOAD_I32) ((int32_t*)out)[j] = q;
            else ((int8_t*)out)[j] = (int8_t)q;
        }
    }
    counters_flush(s_cnt, st);
}

// ----------------------------------------------------------------------------------------
// Aggregate + decode + update + next-norm partial, one pass.
// One unit (4 coordinates) per thread iteration: a 16-byte load per worker on the int32 wire, one packed 32-bit
// word per worker on the int8 wire.
// ----------------------------------------------------------------------------------------
template <bool ALIGNED>
__device__ __forceinline__ void apply_unit(const VecParams& P, int64_t unit, int4 S, float c, ThreadAcc& acc) {
    const float4 xo = load_f4<ALIGNED>(P.x, unit);
    float4 xn;
    xn.x = update_coord(xo.x, S.x, c, acc.dx2);
    xn.y = update_coord(xo.y, S.y, c, acc.dx2);
    xn.z = update_coord(xo.z, S.z, c, acc.dx2);
    xn.w = update_coord(xo.w, S.w, c, acc.dx2);
    store_f4<ALIGNED>(P.x, unit, xn);
    if (P.agg) store_i4<ALIGNED>(P.agg, unit, S);
    note_sum(S.x, P.agg_limit, acc);
    note_sum(S.y, P.agg_limit, acc);
    note_sum(S.z, P.agg_limit, acc);
    note_sum(S.w, P.agg_limit, acc);
}

__device__ __forceinline__ void apply_coord(const VecParams& P, int64_t j, int S, float c, ThreadAcc& acc) {
    P.x[j] = update_coord(P.x[j], S, c, acc.dx2);
    if (P.agg) P.agg[j] = S;
    note_sum(S, P.agg_limit, acc);
}

template <int PAY, bool ALIGNED>
__global__ void __launch_bounds__(kMaxThreads) aggregate_kernel(const __grid_constant__ VecParams P) {
    DevState* st = P.st;
    if (st->status != INTSGD_OK) return;
    const float c = st->c;
    const int n = P.n;
    ThreadAcc acc = {0.0, 0, 0u};
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int64_t first = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    int64_t done;   // coordinates covered by the vector loop
    if (PAY == INTSGD_PAYLOAD_I32) {
        const int64_t full = P.d >> 2;
        for (int64_t unit = first; unit < full; unit += stride) {
            int4 S = make_int4(0, 0, 0, 0);
#pragma unroll 4
            for (int i = 0; i < n; ++i) {
                const int4 q = load_i4<ALIGNED>((const int32_t*)P.in[i], unit);
                S.x += q.x; S.y += q.y; S.z += q.z; S.w += q.w;
            }
            apply_unit<ALIGNED>(P, unit, S, c, acc);
        }
        done = full << 2;
    } else if (ALIGNED) {
        // int8 wire: one unit = one packed 32-bit word per worker; consecutive lanes take consecutive units, so every
        // access of a warp (payload words, x, aggregate) is one contiguous run
        const int64_t full = P.d >> 2;
        for (int64_t unit = first; unit < full; unit += stride) {
            int4 S = make_int4(0, 0, 0, 0);
#pragma unroll 8
            for (int i = 0; i < n; ++i) add_bytes(S, __ldcs((const uint32_t*)P.in[i] + unit));
            apply_unit<ALIGNED>(P, unit, S, c, acc);
        }
        done = full << 2;
    } else {   // element-wise path for unaligned int8 payloads
        for (int64_t j = first; j < P.d; j += stride) {
            int S = 0;
            for (int i = 0; i < n; ++i) S += (int)((const int8_t*)P.in[i])[j];
            apply_coord(P, j, S, c, acc);
        }
        done = P.d;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        for (int64_t j = done; j < P.d; ++j) {
            int S = 0;
            for (int i = 0; i < n; ++i)
                S += (PAY == INTSGD_PAYLOAD_I32) ? ((const int32_t*)P.in[i])[j] : (int)((const int8_t*)P.in[i])[j];
            apply_coord(P, j, S, c, acc);
        }
    }
    grid_finalize(acc, st, P.partials, true);
}

// ----------------------------------------------------------------------------------------
// Fused step: encode -> integer sum -> decode -> update -> next-norm partial.  Each thread owns
// a unit, walks the n gradient streams, rounds in registers and keeps the int32 sums in
// registers; payloads never reach memory.
// ----------------------------------------------------------------------------------------
template <int GRAD, bool ALIGNED, int ROUND>
__global__ void __launch_bounds__(kMaxThreads) fused_step_kernel(const __grid_constant__ VecParams P) {
    __shared__ cnt_t s_cnt[INTSGD_MAX_WORKERS + 1];
    DevState* st = P.st;
    if (st->status != INTSGD_OK) return;
    counters_init(s_cnt);
    const float alpha = st->alpha, c = st->c;
    const uint32_t step = st->step;
    const int n = P.n;
    cnt_t* nonf_slot = &s_cnt[INTSGD_MAX_WORKERS];
    ThreadAcc acc = {0.0, 0, 0u};

    const int64_t full = P.d >> 2;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t unit = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; unit < full; unit += stride) {
        int4 S = make_int4(0, 0, 0, 0);
        // the unit's half of Philox rounds 1-2 serves all n workers
        PhiloxThreadPart tp = {0u, 0u, 0u};
        if (ROUND != INTSGD_ROUND_NEAREST) tp = draw_thread_part<ROUND>(unit + P.unit_base, step, P.keys);
#pragma unroll 4
        for (int i = 0; i < n; ++i) {
            const float4 gv = load_grad4<GRAD, ALIGNED>(P.in[i], unit);
            uint4 w = make_uint4(0, 0, 0, 0);
            if (ROUND != INTSGD_ROUND_NEAREST)
                w = draw_unit_folded<ROUND>(tp, unit + P.unit_base, P.tab.e[i], (uint32_t)i, step, P.keys);
            const int4 q = round_unit<ROUND>(gv, alpha, w, P.Lf, &s_cnt[i], nonf_slot);
            S.x += q.x; S.y += q.y; S.z += q.z; S.w += q.w;
        }
        apply_unit<ALIGNED>(P, unit, S, c, acc);
    }
    const int tail = (int)(P.d & 3);
    if (tail && blockIdx.x == 0 && threadIdx.x == 0) {
        int S[4] = {0, 0, 0, 0};
        for (int i = 0; i < n; ++i) {
            uint4 w = make_uint4(0, 0, 0, 0);
            if (ROUND != INTSGD_ROUND_NEAREST) w = draw_unit<ROUND>(full + P.unit_base, (uint32_t)i, step, P.keys);
            const uint32_t wv[4] = {w.x, w.y, w.z, w.w};
            for (int e = 0; e < tail; ++e) {
                const float y = __fmul_rn(alpha, grad_at<GRAD>(P.in[i], 4 * full + e));
                S[e] += round_checked<ROUND>(y, wv[e], P.Lf, &s_cnt[i], nonf_slot);
            }
        }
        for (int e = 0; e < tail; ++e) apply_coord(P, 4 * full + e, S[e], c, acc);
    }
    counters_flush(s_cnt, st);
    grid_finalize(acc, st, P.partials, true, P.window_flags);
}

// ----------------------------------------------------------------------------------------
// Exact first step (Algorithm 1, Init line): x <- x - fl32(eta/n) * (((g_0 + g_1) + ...) + g_{n-1}).
// ----------------------------------------------------------------------------------------
__device__ __forceinline__ float exact_coord(float x_old, float m, float c0, double& acc) {
    const float t = __fmul_rn(c0, m);
    const float x_new = __fsub_rn(x_old, t);
    const float dj = __fsub_rn(x_new, x_old);
    acc = __fma_rn((double)dj, (double)dj, acc);
    return x_new;
}

template <int GRAD, bool ALIGNED>
__global__ void __launch_bounds__(kMaxThreads) exact_step_kernel(const __grid_constant__ VecParams P) {
    const int n = P.n;
    const float c0 = P.c_exact;
    ThreadAcc acc = {0.0, 0, 0u};
    const int64_t full = P.d >> 2;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t unit = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; unit < full; unit += stride) {
        float4 m = load_grad4<GRAD, ALIGNED>(P.in[0], unit);
#pragma unroll 4
        for (int i = 1; i < n; ++i) {
            const float4 gv = load_grad4<GRAD, ALIGNED>(P.in[i], unit);
            m.x = __fadd_rn(m.x, gv.x); m.y = __fadd_rn(m.y, gv.y);
            m.z = __fadd_rn(m.z, gv.z); m.w = __fadd_rn(m.w, gv.w);
        }
        const float4 xo = load_f4<ALIGNED>(P.x, unit);
        float4 xn;
        xn.x = exact_coord(xo.x, m.x, c0, acc.dx2);
        xn.y = exact_coord(xo.y, m.y, c0, acc.dx2);
        xn.z = exact_coord(xo.z, m.z, c0, acc.dx2);
        xn.w = exact_coord(xo.w, m.w, c0, acc.dx2);
        store_f4<ALIGNED>(P.x, unit, xn);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        for (int64_t j = full << 2; j < P.d; ++j) {
            float m = grad_at<GRAD>(P.in[0], j);
            for (int i = 1; i < n; ++i) m = __fadd_rn(m, grad_at<GRAD>(P.in[i], j));
            P.x[j] = exact_coord(P.x[j], m, c0, acc.dx2);
        }
    }
    grid_finalize(acc, P.st, P.partials, true, P.window_flags);
}

// ----------------------------------------------------------------------------------------
// state.dx2 = ||x - x_prev||^2 (fp32 differences, fp64 sum).
// ----------------------------------------------------------------------------------------
template <bool ALIGNED>
__global__ void __launch_bounds__(kMaxThreads) sqdiff_kernel(const __grid_constant__ VecParams P) {
    ThreadAcc acc = {0.0, 0, 0u};
    const int64_t full = P.d >> 2;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t unit = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; unit < full; unit += stride) {
        const float4 a = load_f4<ALIGNED>(P.x, unit), b = load_f4<ALIGNED>(P.x_prev, unit);
        const float d0 = __fsub_rn(a.x, b.x), d1 = __fsub_rn(a.y, b.y);
        const float d2 = __fsub_rn(a.z, b.z), d3 = __fsub_rn(a.w, b.w);
        acc.dx2 = __fma_rn((double)d0, (double)d0, acc.dx2);
        acc.dx2 = __fma_rn((double)d1, (double)d1, acc.dx2);
        acc.dx2 = __fma_rn((double)d2, (double)d2, acc.dx2);
        acc.dx2 = __fma_rn((double)d3, (double)d3, acc.dx2);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        for (int64_t j = full << 2; j < P.d; ++j) {
            const float dj = __fsub_rn(P.x[j], P.x_prev[j]);
            acc.dx2 = __fma_rn((double)dj, (double)dj, acc.dx2);
        }
    }
    grid_finalize(acc, P.st, P.partials, false);
}

// ----------------------------------------------------------------------------------------
// Heuristic IntSGD (Section 5.2 of the paper, the SwitchML rule): a profiling pass finds the largest
// |g| over all workers (NaN ignored), then alpha = (2^nb - 1) / (n 2^max_exp) with max_exp the
// smallest integer e such that max|g| <= 2^e.  grid = (blocks, workers).
// ----------------------------------------------------------------------------------------
template <int GRAD, bool ALIGNED>
__global__ void __launch_bounds__(kMaxThreads) maxabs_kernel(const __grid_constant__ VecParams P) {
    const void* g = P.in[blockIdx.y];
    float m = 0.0f;
    const int64_t full = P.d >> 2;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t unit = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; unit < full; unit += stride) {
        const float4 v = load_grad4<GRAD, ALIGNED>(g, unit);
        m = fmaxf(m, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
    }
    if (blockIdx.x == 0 && threadIdx.x == 0)
        for (int64_t j = full << 2; j < P.d; ++j) m = fmaxf(m, fabsf(grad_at<GRAD>(g, j)));
    // non-negative, NaN-free floats order like their bit patterns
    const unsigned bits = __reduce_max_sync(0xFFFFFFFFu, __float_as_uint(m));
    if ((threadIdx.x & 31) == 0 && bits) atomicMax(&P.st->maxabs_bits, bits);
}

__global__ void heuristic_scale_kernel(DevState* st, double n_as_double, double eta, double levels, int32_t n) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    const float max_abs = __uint_as_float(st->maxabs_bits);
    st->maxabs_bits = 0;
    for (int i = 0; i < n; ++i) st->clip_count[i] = 0;
    st->nonfinite = 0;
    st->agg_overflow = 0;
    st->max_abs_agg = 0;
    st->ticket = 0;
    if (!(max_abs > 0.0f) || !(max_abs <= 3.402823466e+38f)) {
        st->status = INTSGD_ERR_SCALE_NONFINITE;
        return;
    }
    int e = 0;
    const float mant = frexpf(max_abs, &e);
    const int max_exp = (mant == 0.5f) ? e - 1 : e;
    const double alpha64 = __ddiv_rn(levels, __dmul_rn(n_as_double, ldexp(1.0, max_exp)));
    const float alpha = __double2float_rn(alpha64);
    const float c = __double2float_rn(__ddiv_rn(eta, __dmul_rn(n_as_double, (double)alpha)));
    const bool ok = (alpha > 0.0f) && (alpha <= 3.402823466e+38f) && (c > 0.0f) && (c <= 3.402823466e+38f);
    if (!ok) {
        st->status = INTSGD_ERR_SCALE_NONFINITE;
        return;
    }
    st->alpha = alpha;
    st->c = c;
    st->ainv = __double2float_rn(__ddiv_rn(1.0, (double)alpha));
    st->cn = __double2float_rn(__ddiv_rn(1.0, __dmul_rn(n_as_double, (double)alpha)));
    st->eta32 = __double2float_rn(eta);
    st->status = INTSGD_OK;
}

}  // namespace intsgd
