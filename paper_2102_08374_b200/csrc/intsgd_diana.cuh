// IntDIANA step (Algorithm 3 of the IntSGD paper): the workers round gradient differences
// g_i - h_i, move their shifts by the decoded message, and the estimator h + (1/(n alpha)) sum_i q_i
// is also the new global shift.  One pass: per coordinate it reads n gradients and n local shifts,
// writes the n local shifts, and reads/writes h and x (12 n + 20 bytes with fp32 gradients and
// the int32 aggregate).
//
// fp32 steps, each rounded once (no FMA): v = g - h_i; y = alpha v; q = clip(Int(y));
// h_i += ainv * float(q); t = cn * float(S); gt = h + t; h = gt; x -= eta32 * gt.
#pragma once

#include "intsgd_device.cuh"

namespace intsgd {

struct DianaFactors {
    float alpha, ainv, cn, eta32;
};

__device__ __forceinline__ float diana_coord(float x_old, float h_old, int S, const DianaFactors& f, float& h_new,
                                             double& acc) {
    const float t = __fmul_rn(f.cn, __int2float_rn(S));
    const float gt = __fadd_rn(h_old, t);
    h_new = gt;
    const float x_new = __fsub_rn(x_old, __fmul_rn(f.eta32, gt));
    const float dj = __fsub_rn(x_new, x_old);
    acc = __fma_rn((double)dj, (double)dj, acc);
    return x_new;
}

template <int ROUND>
__device__ __forceinline__ int diana_worker_coord(float g, float& h, uint32_t w, const DianaFactors& f, float Lf,
                                                  cnt_t* clip_slot, cnt_t* nonf_slot) {
    const float y = __fmul_rn(f.alpha, __fsub_rn(g, h));
    const int q = (fabsf(y) <= Lf) ? round_in_range<ROUND>(y, w) : round_checked<ROUND>(y, w, Lf, clip_slot, nonf_slot);
    h = __fadd_rn(h, __fmul_rn(f.ainv, __int2float_rn(q)));
    return q;
}

// Direct (grid-stride) kernel: one unit of 4 coordinates per thread and iteration.
template <int GRAD, bool ALIGNED, int ROUND>
__global__ void __launch_bounds__(512) diana_step_kernel(const __grid_constant__ VecParams P) {
    __shared__ cnt_t s_cnt[INTSGD_MAX_WORKERS + 1];
    DevState* st = P.st;
    if (st->status != INTSGD_OK) return;
    counters_init(s_cnt);
    const DianaFactors f = {st->alpha, st->ainv, st->cn, st->eta32};
    const uint32_t step = st->step;
    const int n = P.n;
    cnt_t* nonf_slot = &s_cnt[INTSGD_MAX_WORKERS];
    ThreadAcc acc = {0.0, 0, 0u};

    const int64_t full = P.d >> 2;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t unit = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; unit < full; unit += stride) {
        int4 S = make_int4(0, 0, 0, 0);
#pragma unroll 2
        for (int i = 0; i < n; ++i) {
            const float4 gv = load_grad4<GRAD, ALIGNED>(P.in[i], unit);
            float* hl = (float*)P.out[i];
            float4 hv = load_f4<ALIGNED>(hl, unit);
            uint4 w = make_uint4(0, 0, 0, 0);
            if (ROUND != INTSGD_ROUND_NEAREST) w = draw_unit<ROUND>(unit, (uint32_t)i, step, P.keys);
            S.x += diana_worker_coord<ROUND>(gv.x, hv.x, w.x, f, P.Lf, &s_cnt[i], nonf_slot);
            S.y += diana_worker_coord<ROUND>(gv.y, hv.y, w.y, f, P.Lf, &s_cnt[i], nonf_slot);
            S.z += diana_worker_coord<ROUND>(gv.z, hv.z, w.z, f, P.Lf, &s_cnt[i], nonf_slot);
            S.w += diana_worker_coord<ROUND>(gv.w, hv.w, w.w, f, P.Lf, &s_cnt[i], nonf_slot);
            store_f4<ALIGNED>(hl, unit, hv);
        }
        const float4 xo = load_f4<ALIGNED>(P.x, unit), ho = load_f4<ALIGNED>(P.h, unit);
        float4 xn, hn;
        xn.x = diana_coord(xo.x, ho.x, S.x, f, hn.x, acc.dx2);
        xn.y = diana_coord(xo.y, ho.y, S.y, f, hn.y, acc.dx2);
        xn.z = diana_coord(xo.z, ho.z, S.z, f, hn.z, acc.dx2);
        xn.w = diana_coord(xo.w, ho.w, S.w, f, hn.w, acc.dx2);
        store_f4<ALIGNED>(P.x, unit, xn);
        store_f4<ALIGNED>(P.h, unit, hn);
        if (P.agg) store_i4<ALIGNED>(P.agg, unit, S);
        note_sum(S.x, P.agg_limit, acc); note_sum(S.y, P.agg_limit, acc);
        note_sum(S.z, P.agg_limit, acc); note_sum(S.w, P.agg_limit, acc);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        for (int64_t j = full << 2; j < P.d; ++j) {
            int S = 0;
            for (int i = 0; i < n; ++i) {
                uint32_t word = 0;
                if (ROUND != INTSGD_ROUND_NEAREST) {
                    const uint4 w4 = draw_unit<ROUND>(j >> 2, (uint32_t)i, step, P.keys);
                    const uint32_t wv[4] = {w4.x, w4.y, w4.z, w4.w};
                    word = wv[j & 3];
                }
                float* hl = (float*)P.out[i];
                float hv = hl[j];
                S += diana_worker_coord<ROUND>(grad_at<GRAD>(P.in[i], j), hv, word, f, P.Lf, &s_cnt[i], nonf_slot);
                hl[j] = hv;
            }
            float hn;
            P.x[j] = diana_coord(P.x[j], P.h[j], S, f, hn, acc.dx2);
            P.h[j] = hn;
            if (P.agg) P.agg[j] = S;
            note_sum(S, P.agg_limit, acc);
        }
    }
    counters_flush(s_cnt, st);
    grid_finalize(acc, st, P.partials, true);
}

}  // namespace intsgd
