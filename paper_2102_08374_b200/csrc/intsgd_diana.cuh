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
#include "intsgd_pipe.cuh"

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
        PhiloxThreadPart tp = {0u, 0u, 0u};   // the unit's half of Philox rounds 1-2 serves all n workers
        if (ROUND != INTSGD_ROUND_NEAREST) tp = draw_thread_part<ROUND>(unit, step, P.keys);
#pragma unroll 2
        for (int i = 0; i < n; ++i) {
            const float4 gv = load_grad4<GRAD, ALIGNED>(P.in[i], unit);
            float* hl = (float*)P.out[i];
            float4 hv = load_f4<ALIGNED>(hl, unit);
            uint4 w = make_uint4(0, 0, 0, 0);
            if (ROUND != INTSGD_ROUND_NEAREST) w = draw_unit_folded<ROUND>(tp, unit, P.tab.e[i], (uint32_t)i, step, P.keys);
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

// ---------------------------------------------------------------------------------------------
// Pipelined variant (16-byte aligned pointers, d <= 2^34): the ring of fused_pipe_kernel, with a stage
// holding G worker slots of one gradient tile and one local-shift tile each.  Consumers read both out
// of shared memory, store the moved shift straight to global memory and keep the integer sums in
// registers; nothing is deferred (a unit with a value outside [-Lf, Lf] takes the counting rule on the
// spot), because the shift update needs every integer as soon as it exists.
// ---------------------------------------------------------------------------------------------
template <int ROUND>
__device__ __forceinline__ void diana_consume_unit(float4 g, float4 h, uint4 w, const DianaFactors& f, float Lf,
                                                   cnt_t* clip_slot, cnt_t* nonf_slot, int4& S, float4& h_new) {
    const float2 neg1 = make_float2(-1.0f, -1.0f), alpha2 = make_float2(f.alpha, f.alpha);
    const float2 h01 = make_float2(h.x, h.y), h23 = make_float2(h.z, h.w);
    const float2 y01 = __fmul2_rn(alpha2, __ffma2_rn(h01, neg1, make_float2(g.x, g.y)));   // alpha * fl(g - h)
    const float2 y23 = __fmul2_rn(alpha2, __ffma2_rn(h23, neg1, make_float2(g.z, g.w)));
    const float m = absmax3_nan(absmax3_nan(y01.x, y01.y, y23.x), y23.y, y23.y);
    int4 q;
    if (m <= Lf) q = round4_in_range<ROUND>(y01, y23, w);   // false for NaN
    else q = round_unit_checked<ROUND>(y01.x, y01.y, y23.x, y23.y, w, Lf, clip_slot, nonf_slot);
    // h + fl(ainv * q): product and sum each rounded once
    h_new = make_float4(__fadd_rn(h.x, __fmul_rn(f.ainv, __int2float_rn(q.x))), __fadd_rn(h.y, __fmul_rn(f.ainv, __int2float_rn(q.y))),
                        __fadd_rn(h.z, __fmul_rn(f.ainv, __int2float_rn(q.z))), __fadd_rn(h.w, __fmul_rn(f.ainv, __int2float_rn(q.w))));
    S.x += q.x; S.y += q.y; S.z += q.z; S.w += q.w;
}

template <int GRAD, int ROUND, int NC, int UPT, int G, int NS>
__global__ void __launch_bounds__(NC + 32, 1) diana_pipe_kernel(const __grid_constant__ PipeParams PP) {
    constexpr int kGBytes = (GRAD == INTSGD_GRAD_F32) ? 16 : 8;
    constexpr int kTileUnits = NC * UPT;
    constexpr int kGTile = kTileUnits * kGBytes, kHTile = kTileUnits * 16, kSlot = kGTile + kHTile;
    constexpr bool kPairShared = ROUND == INTSGD_ROUND_RANDOM16 && NC == 512 && UPT == 2;
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(16) uint4 s_tab[INTSGD_MAX_WORKERS];
    __shared__ uint64_t full_bar[NS], empty_bar[NS];
    __shared__ cnt_t s_cnt[INTSGD_MAX_WORKERS + 1];
    __shared__ int s_fault;

    const VecParams& P = PP.v;
    DevState* st = P.st;
    asm volatile("griddepcontrol.launch_dependents;");
    if (threadIdx.x == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], NC);
        }
        s_fault = 0;
        mbar_fence_init();
    }
    for (int i = threadIdx.x; i < INTSGD_MAX_WORKERS; i += blockDim.x) s_tab[i] = P.tab.e[i];
    counters_init(s_cnt);   // includes a __syncthreads()
    grid_dependency_wait();
    if (st->status != INTSGD_OK) return;

    const int n = P.n;
    const int64_t tiles = PP.tiles;
    ThreadAcc acc = {0.0, 0, 0u};
    bool ok = true;
    uint32_t it = 0;   // producer thread: stages filled so far

    if (threadIdx.x >= NC) {
        if (threadIdx.x == NC) {   // producer
            uint32_t s = 0, phase = 0;
            for (int64_t tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
                const int64_t left = PP.units - tile * kTileUnits;
                const uint32_t units = (uint32_t)(left < kTileUnits ? left : kTileUnits);
                const uint32_t g_bytes = units * kGBytes, h_bytes = units * 16;
                for (int g0 = 0; g0 < n; g0 += G) {
                    if (it >= NS && !mbar_wait(&empty_bar[s], phase ^ 1u)) { ok = false; break; }
                    const int gw = (n - g0 < G) ? (n - g0) : G;
                    mbar_arrive_expect_tx(&full_bar[s], (uint32_t)gw * (g_bytes + h_bytes));
                    unsigned char* dst = smem + (size_t)s * G * kSlot;
                    for (int w = 0; w < gw; ++w) {
                        bulk_load(dst + w * kSlot, (const unsigned char*)P.in[g0 + w] + (size_t)tile * kGTile, g_bytes, &full_bar[s]);
                        bulk_load(dst + w * kSlot + kGTile, (const unsigned char*)P.out[g0 + w] + (size_t)tile * kHTile, h_bytes,
                                  &full_bar[s]);
                    }
                    ++it;
                    if (++s == NS) { s = 0; phase ^= 1u; }
                }
            }
            if (!ok) atomicExch(&s_fault, 1);
        }
    } else {
        const int c = threadIdx.x;
        const DianaFactors f = {st->alpha, st->ainv, st->cn, st->eta32};
        const uint32_t step = st->step;
        cnt_t* nonf_slot = &s_cnt[INTSGD_MAX_WORKERS];
        uint32_t s = 0, phase = 0;
        const uint32_t full0 = smem_addr(&full_bar[0]), empty0 = smem_addr(&empty_bar[0]);
        for (int64_t tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
            const int64_t unit0 = tile * kTileUnits + c;
            float4 xo[UPT], ho[UPT];
            PhiloxThreadPart tp[UPT];
            int4 S[UPT];
            bool active[UPT], half[UPT];
#pragma unroll
            for (int k = 0; k < UPT; ++k) {
                const int64_t unit = unit0 + (int64_t)k * NC;
                active[k] = unit < PP.units;
                half[k] = ((unit + P.unit_base) >> 9) & 1;
                xo[k] = ho[k] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (active[k]) {
                    xo[k] = load_f4<true>(P.x, unit);
                    ho[k] = load_f4<true>(P.h, unit);
                }
                tp[k].n3 = tp[k].H = tp[k].m1 = 0;
                if (ROUND == INTSGD_ROUND_RANDOM || ROUND == INTSGD_ROUND_RANDOM_COMPARE)
                    tp[k] = philox_thread_part((uint32_t)(unit + P.unit_base), step, P.keys);
                if (ROUND == INTSGD_ROUND_RANDOM16 && !(kPairShared && k > 0))
                    tp[k] = philox_thread_part(pair_index((uint32_t)(unit + P.unit_base)), step, P.keys);
                S[k] = make_int4(0, 0, 0, 0);
            }
            for (int g0 = 0; g0 < n; g0 += G) {
                if (!mbar_wait_at(full0 + 8u * s, phase)) { ok = false; break; }
                const unsigned char* src = smem + (size_t)s * G * kSlot;
                const int gw = (n - g0 < G) ? (n - g0) : G;
                for (int w = 0; w < gw; ++w) {
                    const uint4 e = s_tab[g0 + w];
                    uint4 pw = make_uint4(0, 0, 0, 0);
                    if (kPairShared) pw = philox_finish(tp[0], e, P.keys);
                    float* h_out = (float*)P.out[g0 + w];
#pragma unroll
                    for (int k = 0; k < UPT; ++k) {
                        if (!active[k]) continue;
                        const int u = c + k * NC;
                        const float4 gv = lds_unit<GRAD>(src + w * kSlot, u);
                        const float4 hv = *reinterpret_cast<const float4*>(src + w * kSlot + kGTile + 16 * u);
                        float4 hn;
                        diana_consume_unit<ROUND>(gv, hv, unit_draws<ROUND, kPairShared>(tp[k], e, pw, k, half[k], P.keys), f, P.Lf,
                                                  &s_cnt[g0 + w], nonf_slot, S[k], hn);
                        store_f4<true>(h_out, unit0 + (int64_t)k * NC, hn);
                    }
                }
                mbar_arrive_at(empty0 + 8u * s);
                if (++s == NS) { s = 0; phase ^= 1u; }
            }
            if (!ok) break;
#pragma unroll
            for (int k = 0; k < UPT; ++k) {
                if (!active[k]) continue;
                const int64_t unit = unit0 + (int64_t)k * NC;
                float4 xn, hn;
                xn.x = diana_coord(xo[k].x, ho[k].x, S[k].x, f, hn.x, acc.dx2);
                xn.y = diana_coord(xo[k].y, ho[k].y, S[k].y, f, hn.y, acc.dx2);
                xn.z = diana_coord(xo[k].z, ho[k].z, S[k].z, f, hn.z, acc.dx2);
                xn.w = diana_coord(xo[k].w, ho[k].w, S[k].w, f, hn.w, acc.dx2);
                store_f4<true>(P.x, unit, xn);
                store_f4<true>(P.h, unit, hn);
                if (P.agg) store_i4<true>(P.agg, unit, S[k]);
                note_sum(S[k].x, P.agg_limit, acc); note_sum(S[k].y, P.agg_limit, acc);
                note_sum(S[k].z, P.agg_limit, acc); note_sum(S[k].w, P.agg_limit, acc);
            }
        }
        if (!ok) atomicExch(&s_fault, 1);

        // coordinates after the last pipelined unit (at most 7): element-wise, one thread
        if (blockIdx.x == 0 && c == 0 && ok) {
            for (int64_t j = PP.units << 2; j < P.d; ++j) {
                int Sj = 0;
                for (int i = 0; i < n; ++i) {
                    uint32_t word = 0;
                    if (ROUND != INTSGD_ROUND_NEAREST) {
                        const uint4 w4 = draw_unit<ROUND>((j >> 2) + P.unit_base, (uint32_t)i, step, P.keys);
                        const uint32_t wv[4] = {w4.x, w4.y, w4.z, w4.w};
                        word = wv[j & 3];
                    }
                    float* hl = (float*)P.out[i];
                    float hv = hl[j];
                    Sj += diana_worker_coord<ROUND>(grad_at<GRAD>(P.in[i], j), hv, word, f, P.Lf, &s_cnt[i], nonf_slot);
                    hl[j] = hv;
                }
                float hn;
                P.x[j] = diana_coord(P.x[j], P.h[j], Sj, f, hn, acc.dx2);
                P.h[j] = hn;
                if (P.agg) P.agg[j] = Sj;
                note_sum(Sj, P.agg_limit, acc);
            }
        }
    }
    __syncthreads();
    // whichever side's wait gave up: the producer thread lets the copies it has issued land before the block retires
    if (threadIdx.x == NC && s_fault) drain_issued<NS>(full_bar, it);
    counters_flush(s_cnt, st);   // includes a __syncthreads()
    if (threadIdx.x == 0 && s_fault) atomicExch(&st->fault, 1);
    grid_finalize(acc, st, P.partials, true);
}

}  // namespace intsgd
