// Pipelined encode for sm_100a: payload_i = clip(Int(alpha g_i)) for all the workers of one launch
// (Algorithm 1, "scale and round the local gradient"; Section 5.1 for the clipping).
//
// Same ring as fused_pipe_kernel: one producer thread stages G worker tiles per stage into shared memory
// with bulk asynchronous copies, NC consumer threads round out of shared memory.  A consumer owns the
// same UPT units of every worker's tile, so the unit-dependent half of Philox rounds 1-2 is computed once
// per tile and thread and serves all workers (16 wide multiplies per worker unit instead of 20), and the
// loads in flight do not depend on the consumers' registers.  Payload values go straight to global
// memory: 16 bytes (int32 wire) or 4 packed bytes (int8 wire) per unit, consecutive lanes consecutive units.
//
// Requirements checked by the host: every pointer 16-byte aligned, d <= 2^34.  Everything else runs in
// encode_kernel.
#pragma once

#include "intsgd_blocks.cuh"
#include "intsgd_device.cuh"
#include "intsgd_kernels.cuh"
#include "intsgd_pipe.cuh"

namespace intsgd {

// Exact redo of one worker's unit from global memory with the full clipping rule and the counters (rare: some
// |alpha g| outside [-Lf, Lf], or a NaN/Inf).  Overwrites the payload the fast path stored for the unit.
template <int GRAD, int PAY, int ROUND>
__device__ __noinline__ void redo_encode_unit(const VecParams& P, int slot, int64_t unit, float4 alpha4, uint32_t step,
                                              cnt_t* s_cnt) {
    const int worker = P.worker_base + slot;
    const float4 g = load_grad4<GRAD, true>(P.in[slot], unit);
    uint4 w = make_uint4(0, 0, 0, 0);
    if (ROUND != INTSGD_ROUND_NEAREST) w = draw_unit<ROUND>(unit + P.unit_base, (uint32_t)worker, step, P.keys);
    const int4 q = round_unit_checked<ROUND>(__fmul_rn(alpha4.x, g.x), __fmul_rn(alpha4.y, g.y), __fmul_rn(alpha4.z, g.z),
                                             __fmul_rn(alpha4.w, g.w), w, P.Lf, &s_cnt[worker], &s_cnt[INTSGD_MAX_WORKERS]);
    store_payload4<PAY>(P.out[slot], unit, q, true);
}

template <int GRAD, int PAY, int ROUND, bool BLOCKS, int NC, int UPT, int G, int NS>
__global__ void __launch_bounds__(NC + 32, 1) encode_pipe_kernel(const __grid_constant__ PipeParams PP) {
    constexpr int kUnitBytes = (GRAD == INTSGD_GRAD_F32) ? 16 : 8;
    constexpr int kTileUnits = NC * UPT;
    constexpr int kTileBytes = kTileUnits * kUnitBytes;
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
    grid_dependency_wait();  // the step's scale kernel, when this launch was allowed to start early
    if (st->status != INTSGD_OK) return;

    const int n = P.n;   // workers of this launch: slot i is worker P.worker_base + i
    const int64_t tiles = PP.tiles;
    bool ok = true;
    uint32_t issued = 0;   // producer: stages filled so far

    if (threadIdx.x >= NC) {
        if (threadIdx.x == NC) {   // producer
            uint32_t s = 0, phase = 0;
            for (int64_t tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
                const int64_t left = PP.units - tile * kTileUnits;
                const uint32_t bytes = (uint32_t)(left < kTileUnits ? left : kTileUnits) * kUnitBytes;
                const size_t offset = (size_t)tile * kTileBytes;
                for (int g0 = 0; g0 < n; g0 += G) {
                    if (issued >= NS && !mbar_wait(&empty_bar[s], phase ^ 1u)) { ok = false; break; }
                    const int gw = (n - g0 < G) ? (n - g0) : G;
                    mbar_arrive_expect_tx(&full_bar[s], (uint32_t)gw * bytes);
                    unsigned char* dst = smem + (size_t)s * G * kTileBytes;
                    for (int w = 0; w < gw; ++w)
                        bulk_load(dst + w * kTileBytes, (const unsigned char*)P.in[g0 + w] + offset, bytes, &full_bar[s]);
                    ++issued;
                    if (++s == NS) { s = 0; phase ^= 1u; }
                }
            }
            if (!ok) atomicExch(&s_fault, 1);
        }
    } else {
        const int c = threadIdx.x;
        const int lane = c & 31;
        const float alpha = (P.alpha_override == P.alpha_override) ? P.alpha_override : st->alpha;
        const uint32_t step = st->step;
        const BlockParams& bp = P.bp;
        uint32_t s = 0, phase = 0;
        const uint32_t full0 = smem_addr(&full_bar[0]), empty0 = smem_addr(&empty_bar[0]);
        for (int64_t tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
            const int64_t unit0 = tile * kTileUnits + c;
            PhiloxThreadPart tp[UPT];
            float2 a01[UPT], a23[UPT];
            bool active[UPT], half[UPT];
#pragma unroll
            for (int k = 0; k < UPT; ++k) {
                const int64_t unit = unit0 + (int64_t)k * NC;
                active[k] = unit < PP.units;
                half[k] = ((unit + P.unit_base) >> 9) & 1;
                tp[k].n3 = tp[k].H = tp[k].m1 = 0;
                if (ROUND == INTSGD_ROUND_RANDOM || ROUND == INTSGD_ROUND_RANDOM_COMPARE)
                    tp[k] = philox_thread_part((uint32_t)(unit + P.unit_base), step, P.keys);
                if (ROUND == INTSGD_ROUND_RANDOM16 && !(kPairShared && k > 0))
                    tp[k] = philox_thread_part(pair_index((uint32_t)(unit + P.unit_base)), step, P.keys);
                a01[k] = make_float2(alpha, alpha);
                a23[k] = a01[k];
                if (BLOCKS && active[k]) {
                    // the warp's 32 units form one chunk of the partition's table
                    int s_lo, s_hi;
                    chunk_segments(bp, unit - lane + P.unit_base, s_lo, s_hi);
                    const UnitScale us = unit_scale(bp, unit + P.unit_base, s_lo, s_hi);
                    a01[k] = us.a01;
                    a23[k] = us.a23;
                }
            }
            for (int g0 = 0; g0 < n; g0 += G) {
                if (!mbar_wait_at(full0 + 8u * s, phase)) { ok = false; break; }
                const unsigned char* src = smem + (size_t)s * G * kTileBytes;
                const int gw = (n - g0 < G) ? (n - g0) : G;
                // One worker's unit on the fast path: scale, round, store -- no branch, so that the G * UPT independent
                // Philox chains of a stage overlap.  A unit with a value outside [-Lf, Lf] (or a NaN) is only noted
                // (bit w of bad[k]); it is redone with the counting rule once the stage's fast path is through.
                uint32_t bad[UPT];
#pragma unroll
                for (int k = 0; k < UPT; ++k) bad[k] = 0u;
                auto encode_unit = [&](int w, int k, const uint4& e, const uint4& pw) {
                    const float4 gv = lds_unit<GRAD>(src + w * kTileBytes, c + k * NC);
                    const uint4 dr = unit_draws<ROUND, kPairShared>(tp[k], e, pw, k, half[k], P.keys);
                    const float2 y01 = __fmul2_rn(a01[k], make_float2(gv.x, gv.y));
                    const float2 y23 = __fmul2_rn(a23[k], make_float2(gv.z, gv.w));
                    const float m = absmax3_nan(absmax3_nan(y01.x, y01.y, y23.x), y23.y, y23.y);
                    bad[k] |= (m <= P.Lf) ? 0u : (1u << w);   // set for NaN too
                    store_payload4<PAY>(P.out[g0 + w], unit0 + (int64_t)k * NC, round4_in_range<ROUND>(y01, y23, dr), true);
                };
                if (active[UPT - 1] && gw == G) {
#pragma unroll
                    for (int w = 0; w < G; ++w) {
                        const uint4 e = s_tab[P.worker_base + g0 + w];
                        uint4 pw = make_uint4(0, 0, 0, 0);
                        if (kPairShared) pw = philox_finish(tp[0], e, P.keys);   // one block for both units
#pragma unroll
                        for (int k = 0; k < UPT; ++k) encode_unit(w, k, e, pw);
                    }
                } else {
                    for (int w = 0; w < gw; ++w) {
                        const uint4 e = s_tab[P.worker_base + g0 + w];
                        uint4 pw = make_uint4(0, 0, 0, 0);
                        if (kPairShared) pw = philox_finish(tp[0], e, P.keys);
#pragma unroll
                        for (int k = 0; k < UPT; ++k)
                            if (active[k]) encode_unit(w, k, e, pw);
                    }
                }
#pragma unroll
                for (int k = 0; k < UPT; ++k) {
                    while (bad[k]) {   // rare
                        const int w = __ffs(bad[k]) - 1;
                        bad[k] &= bad[k] - 1u;
                        redo_encode_unit<GRAD, PAY, ROUND>(P, g0 + w, unit0 + (int64_t)k * NC,
                                                           make_float4(a01[k].x, a01[k].y, a23[k].x, a23[k].y), step, s_cnt);
                    }
                }
                mbar_arrive_at(empty0 + 8u * s);
                if (++s == NS) { s = 0; phase ^= 1u; }
            }
        }
        if (!ok) atomicExch(&s_fault, 1);

        // coordinates after the last pipelined unit (at most 7): element-wise, one thread
        if (blockIdx.x == 0 && c == 0 && ok) {
            for (int64_t j = PP.units << 2; j < P.d; ++j) {
                float aj = alpha, cj = 0.0f;
                if (BLOCKS) coord_scale(bp, j + (P.unit_base << 2), aj, cj);
                for (int i = 0; i < n; ++i) {
                    const int worker = P.worker_base + i;
                    uint32_t word = 0;
                    if (ROUND != INTSGD_ROUND_NEAREST) {
                        const uint4 w4 = draw_unit<ROUND>((j >> 2) + P.unit_base, (uint32_t)worker, step, P.keys);
                        const uint32_t wv[4] = {w4.x, w4.y, w4.z, w4.w};
                        word = wv[j & 3];
                    }
                    const float y = __fmul_rn(aj, grad_at<GRAD>(P.in[i], j));
                    const int q = round_checked<ROUND>(y, word, P.Lf, &s_cnt[worker], &s_cnt[INTSGD_MAX_WORKERS]);
                    if (PAY == INTSGD_PAYLOAD_I32) ((int32_t*)P.out[i])[j] = q;
                    else ((int8_t*)P.out[i])[j] = (int8_t)q;
                }
            }
        }
    }
    __syncthreads();
    // A wait gave up somewhere in this block: before the block can retire, the producer thread lets every
    // copy it has issued land (bounded), whichever side noticed.
    if (threadIdx.x == NC && s_fault) drain_issued<NS>(full_bar, issued);
    counters_flush(s_cnt, st);   // includes a __syncthreads()
    if (threadIdx.x == 0 && s_fault) atomicExch(&st->fault, 1);
}

}  // namespace intsgd
