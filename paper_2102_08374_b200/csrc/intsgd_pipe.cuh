// Pipelined fused IntSGD step for sm_100a: gradient tiles are staged into shared memory by bulk
// asynchronous copies (cp.async.bulk, completion counted on mbarriers) issued by one producer
// thread, while the consumer warps round, sum and update out of shared memory.  The ring of stages
// keeps ~200 KB of loads in flight per SM independently of the consumers' register use, which is
// what a 17-stream read at HBM3e speed needs.
//
// Layout of one stage: G worker tiles back to back, each NC * UPT units of 16 (fp32) or 8 (bf16)
// bytes; consumer thread c owns units c, c + NC, ... of every tile, so shared-memory reads are
// conflict-free 16-byte (8-byte) accesses and the Philox counters of a thread are fixed for a whole tile.
//
// Requirements checked by the host: every pointer 16-byte aligned, d <= 2^34.  Everything else
// (unaligned pointers, larger d) runs in fused_step_kernel.  A launch may cover a window of the vector: `unit`
// indexes the launch's pointers, `unit + unit_base` the whole vector (random stream, partition tables, chunk partials).
#pragma once

#include "intsgd_blocks.cuh"
#include "intsgd_device.cuh"
#include "intsgd_kernels.cuh"

namespace intsgd {

// ---- mbarrier / bulk-copy primitives (inline PTX) -------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
// One poll.  The suspend-time hint lets the hardware park the warp for up to that long before the poll returns
// (it returns at once when the phase completes): a waiting warp that polled in a tight loop would take issue
// slots from the warps of its scheduler that still have work, and these kernels are bound by instruction issue.
constexpr uint32_t kPollHintNs = 10000;
__device__ __forceinline__ bool mbar_try_wait_at(uint32_t bar_addr, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar_addr), "r"(parity), "r"(kPollHintNs)
        : "memory");
    return done != 0;
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) { return mbar_try_wait_at(smem_addr(bar), parity); }
// Bounded wait: gives up after kWaitLimit polls (each poll may itself block for up to the hinted interval, so
// the bound is about ten seconds at most), so a lost completion can never hang the GPU.
constexpr uint32_t kWaitLimit = 1u << 20;
__device__ __forceinline__ bool mbar_wait_at(uint32_t bar_addr, uint32_t parity) {
    for (uint32_t i = 0; i < kWaitLimit; ++i)
        if (mbar_try_wait_at(bar_addr, parity)) return true;
    return false;
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) { return mbar_wait_at(smem_addr(bar), parity); }
// The consumers' per-stage calls take the barriers' shared-space addresses, computed once per kernel: converting
// the generic pointer on every call costs instructions, and every instruction of these kernels costs time.
__device__ __forceinline__ void mbar_arrive_at(uint32_t bar_addr) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar_addr) : "memory");
}
// Programmatic dependent launch: blocks until the grids this launch depends on have completed and their
// writes are visible; returns at once for an ordinary launch.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Global -> shared bulk copy, completion signalled on an mbarrier of this CTA (no multicast).
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_addr(dst_smem)),
                 "l"(src_gmem), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}

// Failure path of the pipelined kernels: waits (each wait bounded) until the last min(issued, NS) stages the
// producer has filled have landed, so that no bulk copy is still in flight into the shared memory of a block
// that is about to retire.  Stage j (0-based) completes phase (j / NS) & 1 of barrier j % NS.
template <int NS>
__device__ __forceinline__ void drain_issued(uint64_t* full_bar, uint32_t issued) {
    const uint32_t pending = issued < (uint32_t)NS ? issued : (uint32_t)NS;
    for (uint32_t k = 0; k < pending; ++k) {
        const uint32_t j = issued - 1 - k;
        mbar_wait(&full_bar[j % NS], (j / NS) & 1u);
    }
}

// ---- per-unit arithmetic ------------------------------------------------------------------------
// Fast path of one worker's unit.  The rounded values are accumulated as integer-valued
// floats (exact: the host caps the fast-path magnitude T so that n * (T + 1) <= 2^24, and T never
// exceeds the clip limit); `m` tracks max |alpha g| (NaN-propagating) so that a unit with any value
// outside the fast range -- clipped, huge or not finite -- is redone exactly at the end of its tile.
struct UnitAcc {
    float2 F01, F23;   // running sums of the four coordinates
    float m;           // running max |alpha g| over all workers
};

template <int ROUND>
__device__ __forceinline__ void consume_unit(float4 g, float2 alpha01, float2 alpha23, uint4 w, UnitAcc& u) {
    const float2 y01 = __fmul2_rn(alpha01, make_float2(g.x, g.y));
    const float2 y23 = __fmul2_rn(alpha23, make_float2(g.z, g.w));
    u.m = absmax3_nan(u.m, y01.x, y01.y);
    u.m = absmax3_nan(u.m, y23.x, y23.y);
    if (ROUND == INTSGD_ROUND_NEAREST) {
        u.F01 = __fadd2_rn(u.F01, make_float2(rintf(y01.x), rintf(y01.y)));
        u.F23 = __fadd2_rn(u.F23, make_float2(rintf(y23.x), rintf(y23.y)));
        return;
    }
    if (ROUND == INTSGD_ROUND_RANDOM_COMPARE) {
        // f = floor(y); p = fl32(y - f); up iff (float)(w >> 8) < p * 2^24; every step rounded once
        const float2 f01 = make_float2(floorf(y01.x), floorf(y01.y));
        const float2 f23 = make_float2(floorf(y23.x), floorf(y23.y));
        const float2 neg1 = make_float2(-1.0f, -1.0f), two24 = make_float2(16777216.0f, 16777216.0f);
        const float2 p01 = __fmul2_rn(__ffma2_rn(f01, neg1, y01), two24);
        const float2 p23 = __fmul2_rn(__ffma2_rn(f23, neg1, y23), two24);
        const float2 u01 = make_float2(lt_as_float(draw_as_float<ROUND>(w.x), p01.x), lt_as_float(draw_as_float<ROUND>(w.y), p01.y));
        const float2 u23 = make_float2(lt_as_float(draw_as_float<ROUND>(w.z), p23.x), lt_as_float(draw_as_float<ROUND>(w.w), p23.y));
        u.F01 = __fadd2_rn(__fadd2_rn(u.F01, f01), u01);
        u.F23 = __fadd2_rn(__fadd2_rn(u.F23, f23), u23);
        return;
    }
    // floor(y + u) on the unrounded sum: fused multiply-add rounded down, then floor (see round_in_range)
    const float2 scale = make_float2(draw_scale<ROUND>(), draw_scale<ROUND>());
    const float2 z01 = __ffma2_rd(make_float2(draw_as_float<ROUND>(w.x), draw_as_float<ROUND>(w.y)), scale, y01);
    const float2 z23 = __ffma2_rd(make_float2(draw_as_float<ROUND>(w.z), draw_as_float<ROUND>(w.w)), scale, y23);
    u.F01 = __fadd2_rn(u.F01, make_float2(floorf(z01.x), floorf(z01.y)));
    u.F23 = __fadd2_rn(u.F23, make_float2(floorf(z23.x), floorf(z23.y)));
}

// Exact redo of one unit from global memory with the full clipping rule and the counters (rare:
// some |alpha g| outside the fast range, or a NaN/Inf).  The fast path has counted nothing.
template <int GRAD, int ROUND>
__device__ __noinline__ int4 redo_unit(const VecParams& P, int64_t unit, float4 alpha4, uint32_t step, cnt_t* s_cnt) {
    const float av[4] = {alpha4.x, alpha4.y, alpha4.z, alpha4.w};
    int S[4] = {0, 0, 0, 0};
    for (int i = 0; i < P.n; ++i) {
        const float4 g = load_grad4<GRAD, true>(P.in[i], unit);
        uint4 w = make_uint4(0, 0, 0, 0);
        if (ROUND != INTSGD_ROUND_NEAREST) w = draw_unit<ROUND>(unit + P.unit_base, (uint32_t)i, step, P.keys);
        uint32_t clipped = 0, nonfinite = 0;
        S[0] += round_full<ROUND>(__fmul_rn(av[0], g.x), w.x, P.Lf, clipped, nonfinite);
        S[1] += round_full<ROUND>(__fmul_rn(av[1], g.y), w.y, P.Lf, clipped, nonfinite);
        S[2] += round_full<ROUND>(__fmul_rn(av[2], g.z), w.z, P.Lf, clipped, nonfinite);
        S[3] += round_full<ROUND>(__fmul_rn(av[3], g.w), w.w, P.Lf, clipped, nonfinite);
        if (clipped) atomicAdd(&s_cnt[i], clipped);
        if (nonfinite) atomicAdd(&s_cnt[INTSGD_MAX_WORKERS], nonfinite);
    }
    return make_int4(S[0], S[1], S[2], S[3]);
}

struct PipeParams {
    VecParams v;
    float fast_limit;   // T: fast path handles |alpha g| <= T
    int64_t units;      // units covered by the pipeline (the rest is the scalar tail)
    int64_t tiles;
};

// 16-bit draws: pair index of a unit, and the four draws of its half of the pair's Philox block.
__device__ __forceinline__ uint32_t pair_index(uint32_t unit_lo) { return ((unit_lo >> 10) << 9) | (unit_lo & 511u); }
__device__ __forceinline__ uint4 split16(uint32_t a, uint32_t b) {
    return make_uint4(a & 0xFFFFu, a >> 16, b & 0xFFFFu, b >> 16);
}

// The four draws of one unit of one worker from the thread's folded Philox state.  With 16-bit draws and
// PAIR_SHARED the block `pw` of the thread's pair was computed once and unit k takes its half.
template <int ROUND, bool PAIR_SHARED>
__device__ __forceinline__ uint4 unit_draws(const PhiloxThreadPart& t, const uint4& e, const uint4& pw, int k, bool h,
                                            const PhiloxKeys& K) {
    if (ROUND == INTSGD_ROUND_RANDOM || ROUND == INTSGD_ROUND_RANDOM_COMPARE) return philox_finish(t, e, K);
    if (ROUND == INTSGD_ROUND_RANDOM16) {
        if (PAIR_SHARED) return k == 0 ? split16(pw.x, pw.y) : split16(pw.z, pw.w);
        const uint4 r = philox_finish(t, e, K);
        return h ? split16(r.z, r.w) : split16(r.x, r.y);
    }
    return make_uint4(0, 0, 0, 0);
}

template <int GRAD>
__device__ __forceinline__ float4 lds_unit(const unsigned char* tile, int c) {
    if (GRAD == INTSGD_GRAD_F32) return *reinterpret_cast<const float4*>(tile + 16 * c);
    const uint2 v = *reinterpret_cast<const uint2*>(tile + 8 * c);
    return make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xFFFF0000u),
                       __uint_as_float(v.y << 16), __uint_as_float(v.y & 0xFFFF0000u));
}

// ---- the kernel ----------------------------------------------------------------------------------
// NC consumer threads + one producer warp.  A tile is NC * UPT units; consumer c owns units
// c, c + NC, ... of the tile.  G worker tiles per stage, NS stages.
template <int GRAD, int ROUND, bool BLOCKS, int NC, int UPT, int G, int NS>
__global__ void __launch_bounds__(NC + 32, 1) fused_pipe_kernel(const __grid_constant__ PipeParams PP) {
    constexpr int kUnitBytes = (GRAD == INTSGD_GRAD_F32) ? 16 : 8;
    constexpr int kTileUnits = NC * UPT;
    constexpr int kTileBytes = kTileUnits * kUnitBytes;
    // 16-bit draws with the 2 x 512 tile: a thread's two units are 512 apart in a 1024-aligned tile,
    // i.e. the two halves of one pair, so one Philox block per worker serves both.
    constexpr bool kPairShared = ROUND == INTSGD_ROUND_RANDOM16 && NC == 512 && UPT == 2;
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(16) uint4 s_tab[INTSGD_MAX_WORKERS];
    __shared__ uint64_t full_bar[NS], empty_bar[NS];
    __shared__ cnt_t s_cnt[INTSGD_MAX_WORKERS + 1];
    __shared__ int s_fault;

    const VecParams& P = PP.v;
    DevState* st = P.st;
    // the next step's scale kernel may be scheduled from now on; it waits for this grid to complete
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
    // Everything above needs only the kernel's arguments.  When the launch was allowed to start before
    // the step's scale kernel has finished, wait here for that kernel's writes (a no-op otherwise).
    grid_dependency_wait();
    if (st->status != INTSGD_OK) return;

    const int n = P.n;
    const int64_t tiles = PP.tiles;
    ThreadAcc acc = {0.0, 0, 0u};
    bool ok = true;
    uint32_t it = 0;   // producer thread: stages filled so far

    if (threadIdx.x >= NC) {
        // ------------------------------- producer ---------------------------------------------
        if (threadIdx.x == NC) {
            uint32_t s = 0, phase = 0;   // s = it % NS; phase = (it / NS) & 1
            for (int64_t tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
                const int64_t left = PP.units - tile * kTileUnits;
                const uint32_t bytes = (uint32_t)(left < kTileUnits ? left : kTileUnits) * kUnitBytes;
                const size_t offset = (size_t)tile * kTileBytes;
                for (int g0 = 0; g0 < n; g0 += G) {
                    if (it >= NS && !mbar_wait(&empty_bar[s], phase ^ 1u)) { ok = false; break; }
                    const int gw = (n - g0 < G) ? (n - g0) : G;
                    mbar_arrive_expect_tx(&full_bar[s], (uint32_t)gw * bytes);
                    unsigned char* dst = smem + (size_t)s * G * kTileBytes;
                    for (int w = 0; w < gw; ++w)
                        bulk_load(dst + w * kTileBytes, (const unsigned char*)P.in[g0 + w] + offset, bytes, &full_bar[s]);
                    ++it;
                    if (++s == NS) { s = 0; phase ^= 1u; }
                }
            }
            if (!ok) atomicExch(&s_fault, 1);
        }
    } else {
        // ------------------------------- consumers --------------------------------------------
        const int c = threadIdx.x;
        const int lane = c & 31;
        const float alpha = st->alpha, cdec = st->c;
        const uint32_t step = st->step;
        const BlockParams& bp = P.bp;
        uint32_t s = 0, phase = 0;
        const uint32_t full0 = smem_addr(&full_bar[0]), empty0 = smem_addr(&empty_bar[0]);
        float max_sum = 0.0f;                                            // max |S| over fast-path units
        const bool count_overflow = P.agg_limit != 0x7FFFFFFF;          // int8 wire: count |S| > 127
        // Block-wise scales: the table entry of each of the thread's chunks and the scale of its first
        // segment are fetched one tile ahead, so that no load sits between two tiles.
        int32_t ent[UPT], ent_next[UPT];
        float pre_a[UPT], pre_c[UPT];
#pragma unroll
        for (int k = 0; k < UPT; ++k) {
            ent[k] = ent_next[k] = 0;
            pre_a[k] = pre_c[k] = 0.0f;
            if (BLOCKS) {
                const int64_t chunk0 = (int64_t)blockIdx.x * kTileUnits + c + (int64_t)k * NC - lane;
                if (chunk0 < PP.units) ent[k] = chunk_entry(bp, chunk0 + P.unit_base);
                pre_a[k] = __ldg(&bp.alpha[ent[k] & 0x7FFFFFFF]);
                pre_c[k] = __ldg(&bp.c[ent[k] & 0x7FFFFFFF]);
            }
        }
        for (int64_t tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
            const int64_t unit0 = tile * kTileUnits + c;
            float4 xo[UPT];
            PhiloxThreadPart tp[UPT];
            UnitAcc ua[UPT];
            float2 a01[UPT], a23[UPT];
            int s_lo[UPT], s_hi[UPT];
            float c_uni[UPT];
            bool active[UPT], half[UPT];
#pragma unroll
            for (int k = 0; k < UPT; ++k) {
                const int64_t unit = unit0 + (int64_t)k * NC;
                active[k] = unit < PP.units;
                half[k] = ((unit + P.unit_base) >> 9) & 1;
                xo[k] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (active[k]) xo[k] = load_f4<true>(P.x, unit);
                tp[k].n3 = tp[k].H = tp[k].m1 = 0;
                if (ROUND == INTSGD_ROUND_RANDOM || ROUND == INTSGD_ROUND_RANDOM_COMPARE)
                    tp[k] = philox_thread_part((uint32_t)(unit + P.unit_base), step, P.keys);
                if (ROUND == INTSGD_ROUND_RANDOM16 && !(kPairShared && k > 0))
                    tp[k] = philox_thread_part(pair_index((uint32_t)(unit + P.unit_base)), step, P.keys);
                ua[k].F01 = make_float2(0.f, 0.f);
                ua[k].F23 = make_float2(0.f, 0.f);
                ua[k].m = 0.0f;
                a01[k] = make_float2(alpha, alpha);
                a23[k] = a01[k];
                s_lo[k] = s_hi[k] = 0;
                c_uni[k] = 0.0f;
                if (BLOCKS) {
                    // the warp's 32 units form one chunk; chunks past the covered range are never committed
                    if (unit - lane < PP.units) chunk_segments_from(bp, ent[k], unit - lane + P.unit_base, s_lo[k], s_hi[k]);
                    if (active[k]) {
                        if (s_lo[k] == s_hi[k]) {   // the chunk lies in one segment: scale and decode factor are at hand
                            a01[k] = make_float2(pre_a[k], pre_a[k]);
                            a23[k] = a01[k];
                            c_uni[k] = pre_c[k];
                        } else {
                            const UnitScale us = unit_scale(bp, unit + P.unit_base, s_lo[k], s_hi[k]);
                            a01[k] = us.a01;
                            a23[k] = us.a23;
                        }
                    }
                    const int64_t next_chunk0 = unit - lane + (int64_t)gridDim.x * kTileUnits;
                    ent_next[k] = (next_chunk0 < PP.units) ? chunk_entry(bp, next_chunk0 + P.unit_base) : 0;
                }
            }
            for (int g0 = 0; g0 < n; g0 += G) {
                bool arrived = mbar_wait_at(full0 + 8u * s, phase);
                if (BLOCKS) arrived = __all_sync(0xFFFFFFFFu, arrived);   // keep the warp together for the shuffles below
                if (!arrived) { ok = false; break; }
                const unsigned char* src = smem + (size_t)s * G * kTileBytes;
                const int gw = (n - g0 < G) ? (n - g0) : G;
                if (active[UPT - 1] && gw == G) {
                    // every unit of this thread is inside the vector and the group is full: no checks
#pragma unroll
                    for (int w = 0; w < G; ++w) {
                        const uint4 e = s_tab[g0 + w];
                        uint4 pw = make_uint4(0, 0, 0, 0);
                        if (kPairShared) pw = philox_finish(tp[0], e, P.keys);   // one block for both units
#pragma unroll
                        for (int k = 0; k < UPT; ++k) {
                            const float4 gv = lds_unit<GRAD>(src + w * kTileBytes, c + k * NC);
                            consume_unit<ROUND>(gv, a01[k], a23[k], unit_draws<ROUND, kPairShared>(tp[k], e, pw, k, half[k], P.keys), ua[k]);
                        }
                    }
                } else {
                    for (int w = 0; w < gw; ++w) {
                        const uint4 e = s_tab[g0 + w];
                        uint4 pw = make_uint4(0, 0, 0, 0);
                        if (kPairShared) pw = philox_finish(tp[0], e, P.keys);
#pragma unroll
                        for (int k = 0; k < UPT; ++k) {
                            if (!active[k]) continue;
                            const float4 gv = lds_unit<GRAD>(src + w * kTileBytes, c + k * NC);
                            consume_unit<ROUND>(gv, a01[k], a23[k], unit_draws<ROUND, kPairShared>(tp[k], e, pw, k, half[k], P.keys), ua[k]);
                        }
                    }
                }
                mbar_arrive_at(empty0 + 8u * s);
                if (++s == NS) { s = 0; phase ^= 1u; }
            }
            if (!ok) break;
            float next_a[UPT], next_c[UPT];
#pragma unroll
            for (int k = 0; k < UPT; ++k) {
                next_a[k] = next_c[k] = 0.0f;
                if (BLOCKS) {   // the entries have arrived during the tile; these two loads overlap the epilogue
                    next_a[k] = __ldg(&bp.alpha[ent_next[k] & 0x7FFFFFFF]);
                    next_c[k] = __ldg(&bp.c[ent_next[k] & 0x7FFFFFFF]);
                }
            }
#pragma unroll
            for (int k = 0; k < UPT; ++k) {
                const int64_t unit = unit0 + (int64_t)k * NC;
                if (BLOCKS) {
                    if (unit - lane >= PP.units) continue;   // warp-uniform: this chunk does not exist
                    if (s_lo[k] != s_hi[k]) {
                        // the chunk crosses a segment boundary: per-coordinate scales, one partial per segment
                        double sq[4] = {0.0, 0.0, 0.0, 0.0};
                        int seg[4] = {-1, -1, -1, -1};
                        if (active[k]) {
                            const UnitScale us = unit_scale(bp, unit + P.unit_base, s_lo[k], s_hi[k]);
                            int4 S;
                            if (ua[k].m <= PP.fast_limit)
                                S = make_int4(__float2int_rn(ua[k].F01.x), __float2int_rn(ua[k].F01.y),
                                              __float2int_rn(ua[k].F23.x), __float2int_rn(ua[k].F23.y));
                            else
                                S = redo_unit<GRAD, ROUND>(P, unit, make_float4(us.a01.x, us.a01.y, us.a23.x, us.a23.y), step, s_cnt);
                            float4 xn;
                            xn.x = update_coord_sq(xo[k].x, __int2float_rn(S.x), us.c.x, sq[0]);
                            xn.y = update_coord_sq(xo[k].y, __int2float_rn(S.y), us.c.y, sq[1]);
                            xn.z = update_coord_sq(xo[k].z, __int2float_rn(S.z), us.c.z, sq[2]);
                            xn.w = update_coord_sq(xo[k].w, __int2float_rn(S.w), us.c.w, sq[3]);
                            store_f4<true>(P.x, unit, xn);
                            if (P.agg) store_i4<true>(P.agg, unit, S);
                            note_sum(S.x, P.agg_limit, acc); note_sum(S.y, P.agg_limit, acc);
                            note_sum(S.z, P.agg_limit, acc); note_sum(S.w, P.agg_limit, acc);
#pragma unroll
                            for (int e = 0; e < 4; ++e) seg[e] = us.seg[e];
                        }
                        chunk_commit(bp, unit - lane + P.unit_base, s_lo[k], s_hi[k], sq, seg);
                        continue;
                    }
                } else if (!active[k]) {
                    continue;
                }
                // One scale for the whole unit (always, or a chunk inside one segment).
                double unit_sq = 0.0;   // squared step of the unit: ((d0^2 + d1^2) + d2^2) + d3^2, products exact
                if (active[k]) {
                    const float cu = BLOCKS ? c_uni[k] : cdec;
                    int4 S;
                    float2 S01, S23;   // the sums as floats (exact on the fast path)
                    if (ua[k].m <= PP.fast_limit) {
                        S01 = ua[k].F01;
                        S23 = ua[k].F23;
                        S = make_int4(__float2int_rn(S01.x), __float2int_rn(S01.y), __float2int_rn(S23.x), __float2int_rn(S23.y));
                        max_sum = absmax3_nan(max_sum, S01.x, S01.y);
                        max_sum = absmax3_nan(max_sum, S23.x, S23.y);
                        if (count_overflow)
                            acc.overflow += (fabsf(S01.x) > 127.0f) + (fabsf(S01.y) > 127.0f) + (fabsf(S23.x) > 127.0f) +
                                            (fabsf(S23.y) > 127.0f);
                    } else {
                        S = redo_unit<GRAD, ROUND>(P, unit, make_float4(a01[k].x, a01[k].y, a23[k].x, a23[k].y), step, s_cnt);
                        S01 = make_float2(__int2float_rn(S.x), __int2float_rn(S.y));
                        S23 = make_float2(__int2float_rn(S.z), __int2float_rn(S.w));
                        note_sum(S.x, P.agg_limit, acc); note_sum(S.y, P.agg_limit, acc);
                        note_sum(S.z, P.agg_limit, acc); note_sum(S.w, P.agg_limit, acc);
                    }
                    // t = fl(c S); x_new = fl(x - t); dj = fl(x_new - x): packed, each rounded once
                    const float2 neg1 = make_float2(-1.0f, -1.0f), c2 = make_float2(cu, cu);
                    const float2 xo01 = make_float2(xo[k].x, xo[k].y), xo23 = make_float2(xo[k].z, xo[k].w);
                    const float2 xn01 = __ffma2_rn(__fmul2_rn(c2, S01), neg1, xo01);
                    const float2 xn23 = __ffma2_rn(__fmul2_rn(c2, S23), neg1, xo23);
                    const float2 d01 = __ffma2_rn(xo01, neg1, xn01), d23 = __ffma2_rn(xo23, neg1, xn23);
                    double* sink = BLOCKS ? &unit_sq : &acc.dx2;
                    *sink = __fma_rn((double)d01.x, (double)d01.x, *sink);
                    *sink = __fma_rn((double)d01.y, (double)d01.y, *sink);
                    *sink = __fma_rn((double)d23.x, (double)d23.x, *sink);
                    *sink = __fma_rn((double)d23.y, (double)d23.y, *sink);
                    store_f4<true>(P.x, unit, make_float4(xn01.x, xn01.y, xn23.x, xn23.y));
                    if (P.agg) store_i4<true>(P.agg, unit, S);
                }
                if (BLOCKS) {   // all 32 lanes of the warp: one partial per chunk, fixed order
                    const double t = warp_tree(unit_sq);
                    if (lane == 0) __stcg(&bp.chunk_sum[(unit - lane + P.unit_base) >> 5], t);
                }
            }
#pragma unroll
            for (int k = 0; k < UPT; ++k) {
                ent[k] = ent_next[k];
                pre_a[k] = next_a[k];
                pre_c[k] = next_c[k];
            }
        }
        {   // fold the float-tracked maximum of the fast-path sums (integers below 2^24) into the counters
            const int mf = __float2int_rn(max_sum);
            acc.max_abs = acc.max_abs > mf ? acc.max_abs : mf;
        }
        if (!ok) atomicExch(&s_fault, 1);

        // coordinates after the last pipelined unit (at most 7): element-wise, one thread
        if (blockIdx.x == 0 && c == 0 && ok) {
            const int64_t j0 = PP.units << 2;
            for (int64_t j = j0; j < P.d; ++j) {
                float aj = alpha, cj = cdec;
                if (BLOCKS) coord_scale(bp, j + (P.unit_base << 2), aj, cj);
                int S = 0;
                for (int i = 0; i < n; ++i) {
                    uint32_t word = 0;
                    if (ROUND != INTSGD_ROUND_NEAREST) {
                        const uint4 w4 = draw_unit<ROUND>((j >> 2) + P.unit_base, (uint32_t)i, step, P.keys);
                        const uint32_t wv[4] = {w4.x, w4.y, w4.z, w4.w};
                        word = wv[j & 3];
                    }
                    const float y = __fmul_rn(aj, grad_at<GRAD>(P.in[i], j));
                    S += round_checked<ROUND>(y, word, P.Lf, &s_cnt[i], &s_cnt[INTSGD_MAX_WORKERS]);
                }
                if (BLOCKS) {
                    double sqj;
                    P.x[j] = update_coord_sq(P.x[j], __int2float_rn(S), cj, sqj);
                    if (P.agg) P.agg[j] = S;
                    note_sum(S, P.agg_limit, acc);
                    bp.tail_sq[j + (P.unit_base << 2) - bp.covered_end] = sqj;
                } else {
                    apply_coord(P, j, S, cdec, acc);
                }
            }
        }
    }
    __syncthreads();
    // A wait gave up somewhere in this block (the producer's or a consumer's): before the block can retire,
    // the producer thread lets every copy it has issued land, whichever side noticed.
    if (threadIdx.x == NC && s_fault) drain_issued<NS>(full_bar, it);
    counters_flush(s_cnt, st);   // includes a __syncthreads()
    if (threadIdx.x == 0 && s_fault) atomicExch(&st->fault, 1);
    if (BLOCKS) flush_sum_counters(acc, st);   // the per-segment norms are finished by block_norm_kernel
    else grid_finalize(acc, st, P.partials, true, P.window_flags);
}

// Diagnostic: the rate at which an SM gets through rounds 3-10 of Philox4x32-10 when it does nothing else
// (register-only: no loads, no rounding, no stores).  Every thread runs two independent chains, as a consumer of
// the pipelined kernels does with its two units, each block's output seeding the next one's input.  The measured
// rate of 32x32->64-bit products is the ceiling of the random-rounding kernels' arithmetic.  EXTRA > 0 adds that
// many independent fp32 additions per Philox block (on eight accumulators of their own): the time they add shows
// whether other instructions hide behind the wide multiplies or queue up behind them.
template <int EXTRA>
__global__ void __launch_bounds__(512) philox_rate_kernel(PhiloxKeys keys, uint32_t blocks_per_chain, float step, uint32_t* sink) {
    PhiloxThreadPart a, b;
    a.n3 = threadIdx.x; a.H = blockIdx.x; a.m1 = 0x9E3779B9u;
    b.n3 = ~threadIdx.x; b.H = blockIdx.x * 7919u; b.m1 = 0xBB67AE85u;
    uint4 ea = make_uint4(1u, 2u, 3u, 0u), eb = make_uint4(4u, 5u, 6u, 0u);
    float f[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) f[i] = step * (float)(i + 1) + (float)threadIdx.x;
    for (uint32_t i = 0; i < blocks_per_chain; ++i) {
        const uint4 ra = philox_finish(a, ea, keys), rb = philox_finish(b, eb, keys);
        a.H = ra.x; a.m1 = ra.y; a.n3 = ra.z; ea.z = ra.w;
        b.H = rb.x; b.m1 = rb.y; b.n3 = rb.z; eb.z = rb.w;
#pragma unroll
        for (int e = 0; e < 2 * EXTRA; ++e) f[e & 7] = __fadd_rn(f[e & 7], step);
    }
    float fs = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) fs += f[i];
    // keeps the chains alive; the condition is all but impossible, so nothing is written in practice
    if ((a.H ^ b.H ^ a.n3 ^ b.n3) == 0x5EEDu && (a.m1 ^ b.m1 ^ ea.z ^ eb.z) == 0xFACEu && fs == 12345.0f) *sink = a.H;
}

// Diagnostic: the bounded wait on a barrier that nothing completes.  One thread polls `polls` times, then
// reports the expiry exactly as the step kernels do (sticky fault flag in the state) and returns.
__global__ void wait_expiry_kernel(DevState* st, uint32_t polls) {
    __shared__ uint64_t bar;
    if (threadIdx.x != 0) return;
    mbar_init(&bar, 1);
    mbar_fence_init();
    bool done = false;
    for (uint32_t i = 0; i < polls && !done; ++i) done = mbar_try_wait(&bar, 0u);   // mbar_wait with a short limit
    if (!done) atomicExch(&st->fault, 1);
}

}  // namespace intsgd
