// Block-wise scales (Algorithm 2 of the IntSGD paper, "adaptive block quantization"): the
// coordinates are partitioned into B contiguous blocks ("segments" below, to avoid confusion with
// thread blocks); each has its own moving average r_{k,l}, scale alpha_{k,l} and decode factor c_l.
//
// The vector kernels need two things from this header:
//  * the scale of every coordinate of a unit (UnitScale), looked up once per 32-unit chunk;
//  * the squared step length of every segment, summed in a fixed order: a chunk (32 consecutive
//    units = 128 coordinates, the work of one warp) that lies inside one segment stores one partial
//    in chunk_sum[]; a chunk that straddles segments adds one partial per segment to edge_sum[]
//    (a segment receives at most two such additions -- from the chunk holding its first and the one
//    holding its last coordinate -- so the order of the atomics cannot change the result); the two
//    block_norm kernels then add everything per segment in a fixed order.
#pragma once

#include "intsgd_device.cuh"

namespace intsgd {

constexpr int kChunkCoords = 128;   // 32 units of 4 coordinates: one warp's unit group
constexpr int kMaxTail = 8;

// Index l with offsets[l] <= j < offsets[l + 1].
__device__ __forceinline__ int seg_of(const BlockParams& bp, int64_t j) {
    int lo = 0, hi = bp.B;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(&bp.offsets[mid]) <= j) lo = mid;
        else hi = mid;
    }
    return lo;
}

// Scales of the four coordinates of one unit.
struct UnitScale {
    float2 a01, a23;   // alpha of coordinates 0,1 and 2,3
    float4 c;          // decode factors
    int seg[4];
};

// Segment range [s_lo, s_hi] of the chunk that starts at unit `chunk_unit0` (warp-uniform): one load
// from the table built when the partition was set; only a chunk that crosses a boundary searches.
__device__ __forceinline__ int32_t chunk_entry(const BlockParams& bp, int64_t chunk_unit0) {
    return __ldg(&bp.chunk_seg[chunk_unit0 >> 5]);
}
__device__ __forceinline__ void chunk_segments_from(const BlockParams& bp, int32_t entry, int64_t chunk_unit0, int& s_lo,
                                                    int& s_hi) {
    s_lo = entry & 0x7FFFFFFF;
    s_hi = s_lo;
    if (entry >= 0) return;
    int64_t j_hi = (chunk_unit0 << 2) + kChunkCoords;
    if (j_hi > bp.covered_end) j_hi = bp.covered_end;
    if (j_hi - 1 >= __ldg(&bp.offsets[s_lo + 1])) s_hi = seg_of(bp, j_hi - 1);
}
__device__ __forceinline__ void chunk_segments(const BlockParams& bp, int64_t chunk_unit0, int& s_lo, int& s_hi) {
    chunk_segments_from(bp, chunk_entry(bp, chunk_unit0), chunk_unit0, s_lo, s_hi);
}

// Table of chunk_segments: entry k describes coordinates [128 k, min(128 k + 128, d)).
__global__ void __launch_bounds__(256) chunk_table_kernel(const int64_t* offsets, int32_t B, int64_t d, int32_t* chunk_seg,
                                                          int64_t chunks) {
    const int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= chunks) return;
    BlockParams bp = {};
    bp.offsets = offsets;
    bp.B = B;
    const int64_t j_lo = k * kChunkCoords;
    int64_t j_hi = j_lo + kChunkCoords;
    if (j_hi > d) j_hi = d;
    const int s = seg_of(bp, j_lo);
    const bool crosses = (j_hi - 1) >= offsets[s + 1];
    chunk_seg[k] = s | (crosses ? (int32_t)0x80000000 : 0);
}

__device__ __forceinline__ UnitScale unit_scale(const BlockParams& bp, int64_t unit, int s_lo, int s_hi) {
    UnitScale u;
    if (s_lo == s_hi) {
        const float a = __ldg(&bp.alpha[s_lo]), c = __ldg(&bp.c[s_lo]);
        u.a01 = make_float2(a, a);
        u.a23 = u.a01;
        u.c = make_float4(c, c, c, c);
        u.seg[0] = u.seg[1] = u.seg[2] = u.seg[3] = s_lo;
        return u;
    }
    float a[4], c[4];
    int s = seg_of(bp, unit << 2);
    for (int e = 0; e < 4; ++e) {
        const int64_t j = (unit << 2) + e;
        while (s + 1 < bp.B && __ldg(&bp.offsets[s + 1]) <= j) ++s;
        u.seg[e] = s;
        a[e] = __ldg(&bp.alpha[s]);
        c[e] = __ldg(&bp.c[s]);
    }
    u.a01 = make_float2(a[0], a[1]);
    u.a23 = make_float2(a[2], a[3]);
    u.c = make_float4(c[0], c[1], c[2], c[3]);
    return u;
}

// Commit the squared steps of one chunk.  Must be called by all 32 lanes of a warp whose lanes own
// consecutive units starting at chunk_unit0; lanes without a unit pass zeros.
__device__ __forceinline__ void chunk_commit(const BlockParams& bp, int64_t chunk_unit0, int s_lo, int s_hi,
                                             const double sq[4], const int seg[4]) {
    const int lane = threadIdx.x & 31;
    if (s_lo == s_hi) {
        const double t = warp_tree(((sq[0] + sq[1]) + sq[2]) + sq[3]);
        if (lane == 0) __stcg(&bp.chunk_sum[chunk_unit0 >> 5], t);
        return;
    }
    for (int l = s_lo; l <= s_hi; ++l) {
        double v = 0.0;
#pragma unroll
        for (int e = 0; e < 4; ++e)
            if (seg[e] == l) v += sq[e];
        const double t = warp_tree(v);
        if (lane == 0) atomicAdd(&bp.edge_sum[l], t);
    }
}

// Squared fp32 step of one coordinate (the quantity Algorithm 2 sums per block).
__device__ __forceinline__ float update_coord_sq(float x_old, float S_as_float, float c, double& sq) {
    const float t = __fmul_rn(c, S_as_float);
    const float x_new = __fsub_rn(x_old, t);
    const float dj = __fsub_rn(x_new, x_old);
    sq = (double)dj * (double)dj;   // exact
    return x_new;
}

// ---------------------------------------------------------------------------------------------
// Per-segment state and the two small kernels of a block-wise step.
// ---------------------------------------------------------------------------------------------
struct BlockState {
    const int64_t* offsets;
    double* r;          // B: moving averages
    double* r_new;      // B: scratch of the scale kernel
    double* dx2;        // B: squared step lengths left by the last step
    float* alpha;       // B
    float* c;           // B
    double* chunk_sum;
    const int32_t* chunk_seg;
    double* edge_sum;
    double* tail_sq;
    int32_t B;
};

// Algorithm 2, moving averages and scales, one launch of a single thread block:
// r_l = beta r_l + (1 - beta) dx2_l;  alpha_l = eta sqrt(d_l) / sqrt(2 n r_l + eta^2 (d_l / d) eps^2);
// c_l = eta / (n alpha_l).  All segments or none: if any scale is not finite and positive the state
// keeps its old r and the step's vector kernels do nothing.
__global__ void __launch_bounds__(1024) scale_blocks_kernel(DevState* st, BlockState bs, double d_total, double two_n,
                                                            double n_as_double, double eta, double beta, double eps,
                                                            int32_t n) {
    asm volatile("griddepcontrol.launch_dependents;");   // see scale_kernel
    asm volatile("griddepcontrol.wait;" ::: "memory");   // the per-block norms of the step in front
    int bad = 0;
    for (int l = threadIdx.x; l < bs.B; l += blockDim.x) {
        const double dl = (double)(bs.offsets[l + 1] - bs.offsets[l]);
        const double a = __dmul_rn(beta, bs.r[l]);
        const double b = __dmul_rn(__dsub_rn(1.0, beta), bs.dx2[l]);
        const double r = __dadd_rn(a, b);
        const double num = __dmul_rn(eta, __dsqrt_rn(dl));
        const double two_n_r = __dmul_rn(two_n, r);
        const double share = __ddiv_rn(dl, d_total);
        const double guard = __dmul_rn(__dmul_rn(__dmul_rn(eta, eta), share), __dmul_rn(eps, eps));
        const double alpha64 = __ddiv_rn(num, __dsqrt_rn(__dadd_rn(two_n_r, guard)));
        const float alpha = __double2float_rn(alpha64);
        const float c = __double2float_rn(__ddiv_rn(eta, __dmul_rn(n_as_double, (double)alpha)));
        const bool ok = (alpha > 0.0f) && (alpha <= 3.402823466e+38f) && (c > 0.0f) && (c <= 3.402823466e+38f);
        bad |= ok ? 0 : 1;
        bs.r_new[l] = r;
        bs.alpha[l] = alpha;
        bs.c[l] = c;
        bs.edge_sum[l] = 0.0;
    }
    const int any_bad = __syncthreads_or(bad);
    if (!any_bad)
        for (int l = threadIdx.x; l < bs.B; l += blockDim.x) bs.r[l] = bs.r_new[l];
    if (threadIdx.x == 0) {
        for (int i = 0; i < n; ++i) st->clip_count[i] = 0;
        st->nonfinite = 0;
        st->agg_overflow = 0;
        st->max_abs_agg = 0;
        st->ticket = 0;
        st->status = any_bad ? INTSGD_ERR_SCALE_NONFINITE : INTSGD_OK;
        if (!any_bad) {
            st->alpha = bs.alpha[0];
            st->c = bs.c[0];
        }
    }
}

// Reduction plan for the per-segment norms, built on the host when the partition is set: the chunk
// partials that lie inside a segment are cut into slices of at most kSliceChunks chunks, so that long
// segments are summed by many thread blocks.  Slice w covers chunks [k0[w], k1[w]) of one segment;
// segment l owns slices [seg_slice[l], seg_slice[l + 1]).
constexpr int kSliceChunks = 1024;
struct NormPlan {
    const int64_t* k0;         // device, num_slices
    const int64_t* k1;         // device, num_slices
    const int32_t* seg_slice;  // device, B + 1
    double* slice_sum;         // device, num_slices
    int64_t covered_end;
    int32_t num_slices;
};

// Pass 1: one thread block per slice, fixed summation order.
__global__ void __launch_bounds__(256) block_norm_slices_kernel(const DevState* st, BlockState bs, NormPlan plan,
                                                                int32_t check_status) {
    __shared__ double s_warp[32];
    // launched as a programmatic dependent of the step's vector kernel: may be resident early, reads nothing before
    // that kernel has completed; its own dependent (pass 2) may be scheduled at once
    asm volatile("griddepcontrol.launch_dependents;");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (check_status && st->status != INTSGD_OK) return;
    const int w = blockIdx.x;
    double v = 0.0;
    for (int64_t k = plan.k0[w] + threadIdx.x; k < plan.k1[w]; k += blockDim.x) v += __ldcg(&bs.chunk_sum[k]);
    const double t = block_tree(v, s_warp);
    if (threadIdx.x == 0) plan.slice_sum[w] = t;
}

// Pass 2: thread block l adds the slices of segment l in order, then the (at most two) edge partials
// and the segment's tail coordinates.  The block that finishes last adds the B results into
// state.dx2 and (after a step, not after intsgd_sqdiff) advances the step counter.
__global__ void __launch_bounds__(128) block_norm_kernel(DevState* st, BlockState bs, NormPlan plan, int64_t d,
                                                         int32_t check_status, int32_t advance_step) {
    __shared__ double s_warp[32];
    __shared__ bool s_last;
    asm volatile("griddepcontrol.launch_dependents;");   // the next step's scale kernel; it waits for this grid
    asm volatile("griddepcontrol.wait;" ::: "memory");   // pass 1 (or the vector kernel) has completed
    if (check_status && st->status != INTSGD_OK) return;
    const int l = blockIdx.x;
    double v = 0.0;
    for (int w = plan.seg_slice[l] + threadIdx.x; w < plan.seg_slice[l + 1]; w += blockDim.x) v += __ldcg(&plan.slice_sum[w]);
    double total = block_tree(v, s_warp);
    if (threadIdx.x == 0) {
        total += __ldcg(&bs.edge_sum[l]);
        for (int64_t j = plan.covered_end; j < d; ++j)
            if (j >= bs.offsets[l] && j < bs.offsets[l + 1]) total += __ldcg(&bs.tail_sq[j - plan.covered_end]);
        bs.dx2[l] = total;
        __threadfence();
        s_last = (atomicAdd(&st->ticket, 1u) == gridDim.x - 1);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    double w2 = 0.0;
    for (int m = threadIdx.x; m < bs.B; m += blockDim.x) w2 += __ldcg(&bs.dx2[m]);
    const double sum = block_tree(w2, s_warp);
    if (threadIdx.x == 0) {
        st->dx2 = sum;
        if (advance_step) st->step += 1;
        st->ticket = 0;
    }
}

// ---------------------------------------------------------------------------------------------
// Direct (grid-stride) kernels with block-wise scales.  A warp owns 32 consecutive units per
// iteration (one chunk); the loop condition is warp-uniform so that every lane reaches the shuffles.
// ---------------------------------------------------------------------------------------------
template <int ROUND>
__device__ __forceinline__ int4 round_unit_scaled(float4 g, float2 a01, float2 a23, uint4 w, float Lf, cnt_t* clip_slot,
                                                  cnt_t* nonfinite_slot) {
    const float y0 = __fmul_rn(a01.x, g.x), y1 = __fmul_rn(a01.y, g.y);
    const float y2 = __fmul_rn(a23.x, g.z), y3 = __fmul_rn(a23.y, g.w);
    const bool in_range = (fabsf(y0) <= Lf) & (fabsf(y1) <= Lf) & (fabsf(y2) <= Lf) & (fabsf(y3) <= Lf);
    int4 q;
    if (in_range) {
        q.x = round_in_range<ROUND>(y0, w.x);
        q.y = round_in_range<ROUND>(y1, w.y);
        q.z = round_in_range<ROUND>(y2, w.z);
        q.w = round_in_range<ROUND>(y3, w.w);
    } else {
        q = round_unit_checked<ROUND>(y0, y1, y2, y3, w, Lf, clip_slot, nonfinite_slot);
    }
    return q;
}

// Scale and decode factor of one coordinate (tails only).
__device__ __forceinline__ void coord_scale(const BlockParams& bp, int64_t j, float& alpha, float& c) {
    const int s = seg_of(bp, j);
    alpha = __ldg(&bp.alpha[s]);
    c = __ldg(&bp.c[s]);
}

template <int GRAD, bool ALIGNED, int ROUND>
__global__ void __launch_bounds__(512) fused_step_blocks_kernel(const __grid_constant__ VecParams P) {
    __shared__ cnt_t s_cnt[INTSGD_MAX_WORKERS + 1];
    DevState* st = P.st;
    if (st->status != INTSGD_OK) return;
    counters_init(s_cnt);
    const BlockParams& bp = P.bp;
    const uint32_t step = st->step;
    const int n = P.n;
    const int lane = threadIdx.x & 31;
    cnt_t* nonf_slot = &s_cnt[INTSGD_MAX_WORKERS];
    ThreadAcc acc = {0.0, 0, 0u};

    const int64_t full = P.d >> 2;   // == bp.covered_end / 4
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    // A launch may cover a window of the vector: `unit` indexes the launch's pointers, `unit + P.unit_base` the
    // whole vector (partition tables, chunk partials, random stream).
    for (int64_t base = (int64_t)blockIdx.x * blockDim.x + (threadIdx.x - lane); base < full; base += stride) {
        const int64_t unit = base + lane, gunit = unit + P.unit_base;
        const bool active = unit < full;
        int s_lo, s_hi;
        chunk_segments(bp, base + P.unit_base, s_lo, s_hi);
        double sq[4] = {0.0, 0.0, 0.0, 0.0};
        int seg[4] = {-1, -1, -1, -1};
        if (active) {
            const UnitScale us = unit_scale(bp, gunit, s_lo, s_hi);
            int4 S = make_int4(0, 0, 0, 0);
            PhiloxThreadPart tp = {0u, 0u, 0u};   // the unit's half of Philox rounds 1-2 serves all n workers
            if (ROUND != INTSGD_ROUND_NEAREST) tp = draw_thread_part<ROUND>(gunit, step, P.keys);
#pragma unroll 4
            for (int i = 0; i < n; ++i) {
                const float4 gv = load_grad4<GRAD, ALIGNED>(P.in[i], unit);
                uint4 w = make_uint4(0, 0, 0, 0);
                if (ROUND != INTSGD_ROUND_NEAREST) w = draw_unit_folded<ROUND>(tp, gunit, P.tab.e[i], (uint32_t)i, step, P.keys);
                const int4 q = round_unit_scaled<ROUND>(gv, us.a01, us.a23, w, P.Lf, &s_cnt[i], nonf_slot);
                S.x += q.x; S.y += q.y; S.z += q.z; S.w += q.w;
            }
            const float4 xo = load_f4<ALIGNED>(P.x, unit);
            float4 xn;
            xn.x = update_coord_sq(xo.x, __int2float_rn(S.x), us.c.x, sq[0]);
            xn.y = update_coord_sq(xo.y, __int2float_rn(S.y), us.c.y, sq[1]);
            xn.z = update_coord_sq(xo.z, __int2float_rn(S.z), us.c.z, sq[2]);
            xn.w = update_coord_sq(xo.w, __int2float_rn(S.w), us.c.w, sq[3]);
            store_f4<ALIGNED>(P.x, unit, xn);
            if (P.agg) store_i4<ALIGNED>(P.agg, unit, S);
            note_sum(S.x, P.agg_limit, acc); note_sum(S.y, P.agg_limit, acc);
            note_sum(S.z, P.agg_limit, acc); note_sum(S.w, P.agg_limit, acc);
#pragma unroll
            for (int e = 0; e < 4; ++e) seg[e] = us.seg[e];
        }
        chunk_commit(bp, base + P.unit_base, s_lo, s_hi, sq, seg);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        for (int64_t j = full << 2; j < P.d; ++j) {
            const int64_t gj = j + (P.unit_base << 2);
            float alpha, c;
            coord_scale(bp, gj, alpha, c);
            int S = 0;
            for (int i = 0; i < n; ++i) {
                uint32_t word = 0;
                if (ROUND != INTSGD_ROUND_NEAREST) {
                    const uint4 w4 = draw_unit<ROUND>(gj >> 2, (uint32_t)i, step, P.keys);
                    const uint32_t wv[4] = {w4.x, w4.y, w4.z, w4.w};
                    word = wv[j & 3];
                }
                const float y = __fmul_rn(alpha, grad_at<GRAD>(P.in[i], j));
                S += round_checked<ROUND>(y, word, P.Lf, &s_cnt[i], nonf_slot);
            }
            double sqj;
            P.x[j] = update_coord_sq(P.x[j], __int2float_rn(S), c, sqj);
            if (P.agg) P.agg[j] = S;
            note_sum(S, P.agg_limit, acc);
            bp.tail_sq[gj - bp.covered_end] = sqj;
        }
    }
    counters_flush(s_cnt, st);
    flush_sum_counters(acc, st);
}

// Exact first step with per-segment squared step lengths (Algorithm 2's Input line: x^1 is the
// uncompressed mean step; its block norms start the moving averages).
template <int GRAD, bool ALIGNED>
__global__ void __launch_bounds__(512) exact_step_blocks_kernel(const __grid_constant__ VecParams P) {
    const BlockParams& bp = P.bp;
    const int n = P.n;
    const float c0 = P.c_exact;
    const int lane = threadIdx.x & 31;
    const int64_t full = P.d >> 2;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t base = (int64_t)blockIdx.x * blockDim.x + (threadIdx.x - lane); base < full; base += stride) {
        const int64_t unit = base + lane;
        const bool active = unit < full;
        int s_lo, s_hi;
        chunk_segments(bp, base + P.unit_base, s_lo, s_hi);
        double sq[4] = {0.0, 0.0, 0.0, 0.0};
        int seg[4] = {-1, -1, -1, -1};
        if (active) {
            float4 m = load_grad4<GRAD, ALIGNED>(P.in[0], unit);
#pragma unroll 4
            for (int i = 1; i < n; ++i) {
                const float4 gv = load_grad4<GRAD, ALIGNED>(P.in[i], unit);
                m.x = __fadd_rn(m.x, gv.x); m.y = __fadd_rn(m.y, gv.y);
                m.z = __fadd_rn(m.z, gv.z); m.w = __fadd_rn(m.w, gv.w);
            }
            const float4 xo = load_f4<ALIGNED>(P.x, unit);
            float4 xn;
            xn.x = update_coord_sq(xo.x, m.x, c0, sq[0]);
            xn.y = update_coord_sq(xo.y, m.y, c0, sq[1]);
            xn.z = update_coord_sq(xo.z, m.z, c0, sq[2]);
            xn.w = update_coord_sq(xo.w, m.w, c0, sq[3]);
            store_f4<ALIGNED>(P.x, unit, xn);
            if (s_lo == s_hi) {
                seg[0] = seg[1] = seg[2] = seg[3] = s_lo;
            } else {
                const UnitScale us = unit_scale(bp, unit + P.unit_base, s_lo, s_hi);
#pragma unroll
                for (int e = 0; e < 4; ++e) seg[e] = us.seg[e];
            }
        }
        chunk_commit(bp, base + P.unit_base, s_lo, s_hi, sq, seg);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        for (int64_t j = full << 2; j < P.d; ++j) {
            float m = grad_at<GRAD>(P.in[0], j);
            for (int i = 1; i < n; ++i) m = __fadd_rn(m, grad_at<GRAD>(P.in[i], j));
            double sqj;
            P.x[j] = update_coord_sq(P.x[j], m, c0, sqj);
            bp.tail_sq[j + (P.unit_base << 2) - bp.covered_end] = sqj;
        }
    }
}

// Per-segment ||x - x_prev||^2 for a caller that holds two iterates (the block-wise form of intsgd_sqdiff):
// fp32 differences, exact squares, the same chunk partials and fixed-order sums as a step.
template <bool ALIGNED>
__global__ void __launch_bounds__(512) sqdiff_blocks_kernel(const __grid_constant__ VecParams P) {
    const BlockParams& bp = P.bp;
    const int lane = threadIdx.x & 31;
    const int64_t full = P.d >> 2;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t base = (int64_t)blockIdx.x * blockDim.x + (threadIdx.x - lane); base < full; base += stride) {
        const int64_t unit = base + lane;
        int s_lo, s_hi;
        chunk_segments(bp, base, s_lo, s_hi);
        double sq[4] = {0.0, 0.0, 0.0, 0.0};
        int seg[4] = {-1, -1, -1, -1};
        if (unit < full) {
            const float4 a = load_f4<ALIGNED>(P.x, unit), b = load_f4<ALIGNED>(P.x_prev, unit);
            const float d0 = __fsub_rn(a.x, b.x), d1 = __fsub_rn(a.y, b.y), d2 = __fsub_rn(a.z, b.z), d3 = __fsub_rn(a.w, b.w);
            sq[0] = (double)d0 * (double)d0; sq[1] = (double)d1 * (double)d1;
            sq[2] = (double)d2 * (double)d2; sq[3] = (double)d3 * (double)d3;
            if (s_lo == s_hi) {
                seg[0] = seg[1] = seg[2] = seg[3] = s_lo;
            } else {
                const UnitScale us = unit_scale(bp, unit, s_lo, s_hi);
#pragma unroll
                for (int e = 0; e < 4; ++e) seg[e] = us.seg[e];
            }
        }
        chunk_commit(bp, base, s_lo, s_hi, sq, seg);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        for (int64_t j = full << 2; j < P.d; ++j) {
            const float dj = __fsub_rn(P.x[j], P.x_prev[j]);
            bp.tail_sq[j - bp.covered_end] = (double)dj * (double)dj;
        }
    }
}

// Encode with block-wise scales, direct form (one worker per blockIdx.y): payload = clip(Int(alpha_l g)) with
// the scale of the block each coordinate lies in (Algorithm 2's Int(alpha_{k,l} o g)).
template <int GRAD, int PAY, bool ALIGNED, int ROUND>
__global__ void __launch_bounds__(512) encode_blocks_kernel(const __grid_constant__ VecParams P) {
    __shared__ cnt_t s_cnt[INTSGD_MAX_WORKERS + 1];
    DevState* st = P.st;
    if (st->status != INTSGD_OK) return;
    counters_init(s_cnt);
    const BlockParams& bp = P.bp;
    const uint32_t step = st->step;
    const int slot = blockIdx.y;
    const uint32_t worker = (uint32_t)(P.worker_base + slot);
    const void* g = P.in[slot];
    void* out = P.out[slot];
    cnt_t* clip_slot = &s_cnt[worker];
    cnt_t* nonf_slot = &s_cnt[INTSGD_MAX_WORKERS];
    const uint4 e = P.tab.e[worker];
    const int64_t full = P.d >> 2;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t unit = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; unit < full; unit += stride) {
        int s_lo, s_hi;
        chunk_segments(bp, unit & ~(int64_t)31, s_lo, s_hi);
        const UnitScale us = unit_scale(bp, unit, s_lo, s_hi);
        const float4 gv = load_grad4<GRAD, ALIGNED>(g, unit);
        uint4 w = make_uint4(0, 0, 0, 0);
        if (ROUND != INTSGD_ROUND_NEAREST)
            w = draw_unit_folded<ROUND>(draw_thread_part<ROUND>(unit, step, P.keys), unit, e, worker, step, P.keys);
        store_payload4<PAY>(out, unit, round_unit_scaled<ROUND>(gv, us.a01, us.a23, w, P.Lf, clip_slot, nonf_slot), ALIGNED);
    }
    const int tail = (int)(P.d & 3);
    if (tail && blockIdx.x == 0 && threadIdx.x == 0) {
        uint4 w = make_uint4(0, 0, 0, 0);
        if (ROUND != INTSGD_ROUND_NEAREST) w = draw_unit<ROUND>(full, worker, step, P.keys);
        const uint32_t wv[4] = {w.x, w.y, w.z, w.w};
        for (int t = 0; t < tail; ++t) {
            const int64_t j = 4 * full + t;
            float alpha, c;
            coord_scale(bp, j, alpha, c);
            const int q = round_checked<ROUND>(__fmul_rn(alpha, grad_at<GRAD>(g, j)), wv[t], P.Lf, clip_slot, nonf_slot);
            if (PAY == INTSGD_PAYLOAD_I32) ((int32_t*)out)[j] = q;
            else ((int8_t*)out)[j] = (int8_t)q;
        }
    }
    counters_flush(s_cnt, st);
}

// Aggregate + decode + update with block-wise decode factors and per-segment squared step lengths (Algorithm 2:
// every block is decoded with its own eta / (n alpha_{k,l})).  One unit per thread and iteration for both wire
// types, so that a warp's 32 units are one chunk of the norm reduction.
template <int PAY, bool ALIGNED>
__global__ void __launch_bounds__(512) aggregate_blocks_kernel(const __grid_constant__ VecParams P) {
    DevState* st = P.st;
    if (st->status != INTSGD_OK) return;
    const BlockParams& bp = P.bp;
    const int n = P.n;
    const int lane = threadIdx.x & 31;
    ThreadAcc acc = {0.0, 0, 0u};
    const int64_t full = P.d >> 2;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t base = (int64_t)blockIdx.x * blockDim.x + (threadIdx.x - lane); base < full; base += stride) {
        const int64_t unit = base + lane;
        int s_lo, s_hi;
        chunk_segments(bp, base, s_lo, s_hi);
        double sq[4] = {0.0, 0.0, 0.0, 0.0};
        int seg[4] = {-1, -1, -1, -1};
        if (unit < full) {
            const UnitScale us = unit_scale(bp, unit, s_lo, s_hi);
            int4 S = make_int4(0, 0, 0, 0);
#pragma unroll 4
            for (int i = 0; i < n; ++i) {
                if (PAY == INTSGD_PAYLOAD_I32) {
                    const int4 q = load_i4<ALIGNED>((const int32_t*)P.in[i], unit);
                    S.x += q.x; S.y += q.y; S.z += q.z; S.w += q.w;
                } else if (ALIGNED) {
                    add_bytes(S, __ldcs((const uint32_t*)P.in[i] + unit));
                } else {
                    const int8_t* p = (const int8_t*)P.in[i] + 4 * unit;
                    S.x += (int)p[0]; S.y += (int)p[1]; S.z += (int)p[2]; S.w += (int)p[3];
                }
            }
            const float4 xo = load_f4<ALIGNED>(P.x, unit);
            float4 xn;
            xn.x = update_coord_sq(xo.x, __int2float_rn(S.x), us.c.x, sq[0]);
            xn.y = update_coord_sq(xo.y, __int2float_rn(S.y), us.c.y, sq[1]);
            xn.z = update_coord_sq(xo.z, __int2float_rn(S.z), us.c.z, sq[2]);
            xn.w = update_coord_sq(xo.w, __int2float_rn(S.w), us.c.w, sq[3]);
            store_f4<ALIGNED>(P.x, unit, xn);
            if (P.agg) store_i4<ALIGNED>(P.agg, unit, S);
            note_sum(S.x, P.agg_limit, acc); note_sum(S.y, P.agg_limit, acc);
            note_sum(S.z, P.agg_limit, acc); note_sum(S.w, P.agg_limit, acc);
#pragma unroll
            for (int e = 0; e < 4; ++e) seg[e] = us.seg[e];
        }
        chunk_commit(bp, base, s_lo, s_hi, sq, seg);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        for (int64_t j = full << 2; j < P.d; ++j) {
            float alpha, c;
            coord_scale(bp, j, alpha, c);
            int S = 0;
            for (int i = 0; i < n; ++i)
                S += (PAY == INTSGD_PAYLOAD_I32) ? ((const int32_t*)P.in[i])[j] : (int)((const int8_t*)P.in[i])[j];
            double sqj;
            P.x[j] = update_coord_sq(P.x[j], __int2float_rn(S), c, sqj);
            if (P.agg) P.agg[j] = S;
            note_sum(S, P.agg_limit, acc);
            bp.tail_sq[j - bp.covered_end] = sqj;
        }
    }
    flush_sum_counters(acc, st);
}

}  // namespace intsgd
