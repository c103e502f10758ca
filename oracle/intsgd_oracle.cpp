// IntSGD reference oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
//
// A plain, slow, single-threaded CPU statement of what one IntSGD step computes
// (Mishchenko, Wang, Kovalev, Richtarik, "IntSGD: Adaptive Floatless Compression of
// Stochastic Gradients", Section 2, Eq. 2, Algorithm 1, Proposition 2; the appendix
// variants Algorithm 2 and Algorithm 3).  It exists so that the CUDA library can be
// compared with it bit for bit.  Only the tests, the smoke check and the CPU-baseline
// leg of the benchmark may call it; the product never does.  It shares no code, header,
// table or constant generator with the CUDA path and carries its own Philox4x32-10,
// written from the published description (Salmon, Moraes, Dror, Shaw, SC'11).
//
// Build: g++ -std=c++17 -O2 -ffp-contract=off -fno-fast-math -shared -fPIC
// (no FMA contraction: every fp32/fp64 operation below is a separately rounded IEEE op).
//
// Every function states the passage it follows.  Loops are worker x coordinate in the
// paper's order; there is no blocking, vectorisation or fusion.
//
// Pins (tests marked "not gpu"): Philox known-answer vectors; E[Int(t)] = t, |Int(t)-t| < 1,
// Var <= 1/4 (Lemma 1); floor(t + u) against exact rationals; the decode identity below Eq. 2; the hand-worked 4-element alpha and
// encode/aggregate/update examples; the closed form d*eta^2/alpha^2 = eta^2 eps^2 + 2 n r
// (proof of Proposition 2); Proposition 3 as the beta = eps = 0 special case; Algorithm 2 with
// one block equal to Algorithm 1; brute force against exact rational arithmetic on tiny
// inputs.  Nothing here is "parity unpinned".

#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>

namespace {

// ---------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11, Section 3.3 and Table 2): a 4x32-bit counter and a
// 2x32-bit key; ten rounds; each round multiplies counter words 0 and 2 by two fixed odd
// constants, keeps both halves of the 64-bit products and mixes in the other two words and
// the key; the key advances by two Weyl constants between rounds.
// ---------------------------------------------------------------------------------------
constexpr uint32_t kMul0 = 0xD2511F53u;   // multiplier applied to counter word 0
constexpr uint32_t kMul1 = 0xCD9E8D57u;   // multiplier applied to counter word 2
constexpr uint32_t kWeyl0 = 0x9E3779B9u;  // key word 0 increment (golden ratio)
constexpr uint32_t kWeyl1 = 0xBB67AE85u;  // key word 1 increment (sqrt(3) - 1)

void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        const uint64_t prod0 = (uint64_t)kMul0 * (uint64_t)c0;
        const uint64_t prod1 = (uint64_t)kMul1 * (uint64_t)c2;
        const uint32_t hi0 = (uint32_t)(prod0 >> 32), lo0 = (uint32_t)prod0;
        const uint32_t hi1 = (uint32_t)(prod1 >> 32), lo1 = (uint32_t)prod1;
        const uint32_t n0 = hi1 ^ c1 ^ k0;
        const uint32_t n1 = lo1;
        const uint32_t n2 = hi0 ^ c3 ^ k1;
        const uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += kWeyl0;
        k1 += kWeyl1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// The random word of coordinate j of worker `worker` at step `step`.
// Stream layout (the paper only says "with probability p_t"; the layout is this library's
// contract): key = (seed low, seed high); counter = (b low, b high, worker, step) with
// b = j / 4; coordinate j takes output word j mod 4.
uint32_t draw_word(uint64_t seed, uint32_t step, uint32_t worker, uint64_t j) {
    const uint64_t b = j >> 2;
    const uint32_t ctr[4] = {(uint32_t)b, (uint32_t)(b >> 32), worker, step};
    const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t out[4];
    philox4x32_10(ctr, key, out);
    return out[j & 3];
}

// Optional coarser stream ("16-bit draws", rounding mode 2): one Philox block serves 8 coordinates.
// Unit u = j / 4 is paired with the unit 512 places away: pair index P = ((u >> 10) << 9) | (u & 511),
// half h = (u >> 9) & 1; the block of counter (P low, P high, worker, step) gives words 2h and 2h + 1
// to the unit, and coordinate e = j mod 4 takes the low (e even) or high (e odd) 16 bits of word
// 2h + e / 2.  The uniform is that value times 2^-16.
float draw_uniform16(uint64_t seed, uint32_t step, uint32_t worker, uint64_t j) {
    const uint64_t u = j >> 2;
    const uint32_t e = (uint32_t)(j & 3);
    const uint64_t pair = ((u >> 10) << 9) | (u & 511);
    const uint32_t h = (uint32_t)((u >> 9) & 1);
    const uint32_t ctr[4] = {(uint32_t)pair, (uint32_t)(pair >> 32), worker, step};
    const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t out[4];
    philox4x32_10(ctr, key, out);
    const uint32_t word = out[2 * h + (e >> 1)];
    const uint32_t v = (e & 1) ? (word >> 16) : (word & 0xFFFFu);
    return (float)v * 1.52587890625e-5f;  // 2^-16
}

// Uniform in [0, 1) from a 32-bit word: w * 2^-32 truncated (toward zero) to fp32, i.e. the word
// with everything below its 24 leading significant bits cleared.  Always below 1 (at most
// 1 - 2^-24), and exact in fp32 by construction.
float uniform_from_word(uint32_t w) {
    int len = 0;
    while (len < 32 && (w >> len) != 0) ++len;           // number of significant bits of w
    if (len > 24) w &= ~((1u << (len - 24)) - 1u);       // keep the 24 leading ones
    return (float)w * 2.3283064365386963e-10f;           // 2^-32; at most 24 significant bits: exact
}

// 24-bit uniform in [0, 1) of rounding mode 3: the top 24 bits of the word times 2^-24; exact in fp32.
float uniform24_from_word(uint32_t w) {
    return (float)(w >> 8) * 5.9604644775390625e-8f;  // 2^-24
}

float widen_bf16(uint16_t h) {
    const uint32_t bits = (uint32_t)h << 16;
    float f;
    std::memcpy(&f, &bits, sizeof f);
    return f;
}

float load_grad(const void* grad, int grad_dtype, int64_t j) {
    if (grad_dtype == 1) return widen_bf16(((const uint16_t*)grad)[j]);
    return ((const float*)grad)[j];
}

// Largest fp32 value that does not exceed the integer limit L.
float limit_as_float(int64_t L) {
    float Lf = (float)L;
    if ((double)Lf > (double)L) Lf = std::nextafterf(Lf, 0.0f);
    return Lf;
}

// Int(t) of Section 2: floor(t) + 1 with probability t - floor(t), else floor(t); the floor
// is toward minus infinity.  Realised as floor(t + u) with u uniform on [0, 1): the sum reaches
// floor(t) + 1 exactly when u >= 1 - (t - floor(t)), an event of probability t - floor(t).
// The sum is never rounded: with k = floor(t), "t + u >= k + 1" is decided as u >= (k + 1) - t in
// fp64.  That difference lies in (0, 1] and is exact whenever |t| >= 2^-28 (its bits span at most
// 2^0 .. 2^-51) and for every negative t above -1 (it is -t); for 0 <= t < 2^-28 it is within
// 2^-28 of 1, above every possible u (u <= 1 - 2^-24), exactly as the unrounded difference is.
// Returned as an integer-valued float (no clipping here).
float int_round_random(float y, float u) {
    const float k = std::floor(y);
    const double need = ((double)k + 1.0) - (double)y;
    return ((double)u >= need) ? (float)((double)k + 1.0) : k;
}

// The same Int(t) drawn by comparison (rounding mode 3): floor(t) + 1 iff u < p with
// p = fl32(t - floor(t)), the fractional part as fp32 arithmetic gives it (rounded only for
// -1 < t < 0 with bits below 2^-24, where fl32(t + 1) can reach 1).
float int_round_random_compare(float y, float u) {
    const float f = std::floor(y);
    const float p = y - f;
    return f + ((u < p) ? 1.0f : 0.0f);
}

// Deterministic variant named in Section 5.1 ("IntSGD (Determ.)"): round to nearest, ties
// to even.
float int_round_nearest(float y) {
    return std::nearbyintf(y);  // default rounding mode: to nearest even
}

// Clipping (Section 5.1: local values are clipped so that the aggregate fits the wire type).
// Symmetric limit Lf; NaN maps to 0; the clipped flag is defined on y, not on the draw.
struct Rounded { int32_t q; bool clipped; bool nonfinite; };

Rounded round_and_clip(float y, float u, float Lf, int rounding) {
    Rounded r;
    float qf;
    if (rounding == 1) qf = int_round_nearest(y);
    else if (rounding == 3) qf = int_round_random_compare(y, u);
    else qf = int_round_random(y, u);
    r.clipped = !(std::fabs(y) <= Lf);
    r.nonfinite = !std::isfinite(y);
    if (y > Lf) qf = Lf;
    if (y < -Lf) qf = -Lf;
    if (y != y) qf = 0.0f;
    r.q = (int32_t)qf;
    return r;
}

}  // namespace

extern "C" {

// ---- random stream --------------------------------------------------------------------
void orc_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) {
    philox4x32_10(ctr, key, out);
}
uint32_t orc_draw_word(uint64_t seed, uint32_t step, uint32_t worker, uint64_t j) {
    return draw_word(seed, step, worker, j);
}
float orc_uniform_from_word(uint32_t w) { return uniform_from_word(w); }
float orc_draw_uniform16(uint64_t seed, uint32_t step, uint32_t worker, uint64_t j) {
    return draw_uniform16(seed, step, worker, j);
}

// ---- Int(t), Section 2 ------------------------------------------------------------------
int32_t orc_int_round(float y, float u) { return (int32_t)int_round_random(y, u); }
int32_t orc_int_round_nearest(float y) { return (int32_t)int_round_nearest(y); }
int32_t orc_int_round_compare(float y, float u) { return (int32_t)int_round_random_compare(y, u); }
float orc_uniform24_from_word(uint32_t w) { return uniform24_from_word(w); }
float orc_limit_as_float(int64_t L) { return limit_as_float(L); }

// ---- Algorithm 1, the two scalar lines: moving average r_k and scale alpha_k ------------
// r_k = beta r_{k-1} + (1 - beta) ||x^k - x^{k-1}||^2
// alpha_k = sqrt(d) / sqrt(2 n r_k / eta_k^2 + eps^2)            (Proposition 2)
// c_k = eta_k / (n alpha_k) with the fp32-rounded alpha_k, the factor of the decode line.
void orc_scale(int64_t d, int32_t n, double eta, double beta, double eps, double r_prev,
               double dx2, double* r_out, double* alpha64_out, float* alpha_out, float* c_out) {
    const double a = beta * r_prev;
    const double b = (1.0 - beta) * dx2;
    const double r = a + b;
    const double num = std::sqrt((double)d);
    const double two_n_r = (2.0 * (double)n) * r;
    const double eta2 = eta * eta;
    const double eps2 = eps * eps;
    const double inner = two_n_r / eta2 + eps2;
    const double alpha64 = num / std::sqrt(inner);
    const float alpha = (float)alpha64;
    const float c = (float)(eta / ((double)n * (double)alpha));
    *r_out = r;
    *alpha64_out = alpha64;
    *alpha_out = alpha;
    *c_out = c;
}

// Algorithm 2's form of the same rule for one block of size d_l out of d:
// alpha_{k,l} = eta_k sqrt(d_l) / sqrt(2 n r_{k,l} + eta_k^2 (d_l / d) eps^2).
void orc_scale_block(int64_t d, int64_t d_l, int32_t n, double eta, double beta, double eps,
                     double r_prev, double dx2, double* r_out, double* alpha64_out,
                     float* alpha_out, float* c_out) {
    const double a = beta * r_prev;
    const double b = (1.0 - beta) * dx2;
    const double r = a + b;
    const double num = eta * std::sqrt((double)d_l);
    const double two_n_r = (2.0 * (double)n) * r;
    const double share = (double)d_l / (double)d;
    const double guard = ((eta * eta) * share) * (eps * eps);
    const double alpha64 = num / std::sqrt(two_n_r + guard);
    const float alpha = (float)alpha64;
    const float c = (float)(eta / ((double)n * (double)alpha));
    *r_out = r;
    *alpha64_out = alpha64;
    *alpha_out = alpha;
    *c_out = c;
}

// ---- Algorithm 1, "scale and round the local gradient": Int(alpha_k g_i) ----------------
// One worker, coordinates [j0, j0 + count) of a vector whose element 0 is grad[0]
// (grad, payload and u_inject are indexed relative to j0; the random stream by j0 + t).
// grad_dtype 0 = fp32, 1 = bf16; payload_dtype 0 = int32, 1 = int8; rounding 0 = random (one Philox word per draw),
// 2 = random with the 16-bit draws of draw_uniform16, 3 = random by comparison with a 24-bit draw,
// 1 = nearest-even.  u_inject (nullable) replaces the Philox draw, for hand examples.
void orc_encode(const void* grad, int grad_dtype, int64_t j0, int64_t count, float alpha,
                int64_t L, int payload_dtype, int rounding, uint64_t seed, uint32_t step,
                uint32_t worker, const float* u_inject, void* payload, uint64_t* clip_count,
                uint64_t* nonfinite_count) {
    const float Lf = limit_as_float(L);
    for (int64_t t = 0; t < count; ++t) {
        const float g = load_grad(grad, grad_dtype, t);
        const float y = alpha * g;
        float u = 0.0f;
        if (rounding != 1) {
            if (u_inject) u = u_inject[t];
            else if (rounding == 2) u = draw_uniform16(seed, step, worker, (uint64_t)(j0 + t));
            else if (rounding == 3) u = uniform24_from_word(draw_word(seed, step, worker, (uint64_t)(j0 + t)));
            else u = uniform_from_word(draw_word(seed, step, worker, (uint64_t)(j0 + t)));
        }
        const Rounded r = round_and_clip(y, u, Lf, rounding);
        if (r.clipped) *clip_count += 1;
        if (r.nonfinite) *nonfinite_count += 1;
        if (payload_dtype == 1) ((int8_t*)payload)[t] = (int8_t)r.q;
        else ((int32_t*)payload)[t] = r.q;
    }
}

// ---- Algorithm 1, aggregate + estimator + update ------------------------------------------
// S_j = sum_i Int(alpha g_i)_j exactly; x_j <- x_j - c S_j (c = eta / (n alpha));
// dx2 = sum_j (x_new_j - x_j)^2 accumulated serially in fp64 for the next r_k.
void orc_aggregate(const void* const* payloads, int payload_dtype, int32_t n, int64_t count,
                   float c, float* x, int32_t* agg, double* dx2_out, uint64_t* agg_overflow,
                   int32_t* max_abs_agg) {
    double dx2 = 0.0;
    for (int64_t j = 0; j < count; ++j) {
        int32_t S = 0;
        for (int32_t i = 0; i < n; ++i) {
            S += (payload_dtype == 1) ? (int32_t)((const int8_t*)payloads[i])[j]
                                      : ((const int32_t*)payloads[i])[j];
        }
        const int32_t mag = S < 0 ? -S : S;
        if (payload_dtype == 1 && mag > 127) *agg_overflow += 1;
        if (mag > *max_abs_agg) *max_abs_agg = mag;
        if (agg) agg[j] = S;
        const float t = c * (float)S;
        const float x_old = x[j];
        const float x_new = x_old - t;
        const float dj = x_new - x_old;
        dx2 += (double)dj * (double)dj;
        x[j] = x_new;
    }
    *dx2_out = dx2;
}

// ---- Algorithm 1, Init line: the first, uncompressed step --------------------------------
// x^1 = x^0 - eta_0 (1/n) sum_i g_i^0, the sum taken left to right in fp32.
void orc_exact_step(const void* const* grads, int grad_dtype, int32_t n, int64_t count,
                    double eta, float* x, double* dx2_out) {
    const float c0 = (float)(eta / (double)n);
    double dx2 = 0.0;
    for (int64_t j = 0; j < count; ++j) {
        float m = load_grad(grads[0], grad_dtype, j);
        for (int32_t i = 1; i < n; ++i) m = m + load_grad(grads[i], grad_dtype, j);
        const float t = c0 * m;
        const float x_old = x[j];
        const float x_new = x_old - t;
        const float dj = x_new - x_old;
        dx2 += (double)dj * (double)dj;
        x[j] = x_new;
    }
    *dx2_out = dx2;
}

// ||x - x_prev||^2 from two stored iterates: fp32 difference, fp64 serial sum.
double orc_sqdiff(const float* x, const float* x_prev, int64_t count) {
    double s = 0.0;
    for (int64_t j = 0; j < count; ++j) {
        const float dj = x[j] - x_prev[j];
        s += (double)dj * (double)dj;
    }
    return s;
}

// ---- One whole compressed step over a coordinate window ---------------------------------
// The four loops of Algorithm 1 in order (encode every worker, sum, decode, update) with the
// scale (alpha, c) given.  scratch_payload: n * count int32 values of caller memory.
void orc_step_window(const void* const* grads, int grad_dtype, int32_t n, int64_t j0,
                     int64_t count, float alpha, float c, int64_t L, int payload_dtype,
                     int rounding, uint64_t seed, uint32_t step, float* x, int32_t* agg,
                     int32_t* scratch_payload, double* dx2_out, uint64_t* clip_count,
                     uint64_t* nonfinite_count, uint64_t* agg_overflow, int32_t* max_abs_agg) {
    for (int32_t i = 0; i < n; ++i) {
        int32_t* pay = scratch_payload + (int64_t)i * count;
        orc_encode(grads[i], grad_dtype, j0, count, alpha, L, 0, rounding, seed, step,
                   (uint32_t)i, nullptr, pay, &clip_count[i], nonfinite_count);
    }
    // Payload values already lie in [-L, L]; the int8 wire type only changes the overflow
    // rule of the aggregate, so the sum is taken over the int32 copies and the rule applied.
    double dx2 = 0.0;
    for (int64_t j = 0; j < count; ++j) {
        int32_t S = 0;
        for (int32_t i = 0; i < n; ++i) S += scratch_payload[(int64_t)i * count + j];
        const int32_t mag = S < 0 ? -S : S;
        if (payload_dtype == 1 && mag > 127) *agg_overflow += 1;
        if (mag > *max_abs_agg) *max_abs_agg = mag;
        if (agg) agg[j] = S;
        const float t = c * (float)S;
        const float x_old = x[j];
        const float x_new = x_old - t;
        const float dj = x_new - x_old;
        dx2 += (double)dj * (double)dj;
        x[j] = x_new;
    }
    *dx2_out = dx2;
}

// ---- IntDIANA (Algorithm 3): compress gradient differences ---------------------------------
// Worker i rounds alpha (g_i - h_i); its shift moves by the decoded message,
// h_i <- h_i + (1/alpha) Int(alpha (g_i - h_i)) (the proof of the IntDIANA theorem defines
// Q(g_i) = (1/alpha) Int(alpha (g_i - h_i)) for this line); the estimator and the new global
// shift are the same vector, g~ = h + (1/(n alpha)) sum_i Int(...); x <- x - eta g~.
// fp32 steps, each rounded once: v = g - h_i; y = alpha v; q = clip(Int(y));
// h_i = h_i + ainv * float(q); t = cn * float(S); gt = h + t; x = x - eta32 * gt.
// ainv = fp32(1/alpha), cn = fp32(1/(n alpha)), eta32 = fp32(eta) are given by the caller.
void orc_diana_step_window(const void* const* grads, int grad_dtype, int32_t n, int64_t j0, int64_t count,
                           float alpha, float ainv, float cn, float eta32, int64_t L, int payload_dtype,
                           int rounding, uint64_t seed, uint32_t step, float* const* h_local, float* h_global,
                           float* x, int32_t* agg, double* dx2_out, uint64_t* clip_count,
                           uint64_t* nonfinite_count, uint64_t* agg_overflow, int32_t* max_abs_agg) {
    const float Lf = limit_as_float(L);
    double dx2 = 0.0;
    for (int64_t t = 0; t < count; ++t) {
        int32_t S = 0;
        for (int32_t i = 0; i < n; ++i) {
            const float g = load_grad(grads[i], grad_dtype, t);
            const float v = g - h_local[i][t];
            const float y = alpha * v;
            float u = 0.0f;
            if (rounding == 2) u = draw_uniform16(seed, step, (uint32_t)i, (uint64_t)(j0 + t));
            else if (rounding == 3) u = uniform24_from_word(draw_word(seed, step, (uint32_t)i, (uint64_t)(j0 + t)));
            else if (rounding == 0) u = uniform_from_word(draw_word(seed, step, (uint32_t)i, (uint64_t)(j0 + t)));
            const Rounded r = round_and_clip(y, u, Lf, rounding);
            if (r.clipped) clip_count[i] += 1;
            if (r.nonfinite) *nonfinite_count += 1;
            const float dq = ainv * (float)r.q;
            h_local[i][t] = h_local[i][t] + dq;
            S += r.q;
        }
        const int32_t mag = S < 0 ? -S : S;
        if (payload_dtype == 1 && mag > 127) *agg_overflow += 1;
        if (mag > *max_abs_agg) *max_abs_agg = mag;
        if (agg) agg[t] = S;
        const float dec = cn * (float)S;
        const float gt = h_global[t] + dec;
        h_global[t] = gt;
        const float stepv = eta32 * gt;
        const float x_old = x[t];
        const float x_new = x_old - stepv;
        const float dj = x_new - x_old;
        dx2 += (double)dj * (double)dj;
        x[t] = x_new;
    }
    *dx2_out = dx2;
}

// ---- Heuristic IntSGD (Section 5.2, the SwitchML rule the paper compares against) ---------------
// alpha = (2^nb - 1) / (n 2^max_exp), where max_exp is the exponent of the largest absolute value
// in the package rounded up: the smallest integer e with max|g| <= 2^e.  Then |alpha g| <=
// (2^nb - 1) / n for every entry.  c = eta / (n alpha) as in Algorithm 1.  Returns 0, or -1 when
// max_abs is zero, negative or not finite (no scale exists).
int orc_heuristic_scale(float max_abs, int32_t n, int32_t nb, double eta, int32_t* max_exp_out, float* alpha_out,
                        float* c_out) {
    if (!(max_abs > 0.0f) || !std::isfinite(max_abs)) return -1;
    int e = 0;
    const float m = std::frexp(max_abs, &e);   // max_abs = m 2^e, m in [0.5, 1)
    const int max_exp = (m == 0.5f) ? e - 1 : e;
    const double levels = std::ldexp(1.0, nb) - 1.0;
    const double alpha64 = levels / ((double)n * std::ldexp(1.0, max_exp));
    const float alpha = (float)alpha64;
    *max_exp_out = max_exp;
    *alpha_out = alpha;
    *c_out = (float)(eta / ((double)n * (double)alpha));
    return 0;
}

}  // extern "C"
