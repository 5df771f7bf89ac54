// Fixed-point arithmetic of the integer LSTM, shared by all CUDA kernels of this library.
//
// Everything here is exact integer arithmetic; where a floating-point unit is used it only
// produces an estimate that an integer remainder check then corrects, so results never depend
// on floating-point rounding.  Functions are __host__ __device__ so that the host test harness
// (csrc/host_check/qmath_host.cpp) can sweep them on a CPU against fp64 closed forms and exact
// rational arithmetic.
//
// Rounding rule everywhere: to nearest, ties away from zero.
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define QL_HD __host__ __device__ __forceinline__
#else
#define QL_HD inline
#endif

namespace ql {

struct Scale { int32_t mult; int32_t shift; };   // real = mult * 2^(shift-31)

QL_HD int32_t sat32(int64_t v) { return v > INT32_MAX ? INT32_MAX : (v < INT32_MIN ? INT32_MIN : (int32_t)v); }
QL_HD int32_t sat16(int32_t v) { return v > 32767 ? 32767 : (v < -32768 ? -32768 : v); }
QL_HD int32_t sat8(int32_t v) { return v > 127 ? 127 : (v < -128 ? -128 : v); }

// "rescale" (Section 3.2.4): saturating left shift, rounding doubling high multiply, rounding right shift.
// The multiplier is 0 or in [2^30, 2^31), so the high multiply cannot overflow.
QL_HD int32_t mbqm(int32_t x, Scale s)
{
    int left = s.shift > 0 ? s.shift : 0;
    int right = s.shift < 0 ? -s.shift : 0;
    int64_t xl = (int64_t)x << left;
    int32_t xs = sat32(xl);
    int64_t p = (int64_t)xs * (int64_t)s.mult;
    uint64_t ap = p < 0 ? (uint64_t)0 - (uint64_t)p : (uint64_t)p;
    uint64_t q = (ap + ((uint64_t)1 << 30)) >> 31;
    if (right) q = (q + ((uint64_t)1 << (right - 1))) >> right;
    return p < 0 ? -(int32_t)q : (int32_t)q;
}

// Rarely taken paths of the hot loops (a scale with a left shift; a layer-norm quotient beyond 16 bits), out of line
// on the device so that they stay out of those loops' register budget.
#if defined(__CUDACC__)
static __device__ __noinline__ int32_t mbqm_rare(int32_t x, Scale s) { return mbqm(x, s); }
static __device__ __noinline__ uint64_t div_rare(uint64_t n, uint32_t d) { return n / d; }
#endif
QL_HD int32_t mbqm_cold(int32_t x, Scale s)
{
#if defined(__CUDA_ARCH__)
    return mbqm_rare(x, s);
#else
    return mbqm(x, s);
#endif
}

// The same rescale for shift <= 0 with its constants pre-computed, in 32-bit registers:
//   round(round(|x| M / 2^31) / 2^R) = floor((2 |x| M + 2^31 + [R>0] 2^(31+R)) / 2^(32+R))
// (nested floors collapse), i.e. the high word of one 32x32+64 multiply-add, shifted right by R.
struct FastScale { uint32_t m2, add_hi; int32_t rshift; };

QL_HD FastScale make_fast_scale(Scale s)
{
    int R = s.shift < 0 ? -s.shift : 0;
    FastScale f;
    f.m2 = (uint32_t)s.mult * 2u;
    f.add_hi = R > 0 ? (1u << (R - 1)) : 0u;
    f.rshift = R;
    return f;
}

QL_HD int32_t fast_rescale(int32_t x, const FastScale &f)
{
    uint32_t a = x < 0 ? (uint32_t)0 - (uint32_t)x : (uint32_t)x;
    uint64_t p = (uint64_t)a * f.m2 + (((uint64_t)f.add_hi << 32) | 0x80000000ull);
    uint32_t q = (uint32_t)(p >> 32) >> f.rshift;
    return x < 0 ? (int32_t)((uint32_t)0 - q) : (int32_t)q;
}

// n / d, d > 0, |n| + d/2 < 2^63
QL_HD int64_t rdiv(int64_t n, int64_t d)
{
    uint64_t an = n < 0 ? (uint64_t)0 - (uint64_t)n : (uint64_t)n;
    uint64_t q = (an + ((uint64_t)d >> 1)) / (uint64_t)d;
    return n < 0 ? -(int64_t)q : (int64_t)q;
}

// floor(sqrt(v)) for v < 2^62: fp64 estimate, integer correction.
QL_HD uint64_t isqrt64(uint64_t v)
{
#if defined(__CUDA_ARCH__)
    uint64_t r = (uint64_t)__dsqrt_rn((double)v);
#else
    uint64_t r = (uint64_t)__builtin_sqrt((double)v);
#endif
    while (r * r > v) --r;
    while ((r + 1) * (r + 1) <= v) ++r;
    return r;
}

// ---- integer sigmoid / tanh (Section 3.2.1): int16 Q_{m.15-m} in, Q0.15 out ----------------
// exp(-k|x|) = 2^-t with t = k|x|log2(e) in Q26; 2^-frac(t) by a degree-6 polynomial around 1/2 in Q30
// (coefficients round(2^30 2^-1/2 (-ln 2)^j / j!)), then one division rounded half up.  Written for
// the GPU's 32-bit integer pipes (swept exhaustively on the host and on the GPU):
//  * the polynomial variable is pre-shifted by 6 bits so that "/ 2^26" is "take the high word" of one
//    32x32+64 multiply-add, whose 64-bit addend carries the next coefficient (high word) and the
//    rounding term (low word).  Rounding half away from zero on a signed product p is
//    (p + 2^25 - [p < 0]) >> 26, and the sign of the accumulator alternates deterministically down the
//    Horner chain (|c_k| dominates the term added to it), so [p < 0] depends on the sign of g alone;
//  * the final division is estimated in fp32 (biased low so that the estimate is q or q - 1) and fixed
//    by one exact remainder test, evaluated modulo 2^32 because the remainder is known to be small.
// sigmoid and tanh are one routine: tanh uses k = 2 and the numerator 2^30 - E instead of 2^30.

QL_HD float rcp_est(float x)            // reciprocal estimate, relative error <= 2^-22
{
#if defined(__CUDA_ARCH__)
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
#else
    return 1.0f / x;
#endif
}
QL_HD float fma_rn(float a, float b, float c)
{
#if defined(__CUDA_ARCH__)
    return __fmaf_rn(a, b, c);
#else
    return __builtin_fmaf(a, b, c);
#endif
}
QL_HD float mul_rn(float a, float b)
{
#if defined(__CUDA_ARCH__)
    return __fmul_rn(a, b);
#else
    volatile float r = a * b;
    return r;
#endif
}

QL_HD uint32_t shr_clamp(uint32_t v, uint32_t s)     // v >> s, 0 for s >= 32
{
#if defined(__CUDA_ARCH__)
    uint32_t r;
    asm("shr.b32 %0, %1, %2;" : "=r"(r) : "r"(v), "r"(s));
    return r;
#else
    return s >= 32 ? 0u : v >> s;
#endif
}

template <bool TANH>
QL_HD int32_t act_q_fast(int32_t x, int m)
{
    const int32_t c0 = 759250125, c1 = -526272083, c2 = 182392005, c3 = -42141501,
                  c4 = 7302566, c5 = -1012351, c6 = 116951;
    const uint32_t ck = TANH ? 3098164010u : 1549082005u;         // k * round(2^30 log2 e)
    const uint32_t a = (uint32_t)(x < 0 ? -x : x);
    const int sh = 19 - m;
    const uint64_t t = ((uint64_t)a * ck + ((uint64_t)1 << (sh - 1))) >> sh;
    const uint32_t n = (uint32_t)(t >> 26);
    // 64 * g with g = frac(t) - 2^25: the shift drops the integer part, subtracting 2^31 flips the top bit
    const int32_t g6 = (int32_t)(((uint32_t)t << 6) ^ 0x80000000u);
    const uint32_t s = (uint32_t)(g6 >> 31);                       // all ones iff g < 0
    const uint32_t lo_pos = 0x80000000u + (s & 0xFFFFFFC0u);       // 64 * (2^25 - [g < 0]): accumulator > 0
    const uint32_t lo_neg = lo_pos ^ 0xFFFFFFC0u;                  // 64 * (2^25 - [g >= 0]): accumulator < 0
#define QL_HORNER(acc, ck_, lo_) (int32_t)(((int64_t)(acc) * g6 + (int64_t)(((uint64_t)(uint32_t)(ck_) << 32) | (lo_))) >> 32)
    int32_t acc = c6;
    acc = QL_HORNER(acc, c5, lo_pos);
    acc = QL_HORNER(acc, c4, lo_neg);
    acc = QL_HORNER(acc, c3, lo_pos);
    acc = QL_HORNER(acc, c2, lo_neg);
    acc = QL_HORNER(acc, c1, lo_pos);
    acc = QL_HORNER(acc, c0, lo_neg);
#undef QL_HORNER
    // E = round(acc / 2^n): for n >= 1 the high word of acc * 2^(32-n) + 2^31 (0 once n > 32); for n = 0 acc itself,
    // clamped to 2^30 (only x = 0 exceeds it, by a few units, and the quotient is the same)
    const uint32_t p = (uint32_t)acc;
    const uint32_t scaled = (uint32_t)(((uint64_t)p * shr_clamp(0x80000000u, n - 1u) + 0x80000000ull) >> 32);
    const uint32_t E = n == 0 ? (p > (1u << 30) ? (1u << 30) : p) : scaled;
    const uint32_t D = (1u << 30) + E;
    const uint32_t N = TANH ? (1u << 30) - E : (1u << 30);
    // q = floor(2^15 N / D + 1/2); the estimate is biased low by more than its error: it is q or q - 1
    const float est = fma_rn(mul_rn((float)N, 32768.0f), rcp_est((float)D), 0.47f);
    uint32_t q = (uint32_t)est;
    // q + 1 is admissible iff D q + ceil(D / 2) <= 2^15 N; the difference lies in [-D, D), so mod 2^32 suffices
    const int32_t rem = (int32_t)((N << 15) - D * q - ((D + 1u) >> 1));
    q += rem >= 0 ? 1u : 0u;
    const int32_t pos = q > 32767u ? 32767 : (int32_t)q;
    return x >= 0 ? pos : (TANH ? -(int32_t)q : 32768 - (int32_t)q);
}

QL_HD int32_t sigmoid_q_fast(int32_t x, int m) { return act_q_fast<false>(x, m); }
QL_HD int32_t tanh_q_fast(int32_t x, int m) { return act_q_fast<true>(x, m); }

// ---- integer layer normalisation (Section 3.2.6) --------------------------------------------

struct LnStats { int64_t mean; int64_t sigma; };   // mean at scale 2^-10 of the input grid; sigma = 2^10 * std

QL_HD LnStats ln_stats(int64_t sum, int64_t sumsq, int n)
{
    LnStats s;
    s.mean = rdiv(sum * 1024, n);
    int64_t var = rdiv(sumsq * 1048576, n) - s.mean * s.mean;
    s.sigma = (int64_t)isqrt64(var > 0 ? (uint64_t)var : 0);
    return s;
}

// The same statistics without a hardware-less 64-bit division or an fp64 square root on the way (in the kernels one
// thread per (row, gate) computes them while the whole block waits): the divisor n is fixed per layer, so x / n is the
// high half of x * ceil(2^64 / n), exact for x < 2^50 and n < 2^14; the square root starts from an fp32 estimate.
// Requires n < 2^14 and |q| <= 2^15 (then sum 2^10 < 2^39 and sumsq < 2^44).
struct DivMagic { uint64_t m; uint32_t n; };

QL_HD DivMagic make_div_magic(uint32_t n)
{
    DivMagic d;
    d.n = n;
    d.m = n > 1 ? ~(uint64_t)0 / n + 1 : 0;          // floor((2^64 - 1) / n) + 1 = floor(2^64 / n) + 1 unless n divides 2^64,
                                                     // where it is 2^64 / n exactly: both are valid multipliers
    return d;
}

QL_HD uint64_t umul64hi_hd(uint64_t a, uint64_t b)
{
#if defined(__CUDA_ARCH__)
    return __umul64hi(a, b);
#else
    return (uint64_t)(((unsigned __int128)a * b) >> 64);
#endif
}

QL_HD uint64_t div_by_magic(uint64_t x, const DivMagic &d) { return d.n > 1 ? umul64hi_hd(x, d.m) : x; }   // x < 2^50

QL_HD uint64_t isqrt_from_f32(uint64_t v)           // floor(sqrt(v)), v < 2^52
{
#if defined(__CUDA_ARCH__)
    uint64_t r = (uint64_t)__fsqrt_rn((float)v);
#else
    uint64_t r = (uint64_t)__builtin_sqrtf((float)v);
#endif
    while (r * r > v) --r;
    while ((r + 1) * (r + 1) <= v) ++r;
    return r;
}

QL_HD LnStats ln_stats_fast(int64_t sum, int64_t sumsq, const DivMagic &d)
{
    LnStats s;
    const uint64_t half = d.n >> 1;
    const uint64_t as = (uint64_t)(sum < 0 ? -sum : sum) * 1024u;
    const int64_t am = (int64_t)div_by_magic(as + half, d);
    s.mean = sum < 0 ? -am : am;
    // round(sumsq 2^20 / n) = floor(sumsq / n) 2^20 + floor(((sumsq mod n) 2^20 + n / 2) / n)
    const uint64_t q1 = div_by_magic((uint64_t)sumsq, d);
    const uint64_t r1 = (uint64_t)sumsq - q1 * d.n;
    const uint64_t msq = (q1 << 20) + div_by_magic((r1 << 20) + half, d);
    const int64_t var = (int64_t)msq - s.mean * s.mean;
    s.sigma = (int64_t)isqrt_from_f32(var > 0 ? (uint64_t)var : 0);
    return s;
}

// One element: q' = round(2^10 (2^10 q - mean) / sigma); out = sat16(rescale(sat32(q' L + b), eff_ln)).
// Per (row, gate) constants: mean, sigma and the fp32 reciprocal of sigma for the quotient estimate.
struct LnRow { int32_t mean; uint32_t sigma; float inv_sigma; };

QL_HD LnRow make_ln_row(LnStats s)
{
    LnRow r;
    r.mean = (int32_t)s.mean;                      // |mean| <= 2^25
    r.sigma = (uint32_t)s.sigma;                   // < 2^26
    r.inv_sigma = s.sigma > 0 ? 1.0f / (float)r.sigma : 0.0f;
    return r;
}

// q' = round(2^10 (2^10 q - mean) / sigma), exact.  Quotients up to 2^16 (|z-score| <= 64) take the fp32
// estimate (biased low: q' or q' - 1) and one remainder test modulo 2^32; anything larger - a tiny sigma
// against a large deviation - takes the plain 64-bit division.  fast: the quotient fits 17 bits, so that its product
// with an int16 weight fits an int32.
QL_HD int64_t ln_quotient_core(int32_t q, const LnRow &r, bool &fast)
{
    const int32_t d = 1024 * q - r.mean;
    const uint32_t ad = (uint32_t)(d < 0 ? -d : d);
    const uint32_t half = r.sigma >> 1;
    const float est = fma_rn(fma_rn((float)ad, 1024.0f, (float)half), r.inv_sigma, -0.05f);
    fast = est < 65536.0f;
    if (fast) {
#if defined(__CUDA_ARCH__)
        uint32_t qe = __float2uint_rz(est);                        // a negative estimate (ad = 0) converts to 0
#else
        uint32_t qe = est > 0.0f ? (uint32_t)est : 0u;
#endif
        const uint32_t rem = (ad << 10) + half - qe * r.sigma;     // in [0, 2 sigma), exact modulo 2^32
        qe += (rem >= r.sigma && r.sigma != 0u) ? 1u : 0u;
        return d < 0 ? -(int32_t)qe : (int32_t)qe;
    }
#if defined(__CUDA_ARCH__)
    const uint64_t quo = r.sigma ? div_rare((uint64_t)ad * 1024u + half, r.sigma) : 0u;
#else
    const uint64_t quo = r.sigma ? ((uint64_t)ad * 1024u + half) / r.sigma : 0u;
#endif
    return d < 0 ? -(int64_t)quo : (int64_t)quo;
}

QL_HD int64_t ln_quotient_fast(int32_t q, const LnRow &r)
{
    bool fast;
    return ln_quotient_core(q, r, fast);
}

QL_HD int32_t sat32_halves(int64_t v)              // saturate through the two 32-bit halves
{
    const int32_t lo = (int32_t)v, hi = (int32_t)(v >> 32);
    return hi == (lo >> 31) ? lo : (int32_t)(0x7fffffff ^ (hi >> 31));
}

QL_HD int32_t add_sat_s32(int32_t a, int32_t b)
{
#if defined(__CUDA_ARCH__)
    int32_t d;
    asm("add.sat.s32 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
#else
    return sat32((int64_t)a + b);
#endif
}

// sat32(q' L + b): in 32 bits on the fast path (|q'| <= 2^16 and -2^15 <= L < 2^15: the product is exact, the sum
// saturates), in 64 bits otherwise
QL_HD int32_t ln_scaled_sat32(int32_t q, const LnRow &r, int32_t L, int32_t b)
{
    bool fast;
    const int64_t qp = ln_quotient_core(q, r, fast);
    if (fast) return add_sat_s32((int32_t)qp * L, b);
    return sat32_halves(qp * (int64_t)L + (int64_t)b);
}

QL_HD int32_t ln_apply_fast(int32_t q, const LnRow &r, int32_t L, int32_t b, Scale eff_ln, const FastScale &f_ln)
{
    const int32_t v32 = ln_scaled_sat32(q, r, L, b);
    return sat16(eff_ln.shift <= 0 ? fast_rescale(v32, f_ln) : mbqm_cold(v32, eff_ln));
}

// The same for a scale known to shift right (eff_ln.shift <= 0): no rarely taken call in the caller's loop, which the
// instruction scheduler does not move work across.
QL_HD int32_t ln_apply_noshift(int32_t q, const LnRow &r, int32_t L, int32_t b, const FastScale &f_ln)
{
    return sat16(fast_rescale(ln_scaled_sat32(q, r, L, b), f_ln));
}

// ---- cell update and hidden state (Section 3.2.7) -------------------------------------------

// x / 2^e for |x| <= 2^30 and 1 <= e <= 30, ties away from zero, in 32 bits
QL_HD int32_t rdivpot32(int32_t x, int e) { return (x + (1 << (e - 1)) + (x >> 31)) >> e; }

QL_HD int32_t cell_update_fast(int32_t i, int32_t z, int32_t f, int32_t c_old, int m)
{
    return sat16(rdivpot32(i * z, 15 + m) + rdivpot32(f * c_old, 15));
}

QL_HD int32_t hidden_q_fast(int32_t o, int32_t c_new, int m, Scale eff_m, const FastScale &f_m, int32_t zp_m)
{
    int32_t prod = o * tanh_q_fast(c_new, m);
    return sat8((eff_m.shift <= 0 ? fast_rescale(prod, f_m) : mbqm_cold(prod, eff_m)) + zp_m);
}

}  // namespace ql
