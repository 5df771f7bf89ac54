// Fixed-point arithmetic of the integer LSTM, shared by all CUDA kernels of this library.
//
// Everything here is exact integer arithmetic; where a floating-point unit is used it only
// produces an estimate that an integer remainder check then corrects, so results never depend
// on floating-point rounding.  Functions are __host__ __device__ so that the host test harness
// (csrc/qmath_host_check.cpp) can sweep them on a CPU.
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

// x / 2^e (0 <= e <= 62), |x| < 2^62
QL_HD int64_t rdivpot(int64_t x, int e)
{
    if (e == 0) return x;
    uint64_t ax = x < 0 ? (uint64_t)0 - (uint64_t)x : (uint64_t)x;
    uint64_t q = (ax + ((uint64_t)1 << (e - 1))) >> e;
    return x < 0 ? -(int64_t)q : (int64_t)q;
}

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
// exp(-k|x|) = 2^-t with t = k|x|log2(e) in Q26; 2^-frac(t) by a degree-6 polynomial around 1/2 in Q30.

QL_HD int64_t exp_neg_q30(int32_t absx, int m, int k)
{
    const int64_t LOG2E_Q30 = 1549082005;      // round(2^30 log2 e)
    const int64_t c0 = 759250125, c1 = -526272083, c2 = 182392005, c3 = -42141501,
                  c4 = 7302566, c5 = -1012351, c6 = 116951;   // round(2^30 2^-1/2 (-ln 2)^j / j!)
    int64_t t = rdivpot((int64_t)absx * LOG2E_Q30 * k, 15 - m + 4);
    int64_t n = t >> 26;
    if (n > 40) n = 40;
    int64_t g = (t & (((int64_t)1 << 26) - 1)) - ((int64_t)1 << 25);
    int64_t acc = c6;
    acc = rdivpot(acc * g, 26) + c5;
    acc = rdivpot(acc * g, 26) + c4;
    acc = rdivpot(acc * g, 26) + c3;
    acc = rdivpot(acc * g, 26) + c2;
    acc = rdivpot(acc * g, 26) + c1;
    acc = rdivpot(acc * g, 26) + c0;
    return rdivpot(acc, (int)n);
}

QL_HD int32_t sigmoid_q(int32_t x, int m)
{
    int32_t a = x < 0 ? -x : x;
    int64_t E = exp_neg_q30(a, m, 1);
    uint64_t D = ((uint64_t)1 << 30) + (uint64_t)E;
    int32_t S = (int32_t)((((uint64_t)1 << 46) + D) / (2 * D));
    return x >= 0 ? (S > 32767 ? 32767 : S) : 32768 - S;
}

QL_HD int32_t tanh_q(int32_t x, int m)
{
    int32_t a = x < 0 ? -x : x;
    int64_t E = exp_neg_q30(a, m, 2);
    uint64_t D = ((uint64_t)1 << 30) + (uint64_t)E;
    uint64_t N = ((uint64_t)1 << 30) - (uint64_t)E;
    int32_t T = (int32_t)((N * 65536 + D) / (2 * D));
    return x >= 0 ? (T > 32767 ? 32767 : T) : -T;
}

// ---- the same two functions in 32-bit registers ------------------------------------------------
// Bit-identical to sigmoid_q / tanh_q above (swept exhaustively on the host), but written for the
// GPU's integer pipes: 32x32->64 multiply-adds, funnel shifts, and one fp32 reciprocal whose result
// is only an estimate of the final quotient - an exact 64-bit remainder test then fixes it.
//
// Rounding x / 2^26 half away from zero on a signed product p: (p + 2^25 - [p < 0]) >> 26.  In the
// Horner chain the sign of the accumulator alternates deterministically (|c_k| dominates the term
// it is added to), so [p < 0] depends on the sign of g alone and costs nothing per step.

QL_HD float rcp_rn(float x)
{
#if defined(__CUDA_ARCH__)
    return __frcp_rn(x);
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

// 2^30 * exp(-k |x|), k folded into ck = k * round(2^30 log2 e); sh = 19 - m.
QL_HD uint32_t exp_neg_q30_fast(uint32_t a, int sh, uint32_t ck)
{
    const int32_t c0 = 759250125, c1 = -526272083, c2 = 182392005, c3 = -42141501,
                  c4 = 7302566, c5 = -1012351, c6 = 116951;
    uint64_t t = ((uint64_t)a * ck + ((uint64_t)1 << (sh - 1))) >> sh;
    uint32_t n = (uint32_t)(t >> 26);
    int32_t g = (int32_t)((uint32_t)t & 0x3FFFFFFu) - (1 << 25);
    int32_t sg = g >> 31;
    const int64_t add_pos = (int64_t)((1 << 25) + sg);      // accumulator > 0: product negative iff g < 0
    const int64_t add_neg = (int64_t)((1 << 25) + ~sg);     // accumulator < 0: product negative iff g > 0
    int32_t acc = c6;
    acc = (int32_t)(((int64_t)acc * g + add_pos) >> 26) + c5;
    acc = (int32_t)(((int64_t)acc * g + add_neg) >> 26) + c4;
    acc = (int32_t)(((int64_t)acc * g + add_pos) >> 26) + c3;
    acc = (int32_t)(((int64_t)acc * g + add_neg) >> 26) + c2;
    acc = (int32_t)(((int64_t)acc * g + add_pos) >> 26) + c1;
    acc = (int32_t)(((int64_t)acc * g + add_neg) >> 26) + c0;
    uint32_t p = (uint32_t)acc;                              // in (2^29, 2^30 + small]
    if (n == 0) return p;
    if (n > 31) return 0;
    return (p + (1u << (n - 1))) >> n;
}

// largest q with d * (2q - 1) <= rhs, given an estimate within +-1
QL_HD uint32_t fix_quotient(uint32_t q, uint32_t d, uint64_t rhs)
{
    if (q > 0 && (uint64_t)d * (2 * q - 1) > rhs) return q - 1;
    if ((uint64_t)d * (2 * q + 1) <= rhs) return q + 1;
    return q;
}

QL_HD int32_t sigmoid_q_fast(int32_t x, int m)
{
    uint32_t a = (uint32_t)(x < 0 ? -x : x);
    uint32_t E = exp_neg_q30_fast(a, 19 - m, 1549082005u);
    uint32_t D = (1u << 30) + E;
    float r = rcp_rn((float)D);
    uint32_t q = (uint32_t)fma_rn(35184372088832.0f, r, 0.5f);          // 2^45 / D + 1/2
    int32_t S = (int32_t)fix_quotient(q, D, (uint64_t)1 << 46);
    return x >= 0 ? (S > 32767 ? 32767 : S) : 32768 - S;
}

QL_HD int32_t tanh_q_fast(int32_t x, int m)
{
    uint32_t a = (uint32_t)(x < 0 ? -x : x);
    uint32_t E = exp_neg_q30_fast(a, 19 - m, 3098164010u);
    uint32_t D = (1u << 30) + E;
    int32_t N = (1 << 30) - (int32_t)E;             // E can exceed 2^30 by a few units at x = 0: the quotient is 0 there
    if (N <= 0) return 0;
    float r = rcp_rn((float)D);
    uint32_t q = (uint32_t)fma_rn(mul_rn((float)N, 32768.0f), r, 0.5f);  // 2^15 N / D + 1/2
    int32_t T = (int32_t)fix_quotient(q, D, (uint64_t)(uint32_t)N << 16);
    return x >= 0 ? (T > 32767 ? 32767 : T) : -T;
}

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

// one element: q' = round(2^10 (2^10 q - mean) / sigma); out = sat16(rescale(sat32(q' L + b), eff_ln))
QL_HD int32_t ln_apply(int32_t q, LnStats s, int32_t L, int32_t b, Scale eff_ln)
{
    int64_t qp = s.sigma == 0 ? 0 : rdiv(1024 * (1024 * (int64_t)q - s.mean), s.sigma);
    return sat16(mbqm(sat32(qp * (int64_t)L + (int64_t)b), eff_ln));
}

// Per (row, gate) constants of the fast path: fp32 reciprocal of sigma for the quotient estimate.
struct LnRow { int32_t mean; uint32_t sigma; float inv_sigma; };

QL_HD LnRow make_ln_row(LnStats s)
{
    LnRow r;
    r.mean = (int32_t)s.mean;                      // |mean| <= 2^25
    r.sigma = (uint32_t)s.sigma;                   // < 2^26
    r.inv_sigma = s.sigma > 0 ? rcp_rn((float)r.sigma) : 0.0f;
    return r;
}

// q' = round(2^10 (2^10 q - mean) / sigma), exact: fp32 estimate, 64-bit remainder check, and the plain
// division as a fallback where the estimate could be more than one off (tiny sigma against large deviations).
QL_HD int64_t ln_quotient_fast(int32_t q, const LnRow &r)
{
    if (r.sigma == 0) return 0;
    int32_t d = 1024 * q - r.mean;
    uint32_t ad = (uint32_t)(d < 0 ? -d : d);
    uint64_t num = (uint64_t)ad * 1024u + (r.sigma >> 1);
    float est = mul_rn(fma_rn((float)ad, 1024.0f, (float)(r.sigma >> 1)), r.inv_sigma);
    uint64_t quo;
    if (est < 2.0e9f) {
        uint32_t qe = (uint32_t)est;
        int64_t rem = (int64_t)num - (int64_t)((uint64_t)qe * r.sigma);
        if (rem < 0) { --qe; rem += r.sigma; }
        else if (rem >= (int64_t)r.sigma) { ++qe; rem -= r.sigma; }
        quo = (rem < 0 || rem >= (int64_t)r.sigma) ? num / r.sigma : (uint64_t)qe;
    } else {
        quo = num / r.sigma;
    }
    return d < 0 ? -(int64_t)quo : (int64_t)quo;
}

QL_HD int32_t ln_apply_fast(int32_t q, const LnRow &r, int32_t L, int32_t b, Scale eff_ln, const FastScale &f_ln)
{
    int64_t v = ln_quotient_fast(q, r) * (int64_t)L + (int64_t)b;
    int32_t v32 = sat32(v);
    return sat16(eff_ln.shift <= 0 ? fast_rescale(v32, f_ln) : mbqm(v32, eff_ln));
}

// ---- cell update and hidden state (Section 3.2.7) -------------------------------------------

// x / 2^e on a 32-bit product, ties away from zero, 1 <= e <= 31
QL_HD int32_t rdivpot32(int32_t x, int e) { return (int32_t)(((int64_t)x + ((int64_t)1 << (e - 1)) + (x >> 31)) >> e); }

QL_HD int32_t cell_update_fast(int32_t i, int32_t z, int32_t f, int32_t c_old, int m)
{
    return sat16(rdivpot32(i * z, 15 + m) + rdivpot32(f * c_old, 15));
}

QL_HD int32_t hidden_q_fast(int32_t o, int32_t c_new, int m, Scale eff_m, const FastScale &f_m, int32_t zp_m)
{
    int32_t prod = o * tanh_q_fast(c_new, m);
    return sat8((eff_m.shift <= 0 ? fast_rescale(prod, f_m) : mbqm(prod, eff_m)) + zp_m);
}

QL_HD int32_t cell_update(int32_t i, int32_t z, int32_t f, int32_t c_old, int m)
{
    int64_t iz = rdivpot((int64_t)i * z, 15 + m);
    int64_t fc = rdivpot((int64_t)f * c_old, 15);
    return sat16((int32_t)(iz + fc));
}

QL_HD int32_t hidden_q(int32_t o, int32_t c_new, int m, Scale eff_m, int32_t zp_m)
{
    return sat8(mbqm(o * tanh_q(c_new, m), eff_m) + zp_m);
}

}  // namespace ql
