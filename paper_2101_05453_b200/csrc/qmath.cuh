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

// ---- cell update and hidden state (Section 3.2.7) -------------------------------------------

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
