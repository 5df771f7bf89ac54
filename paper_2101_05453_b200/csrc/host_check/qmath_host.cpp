// Host build of the kernels' fixed-point arithmetic (qmath.cuh) so that CPU-only tests can sweep it
// exhaustively.  Not part of libqlstm.so and not used by any product path.
#include "../qmath.cuh"

extern "C" {
int32_t qmh_mbqm(int32_t x, int32_t mult, int32_t shift) { return ql::mbqm(x, ql::Scale{mult, shift}); }
void qmh_mbqm_many(const int32_t *x, int n, int32_t mult, int32_t shift, int32_t *out)
{
    for (int i = 0; i < n; ++i) out[i] = ql::mbqm(x[i], ql::Scale{mult, shift});
}
void qmh_fast_rescale_many(const int32_t *x, int n, int32_t mult, int32_t shift, int32_t *out)
{
    ql::FastScale f = ql::make_fast_scale(ql::Scale{mult, shift});
    for (int i = 0; i < n; ++i) out[i] = ql::fast_rescale(x[i], f);
}
void qmh_sigmoid_fast_all(int m, int32_t *out) { for (int x = -32768; x < 32768; ++x) out[x + 32768] = ql::sigmoid_q_fast(x, m); }
void qmh_tanh_fast_all(int m, int32_t *out) { for (int x = -32768; x < 32768; ++x) out[x + 32768] = ql::tanh_q_fast(x, m); }
void qmh_layernorm_row_fast(const int16_t *q, int n, const int16_t *L, const int32_t *b, int32_t mult, int32_t shift, int16_t *out)
{
    int64_t s = 0, s2 = 0;
    for (int i = 0; i < n; ++i) { s += q[i]; s2 += (int64_t)q[i] * q[i]; }
    ql::LnRow r = ql::make_ln_row(ql::ln_stats(s, s2, n));
    ql::Scale sc{mult, shift};
    ql::FastScale f = ql::make_fast_scale(sc);
    for (int i = 0; i < n; ++i) out[i] = (int16_t)ql::ln_apply_fast(q[i], r, L[i], b[i], sc, f);
}
// the quotient alone, with hand-picked statistics (tiny sigma against large deviations)
int64_t qmh_ln_quotient_fast(int32_t q, int64_t mean, int64_t sigma)
{
    ql::LnStats st{mean, sigma};
    return ql::ln_quotient_fast(q, ql::make_ln_row(st));
}
int32_t qmh_cell_update_fast(int32_t i, int32_t z, int32_t f, int32_t c, int m) { return ql::cell_update_fast(i, z, f, c, m); }
int32_t qmh_hidden_fast(int32_t o, int32_t c, int m, int32_t mult, int32_t shift, int32_t zp)
{
    ql::Scale sc{mult, shift};
    return ql::hidden_q_fast(o, c, m, sc, ql::make_fast_scale(sc), zp);
}
uint64_t qmh_isqrt(uint64_t v) { return ql::isqrt64(v); }
uint64_t qmh_isqrt_from_f32(uint64_t v) { return ql::isqrt_from_f32(v); }
uint64_t qmh_div_by_magic(uint64_t x, uint32_t n) { return ql::div_by_magic(x, ql::make_div_magic(n)); }
void qmh_ln_stats(int64_t sum, int64_t sumsq, int n, int fast, int64_t *mean_sigma)
{
    ql::LnStats s = fast ? ql::ln_stats_fast(sum, sumsq, ql::make_div_magic((uint32_t)n)) : ql::ln_stats(sum, sumsq, n);
    mean_sigma[0] = s.mean; mean_sigma[1] = s.sigma;
}
}
