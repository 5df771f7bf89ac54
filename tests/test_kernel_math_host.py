"""The kernels' integer arithmetic (csrc/qmath.cuh), compiled for the host and swept on the CPU.

This runs the very source the CUDA kernels compile, so that a wrong shift or rounding in the device
code shows up without a GPU.  Two kinds of check: against the oracle (the reference; nothing here feeds
it), and - so that agreement does not rest on the oracle alone - directly against what the mathematics
fixes: exact rational arithmetic for the rescale, fp64 closed forms for the nonlinearities.
"""
import ctypes as C
import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import qlstm_ref as R
from paper_2101_05453_b200 import build as B


@pytest.fixture(scope="module")
def H():
    lib = C.CDLL(B.build_host_check())
    lib.qmh_mbqm.restype = C.c_int32
    lib.qmh_mbqm.argtypes = [C.c_int32] * 3
    lib.qmh_isqrt.restype = C.c_uint64
    lib.qmh_isqrt.argtypes = [C.c_uint64]
    lib.qmh_isqrt_from_f32.restype = C.c_uint64
    lib.qmh_isqrt_from_f32.argtypes = [C.c_uint64]
    lib.qmh_div_by_magic.restype = C.c_uint64
    lib.qmh_div_by_magic.argtypes = [C.c_uint64, C.c_uint32]
    lib.qmh_ln_stats.restype = None
    lib.qmh_ln_stats.argtypes = [C.c_int64, C.c_int64, C.c_int, C.c_int, C.POINTER(C.c_int64)]
    return lib


def test_rescale_against_oracle(H):
    rng = np.random.default_rng(0)
    xs = np.concatenate([rng.integers(-2 ** 31, 2 ** 31, 20000), np.arange(-40000, 40000, 7),
                         [-2 ** 31, 2 ** 31 - 1, 0, 1, -1, 2 ** 30, -2 ** 30]]).astype(np.int32)
    scales = [(1 << 30, 1), ((1 << 31) - 1, 0), (1 << 30, -31), (0, 0)] + \
        [(int(rng.integers(1 << 30, 1 << 31)), int(s)) for s in range(-31, 31, 3)]
    out = np.empty_like(xs)
    for M, s in scales:
        H.qmh_mbqm_many(xs.ctypes.data_as(C.c_void_p), len(xs), M, s, out.ctypes.data_as(C.c_void_p))
        want = np.array([R.mbqm(int(x), (M, s)) for x in xs[::17]], np.int32)
        assert np.array_equal(out[::17], want), (M, s)


def test_fast_rescale_against_oracle(H):
    """The pre-computed single multiply-add form used in the kernels' epilogues (shift <= 0)."""
    rng = np.random.default_rng(3)
    xs = np.concatenate([rng.integers(-2 ** 31, 2 ** 31, 30000), np.arange(-70000, 70000, 3),
                         [-2 ** 31, 2 ** 31 - 1, 0, 1, -1, 2 ** 30, -2 ** 30, 2 ** 30 + 1]]).astype(np.int32)
    scales = [((1 << 31) - 1, 0), (1 << 30, 0), (1 << 30, -1), (1 << 30, -31), (0, 0), ((1 << 31) - 1, -31)] + \
        [(int(rng.integers(1 << 30, 1 << 31)), int(s)) for s in range(-31, 1)]
    out = np.empty_like(xs)
    ref = np.empty_like(xs)
    for M, s in scales:
        H.qmh_fast_rescale_many(xs.ctypes.data_as(C.c_void_p), len(xs), M, s, out.ctypes.data_as(C.c_void_p))
        H.qmh_mbqm_many(xs.ctypes.data_as(C.c_void_p), len(xs), M, s, ref.ctypes.data_as(C.c_void_p))
        assert np.array_equal(out, ref), (M, s)            # all points: against the plain form (itself checked above)
        want = np.array([R.mbqm(int(x), (M, s)) for x in xs[::23]], np.int32)
        assert np.array_equal(out[::23], want), (M, s)     # a subsample directly against the oracle
    # ties: x * M / 2^31 exactly half-way, then a second half-way in the right shift
    for x in (1, -1, 3, -3, 5, -5, 7, -7, 1 << 20, -(1 << 20)):
        for s in (0, -1, -2, -5):
            xs1 = np.array([x], np.int32)
            H.qmh_fast_rescale_many(xs1.ctypes.data_as(C.c_void_p), 1, 1 << 30, s, out.ctypes.data_as(C.c_void_p))
            assert out[0] == R.mbqm(x, (1 << 30, s))


def test_isqrt(H):
    import math
    rng = np.random.default_rng(1)
    for v in list(range(2000)) + [int(x) for x in rng.integers(0, 1 << 61, 5000)] + [(1 << 61) - 1, (1 << 50) + 1]:
        assert H.qmh_isqrt(v) == math.isqrt(v)
    for r in [3, 1 << 20, (1 << 25) + 3, (1 << 30) - 1]:
        assert H.qmh_isqrt(r * r) == r and H.qmh_isqrt(r * r - 1) == r - 1


# ---------------------------------------------------------------- the 32-bit / fp32-assisted forms the kernels run

@pytest.mark.parametrize("m", [0, 1, 2, 3, 4, 5, 6, 9, 12, 15])
def test_fast_activations_exhaustive(H, m):
    out = np.empty(65536, np.int32)
    H.qmh_sigmoid_fast_all(m, out.ctypes.data_as(C.c_void_p))
    assert np.array_equal(out, R.sigmoid_all(m))
    H.qmh_tanh_fast_all(m, out.ctypes.data_as(C.c_void_p))
    assert np.array_equal(out, R.tanh_all(m))


@pytest.mark.parametrize("seed", range(12))
def test_fast_layernorm_rows(H, seed):
    rng = np.random.default_rng(500 + seed)
    n = int(rng.integers(1, 2100))
    q = (rng.integers(-32768, 32768, n) // int(rng.integers(1, 60))).astype(np.int16)
    if seed == 0:
        q[:] = -5
    if seed == 1:                                   # one outlier: the largest z-score
        q[:] = 0
        q[3] = 32767
    if seed == 2:
        q = np.where(np.arange(n) % 2 == 0, 32767, -32768).astype(np.int16)
    L = rng.integers(-32767, 32768, n).astype(np.int16)
    b = (rng.integers(-2 ** 31 + 1, 2 ** 31, n) // int(rng.integers(1, 3000))).astype(np.int32)
    eff = (int(rng.integers(1 << 30, 1 << 31)), int(rng.integers(-14, 2)))
    out = np.empty(n, np.int16)
    H.qmh_layernorm_row_fast(q.ctypes.data_as(C.c_void_p), n, L.ctypes.data_as(C.c_void_p), b.ctypes.data_as(C.c_void_p),
                             eff[0], eff[1], out.ctypes.data_as(C.c_void_p))
    assert np.array_equal(out, R.layernorm_row(q, L, b, eff))


def test_fast_ln_quotient_with_adversarial_statistics(H):
    """Statistics that cannot come from a real row still must divide exactly (tiny sigma, huge deviation)."""
    H.qmh_ln_quotient_fast.restype = C.c_int64
    H.qmh_ln_quotient_fast.argtypes = [C.c_int32, C.c_int64, C.c_int64]
    rng = np.random.default_rng(9)
    cases = [(32767, -(1 << 25), 1), (-32768, (1 << 25), 1), (5000, 0, 3), (123, 125000, 7), (0, 0, 0), (77, 5, (1 << 26) - 1)]
    cases += [(int(rng.integers(-32768, 32768)), int(rng.integers(-(1 << 25), 1 << 25)), int(rng.integers(1, 1 << int(rng.integers(1, 27)))))
              for _ in range(20000)]
    for q, mean, sigma in cases:
        want = 0 if sigma == 0 else R.rdiv(1024 * (1024 * q - mean), sigma)
        assert H.qmh_ln_quotient_fast(q, mean, sigma) == want, (q, mean, sigma)


def test_fast_cell_update_and_hidden(H):
    H.qmh_cell_update_fast.restype = C.c_int32
    H.qmh_cell_update_fast.argtypes = [C.c_int32] * 5
    H.qmh_hidden_fast.restype = C.c_int32
    H.qmh_hidden_fast.argtypes = [C.c_int32] * 6
    rng = np.random.default_rng(12)
    edge = [(32767, 32767, 32767, 32767), (32767, -32768, 32767, -32768), (1, -1, 1, -1), (0, 0, 0, 0), (16384, 1, 16384, -1)]
    rand = [tuple(int(v) for v in (rng.integers(0, 32768), rng.integers(-32768, 32768), rng.integers(0, 32768),
                                   rng.integers(-32768, 32768))) for _ in range(5000)]
    for i, z, f, c in edge + rand:
        for m in (0, 3, 5):
            want = max(-32768, min(32767, R.rdivpot(i * z, 15 + m) + R.rdivpot(f * c, 15)))
            assert H.qmh_cell_update_fast(i, z, f, c, m) == want
    for _ in range(3000):
        o = int(rng.integers(0, 32768)); c = int(rng.integers(-32768, 32768)); m = int(rng.integers(0, 7))
        eff = (int(rng.integers(1 << 30, 1 << 31)), int(rng.integers(-24, -18))); zp = int(rng.integers(-128, 128))
        want = max(-128, min(127, R.mbqm(o * R.tanh(c, m), eff) + zp))
        assert H.qmh_hidden_fast(o, c, m, eff[0], eff[1], zp) == want


# ---------------------------------------------------------------- directly against the mathematics

def _round_half_away(fr: Fraction) -> int:
    n = abs(fr)
    q = (n.numerator * 2 + n.denominator) // (2 * n.denominator)
    return -q if fr < 0 else q


def test_rescale_forms_against_exact_rationals(H):
    """rescale(x, (M, s)) = round(round(x 2^max(s,0) M / 2^31) / 2^max(-s,0)), both roundings half away from zero."""
    rng = np.random.default_rng(21)
    xs = [int(v) for v in rng.integers(-2 ** 31, 2 ** 31, 400)] + [0, 1, -1, 5, -5, 2 ** 31 - 1, -2 ** 31, 12345, -32768]
    scales = [(1 << 30, 0), ((1 << 31) - 1, -7), (1 << 30, -1), (1 << 30, 1)] + \
        [(int(rng.integers(1 << 30, 1 << 31)), int(s)) for s in (-31, -20, -12, -5, -1, 0, 2, 6)]
    out = np.empty(len(xs), np.int32)
    xa = np.array(xs, np.int32)
    for M, s in scales:
        def exact(x):
            left, right = max(s, 0), max(-s, 0)
            xl = max(-2 ** 31, min(2 ** 31 - 1, x << left))
            first = _round_half_away(Fraction(xl * M, 2 ** 31))
            return _round_half_away(Fraction(first, 2 ** right))
        want = np.array([exact(x) for x in xs], np.int64)
        H.qmh_mbqm_many(xa.ctypes.data_as(C.c_void_p), len(xs), M, s, out.ctypes.data_as(C.c_void_p))
        assert np.array_equal(out, want), (M, s)
        if s <= 0:
            H.qmh_fast_rescale_many(xa.ctypes.data_as(C.c_void_p), len(xs), M, s, out.ctypes.data_as(C.c_void_p))
            assert np.array_equal(out, want), (M, s)


@pytest.mark.parametrize("m", [0, 3, 4, 6])
def test_fast_activations_against_fp64_closed_forms(H, m):
    """Section 3.2.1: Q_{m.15-m} in, Q0.15 out, clamped to [-1, 32767/32768]."""
    x = np.arange(-32768, 32768, dtype=np.float64) * 2.0 ** (m - 15)
    out = np.empty(65536, np.int32)
    for fn, f64 in ((H.qmh_sigmoid_fast_all, 1.0 / (1.0 + np.exp(-x))), (H.qmh_tanh_fast_all, np.tanh(x))):
        fn(m, out.ctypes.data_as(C.c_void_p))
        true = 32768.0 * f64
        err = np.abs(out - true)
        assert err.max() <= 1.0                                  # the forced clamp at +32767 costs up to one step
        assert err[true <= 32767.0].max() <= 0.51
        assert np.all(np.diff(out) >= 0)                         # monotone
    H.qmh_sigmoid_fast_all(m, out.ctypes.data_as(C.c_void_p))
    assert out[32768] == 16384 and out.min() >= 0 and out.max() <= 32767
    H.qmh_tanh_fast_all(m, out.ctypes.data_as(C.c_void_p))
    assert out[32768] == 0 and out.min() >= -32768 and out.max() <= 32767


def test_fast_layernorm_against_fp64_layer_norm(H):
    """Section 3.2.6: out = (x - mean) / std * L + b in Q3.12, within the quantization of its parts."""
    rng = np.random.default_rng(5)
    n = 1536
    q = np.clip(np.rint(rng.normal(300.0, 4000.0, n)), -32768, 32767).astype(np.int16)
    s_L = 1.3 / 32767.0
    Lr, br = rng.normal(1.0, 0.1, n), rng.normal(0.0, 0.1, n)
    L = np.rint(Lr / s_L).astype(np.int16)
    b = np.rint(br / (s_L * 2.0 ** -10)).astype(np.int32)
    real = s_L * 2.0 ** -10 / 2.0 ** -12
    frac, exp = math.frexp(real)
    eff = (int(round(frac * (1 << 31))), exp)
    out = np.empty(n, np.int16)
    H.qmh_layernorm_row_fast(q.ctypes.data_as(C.c_void_p), n, L.ctypes.data_as(C.c_void_p), b.ctypes.data_as(C.c_void_p),
                             eff[0], eff[1], out.ctypes.data_as(C.c_void_p))
    qf = q.astype(float)
    want = (qf - qf.mean()) / qf.std() * (L * s_L) + b * (s_L * 2.0 ** -10)
    assert np.abs(out / 4096.0 - want).max() <= 3e-3             # q' is on a 2^-10 grid: about 1e-3 per unit of L


def test_division_by_fixed_divisor_and_fp32_seeded_root(H):
    """The statistics' division by the row length as a multiplication (exact below 2^50 for lengths below 2^14) and
    the integer square root from an fp32 estimate, against Python integers."""
    rng = np.random.default_rng(41)
    for n in [1, 2, 3, 7, 16, 48, 640, 1000, 1024, 2048, 4095, 4096, 8191, 16383]:
        xs = [0, 1, n - 1, n, n + 1, 2 ** 50 - 1, 2 ** 50 - n, (2 ** 50 - 1) // n * n, (2 ** 50 - 1) // n * n - 1]
        xs += [int(v) for v in rng.integers(0, 2 ** 50, 300)] + [int(v) * n for v in rng.integers(0, 2 ** 36, 100)]
        xs += [int(v) * n - 1 for v in rng.integers(1, 2 ** 36, 100)]
        for x in xs:
            assert H.qmh_div_by_magic(x, n) == x // n, (x, n)
    vs = [0, 1, 2, 3, 4, 2 ** 52 - 1, 2 ** 50, 2 ** 50 - 1] + [int(v) for v in rng.integers(0, 2 ** 52, 2000)]
    for r in [1, 2, 4095, 4096, 2 ** 24 - 1, 2 ** 24, 2 ** 24 + 1, 2 ** 25 - 1, 2 ** 25, 2 ** 26 - 1, 33554431, 47453132]:
        vs += [r * r - 1, r * r, r * r + 1, r * r + r, r * r + 2 * r]
    for v in vs:
        assert H.qmh_isqrt_from_f32(v) == math.isqrt(v), v


def test_fast_statistics_equal_the_plain_ones_and_the_definition(H):
    """ln_stats_fast (no 64-bit division, no fp64 root) against ln_stats and against the definition in Python integers
    (Section 3.2.6): mean = round(2^10 sum / n), sigma = floor(sqrt(round(2^20 sumsq / n) - mean^2))."""
    rng = np.random.default_rng(42)

    def rdiv(a, b):
        q = (abs(a) + b // 2) // b
        return -q if a < 0 else q

    out_f, out_p = (C.c_int64 * 2)(), (C.c_int64 * 2)()
    cases = []
    for n in [1, 2, 16, 48, 640, 1024, 2048, 3000, 8191]:
        for kind in range(40):
            if kind == 0:
                q = np.full(n, 32767)
            elif kind == 1:
                q = np.full(n, -32768)
            elif kind == 2:
                q = np.where(np.arange(n) % 2 == 0, 32767, -32768)
            elif kind == 3:
                q = np.zeros(n, dtype=np.int64); q[0] = -32768
            elif kind == 4:
                q = np.full(n, 123)
            else:
                q = rng.integers(-32768, 32768, n) // int(rng.integers(1, 3000))
            q = q.astype(np.int64)
            cases.append((int(q.sum()), int((q * q).sum()), n))
    for s, s2, n in cases:
        H.qmh_ln_stats(s, s2, n, 1, out_f)
        H.qmh_ln_stats(s, s2, n, 0, out_p)
        mean = rdiv(s * 1024, n)
        var = rdiv(s2 * 1048576, n) - mean * mean
        sigma = math.isqrt(max(var, 0))
        assert (out_f[0], out_f[1]) == (mean, sigma), (s, s2, n)
        assert (out_p[0], out_p[1]) == (mean, sigma), (s, s2, n)
