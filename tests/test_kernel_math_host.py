"""The kernels' integer arithmetic (csrc/qmath.cuh), compiled for the host, swept against the oracle.

This runs the very source the CUDA kernels compile, on the CPU, so that a wrong shift or rounding in
the device code shows up without a GPU.  The oracle stays the reference; nothing here feeds it.
"""
import ctypes as C

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
    lib.qmh_cell_update.restype = C.c_int32
    lib.qmh_cell_update.argtypes = [C.c_int32] * 5
    lib.qmh_hidden.restype = C.c_int32
    lib.qmh_hidden.argtypes = [C.c_int32] * 6
    return lib


@pytest.mark.parametrize("m", [0, 1, 2, 3, 4, 5, 6, 9, 15])
def test_activations_exhaustive(H, m):
    out = np.empty(65536, np.int32)
    H.qmh_sigmoid_all(m, out.ctypes.data_as(C.c_void_p))
    assert np.array_equal(out, R.sigmoid_all(m))
    H.qmh_tanh_all(m, out.ctypes.data_as(C.c_void_p))
    assert np.array_equal(out, R.tanh_all(m))


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


@pytest.mark.parametrize("seed", range(8))
def test_layernorm_rows(H, seed):
    rng = np.random.default_rng(50 + seed)
    n = int(rng.integers(1, 2100))
    q = (rng.integers(-32768, 32768, n) // int(rng.integers(1, 60))).astype(np.int16)
    if seed == 0:
        q[:] = 77
    L = rng.integers(-32767, 32768, n).astype(np.int16)
    b = (rng.integers(-2 ** 31 + 1, 2 ** 31, n) // int(rng.integers(1, 3000))).astype(np.int32)
    eff = (int(rng.integers(1 << 30, 1 << 31)), int(rng.integers(-14, -6)))
    out = np.empty(n, np.int16)
    H.qmh_layernorm_row(q.ctypes.data_as(C.c_void_p), n, L.ctypes.data_as(C.c_void_p), b.ctypes.data_as(C.c_void_p),
                        eff[0], eff[1], out.ctypes.data_as(C.c_void_p))
    assert np.array_equal(out, R.layernorm_row(q, L, b, eff))


def test_cell_update_and_hidden(H):
    rng = np.random.default_rng(2)
    for _ in range(3000):
        i, f, o = (int(v) for v in rng.integers(0, 32768, 3))
        z, c = (int(v) for v in rng.integers(-32768, 32768, 2))
        m = int(rng.integers(0, 7))
        want_c = R.rdivpot(i * z, 15 + m) + R.rdivpot(f * c, 15)
        want_c = max(-32768, min(32767, want_c))
        assert H.qmh_cell_update(i, z, f, c, m) == want_c
        eff = (int(rng.integers(1 << 30, 1 << 31)), -22)
        zp = int(rng.integers(-128, 128))
        want_m = max(-128, min(127, R.mbqm(o * R.tanh(want_c, m), eff) + zp))
        assert H.qmh_hidden(o, want_c, m, eff[0], eff[1], zp) == want_m


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
