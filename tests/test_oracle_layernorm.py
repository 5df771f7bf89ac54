"""Pins for the oracle's integer layer normalisation (Section 3.2.6)."""
import numpy as np
import pytest

from oracle import qlstm_ref as R
from oracle import qlstm_np as NP
from workloads.quantize import encode_scale


def float_ln(x, L, b):
    mean = x.mean()
    std = np.sqrt((x * x).mean() - mean * mean)
    return (x - mean) / std * L + b


@pytest.mark.parametrize("n,seed", [(32, 0), (256, 1), (2048, 2), (1000, 3)])
def test_matches_float_layer_norm(n, seed):
    rng = np.random.default_rng(seed)
    s_in = 3.7e-4                                     # any input scale: it cancels (Section 3.2.6)
    x = rng.normal(0.3, 1.5, n)
    q = np.clip(np.rint(x / s_in), -32767, 32767).astype(np.int16)
    Lf = rng.normal(1.0, 0.1, n)
    bf = rng.normal(0.0, 0.1, n)
    s_L = np.abs(Lf).max() / 32767
    Lq = np.rint(Lf / s_L).astype(np.int16)
    bq = np.rint(bf / (s_L * 2.0 ** -10)).astype(np.int32)
    eff = encode_scale(s_L * 2.0 ** -10 / 2.0 ** -12)
    got = R.layernorm_row(q, Lq, bq, eff).astype(float) / 4096.0
    want = float_ln(q.astype(float), Lf, bf)
    # q' carries 10 fractional bits, the output 12: error well below 2^-9 per element
    assert np.abs(got - want).max() < 4e-3
    assert np.abs(got - want).mean() < 1e-3


def test_input_scale_cancels():
    rng = np.random.default_rng(4)
    q = rng.integers(-2000, 2000, 128).astype(np.int16)
    L = np.full(128, 30000, np.int16)
    b = np.zeros(128, np.int32)
    eff = encode_scale(4.0 * 1.1 / 32767)
    a = R.layernorm_row(q, L, b, eff).astype(int)
    c = R.layernorm_row((q * 8).astype(np.int16), L, b, eff).astype(int)
    assert np.abs(a - c).max() <= 2


def test_constant_row_gives_bias_only():
    n = 64
    q = np.full(n, 1234, np.int16)
    L = np.arange(1, n + 1, dtype=np.int16) * 100
    b = (np.arange(n, dtype=np.int32) - 32) * 5000
    eff = (1 << 30, -3)                              # 0.5 * 2^-3 = 1/16
    got = R.layernorm_row(q, L, b, eff)
    want = [R.mbqm(int(v), eff) for v in b]
    assert list(got) == want


def test_extreme_rows_do_not_overflow():
    n = 8191                                          # largest width the int64 sum of squares admits
    for pattern in ("alt", "one", "max"):
        if pattern == "alt":
            q = np.where(np.arange(n) % 2 == 0, 32767, -32768).astype(np.int16)
        elif pattern == "one":
            q = np.zeros(n, np.int16)
            q[17] = 32767
        else:
            q = np.full(n, -32768, np.int16)
            q[0] = 32767
        L = np.full(n, 32767, np.int16)
        b = np.full(n, 2 ** 31 - 1, np.int32)
        eff = (1 << 30, -8)
        got = R.layernorm_row(q, L, b, eff)
        want = NP.layernorm_q([int(v) for v in q], [int(v) for v in L], [int(v) for v in b], eff)
        assert list(got) == want


@pytest.mark.parametrize("seed", range(6))
def test_agrees_with_python_integers(seed):
    rng = np.random.default_rng(100 + seed)
    n = int(rng.integers(1, 300))
    q = rng.integers(-32768, 32768, n).astype(np.int16) // int(rng.integers(1, 50))
    L = rng.integers(-32767, 32768, n).astype(np.int16)
    b = rng.integers(-2 ** 31 + 1, 2 ** 31, n).astype(np.int32) // int(rng.integers(1, 4000))
    eff = (int(rng.integers(1 << 30, 1 << 31)), int(rng.integers(-14, -6)))
    got = R.layernorm_row(q, L, b, eff)
    want = NP.layernorm_q([int(v) for v in q], [int(v) for v in L], [int(v) for v in b], eff)
    assert list(got) == want


def test_normalised_values_fit_the_extra_scale():
    """s' = 2^-10: |q'| <= 2^10 * sqrt(n - 1) (the largest possible z-score), far inside int32."""
    n = 2048
    q = np.zeros(n, np.int16)
    q[5] = 32767                                      # one outlier: z-score sqrt(n - 1)
    L = np.full(n, 1, np.int16)
    b = np.zeros(n, np.int32)
    out = R.layernorm_row(q, L, b, (1 << 30, 1))      # identity scale: out = sat16(q' * 1)
    assert out[5] == 32767 or abs(int(out[5]) - round(1024 * np.sqrt(n - 1))) <= 2
    assert 1024 * np.sqrt(n - 1) < 2 ** 31
