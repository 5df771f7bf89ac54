"""Pins for the oracle's integer sigmoid / tanh: exhaustive int16 sweeps against fp64 closed forms."""
import math

import numpy as np
import pytest

from oracle import qlstm_ref as R
from oracle import qlstm_np as NP
from tests.util import paper_values

XS = np.arange(-32768, 32768)


@pytest.mark.parametrize("m", range(0, 7))
def test_sigmoid_exhaustive_against_double(m):
    got = R.sigmoid_all(m)
    real = XS * 2.0 ** -(15 - m)
    want = 32768.0 / (1.0 + np.exp(-real))
    err = np.abs(got - want)
    assert got.min() >= 0 and got.max() <= 32767
    assert err.max() <= 1.0                                   # everywhere, incl. the forced clamp at 32767/32768
    assert err[want < 32767.0].max() <= 0.51                  # away from the clamp
    assert np.all(np.diff(got) >= 0)                          # monotone
    assert got[32768] == 16384                                # sigmoid(0) = 1/2
    unclamped = got[32768 + 1:] < 32767
    sym = got[32768 + 1:] + got[32768 - 1:0:-1]               # s(x) + s(-x) = 1
    assert np.all(sym[unclamped] == 32768)


@pytest.mark.parametrize("m", range(0, 7))
def test_tanh_exhaustive_against_double(m):
    got = R.tanh_all(m)
    real = XS * 2.0 ** -(15 - m)
    want = 32768.0 * np.tanh(real)
    err = np.abs(got - want)
    assert got.min() >= -32768 and got.max() <= 32767
    assert err.max() <= 1.0
    assert err[want < 32767.0].max() <= 0.51
    assert np.all(np.diff(got) >= 0)
    assert got[32768] == 0
    pos, neg = got[32768 + 1:], got[32768 - 1:0:-1]
    assert np.all((pos == -neg) | ((pos == 32767) & (neg == -32768)))   # odd except at the clamp


@pytest.mark.parametrize("m", [7, 10, 15])
def test_wide_cell_formats_stay_in_range(m):
    """tanh of the cell takes the cell's own Q_{m.15-m}; large m must still be total and accurate."""
    got = R.tanh_all(m)
    want = 32768.0 * np.tanh(XS * 2.0 ** -(15 - m))
    assert np.abs(got - want).max() <= 1.0 and np.all(np.diff(got) >= 0)


def test_paper_printed_values():
    pv = paper_values()
    # clamping error of Q3.12: 1 - tanh(8)
    # (fp64 gives 2.25e-7; the printed 2.35e-7 is within 5 % of it)
    assert math.isclose(1.0 - math.tanh(8.0), pv["tanh_clamp_error_at_8"], rel_tol=5e-2)
    # the largest Q3.12 input is just below 8: the integer tanh reaches the top code there
    assert R.tanh(32767, 3) == int(pv["activation_out_max_q"])
    assert R.tanh(-32768, 3) == int(pv["activation_out_min_q"])
    # resolution error at 0: tanh(2^-12); one input LSB moves the Q0.15 output by round(32768 * that) = 8
    assert math.isclose(math.tanh(2.0 ** -12), pv["tanh_resolution_error_at_0"], rel_tol=5e-3)
    assert R.tanh(1, 3) == round(32768 * math.tanh(2.0 ** -12)) == 8
    assert R.sigmoid(1, 3) - R.sigmoid(0, 3) == round(32768 * 0.25 * 2.0 ** -12)


def test_q3_12_balances_clamping_and_resolution_error():
    """Section 3.2.1: clamping error f(inf) - f(2^m) vs resolution error 2^-n max f'; Q3.12 is best overall."""
    pv = paper_values()

    def total(m):
        n = 15 - m
        tanh_err = max(1.0 - math.tanh(2.0 ** m), math.tanh(2.0 ** -n))
        sig = lambda v: 1.0 / (1.0 + math.exp(-v))
        sig_err = max(1.0 - sig(2.0 ** m), sig(2.0 ** -n) - 0.5)
        return tanh_err + sig_err

    best = min(range(0, 8), key=total)
    assert best == int(pv["best_activation_int_bits"])


def test_python_restatement_agrees_on_a_sample():
    rng = np.random.default_rng(5)
    xs = list(rng.integers(-32768, 32768, 3000)) + [-32768, -1, 0, 1, 32767]
    for m in (0, 2, 3, 4, 5):
        for x in xs:
            assert R.sigmoid(int(x), m) == NP.sigmoid_q(int(x), m)
            assert R.tanh(int(x), m) == NP.tanh_q(int(x), m)
