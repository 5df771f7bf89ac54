"""Pins for the oracle's cell step and sequence loop: float LSTM agreement, an independent
restatement on tiny inputs, invariants, hand-built saturation cases, streaming equivalence."""
import numpy as np
import pytest

from oracle import qlstm_ref as R
from oracle import qlstm_np as NP
from tests.util import paper_values
from workloads import make_workload, random_layer_stack
from workloads.float_lstm import run_sequence
from workloads.quantize import QLayer, cell_int_bits


# ------------------------------------------------------------------ float LSTM (Eq. 1-7)

@pytest.mark.parametrize("index", [1, 2])
def test_agrees_with_float_lstm(index):
    w = make_workload(index)
    h0, c0 = w.initial_state()
    y, _, _, tr = R.run(w.layers, w.x, h0, c0, trace=True)
    yf, outs, cells = run_sequence(w.float_layers, w.x_float, keep_cell=True)
    q = w.layers[-1]
    err = np.abs(q.s_h * (y.astype(float) - q.zp_h) - yf)
    # stated quantization-error bound (measured: 0.0072 / 0.030 max, 0.4 / 0.65 int8 steps mean)
    assert err.max() <= 0.05
    assert err.mean() <= 1.0 * q.s_h
    quarter = max(1, w.T // 4)
    assert err[-quarter:].mean() <= 1.5 * q.s_h                       # no growth with t
    for l, ql in enumerate(w.layers):
        cerr = np.abs(ql.s_c * tr[l]["c"].astype(float) - cells[l])
        # the cell's error comes from the int8 x / h feeding it, not from its own 16-bit grid
        assert cerr.max() <= 0.25 and cerr.mean() <= 0.01, (cerr.max(), cerr.mean())   # measured 0.18 / 0.0068


@pytest.mark.parametrize("kw", [
    dict(projection=True, peephole=True, layernorm=True),
    dict(cifg=True),
    dict(peephole=True),
    dict(layernorm=True, cifg=True),
    dict(projection=True, cifg=True, peephole=True),
])
def test_variants_agree_with_float_lstm(kw):
    w = random_layer_stack(31, 1, 24, 64, 40, T=12, B=4, **kw)
    h0, c0 = w.initial_state()
    y, _, _, _ = R.run(w.layers, w.x, h0, c0)
    yf, _, _ = run_sequence(w.float_layers, w.x_float)
    q = w.layers[-1]
    err = np.abs(q.s_h * (y.astype(float) - q.zp_h) - yf)
    assert err.max() <= 0.06 and err.mean() <= 1.5 * q.s_h


# ------------------------------------------------------------------ independent restatement

def test_python_restatement_bit_equal_config1():
    w = make_workload(1)
    h0, c0 = w.initial_state()
    y, h, c, _ = R.run(w.layers, w.x, h0, c0)
    y2, h2, c2 = NP.run(w.layers, w.x, h0, c0)
    assert np.array_equal(y, y2) and np.array_equal(h, h2) and np.array_equal(c, c2)


def test_python_restatement_bit_equal_config2_prefix():
    w = make_workload(2, batch=2, T=3)
    h0, c0 = w.initial_state()
    y, h, c, _ = R.run(w.layers, w.x, h0, c0)
    y2, h2, c2 = NP.run(w.layers, w.x, h0, c0)
    assert np.array_equal(y, y2) and np.array_equal(h, h2) and np.array_equal(c, c2)


@pytest.mark.parametrize("seed,kw", [
    (1, dict(projection=True, peephole=True, layernorm=True)),
    (2, dict(cifg=True)),
    (3, dict(layernorm=True, projection=True)),
    (4, dict(peephole=True, cifg=True, layernorm=True)),
    (5, dict()),
])
def test_python_restatement_bit_equal_variants(seed, kw):
    w = random_layer_stack(seed, 2, 7, 12, 9, T=4, B=2, **kw)
    h0, c0 = w.initial_state()
    y, h, c, _ = R.run(w.layers, w.x, h0, c0)
    y2, h2, c2 = NP.run(w.layers, w.x, h0, c0)
    assert np.array_equal(y, y2) and np.array_equal(h, h2) and np.array_equal(c, c2)


# ------------------------------------------------------------------ invariants

def test_step_invariants_and_cifg_range():
    pv = paper_values()
    w = random_layer_stack(8, 2, 16, 48, 48, cifg=True, T=30, B=3)
    h0, c0 = w.initial_state()
    _, _, _, tr = R.run(w.layers, w.x, h0, c0, trace=True)
    for d in tr:
        g = d["gate"].astype(int)
        i, f, z, o = g[:, 0], g[:, 1], g[:, 2], g[:, 3]
        assert f.min() >= 0 and f.max() <= 32767 and o.min() >= 0 and o.max() <= 32767
        assert np.array_equal(i, np.minimum(32768 - f, 32767))
        assert i.min() >= int(pv["cifg_input_gate_min_q"]) and i.max() <= int(pv["cifg_input_gate_max_q"])
        assert z.min() >= -32768 and z.max() <= 32767
        assert np.all(d["acc"][:, 0] == 0) and np.all(d["xg"][:, 0] == 0)      # no i-gate matmul with CIFG


def test_cifg_coupling_exhaustive():
    pv = paper_values()
    f = np.arange(0, 32768)
    i = np.minimum(32768 - f, 32767)
    assert i.min() == int(pv["cifg_input_gate_min_q"]) and i.max() == int(pv["cifg_input_gate_max_q"])


def test_streaming_equivalence():
    """The state (h int8, c int16) carried across calls is the whole recurrent state (Section 3.2.2)."""
    w = random_layer_stack(9, 2, 10, 20, 14, projection=True, layernorm=True, T=9, B=3)
    h0, c0 = w.initial_state()
    y, h, c, _ = R.run(w.layers, w.x, h0, c0)
    y1, h1, c1, _ = R.run(w.layers, w.x[:4], h0, c0)
    y2, h2, c2, _ = R.run(w.layers, w.x[4:], h1, c1)
    assert np.array_equal(y, np.concatenate([y1, y2])) and np.array_equal(h, h2) and np.array_equal(c, c2)


def test_batch_rows_are_independent():
    w = random_layer_stack(10, 1, 10, 24, 24, layernorm=True, peephole=True, T=6, B=5)
    h0, c0 = w.initial_state()
    y, _, _, _ = R.run(w.layers, w.x, h0, c0)
    q = w.layers[0]
    for b in (0, 3):
        yb, _, _, _ = R.run(w.layers, w.x[:, b:b + 1], h0[:q.n_output], c0[:q.n_cell])
        assert np.array_equal(y[:, b], yb[:, 0])


def test_zero_point_identity():
    """Section 6: sum W (x - zp) = sum W x - zp sum W, exactly, in int32."""
    rng = np.random.default_rng(11)
    W = rng.integers(-127, 128, (64, 4096)).astype(np.int64)
    x = rng.integers(-128, 128, 4096).astype(np.int64)
    for zp in (-128, -7, 0, 127):
        unfolded = W @ (x - zp)
        folded = W @ x + (-zp * W.sum(axis=1))
        assert np.array_equal(unfolded, folded)
        assert np.abs(unfolded).max() < 2 ** 31 and np.abs(W @ x).max() < 2 ** 31


def test_cell_format_example_from_paper():
    pv = paper_values()
    assert cell_int_bits(max(abs(pv["cell_range_example_lo"]), abs(pv["cell_range_example_hi"]))) \
        == int(pv["cell_range_example_int_bits"])


# ------------------------------------------------------------------ hand-built extremes

def hand_layer(C=1, I=1, **kw) -> QLayer:
    q = QLayer(I, C, C, 0, 3, 0, 0, 0)
    one = (1 << 30, 1)
    for g in range(4):
        q.W[g] = np.zeros((C, I), np.int8)
        q.R[g] = np.zeros((C, C), np.int8)
        q.b[g] = np.zeros(C, np.int32)
        q.eff_x[g] = one
        q.eff_h[g] = one
    q.eff_m = (1 << 30, -21)                       # 2^-22: o * tanh(c) of 2^30 -> 256
    for k, v in kw.items():
        setattr(q, k, v)
    return q


def test_gate_sum_saturates_per_term_and_in_total():
    q = hand_layer(zp_x=-128, zp_h=-128)
    for g in range(4):
        q.W[g][:] = 127
        q.R[g][:] = 127
        q.eff_x[g] = (1 << 30, 3)                  # x4
        q.eff_h[g] = (1 << 30, 3)
    x = np.full((1, 1, 1), 127, np.int8)           # x - zp = 255 -> 127 * 255 * 4 > 32767
    h0 = np.full(1, 127, np.int8)
    _, _, _, tr = R.run([q], x, h0, np.zeros(1, np.int16), trace=True)
    d = tr[0]
    assert np.all(d["acc"][0] == 127 * 255)
    assert np.all(d["xg"][0] == 32767) and np.all(d["pre"][0] == 32767)
    assert d["gate"][0, 1, 0, 0] == R.sigmoid(32767, 3) and d["gate"][0, 2, 0, 0] == 32767
    # and the negative side reaches -32768, not -32767
    x = np.full((1, 1, 1), -128, np.int8)
    q.zp_x, q.zp_h = 127, 127
    _, _, _, tr = R.run([q], x, np.full(1, -128, np.int8), np.zeros(1, np.int16), trace=True)
    assert np.all(tr[0]["xg"][0] == -32768) and np.all(tr[0]["pre"][0] == -32768)
    assert tr[0]["gate"][0, 2, 0, 0] == -32768


def test_bias_rides_on_the_recurrent_accumulator_and_saturates():
    q = hand_layer()
    for g in range(4):
        q.R[g][:] = 127
        q.b[g][:] = 2 ** 31 - 1
        q.eff_h[g] = (1 << 30, -16)                # 2^-17
    _, _, _, tr = R.run([q], np.zeros((1, 1, 1), np.int8), np.full(1, 100, np.int8), np.zeros(1, np.int16), trace=True)
    assert np.all(tr[0]["acc"][0] == 2 ** 31 - 1)  # 12700 + (2^31 - 1) saturates
    assert np.all(tr[0]["pre"][0] == R.mbqm(2 ** 31 - 1, (1 << 30, -16)))


def test_cell_update_shifts_and_clamp():
    # i = sigmoid(+big) = 32767, z = tanh(+big) = 32767, f = 32767, c_old = 32767, m = 0:
    # round(32767^2 / 2^15) = 32766 twice -> 65532 -> clamps to 32767
    q = hand_layer(cell_int_bits=0)
    for g in range(4):
        q.b[g][:] = 32767
    c0 = np.full(1, 32767, np.int16)
    _, _, c, tr = R.run([q], np.zeros((1, 1, 1), np.int8), np.zeros(1, np.int8), c0, trace=True)
    assert c[0] == 32767
    # with m = 3 the i*z term is shifted by 18: round(32767^2 / 2^18) = 4096; f*c by 15
    q = hand_layer(cell_int_bits=3)
    for g in range(4):
        q.b[g][:] = 32767
    i_q, z_q = R.sigmoid(32767, 3), R.tanh(32767, 3)
    c0 = np.full(1, -1000, np.int16)
    _, _, c, tr = R.run([q], np.zeros((1, 1, 1), np.int8), np.zeros(1, np.int8), c0, trace=True)
    want = R.rdivpot(i_q * z_q, 18) + R.rdivpot(R.sigmoid(32767, 3) * -1000, 15)
    assert c[0] == want and want == 4095 - 1000
    # hidden state: o * tanh(c; m) rescaled by eff_m, plus zero point
    o_q = tr[0]["gate"][0, 3, 0, 0]
    assert tr[0]["m"][0, 0, 0] == max(-128, min(127, R.mbqm(int(o_q) * R.tanh(int(c[0]), 3), q.eff_m)))


def test_invalid_arguments_are_rejected():
    q = hand_layer()
    q.n_output = 2                                  # no projection but n_output != n_cell
    with pytest.raises(ValueError):
        R.run([q], np.zeros((1, 1, 1), np.int8), np.zeros(2, np.int8), np.zeros(1, np.int16))


def test_empty_batch_and_sequence():
    q = hand_layer()
    y, h, c, _ = R.run([q], np.zeros((0, 1, 1), np.int8), np.full(1, 5, np.int8), np.full(1, 9, np.int16))
    assert y.shape == (0, 1, 1) and h[0] == 5 and c[0] == 9
