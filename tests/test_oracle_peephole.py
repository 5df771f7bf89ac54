"""Pins for the oracle's peephole terms (Eq. 1, 2, 5; Section 3.2.3, 3.2.5).

Which cell state each gate's peephole sees is fixed by the float equations: the input and forget
gates read c^{t-1} (Eq. 1-2), the output gate reads c^t (Eq. 5), the update gate has none (Eq. 3).
The cases below are built so that the gate value changes by thousands of Q0.15 steps if a term is
dropped or reads the other cell state, and the expected values come from the float equations in
fp64, never from the integer code.  None of them uses the pure-Python restatement.
"""
import math

import numpy as np
import pytest

from oracle import qlstm_ref as R
from workloads.configs import Config, _draw_layers, _draw_x
from workloads.float_lstm import LayerStats, layer_norm, run_sequence, sigmoid
from workloads.quantize import FLAG_PEEPHOLE, QLayer, encode_scale, quantize_asym_int8, quantize_model


def sig(v):
    return 1.0 / (1.0 + math.exp(-v))


# ------------------------------------------------------------------ one cell, one step, by hand

def one_cell_layer(m_bits, b_real, P_real):
    """A single cell with no matmul contribution: every gate's pre-activation is its bias plus its
    peephole term.  Gate inputs are Q3.12 (scale 2^-12), the cell is Q_{m.15-m}; P is stored at
    scale |P| / 32767 and its product with c is rescaled to Q3.12 (Section 3.2.3)."""
    q = QLayer(1, 1, 1, FLAG_PEEPHOLE, m_bits, 0, 0, 0)
    s_c = 2.0 ** (m_bits - 15)
    for g in range(4):
        q.W[g] = np.zeros((1, 1), np.int8)
        q.R[g] = np.zeros((1, 1), np.int8)
        q.b[g] = np.array([round(b_real[g] * 4096)], np.int32)
        q.eff_x[g] = (1 << 30, 1)                       # identity: the accumulator is already Q3.12
        q.eff_h[g] = (1 << 30, 1)
        if g != 2:
            s_P = abs(P_real[g]) / 32767.0
            q.P[g] = np.array([round(P_real[g] / s_P)], np.int16)
            q.eff_c[g] = encode_scale(s_P * s_c / 2.0 ** -12)
    q.eff_m = encode_scale(2.0 ** -30 / (1.0 / 127.0))  # m at scale 1/127, zero point 0
    return q


@pytest.mark.parametrize("P_o", [-6.0, -1.0, 2.5])
def test_output_gate_peephole_reads_the_new_cell_state(P_o):
    # c^{t-1} = 0; i and z saturate high so that c^t = i z is close to 1; the output gate has no bias:
    # Eq. 5 gives o = sigmoid(P_o c^t), while c^{t-1} in its place would give sigmoid(0) = 1/2.
    m_bits = 3
    q = one_cell_layer(m_bits, b_real=[7.5, 0.0, 7.5, 0.0], P_real=[1.0, 1.0, None, P_o])
    _, _, c, tr = R.run([q], np.zeros((1, 1, 1), np.int8), np.zeros(1, np.int8), np.zeros(1, np.int16), trace=True)
    i, z = sig(7.5), math.tanh(7.5)
    c_new = i * z                                        # f c^{t-1} = 0
    assert abs(c[0] * 2.0 ** (m_bits - 15) - c_new) <= 2.0 ** (m_bits - 15)
    o = sig(P_o * c_new)
    o_q = int(tr[0]["gate"][0, 3, 0, 0])
    assert abs(o_q - 32768 * o) <= 4, (o_q, 32768 * o)   # a Q3.12 input step moves sigmoid by at most 2 steps of Q0.15
    assert abs(o_q - 16384) > 2000                       # far from what c^{t-1} = 0 would give
    # and the hidden state follows Eq. 6 with that o
    m_q = int(tr[0]["m"][0, 0, 0])
    assert abs(m_q - 127 * o * math.tanh(c_new)) <= 1.0


@pytest.mark.parametrize("c_prev,P_i,P_f", [(2.0, 1.0, -1.5), (-1.25, 2.0, 2.0), (3.0, -0.75, 0.5)])
def test_input_and_forget_peepholes_read_the_previous_cell_state(c_prev, P_i, P_f):
    # i = sigmoid(b_i + P_i c^{t-1}), f = sigmoid(b_f + P_f c^{t-1}) (Eq. 1-2); z has no peephole (Eq. 3)
    m_bits = 3
    b = [0.25, -0.5, 0.75, 0.0]
    q = one_cell_layer(m_bits, b_real=b, P_real=[P_i, P_f, None, 1.0])
    c0 = np.array([round(c_prev * 2 ** (15 - m_bits))], np.int16)
    _, _, c, tr = R.run([q], np.zeros((1, 1, 1), np.int8), np.zeros(1, np.int8), c0, trace=True)
    gate = tr[0]["gate"][0, :, 0, 0].astype(int)
    i, f, z = sig(b[0] + P_i * c_prev), sig(b[1] + P_f * c_prev), math.tanh(b[2])
    assert abs(gate[0] - 32768 * i) <= 4 and abs(gate[1] - 32768 * f) <= 4
    assert abs(gate[2] - 32768 * z) <= 9                 # tanh moves up to 8 steps of Q0.15 per Q3.12 input step
    # without their peephole terms the two gates would sit at sigmoid(b): thousands of steps away
    assert abs(gate[0] - 32768 * sig(b[0])) > 1500 and abs(gate[1] - 32768 * sig(b[1])) > 1500
    c_new = i * z + f * c_prev
    assert abs(c[0] * 2.0 ** (m_bits - 15) - c_new) <= 4 * 2.0 ** (m_bits - 15)
    o = sig(b[3] + 1.0 * c_new)                          # Eq. 5 again, now with c^{t-1} != 0 != c^t
    assert abs(int(tr[0]["gate"][0, 3, 0, 0]) - 32768 * o) <= 6
    assert abs(32768 * sig(b[3] + 1.0 * c_prev) - 32768 * o) > 300


# ------------------------------------------------------------------ random layers with strong peepholes

def strong_peephole_workload(seed, layernorm, projection=False, cifg=False, C=48, T=10, B=3):
    """One layer drawn by the usual recipe, its peephole weights scaled up to N(0, 1) so that
    P (.) c is of the order of the matmul terms (the recipe's N(0, 0.1) hides it under the
    quantization error)."""
    n_out = 32 if projection else C
    cfg = Config(0, "peephole-pin", 1, 20, C, n_out, projection, True, layernorm, cifg, T, (B,), "normal", True)
    rng = np.random.default_rng(seed)
    fls = _draw_layers(cfg, rng)
    for fl in fls:
        for g in fl.P:
            fl.P[g] = fl.P[g] * 10.0
    xf = _draw_x(cfg, rng, T, B)
    stats = [LayerStats() for _ in fls]
    run_sequence(fls, xf, stats)
    qls = quantize_model(fls, stats)
    return fls[0], qls[0], quantize_asym_int8(xf, qls[0].s_x, qls[0].zp_x)


def float_pre(fl, g, x, h, c_peep):
    """Pre-activation of gate g by Eq. 1-5 in fp64 (with the norm() of the layer-norm variant)."""
    a = x @ fl.W[g].T + h @ fl.R[g].T
    if c_peep is not None:
        a = a + fl.P[g] * c_peep
    if fl.layernorm:
        a = layer_norm(a) * fl.L[g]
    return a + fl.b[g]


@pytest.mark.parametrize("layernorm,projection,cifg", [(False, False, False), (True, False, False),
                                                       (True, True, False), (True, False, True)])
def test_gate_inputs_follow_the_float_equations_step_by_step(layernorm, projection, cifg):
    """Teacher-forced: at every step the float equations are evaluated on the oracle's own
    de-quantized x, h^{t-1}, c^{t-1} and c^t, so nothing accumulates and the bound is tight enough
    to tell c^t from c^{t-1} in the output gate and to see each peephole term, with layer norm too."""
    fl, q, xq = strong_peephole_workload(77, layernorm, projection, cifg)
    T, B = xq.shape[0], xq.shape[1]
    h0 = np.full(B * q.n_output, q.zp_h, np.int8)
    c0 = np.zeros(B * q.n_cell, np.int16)
    _, _, _, tr = R.run([q], xq, h0, c0, trace=True)
    d = tr[0]
    worst = {g: 0.0 for g in "ifzo"}
    gap_old_c, gap_no_peep = 0.0, {g: 0.0 for g in "ifo"}
    for t in range(T):
        x = q.s_x * (xq[t].astype(float) - q.zp_x)
        h_prev = q.s_h * ((d["h"][t - 1] if t else h0.reshape(B, -1)).astype(float) - q.zp_h)
        c_prev = q.s_c * (d["c"][t - 1] if t else c0.reshape(B, -1)).astype(float)
        c_new = q.s_c * d["c"][t].astype(float)
        for gi, g in enumerate("ifzo"):
            if cifg and g == "i":
                continue
            c_peep = None if g == "z" else (c_new if g == "o" else c_prev)
            want = float_pre(fl, g, x, h_prev, c_peep)
            got = d["ain"][t, gi].astype(float) / 4096.0
            worst[g] = max(worst[g], float(np.abs(np.clip(want, -8, 8) - got).max()))
            if g != "z":
                gap_no_peep[g] = max(gap_no_peep[g], float(np.abs(float_pre(fl, g, x, h_prev, None) - want).max()))
            if g == "o":
                gap_old_c = max(gap_old_c, float(np.abs(float_pre(fl, g, x, h_prev, c_prev) - want).max()))
    # measured: at most 0.034 over the four variants; the other readings are 1.9 or more away
    bound = 0.05
    for g, w in worst.items():
        assert w <= bound, (g, w)
    # the test has teeth: the other readings are several times the bound away
    assert gap_old_c >= 5 * bound
    for g, gap in gap_no_peep.items():
        if not (cifg and g == "i"):
            assert gap >= 5 * bound, (g, gap)


@pytest.mark.parametrize("layernorm", [False, True])
def test_strong_peephole_sequence_agrees_with_float_lstm(layernorm):
    """Free-running: the whole sequence against the float LSTM, peephole weights of order 1."""
    fl, q, xq = strong_peephole_workload(78, layernorm, T=8)
    T, B = xq.shape[0], xq.shape[1]
    y, _, _, _ = R.run([q], xq, np.full(B * q.n_output, q.zp_h, np.int8), np.zeros(B * q.n_cell, np.int16))
    xf = q.s_x * (xq.astype(float) - q.zp_x)             # the float model sees the same quantized input
    yf, _, _ = run_sequence([fl], xf)
    err = np.abs(q.s_h * (y.astype(float) - q.zp_h) - yf)
    assert err.max() <= 0.03, err.max()                  # measured 0.0154 / 0.0136
