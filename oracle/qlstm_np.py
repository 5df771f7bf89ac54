"""Second, independent restatement of the integer LSTM in pure Python integers.

TEST INFRASTRUCTURE ONLY.  Written from the step list of the integer execution graph
(Section 3.2 of the paper), not from the C oracle: unbounded Python ints and exact
`fractions.Fraction` rounding instead of shifts and masks, whole-vector passes instead
of a per-row step function.  It is slow and meant for tiny cases; its only job is to
fail when the C oracle drops a term, flips a sign or transposes an operand.
"""
from __future__ import annotations

import math
from fractions import Fraction
from typing import List, Sequence

import numpy as np


def rnd(v: Fraction) -> int:
    """Nearest integer, ties away from zero."""
    if v >= 0:
        return math.floor(v + Fraction(1, 2))
    return -math.floor(-v + Fraction(1, 2))


def clamp(v: int, bits: int) -> int:
    lo, hi = -(1 << (bits - 1)), (1 << (bits - 1)) - 1
    return max(lo, min(hi, v))


def rescale(x: int, scale) -> int:
    """int32 x times multiplier * 2^(shift-31): saturating left shift, rounded high multiply, rounded right shift."""
    mult, shift = int(scale[0]), int(scale[1])
    if shift > 0:
        x = clamp(x << shift, 32)
    hi = (1 << 31) - 1 if (x == -(1 << 31) and mult == -(1 << 31)) else rnd(Fraction(x * mult, 1 << 31))
    return rnd(Fraction(hi, 1 << -shift)) if shift < 0 else hi


_LOG2E = 1549082005
_POLY = [759250125, -526272083, 182392005, -42141501, 7302566, -1012351, 116951]


def _exp_neg(a: int, m: int, k: int) -> int:
    t = rnd(Fraction(a * _LOG2E * k, 1 << (15 - m + 4)))
    n, f = divmod(t, 1 << 26)
    n = min(n, 40)
    g = f - (1 << 25)
    acc = _POLY[6]
    for ck in reversed(_POLY[:6]):
        acc = rnd(Fraction(acc * g, 1 << 26)) + ck
    return rnd(Fraction(acc, 1 << n))


def sigmoid_q(x: int, m: int = 3) -> int:
    E = _exp_neg(abs(x), m, 1)
    S = math.floor(Fraction(1 << 45, (1 << 30) + E) + Fraction(1, 2))
    return min(S, 32767) if x >= 0 else 32768 - S


def tanh_q(x: int, m: int = 3) -> int:
    E = _exp_neg(abs(x), m, 2)
    Tq = math.floor(Fraction(((1 << 30) - E) << 15, (1 << 30) + E) + Fraction(1, 2))
    return min(Tq, 32767) if x >= 0 else -Tq


def layernorm_q(q: Sequence[int], L: Sequence[int], b: Sequence[int], eff_ln) -> List[int]:
    n = len(q)
    mean = rnd(Fraction(1024 * sum(q), n))
    var = rnd(Fraction((1 << 20) * sum(v * v for v in q), n)) - mean * mean
    sigma = math.isqrt(max(var, 0))
    out = []
    for qi, Li, bi in zip(q, L, b):
        qp = 0 if sigma == 0 else rnd(Fraction(1024 * (1024 * qi - mean), sigma))
        out.append(clamp(rescale(clamp(qp * Li + bi, 32), eff_ln), 16))
    return out


def run(layers: Sequence, x: np.ndarray, h0: np.ndarray, c0: np.ndarray):
    """Same contract as oracle.qlstm_ref.run without the trace: returns (y, h, c)."""
    T, B, _ = x.shape
    seq = [[[int(v) for v in x[t, b]] for b in range(B)] for t in range(T)]
    h_out, c_out = [], []
    ho = co = 0
    for q in layers:
        C, O, I = q.n_cell, q.n_output, q.n_input
        LN, PH, PR, CIFG = q.layernorm, q.peephole, q.projection, q.cifg
        W = [None if w is None else w.astype(object) for w in q.W]
        R = [None if r is None else r.astype(object) for r in q.R]
        hs = [[int(v) for v in h0[ho + b * O: ho + (b + 1) * O]] for b in range(B)]
        cs = [[int(v) for v in c0[co + b * C: co + (b + 1) * C]] for b in range(B)]
        nxt = []
        for t in range(T):
            row_out = []
            for b in range(B):
                xin = np.array([v - q.zp_x for v in seq[t][b]], dtype=object)
                hin = np.array([v - q.zp_h for v in hs[b]], dtype=object)
                c_old = cs[b]

                def gate(g, c_peep):
                    ax = W[g].dot(xin)
                    ah = R[g].dot(hin)
                    pre = []
                    for u in range(C):
                        a = int(ah[u]) + (0 if LN else int(q.b[g][u]))
                        s = clamp(rescale(clamp(int(ax[u]), 32), q.eff_x[g]), 16)
                        s += clamp(rescale(clamp(a, 32), q.eff_h[g]), 16)
                        if PH and c_peep is not None:
                            s += clamp(rescale(int(q.P[g][u]) * c_peep[u], q.eff_c[g]), 16)
                        pre.append(clamp(s, 16))
                    if LN:
                        pre = layernorm_q(pre, [int(v) for v in q.L[g]], [int(v) for v in q.b[g]], q.eff_ln[g])
                    return pre

                f = [sigmoid_q(v) for v in gate(1, c_old)]
                if CIFG:
                    i = [min(32768 - v, 32767) for v in f]
                else:
                    i = [sigmoid_q(v) for v in gate(0, c_old)]
                z = [tanh_q(v) for v in gate(2, None)]
                mb = q.cell_int_bits
                c_new = [clamp(rnd(Fraction(i[u] * z[u], 1 << (15 + mb))) + rnd(Fraction(f[u] * c_old[u], 1 << 15)), 16)
                         for u in range(C)]
                o = [sigmoid_q(v) for v in gate(3, c_new)]
                m = [clamp(rescale(o[u] * tanh_q(c_new[u], mb), q.eff_m) + q.zp_m, 8) for u in range(C)]
                if PR:
                    mz = np.array([v - q.zp_m for v in m], dtype=object)
                    acc = q.W_proj.astype(object).dot(mz)
                    hn = [clamp(rescale(clamp(int(acc[p]) + int(q.b_proj[p]), 32), q.eff_proj) + q.zp_h, 8)
                          for p in range(O)]
                else:
                    hn = m
                hs[b], cs[b] = hn, c_new
                row_out.append(list(hn))
            nxt.append(row_out)
        seq = nxt
        h_out += [v for b in range(B) for v in hs[b]]
        c_out += [v for b in range(B) for v in cs[b]]
        ho += B * O
        co += B * C
    y = np.array(seq, dtype=np.int8).reshape(T, B, layers[-1].n_output)
    return y, np.array(h_out, np.int8), np.array(c_out, np.int16)
