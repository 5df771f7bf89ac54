"""Offline quantizer: float LSTM + logged ranges -> integer tensors and scales (Table 2).

Everything here happens before the integer hot path runs: it produces the
*inputs* of that path (int8 weights, int32 biases, int16 peephole / layer-norm
weights, zero points, and effective scales encoded as (multiplier, shift)).
None of the integer execution arithmetic (rescale, integer activations, integer
layer norm, cell update) lives in this module.

Readings of the paper taken here:
* affine convention real = scale * (q - zero_point);
* int8 asymmetric tensors: scale = range / 255 with the range first widened to
  contain 0, zero point rounded and clamped so that float 0 maps to an integer
  (the "nudging" of Section 3.2.4);
* symmetric tensors: max|.| / 127 (int8), max|.| / 32767 (int16);
* cell state: measured max|c| extended to the next power of two 2^m, scale
  2^m / 32768, i.e. Q_{m.15-m} (Section 3.2.2);
* "range" in the caption of Table 2 is max - min (the absolute values printed
  there are a typo).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np

from .float_lstm import GATES, FloatLayer, LayerStats

FLAG_PROJECTION = 1
FLAG_PEEPHOLE = 2
FLAG_LAYERNORM = 4
FLAG_CIFG = 8


def encode_scale(real: float) -> Tuple[int, int]:
    """real > 0 -> (multiplier, shift) with real ~= multiplier * 2^(shift-31), multiplier in [2^30, 2^31)."""
    if real == 0.0:
        return 0, 0
    assert real > 0.0 and math.isfinite(real)
    frac, exp = math.frexp(real)          # real = frac * 2^exp, frac in [0.5, 1)
    mult = int(round(frac * (1 << 31)))
    if mult == (1 << 31):
        mult //= 2
        exp += 1
    assert (1 << 30) <= mult < (1 << 31)
    assert -31 <= exp <= 30, f"effective scale {real} outside the encodable window"
    return mult, exp


def decode_scale(ms: Tuple[int, int]) -> float:
    return ms[0] * 2.0 ** (ms[1] - 31)


def asym_int8_params(lo: float, hi: float) -> Tuple[float, int]:
    lo, hi = min(lo, 0.0), max(hi, 0.0)
    if hi == lo:
        hi = lo + 1.0
    scale = (hi - lo) / 255.0
    zp = int(round(-128.0 - lo / scale))
    return scale, max(-128, min(127, zp))


def quantize_asym_int8(v: np.ndarray, scale: float, zp: int) -> np.ndarray:
    return np.clip(np.rint(v / scale) + zp, -128, 127).astype(np.int8)


def sym_scale(v: np.ndarray, qmax: int) -> float:
    m = float(np.abs(v).max())
    return (m if m > 0.0 else 1.0) / qmax


def quantize_sym(v: np.ndarray, scale: float, qmax: int, dtype) -> np.ndarray:
    return np.clip(np.rint(v / scale), -qmax, qmax).astype(dtype)


def cell_int_bits(absmax: float) -> int:
    """m of Q_{m.15-m}: smallest m >= 0 with 2^m >= max|c| (Section 3.2.2)."""
    m = 0
    while (1 << m) < absmax:
        m += 1
    return m


@dataclass
class QLayer:
    """One integer LSTM layer as the C-ABI's create call takes it."""

    n_input: int
    n_cell: int
    n_output: int
    flags: int
    cell_int_bits: int
    zp_x: int
    zp_m: int
    zp_h: int
    W: List[Optional[np.ndarray]] = field(default_factory=lambda: [None] * 4)   # int8 [C, I]
    R: List[Optional[np.ndarray]] = field(default_factory=lambda: [None] * 4)   # int8 [C, O]
    P: List[Optional[np.ndarray]] = field(default_factory=lambda: [None] * 4)   # int16 [C]
    b: List[Optional[np.ndarray]] = field(default_factory=lambda: [None] * 4)   # int32 [C]
    L: List[Optional[np.ndarray]] = field(default_factory=lambda: [None] * 4)   # int16 [C]
    W_proj: Optional[np.ndarray] = None                                          # int8 [O, C]
    b_proj: Optional[np.ndarray] = None                                          # int32 [O]
    eff_x: List[Tuple[int, int]] = field(default_factory=lambda: [(0, 0)] * 4)
    eff_h: List[Tuple[int, int]] = field(default_factory=lambda: [(0, 0)] * 4)
    eff_c: List[Tuple[int, int]] = field(default_factory=lambda: [(0, 0)] * 4)
    eff_ln: List[Tuple[int, int]] = field(default_factory=lambda: [(0, 0)] * 4)
    eff_m: Tuple[int, int] = (0, 0)
    eff_proj: Tuple[int, int] = (0, 0)
    # real scales, kept for de-quantizing in tests; not consumed by the integer path
    s_x: float = 0.0
    s_h: float = 0.0
    s_m: float = 0.0
    s_c: float = 0.0

    @property
    def projection(self):
        return bool(self.flags & FLAG_PROJECTION)

    @property
    def peephole(self):
        return bool(self.flags & FLAG_PEEPHOLE)

    @property
    def layernorm(self):
        return bool(self.flags & FLAG_LAYERNORM)

    @property
    def cifg(self):
        return bool(self.flags & FLAG_CIFG)

    @property
    def gate_ids(self):
        return tuple(g for g in range(4) if not (self.cifg and g == 0))


def quantize_layer(fl: FloatLayer, st: LayerStats, x_scale_zp: Tuple[float, int]) -> QLayer:
    """Apply Table 2 to one layer.  x_scale_zp is the (scale, zero point) of this layer's input."""
    s_x, zp_x = x_scale_zp
    s_h, zp_h = asym_int8_params(st.h_min, st.h_max)
    if fl.projection:
        s_m, zp_m = asym_int8_params(st.m_min, st.m_max)
    else:
        s_m, zp_m = s_h, zp_h
    m_bits = cell_int_bits(st.c_absmax)
    s_c = 2.0 ** (m_bits - 15)
    flags = ((FLAG_PROJECTION if fl.projection else 0) | (FLAG_PEEPHOLE if fl.peephole else 0)
             | (FLAG_LAYERNORM if fl.layernorm else 0) | (FLAG_CIFG if fl.cifg else 0))
    q = QLayer(fl.n_input, fl.n_cell, fl.n_output, flags, m_bits, zp_x, zp_m, zp_h,
               s_x=s_x, s_h=s_h, s_m=s_m, s_c=s_c)
    for gi, g in enumerate(GATES):
        if fl.cifg and g == "i":
            continue
        s_W = sym_scale(fl.W[g], 127)
        s_R = sym_scale(fl.R[g], 127)
        q.W[gi] = quantize_sym(fl.W[g], s_W, 127, np.int8)
        q.R[gi] = quantize_sym(fl.R[g], s_R, 127, np.int8)
        if fl.layernorm:
            gm = st.g_absmax[g]
            s_gate = (gm if gm > 0.0 else 1.0) / 32767.0            # Section 3.2.5
            s_L = sym_scale(fl.L[g], 32767)
            q.L[gi] = quantize_sym(fl.L[g], s_L, 32767, np.int16)
            s_b = s_L * 2.0 ** -10                                  # Section 3.2.6
            q.eff_ln[gi] = encode_scale(s_b / 2.0 ** -12)
        else:
            s_gate = 2.0 ** -12                                     # Q3.12, Section 3.2.4
            s_b = s_R * s_h
        q.b[gi] = np.clip(np.rint(fl.b[g] / s_b), -(2 ** 31 - 1), 2 ** 31 - 1).astype(np.int32)
        q.eff_x[gi] = encode_scale(s_W * s_x / s_gate)
        q.eff_h[gi] = encode_scale(s_R * s_h / s_gate)
        if fl.peephole and g != "z":
            s_P = sym_scale(fl.P[g], 32767)
            q.P[gi] = quantize_sym(fl.P[g], s_P, 32767, np.int16)
            q.eff_c[gi] = encode_scale(s_P * s_c / s_gate)
    q.eff_m = encode_scale(2.0 ** -30 / s_m)                        # Section 3.2.7
    if fl.projection:
        s_Wp = sym_scale(fl.W_proj, 127)
        q.W_proj = quantize_sym(fl.W_proj, s_Wp, 127, np.int8)
        s_bp = s_Wp * s_m
        q.b_proj = np.clip(np.rint(fl.b_proj / s_bp), -(2 ** 31 - 1), 2 ** 31 - 1).astype(np.int32)
        q.eff_proj = encode_scale(s_Wp * s_m / s_h)                 # Section 3.2.8
    return q


def quantize_model(layers: List[FloatLayer], stats: List[LayerStats]) -> List[QLayer]:
    """Quantize a stack; layer l+1 reads layer l's h with that h's (scale, zero point)."""
    out = []
    xq = asym_int8_params(stats[0].x_min, stats[0].x_max)
    for fl, st in zip(layers, stats):
        ql = quantize_layer(fl, st, xq)
        out.append(ql)
        xq = (ql.s_h, ql.zp_h)
    return out
