"""Float (fp64) LSTM cell and sequence loop, Eq. 1-7 of the paper.

This is the high-precision computation that the integer-only LSTM approximates.
It serves two purposes, neither of them on the integer hot path:

* calibration: a run over a representative batch records the min/max of every
  activation tensor whose scale the quantization recipe (Table 2) derives from
  measured ranges (Section 4, post-training statistics collection);
* a pin for the integer oracle: dequantized integer outputs must stay within a
  stated quantization-error bound of this computation.

Gate order everywhere is i, f, z, o.  All weight matrices are row-major
[rows = output unit, cols = input unit].
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np

GATES = ("i", "f", "z", "o")


@dataclass
class FloatLayer:
    """Float parameters of one LSTM layer (Eq. 1-7 and the variants of Section 2)."""

    n_input: int
    n_cell: int
    n_output: int
    projection: bool = False
    peephole: bool = False
    layernorm: bool = False
    cifg: bool = False
    W: Dict[str, np.ndarray] = field(default_factory=dict)   # [n_cell, n_input]
    R: Dict[str, np.ndarray] = field(default_factory=dict)   # [n_cell, n_output]
    P: Dict[str, np.ndarray] = field(default_factory=dict)   # [n_cell]; gates i, f, o
    L: Dict[str, np.ndarray] = field(default_factory=dict)   # [n_cell]; layer-norm weights
    b: Dict[str, np.ndarray] = field(default_factory=dict)   # [n_cell]
    W_proj: Optional[np.ndarray] = None                      # [n_output, n_cell]
    b_proj: Optional[np.ndarray] = None                      # [n_output]

    @property
    def gates(self):
        return tuple(g for g in GATES if not (self.cifg and g == "i"))


@dataclass
class LayerStats:
    """Ranges logged during a float run (the green "log" nodes of the paper's figures)."""

    x_min: float = np.inf
    x_max: float = -np.inf
    h_min: float = np.inf
    h_max: float = -np.inf
    m_min: float = np.inf
    m_max: float = -np.inf
    c_absmax: float = 0.0
    g_absmax: Dict[str, float] = field(default_factory=lambda: {g: 0.0 for g in GATES})

    def see(self, name: str, v: np.ndarray) -> None:
        setattr(self, name + "_min", min(getattr(self, name + "_min"), float(v.min())))
        setattr(self, name + "_max", max(getattr(self, name + "_max"), float(v.max())))


def sigmoid(v: np.ndarray) -> np.ndarray:
    return 1.0 / (1.0 + np.exp(-v))


def layer_norm(v: np.ndarray) -> np.ndarray:
    """norm() of Eq. 1-5: zero mean, unit (population) standard deviation per row (Eq. 10-11)."""
    mean = v.mean(axis=-1, keepdims=True)
    var = (v * v).mean(axis=-1, keepdims=True) - mean * mean
    std = np.sqrt(np.maximum(var, 0.0))
    std = np.where(std == 0.0, 1.0, std)
    return (v - mean) / std


def cell_step(layer: FloatLayer, x: np.ndarray, h: np.ndarray, c: np.ndarray,
              stats: Optional[LayerStats] = None):
    """One time step for a batch: x [B, I], h [B, O], c [B, C] -> (h', c', m')."""

    def pre(g: str, c_peep: Optional[np.ndarray]) -> np.ndarray:
        a = x @ layer.W[g].T + h @ layer.R[g].T
        if layer.peephole and c_peep is not None:
            a = a + layer.P[g] * c_peep
        if layer.layernorm:
            if stats is not None:
                stats.g_absmax[g] = max(stats.g_absmax[g], float(np.abs(a).max()))
            a = layer_norm(a) * layer.L[g]
        return a + layer.b[g]

    f = sigmoid(pre("f", c))
    i = (1.0 - f) if layer.cifg else sigmoid(pre("i", c))
    z = np.tanh(pre("z", None))
    c_new = i * z + f * c
    o = sigmoid(pre("o", c_new))
    m = o * np.tanh(c_new)
    h_new = m @ layer.W_proj.T + layer.b_proj if layer.projection else m
    if stats is not None:
        stats.see("x", x)
        stats.see("h", h_new)
        stats.see("m", m)
        stats.c_absmax = max(stats.c_absmax, float(np.abs(c_new).max()))
    return h_new, c_new, m


def run_sequence(layers: List[FloatLayer], x: np.ndarray,
                 stats: Optional[List[LayerStats]] = None, keep_cell: bool = False):
    """Unidirectional multi-layer loop over time.  x [T, B, I] -> y [T, B, O_last].

    Initial h and c are zero.  Returns (y, per-layer outputs [T,B,O_l], per-layer c [T,B,C_l] or None).
    """
    T, B, _ = x.shape
    inp = x
    outs, cells = [], []
    for li, layer in enumerate(layers):
        h = np.zeros((B, layer.n_output))
        c = np.zeros((B, layer.n_cell))
        y = np.empty((T, B, layer.n_output))
        cs = np.empty((T, B, layer.n_cell)) if keep_cell else None
        st = stats[li] if stats is not None else None
        if st is not None:
            st.see("h", h)  # the initial state is part of the range h takes
        for t in range(T):
            h, c, _ = cell_step(layer, inp[t], h, c, st)
            y[t] = h
            if keep_cell:
                cs[t] = c
        outs.append(y)
        cells.append(cs)
        inp = y
    return inp, outs, cells
