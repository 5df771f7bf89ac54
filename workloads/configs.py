"""Seeded synthetic workloads: the five speech-shaped integer-LSTM configurations.

The paper's own experiments use private speech sets and trained RNN-T weights
(Section 5); neither is available, so every input here is synthetic with the
shapes of those models ("10 layers of LSTM, 2048 hidden units", LSTMx8 encoder)
and the value distributions stated below.

Recipe (deterministic; numpy default_rng(20210105 + config index)):
  draw order, per layer, per gate in order i, f, z, o (gate i skipped with CIFG):
      W ~ N(0, 1/sqrt(n_input)), R ~ N(0, 1/sqrt(n_output)),
      [P ~ N(0, 0.1) for gates i, f, o], [L ~ N(1, 0.1)], b ~ N(0, 0.1) (+1.0 on the forget gate);
  then W_proj ~ N(0, 1/sqrt(n_cell)), b_proj ~ N(0, 0.1); after all layers the input x.
  Calibration: the float LSTM runs on a separate batch (seed + 1000, batch 8, same T and
  distribution; config 1 calibrates on its own input) and the logged ranges fix every scale,
  so scales are model constants shared by all batch sizes.
  Initial state: h = zero point of h (float 0), c = 0.
"""
from __future__ import annotations

import functools
from dataclasses import dataclass
from typing import List, Optional, Tuple

import numpy as np

from .float_lstm import GATES, FloatLayer, LayerStats, run_sequence
from .quantize import QLayer, quantize_asym_int8, quantize_model

BASE_SEED = 20210105


@dataclass(frozen=True)
class Config:
    index: int
    name: str
    n_layers: int
    n_input: int
    n_cell: int
    n_output: int
    projection: bool
    peephole: bool
    layernorm: bool
    cifg: bool
    T: int
    batches: Tuple[int, ...]
    x_dist: str            # "uniform" -> U[-1, 1]; "normal" -> N(0, 1)
    calib_self: bool = False


CONFIGS = {
    1: Config(1, "basic-1x32", 1, 16, 32, 32, False, False, False, False, 20, (1,), "uniform", True),
    2: Config(2, "basic-2x256", 2, 80, 256, 256, False, False, False, False, 100, (8,), "normal"),
    3: Config(3, "ln-peephole-proj-1x2048", 1, 512, 2048, 640, True, True, True, False, 200, (32,), "normal"),
    4: Config(4, "cifg-5x1024", 5, 640, 1024, 1024, False, False, False, True, 500, (64,), "normal"),
    5: Config(5, "ln-proj-8x2048", 8, 640, 2048, 640, True, False, True, False, 300, (1, 8, 64, 256), "normal"),
}


@dataclass
class Workload:
    config: Config
    float_layers: List[FloatLayer]
    layers: List[QLayer]
    x_float: np.ndarray      # [T, B, I] fp64
    x: np.ndarray            # [T, B, I] int8
    T: int
    B: int

    def initial_state(self) -> Tuple[np.ndarray, np.ndarray]:
        """(h int8 [sum_l B*O_l], c int16 [sum_l B*C_l]) flattened layer after layer."""
        h = np.concatenate([np.full(self.B * q.n_output, q.zp_h, np.int8) for q in self.layers])
        c = np.concatenate([np.zeros(self.B * q.n_cell, np.int16) for q in self.layers])
        return h, c


def _draw_layers(cfg: Config, rng: np.random.Generator) -> List[FloatLayer]:
    layers = []
    n_in = cfg.n_input
    for _ in range(cfg.n_layers):
        fl = FloatLayer(n_in, cfg.n_cell, cfg.n_output, cfg.projection, cfg.peephole, cfg.layernorm, cfg.cifg)
        for g in GATES:
            if cfg.cifg and g == "i":
                continue
            fl.W[g] = rng.normal(0.0, 1.0 / np.sqrt(n_in), (cfg.n_cell, n_in))
            fl.R[g] = rng.normal(0.0, 1.0 / np.sqrt(cfg.n_output), (cfg.n_cell, cfg.n_output))
            if cfg.peephole and g != "z":
                fl.P[g] = rng.normal(0.0, 0.1, cfg.n_cell)
            if cfg.layernorm:
                fl.L[g] = rng.normal(1.0, 0.1, cfg.n_cell)
            fl.b[g] = rng.normal(0.0, 0.1, cfg.n_cell) + (1.0 if g == "f" else 0.0)
        if cfg.projection:
            fl.W_proj = rng.normal(0.0, 1.0 / np.sqrt(cfg.n_cell), (cfg.n_output, cfg.n_cell))
            fl.b_proj = rng.normal(0.0, 0.1, cfg.n_output)
        layers.append(fl)
        n_in = cfg.n_output
    return layers


def _draw_x(cfg: Config, rng: np.random.Generator, T: int, B: int) -> np.ndarray:
    if cfg.x_dist == "uniform":
        return rng.uniform(-1.0, 1.0, (T, B, cfg.n_input))
    return rng.normal(0.0, 1.0, (T, B, cfg.n_input))


@functools.lru_cache(maxsize=2)
def _model(index: int):
    cfg = CONFIGS[index]
    rng = np.random.default_rng(BASE_SEED + index)
    fls = _draw_layers(cfg, rng)
    x_full = _draw_x(cfg, rng, cfg.T, max(cfg.batches))
    if cfg.calib_self:
        x_cal = x_full
    else:
        x_cal = _draw_x(cfg, np.random.default_rng(BASE_SEED + index + 1000), cfg.T, 8)
    stats = [LayerStats() for _ in fls]
    run_sequence(fls, x_cal, stats)
    qls = quantize_model(fls, stats)
    return cfg, fls, qls, x_full


def make_workload(index: int, batch: Optional[int] = None, T: Optional[int] = None,
                  rows: Optional[List[int]] = None) -> Workload:
    """Build config `index`.  `batch` picks the first `batch` rows of the largest batch drawn,
    `rows` picks explicit batch rows instead, `T` truncates the sequence."""
    cfg, fls, qls, x_full = _model(index)
    T = cfg.T if T is None else T
    assert 0 < T <= cfg.T
    if rows is not None:
        xf = x_full[:T, rows, :]
    else:
        B = cfg.batches[-1] if batch is None else batch
        assert 0 < B <= x_full.shape[1]
        xf = x_full[:T, :B, :]
    xf = np.ascontiguousarray(xf)
    xq = quantize_asym_int8(xf, qls[0].s_x, qls[0].zp_x)
    return Workload(cfg, fls, qls, xf, xq, T, xf.shape[1])


def random_layer_stack(seed: int, n_layers: int, n_input: int, n_cell: int, n_output: int,
                       projection=False, peephole=False, layernorm=False, cifg=False,
                       T: int = 6, B: int = 3) -> Workload:
    """Small ad-hoc workload for variant sweeps in tests (same recipe, arbitrary shape)."""
    cfg = Config(0, f"adhoc-{seed}", n_layers, n_input, n_cell, n_output if projection else n_cell,
                 projection, peephole, layernorm, cifg, T, (B,), "normal", True)
    rng = np.random.default_rng(seed)
    fls = _draw_layers(cfg, rng)
    xf = _draw_x(cfg, rng, T, B)
    stats = [LayerStats() for _ in fls]
    run_sequence(fls, xf, stats)
    qls = quantize_model(fls, stats)
    xq = quantize_asym_int8(xf, qls[0].s_x, qls[0].zp_x)
    return Workload(cfg, fls, qls, xf, xq, T, B)
