"""Seeded synthetic inputs for the integer LSTM: float model, calibration, quantizer, configs.

Holds none of the integer execution arithmetic; both the CPU oracle's tests and the CUDA
path's tests draw their inputs from here.
"""
from .configs import CONFIGS, Workload, make_workload, random_layer_stack  # noqa: F401
from .quantize import QLayer, decode_scale, encode_scale  # noqa: F401
