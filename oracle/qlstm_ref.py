"""ctypes access to the C oracle (oracle/qlstm_ref.c).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg import this module;
it neither imports nor is imported by the CUDA package.  Layer descriptions are duck
typed: any object with the attributes of workloads.quantize.QLayer works.
"""
from __future__ import annotations

import ctypes as C
from typing import Dict, List, Optional, Sequence

import numpy as np

from . import build as _build


class _Scale(C.Structure):
    _fields_ = [("multiplier", C.c_int32), ("shift", C.c_int32)]


class _Layer(C.Structure):
    _fields_ = [
        ("n_input", C.c_int32), ("n_cell", C.c_int32), ("n_output", C.c_int32),
        ("flags", C.c_uint32), ("cell_int_bits", C.c_int32),
        ("zp_x", C.c_int32), ("zp_m", C.c_int32), ("zp_h", C.c_int32),
        ("W", C.c_void_p * 4), ("R", C.c_void_p * 4), ("P", C.c_void_p * 4),
        ("b", C.c_void_p * 4), ("L", C.c_void_p * 4),
        ("W_proj", C.c_void_p), ("b_proj", C.c_void_p),
        ("eff_x", _Scale * 4), ("eff_h", _Scale * 4), ("eff_c", _Scale * 4), ("eff_ln", _Scale * 4),
        ("eff_m", _Scale), ("eff_proj", _Scale),
    ]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        L.qref_srdhm.restype = C.c_int32
        L.qref_srdhm.argtypes = [C.c_int32, C.c_int32]
        L.qref_rdivpot.restype = C.c_int64
        L.qref_rdivpot.argtypes = [C.c_int64, C.c_int]
        L.qref_mbqm.restype = C.c_int32
        L.qref_mbqm.argtypes = [C.c_int32, _Scale]
        L.qref_rdiv.restype = C.c_int64
        L.qref_rdiv.argtypes = [C.c_int64, C.c_int64]
        L.qref_isqrt.restype = C.c_uint64
        L.qref_isqrt.argtypes = [C.c_uint64]
        L.qref_sigmoid.restype = C.c_int16
        L.qref_sigmoid.argtypes = [C.c_int16, C.c_int]
        L.qref_tanh.restype = C.c_int16
        L.qref_tanh.argtypes = [C.c_int16, C.c_int]
        L.qref_layernorm_row.restype = None
        L.qref_layernorm_row.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, _Scale, C.c_void_p]
        L.qref_trace_bytes.restype = C.c_size_t
        L.qref_trace_bytes.argtypes = [C.POINTER(_Layer), C.c_int, C.c_int, C.c_int]
        L.qref_run.restype = C.c_int
        L.qref_run.argtypes = [C.POINTER(_Layer), C.c_int, C.c_void_p, C.c_int, C.c_int,
                               C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.qref_num_threads.restype = C.c_int
        _lib = L
    return _lib


def srdhm(a: int, b: int) -> int:
    return lib().qref_srdhm(a, b)


def rdivpot(x: int, e: int) -> int:
    return lib().qref_rdivpot(x, e)


def mbqm(x: int, scale) -> int:
    return lib().qref_mbqm(x, _Scale(int(scale[0]), int(scale[1])))


def rdiv(n: int, d: int) -> int:
    return lib().qref_rdiv(n, d)


def isqrt(v: int) -> int:
    return lib().qref_isqrt(v)


def sigmoid(x: int, m: int = 3) -> int:
    return lib().qref_sigmoid(x, m)


def tanh(x: int, m: int = 3) -> int:
    return lib().qref_tanh(x, m)


def sigmoid_all(m: int = 3) -> np.ndarray:
    """sigmoid_q over the whole int16 domain, index = x + 32768."""
    L = lib()
    return np.array([L.qref_sigmoid(x, m) for x in range(-32768, 32768)], dtype=np.int32)


def tanh_all(m: int = 3) -> np.ndarray:
    L = lib()
    return np.array([L.qref_tanh(x, m) for x in range(-32768, 32768)], dtype=np.int32)


def layernorm_row(q: np.ndarray, Lw: np.ndarray, b: np.ndarray, eff_ln) -> np.ndarray:
    q = np.ascontiguousarray(q, np.int16)
    Lw = np.ascontiguousarray(Lw, np.int16)
    b = np.ascontiguousarray(b, np.int32)
    out = np.empty_like(q)
    lib().qref_layernorm_row(q.ctypes.data, q.size, Lw.ctypes.data, b.ctypes.data,
                             _Scale(int(eff_ln[0]), int(eff_ln[1])), out.ctypes.data)
    return out


def _ptr(a: Optional[np.ndarray], dtype, keep: list):
    if a is None:
        return None
    a = np.ascontiguousarray(a, dtype)
    keep.append(a)
    return a.ctypes.data


def _pack(layers: Sequence, keep: list):
    arr = (_Layer * len(layers))()
    for d, q in zip(arr, layers):
        d.n_input, d.n_cell, d.n_output = q.n_input, q.n_cell, q.n_output
        d.flags, d.cell_int_bits = q.flags, q.cell_int_bits
        d.zp_x, d.zp_m, d.zp_h = q.zp_x, q.zp_m, q.zp_h
        for g in range(4):
            d.W[g] = _ptr(q.W[g], np.int8, keep)
            d.R[g] = _ptr(q.R[g], np.int8, keep)
            d.P[g] = _ptr(q.P[g], np.int16, keep)
            d.b[g] = _ptr(q.b[g], np.int32, keep)
            d.L[g] = _ptr(q.L[g], np.int16, keep)
            d.eff_x[g] = _Scale(*map(int, q.eff_x[g]))
            d.eff_h[g] = _Scale(*map(int, q.eff_h[g]))
            d.eff_c[g] = _Scale(*map(int, q.eff_c[g]))
            d.eff_ln[g] = _Scale(*map(int, q.eff_ln[g]))
        d.W_proj = _ptr(q.W_proj, np.int8, keep)
        d.b_proj = _ptr(q.b_proj, np.int32, keep)
        d.eff_m = _Scale(*map(int, q.eff_m))
        d.eff_proj = _Scale(*map(int, q.eff_proj))
    return arr


def parse_trace(buf: np.ndarray, layers: Sequence, T: int, B: int) -> List[Dict[str, np.ndarray]]:
    """Split a trace buffer into per-layer dicts of arrays with a leading T axis."""
    out = []
    off = 0
    for q in layers:
        Cn, O = q.n_cell, q.n_output
        bc, bo = B * Cn, B * O
        fields = [("acc", np.int32, (4, B, Cn)), ("pacc", np.int32, (B, O)),
                  ("xg", np.int16, (4, B, Cn)), ("pre", np.int16, (4, B, Cn)),
                  ("ain", np.int16, (4, B, Cn)), ("gate", np.int16, (4, B, Cn)),
                  ("c", np.int16, (B, Cn)), ("m", np.int8, (B, Cn)), ("h", np.int8, (B, O))]
        raw = 4 * 4 * bc + 4 * bo + 4 * (2 * 4 * bc) + 2 * bc + bc + bo
        rec = (raw + 15) & ~15
        sect = buf[off:off + T * rec].reshape(T, rec)
        d, o = {}, 0
        for name, dt, shape in fields:
            n = int(np.prod(shape)) * np.dtype(dt).itemsize
            d[name] = np.ascontiguousarray(sect[:, o:o + n]).view(dt).reshape((T,) + shape)
            o += n
        out.append(d)
        off += T * rec
    return out


def run(layers: Sequence, x: np.ndarray, h: np.ndarray, c: np.ndarray, trace: bool = False):
    """x int8 [T,B,I]; h int8 / c int16 flat state (updated copies are returned).

    Returns (y int8 [T,B,O_last], h, c, trace list or None).
    """
    keep: list = []
    arr = _pack(layers, keep)
    x = np.ascontiguousarray(x, np.int8)
    T, B, _ = x.shape
    h = np.array(h, np.int8, copy=True)
    c = np.array(c, np.int16, copy=True)
    assert h.size == sum(B * q.n_output for q in layers) and c.size == sum(B * q.n_cell for q in layers)
    y = np.zeros((T, B, layers[-1].n_output), np.int8)
    tbuf = None
    if trace:
        n = lib().qref_trace_bytes(arr, len(layers), T, B)
        tbuf = np.zeros(n, np.uint8)
    rc = lib().qref_run(arr, len(layers), x.ctypes.data, T, B, h.ctypes.data, c.ctypes.data, y.ctypes.data,
                        tbuf.ctypes.data if tbuf is not None else None)
    if rc != 0:
        raise ValueError(f"qref_run rejected its arguments (code {rc})")
    return y, h, c, (parse_trace(tbuf, layers, T, B) if trace else None)


def num_threads() -> int:
    return lib().qref_num_threads()
