"""Thin ctypes binding of libqlstm.so: argument marshalling only.

Every step of the integer LSTM runs inside the library's CUDA kernels; this module only
converts numpy / torch arguments into the plain pointers and sizes of the C ABI
(include/qlstm.h) and turns error codes into exceptions.  There is no fallback: if the
library is missing or no sm_100 device is present, calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

from . import build as _build

OK = 0
ERR_ARG, ERR_DIM, ERR_RANGE, ERR_NOMEM, ERR_CUDA, ERR_LAUNCH, ERR_TIMEOUT = -1, -2, -3, -4, -5, -6, -7
IMPL_AUTO, IMPL_SIMPLE, IMPL_FAST = 0, 1, 2

EXPORTS = ["qlstm_create", "qlstm_run", "qlstm_run_host", "qlstm_input_projection", "qlstm_last_status",
           "qlstm_destroy", "qlstm_strerror", "qlstm_trace_bytes", "qlstm_set_impl", "qlstm_set_profiling",
           "qlstm_get_profile", "qlstm_device_info", "qlstm_eval_activations", "qlstm_eval_layernorm_row",
           "qlstm_eval_activation_tables", "qlstm_debug_activation_tables",
           "qlstm_layernorm_rows_static", "qlstm_debug_barrier_timeout", "qlstm_debug_ring_plan",
           "qlstm_debug_projection_plan", "qlstm_debug_mma_i8_peak", "qlstm_debug_barrier_latency",
           "qlstm_bidir_create", "qlstm_bidir_run", "qlstm_bidir_last_status", "qlstm_bidir_destroy",
           "qlstm_calibrate", "qlstm_quantize_model", "qlstm_quantized_layers", "qlstm_quantized_scales",
           "qlstm_quantized_destroy"]


class Scale(C.Structure):
    _fields_ = [("multiplier", C.c_int32), ("shift", C.c_int32)]


class Layer(C.Structure):
    _fields_ = [
        ("n_input", C.c_int32), ("n_cell", C.c_int32), ("n_output", C.c_int32),
        ("flags", C.c_uint32), ("cell_int_bits", C.c_int32),
        ("zp_x", C.c_int32), ("zp_m", C.c_int32), ("zp_h", C.c_int32),
        ("W", C.c_void_p * 4), ("R", C.c_void_p * 4), ("P", C.c_void_p * 4),
        ("b", C.c_void_p * 4), ("L", C.c_void_p * 4),
        ("W_proj", C.c_void_p), ("b_proj", C.c_void_p),
        ("eff_x", Scale * 4), ("eff_h", Scale * 4), ("eff_c", Scale * 4), ("eff_ln", Scale * 4),
        ("eff_m", Scale), ("eff_proj", Scale),
    ]


class FloatLayer(C.Structure):
    _fields_ = [("n_input", C.c_int32), ("n_cell", C.c_int32), ("n_output", C.c_int32), ("flags", C.c_uint32),
                ("W", C.c_void_p * 4), ("R", C.c_void_p * 4), ("P", C.c_void_p * 4), ("L", C.c_void_p * 4),
                ("b", C.c_void_p * 4), ("W_proj", C.c_void_p), ("b_proj", C.c_void_p)]


class Ranges(C.Structure):
    _fields_ = [("x_min", C.c_double), ("x_max", C.c_double), ("h_min", C.c_double), ("h_max", C.c_double),
                ("m_min", C.c_double), ("m_max", C.c_double), ("c_absmax", C.c_double), ("g_absmax", C.c_double * 4)]


class Profile(C.Structure):
    _fields_ = [("projection_ms", C.c_double), ("projection_launches", C.c_int),
                ("recurrent_ms", C.c_double), ("recurrent_launches", C.c_int),
                ("other_ms", C.c_double), ("other_launches", C.c_int),
                ("phase_a_ms", C.c_double), ("wait_a_ms", C.c_double), ("phase_b_ms", C.c_double),
                ("wait_b_ms", C.c_double), ("phase_c_ms", C.c_double), ("wait_c_ms", C.c_double),
                ("matmul_a_ms", C.c_double)]


class QlstmError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {strerror(code)} ({code})")
        self.code = code


_lib = None


def library_path() -> str:
    return _build.LIB


def lib():
    """Loads libqlstm.so, building it first if the sources are newer.  Raises if that fails."""
    global _lib
    if _lib is None:
        # QLSTM_LIB names a prebuilt library to load instead of the in-tree one
        path = os.environ.get("QLSTM_LIB") or (_build.build() if os.environ.get("QLSTM_NO_BUILD") != "1" else _build.LIB)
        L = C.CDLL(path)
        L.qlstm_create.restype = C.c_int
        L.qlstm_create.argtypes = [C.POINTER(Layer), C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_void_p)]
        L.qlstm_run.restype = C.c_int
        L.qlstm_run.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p,
                                C.c_void_p, C.c_void_p]
        L.qlstm_run_host.restype = C.c_int
        L.qlstm_run_host.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
        L.qlstm_input_projection.restype = C.c_int
        L.qlstm_input_projection.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
        L.qlstm_last_status.restype = C.c_int
        L.qlstm_last_status.argtypes = [C.c_void_p]
        L.qlstm_destroy.restype = None
        L.qlstm_destroy.argtypes = [C.c_void_p]
        L.qlstm_strerror.restype = C.c_char_p
        L.qlstm_strerror.argtypes = [C.c_int]
        L.qlstm_trace_bytes.restype = C.c_size_t
        L.qlstm_trace_bytes.argtypes = [C.c_void_p, C.c_int, C.c_int]
        L.qlstm_set_impl.restype = C.c_int
        L.qlstm_set_impl.argtypes = [C.c_void_p, C.c_int, C.c_int]
        L.qlstm_set_profiling.restype = C.c_int
        L.qlstm_set_profiling.argtypes = [C.c_void_p, C.c_int]
        L.qlstm_get_profile.restype = C.c_int
        L.qlstm_get_profile.argtypes = [C.c_void_p, C.POINTER(Profile), C.c_int]
        L.qlstm_device_info.restype = C.c_int
        L.qlstm_device_info.argtypes = [C.c_void_p, C.POINTER(C.c_int), C.POINTER(C.c_int)]
        L.qlstm_eval_activations.restype = C.c_int
        L.qlstm_eval_activations.argtypes = [C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
        L.qlstm_eval_activation_tables.restype = C.c_int
        L.qlstm_eval_activation_tables.argtypes = [C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(C.c_int),
                                                   C.c_void_p]
        L.qlstm_debug_activation_tables.restype = C.c_int
        L.qlstm_debug_activation_tables.argtypes = [C.c_void_p, C.c_int]
        L.qlstm_eval_layernorm_row.restype = C.c_int
        L.qlstm_eval_layernorm_row.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, Scale, C.c_void_p, C.c_void_p]
        L.qlstm_debug_barrier_timeout.restype = C.c_int
        L.qlstm_debug_barrier_timeout.argtypes = [C.c_void_p, C.c_int, C.c_ulonglong]
        L.qlstm_debug_ring_plan.restype = C.c_int
        L.qlstm_debug_ring_plan.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_int)]
        L.qlstm_debug_projection_plan.restype = C.c_int
        L.qlstm_debug_projection_plan.argtypes = [C.c_longlong, C.c_longlong, C.c_int, C.c_int, C.c_int, C.c_int,
                                                  C.POINTER(C.c_int)]
        L.qlstm_debug_mma_i8_peak.restype = C.c_int
        L.qlstm_debug_mma_i8_peak.argtypes = [C.c_int, C.c_int, C.POINTER(C.c_double)]
        L.qlstm_debug_barrier_latency.restype = C.c_int
        L.qlstm_debug_barrier_latency.argtypes = [C.c_int, C.c_int, C.POINTER(C.c_double)]
        L.qlstm_bidir_create.restype = C.c_int
        L.qlstm_bidir_create.argtypes = [C.POINTER(Layer), C.POINTER(Layer), C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_void_p)]
        L.qlstm_bidir_run.restype = C.c_int
        L.qlstm_bidir_run.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int] + [C.c_void_p] * 6
        L.qlstm_bidir_last_status.restype = C.c_int
        L.qlstm_bidir_last_status.argtypes = [C.c_void_p]
        L.qlstm_bidir_destroy.restype = None
        L.qlstm_bidir_destroy.argtypes = [C.c_void_p]
        L.qlstm_calibrate.restype = C.c_int
        L.qlstm_calibrate.argtypes = [C.POINTER(FloatLayer), C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_int, C.POINTER(Ranges)]
        L.qlstm_quantize_model.restype = C.c_int
        L.qlstm_quantize_model.argtypes = [C.POINTER(FloatLayer), C.POINTER(Ranges), C.c_int, C.c_int, C.POINTER(C.c_void_p)]
        L.qlstm_quantized_layers.restype = C.POINTER(Layer)
        L.qlstm_quantized_layers.argtypes = [C.c_void_p]
        L.qlstm_quantized_scales.restype = C.c_int
        L.qlstm_quantized_scales.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_double)]
        L.qlstm_quantized_destroy.restype = None
        L.qlstm_quantized_destroy.argtypes = [C.c_void_p]
        L.qlstm_layernorm_rows_static.restype = C.c_int
        L.qlstm_layernorm_rows_static.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p, Scale, C.c_void_p,
                                                  C.c_void_p]
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().qlstm_strerror(code).decode()


def _check(code: int, what: str):
    if code != OK:
        raise QlstmError(code, what)


def _ptr(a: Optional[np.ndarray], dtype, keep: list):
    if a is None:
        return None
    a = np.ascontiguousarray(a, dtype)
    keep.append(a)
    return a.ctypes.data


def pack_layers(layers: Sequence, keep: list):
    """Marshals layer descriptions (objects with the fields of qlstm_layer_t) into a C array."""
    arr = (Layer * len(layers))()
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
            d.eff_x[g] = Scale(*map(int, q.eff_x[g]))
            d.eff_h[g] = Scale(*map(int, q.eff_h[g]))
            d.eff_c[g] = Scale(*map(int, q.eff_c[g]))
            d.eff_ln[g] = Scale(*map(int, q.eff_ln[g]))
        d.W_proj = _ptr(q.W_proj, np.int8, keep)
        d.b_proj = _ptr(q.b_proj, np.int32, keep)
        d.eff_m = Scale(*map(int, q.eff_m))
        d.eff_proj = Scale(*map(int, q.eff_proj))
    return arr


def _dev_ptr(t) -> int:
    """Device pointer of a torch CUDA tensor (must be contiguous) or a raw int address."""
    if isinstance(t, int):
        return t
    if t is None:
        return 0
    assert t.is_cuda and t.is_contiguous()
    return t.data_ptr()


class QLSTM:
    """Handle of one integer LSTM stack on one GPU (qlstm_create / qlstm_run / qlstm_destroy)."""

    def __init__(self, layers: Sequence, max_T: int, max_B: int, device: int = 0):
        keep: list = []
        arr = pack_layers(layers, keep)
        h = C.c_void_p()
        _check(lib().qlstm_create(arr, len(layers), max_T, max_B, device, C.byref(h)), "qlstm_create")
        self._h = h
        self.device = device
        self.dims = [(q.n_input, q.n_cell, q.n_output, 3 if (q.flags & 8) else 4) for q in layers]
        self.max_T, self.max_B = max_T, max_B

    def close(self):
        if getattr(self, "_h", None):
            lib().qlstm_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()

    def run(self, x, T: int, B: int, h, c, y, trace=None, stream: int = 0, check: bool = False):
        """qlstm_run on device tensors (torch CUDA tensors or raw addresses).  Asynchronous."""
        _check(lib().qlstm_run(self._h, _dev_ptr(x), T, B, _dev_ptr(h), _dev_ptr(c), _dev_ptr(y), _dev_ptr(trace),
                               stream), "qlstm_run")
        if check:
            self.last_status()

    def run_host(self, x: np.ndarray, h: np.ndarray, c: np.ndarray):
        """qlstm_run_host on numpy arrays: returns (y, h, c) as new arrays."""
        x = np.ascontiguousarray(x, np.int8)
        T, B, _ = x.shape
        h = np.array(h, np.int8, copy=True)
        c = np.array(c, np.int16, copy=True)
        y = np.empty((T, B, self.dims[-1][2]), np.int8)
        _check(lib().qlstm_run_host(self._h, x.ctypes.data, T, B, h.ctypes.data, c.ctypes.data, y.ctypes.data),
               "qlstm_run_host")
        return y, h, c

    def run_host_raw(self, x_ptr: int, T: int, B: int, h_ptr: int, c_ptr: int, y_ptr: int):
        _check(lib().qlstm_run_host(self._h, x_ptr, T, B, h_ptr, c_ptr, y_ptr), "qlstm_run_host")

    def input_projection(self, layer: int, x, rows: int, out, stream: int = 0):
        _check(lib().qlstm_input_projection(self._h, layer, _dev_ptr(x), rows, _dev_ptr(out), stream),
               "qlstm_input_projection")

    def last_status(self):
        _check(lib().qlstm_last_status(self._h), "qlstm_last_status")

    def trace_bytes(self, T: int, B: int) -> int:
        return lib().qlstm_trace_bytes(self._h, T, B)

    def set_impl(self, projection: int = IMPL_AUTO, recurrent: int = IMPL_AUTO):
        _check(lib().qlstm_set_impl(self._h, projection, recurrent), "qlstm_set_impl")

    def activation_tables(self, enable=True) -> int:
        """Memoised sigmoid / tanh in the persistent kernel on (default) or off; 2: the kernel's general instantiation
        (scales with a left shift allowed, no tables).  Returns the number of layers that hold tables."""
        n = lib().qlstm_debug_activation_tables(self._h, int(enable))
        _check(min(n, 0), "qlstm_debug_activation_tables")
        return n

    def set_profiling(self, level: int):
        """0 off, 1 per-kernel event times, 2 also the device phase timers (which slow the kernel they time)."""
        _check(lib().qlstm_set_profiling(self._h, int(level)), "qlstm_set_profiling")

    def get_profile(self, reset: bool = True) -> dict:
        p = Profile()
        _check(lib().qlstm_get_profile(self._h, C.byref(p), int(reset)), "qlstm_get_profile")
        return {k: getattr(p, k) for k, _ in Profile._fields_}

    def debug_barrier_timeout(self, missing_arrivals: int, limit_ns: int = 0):
        _check(lib().qlstm_debug_barrier_timeout(self._h, missing_arrivals, limit_ns), "qlstm_debug_barrier_timeout")

    def device_info(self):
        a, b = C.c_int(), C.c_int()
        _check(lib().qlstm_device_info(self._h, C.byref(a), C.byref(b)), "qlstm_device_info")
        return a.value, b.value


class BiQLSTM:
    """Handle of a bidirectional stack (qlstm_bidir_create / qlstm_bidir_run / qlstm_bidir_destroy)."""

    def __init__(self, fwd_layers: Sequence, bwd_layers: Sequence, max_T: int, max_B: int, device: int = 0):
        assert len(fwd_layers) == len(bwd_layers)
        keep: list = []
        fa, ba = pack_layers(fwd_layers, keep), pack_layers(bwd_layers, keep)
        h = C.c_void_p()
        _check(lib().qlstm_bidir_create(fa, ba, len(fwd_layers), max_T, max_B, device, C.byref(h)), "qlstm_bidir_create")
        self._h = h
        self.n_output = fwd_layers[-1].n_output + bwd_layers[-1].n_output

    def run(self, x, T: int, B: int, h_fwd, c_fwd, h_bwd, c_bwd, y, stream: int = 0):
        _check(lib().qlstm_bidir_run(self._h, _dev_ptr(x), T, B, _dev_ptr(h_fwd), _dev_ptr(c_fwd), _dev_ptr(h_bwd),
                                     _dev_ptr(c_bwd), _dev_ptr(y), stream), "qlstm_bidir_run")

    def last_status(self):
        _check(lib().qlstm_bidir_last_status(self._h), "qlstm_bidir_last_status")

    def close(self):
        if getattr(self, "_h", None):
            lib().qlstm_bidir_destroy(self._h)
            self._h = None

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def eval_activations(cell_int_bits: int, sigmoid_out, tanh_out, stream: int = 0):
    """qlstm_eval_activations on two device int16 [65536] tensors."""
    _check(lib().qlstm_eval_activations(cell_int_bits, _dev_ptr(sigmoid_out), _dev_ptr(tanh_out), stream),
           "qlstm_eval_activations")


def eval_activation_tables(cell_int_bits: int, max_bytes: int, sigmoid_out, tanh_gate_out, tanh_cell_out, stream: int = 0):
    """qlstm_eval_activation_tables on three device int16 [65536] tensors; returns the seven layout numbers."""
    lay = (C.c_int * 7)()
    _check(lib().qlstm_eval_activation_tables(cell_int_bits, max_bytes, _dev_ptr(sigmoid_out), _dev_ptr(tanh_gate_out),
                                              _dev_ptr(tanh_cell_out), lay, stream), "qlstm_eval_activation_tables")
    return list(lay)


def eval_layernorm_row(q, n: int, L, b, eff_ln, out, stream: int = 0):
    _check(lib().qlstm_eval_layernorm_row(_dev_ptr(q), n, _dev_ptr(L), _dev_ptr(b), Scale(int(eff_ln[0]), int(eff_ln[1])),
                                          _dev_ptr(out), stream), "qlstm_eval_layernorm_row")


def layernorm_rows_static(q, rows: int, n: int, L, b, eff_ln, out, stream: int = 0):
    """qlstm_layernorm_rows_static: layer norm of `rows` rows using only the library's built-in scratch
    (for callers that may not allocate device memory).  Raises QlstmError(ERR_DIM) beyond 4096 rows."""
    _check(lib().qlstm_layernorm_rows_static(_dev_ptr(q), rows, n, _dev_ptr(L), _dev_ptr(b),
                                             Scale(int(eff_ln[0]), int(eff_ln[1])), _dev_ptr(out), stream),
           "qlstm_layernorm_rows_static")


def parse_trace(buf: np.ndarray, dims: Sequence, T: int, B: int):
    """Splits a trace buffer (uint8 array, layout of include/qlstm.h) into per-layer dicts of arrays [T, ...]."""
    out, off = [], 0
    for (_, Cn, O, _) in dims:
        bc, bo = B * Cn, B * O
        fields = [("acc", np.int32, (4, B, Cn)), ("pacc", np.int32, (B, O)), ("xg", np.int16, (4, B, Cn)),
                  ("pre", np.int16, (4, B, Cn)), ("ain", np.int16, (4, B, Cn)), ("gate", np.int16, (4, B, Cn)),
                  ("c", np.int16, (B, Cn)), ("m", np.int8, (B, Cn)), ("h", np.int8, (B, O))]
        rec = (16 * bc + 4 * bo + 32 * bc + 2 * bc + bc + bo + 15) & ~15
        sect = buf[off:off + T * rec].reshape(T, rec)
        d, o = {}, 0
        for name, dt, shape in fields:
            n = int(np.prod(shape)) * np.dtype(dt).itemsize
            d[name] = np.ascontiguousarray(sect[:, o:o + n]).view(dt).reshape((T,) + shape)
            o += n
        out.append(d)
        off += T * rec
    return out


def ring_plan(stages: int, n_owners: int, contiguous: bool, chunks_per_tile: int = 0, chunks_total: int = 0):
    """The operand-ring plan of the recurrent kernel for one matmul phase (host logic only; needs no GPU)."""
    out = (C.c_int * 14)()
    _check(lib().qlstm_debug_ring_plan(stages, n_owners, int(contiguous), chunks_per_tile, chunks_total, out),
           "qlstm_debug_ring_plan")
    v = list(out)
    return {"n_own": v[0], "n_max": v[1], "n_chunks": v[2:6], "cnt": v[6:10], "uses": v[10:14]}


def projection_plan(rows: int, n_gate_rows: int, n_input: int, sm_count: int = 148, smem_bytes: int = 232448,
                    max_rows: Optional[int] = None):
    """The tiling of the input-projection kernel for one launch shape, on a handle created for max_rows rows
    (default: rows).  Host logic only; needs no GPU."""
    out = (C.c_int * 5)()
    _check(lib().qlstm_debug_projection_plan(rows if max_rows is None else max_rows, rows, n_gate_rows, n_input,
                                             sm_count, smem_bytes, out),
           "qlstm_debug_projection_plan")
    v = list(out)
    return {"bn": v[0], "stages": v[1], "per_cta": v[2], "m_ranges": v[3], "grid": v[4]}


def mma_i8_peak(device: int = 0, iters: int = 20000) -> float:
    """Measured int8 TOP/s of back-to-back tcgen05.mma kind::i8 from resident operands on every SM."""
    out = C.c_double()
    _check(lib().qlstm_debug_mma_i8_peak(device, iters, C.byref(out)), "qlstm_debug_mma_i8_peak")
    return out.value


def barrier_latency_us(device: int = 0, n_barriers: int = 2000) -> float:
    """Microseconds per grid-wide barrier of the persistent kernel's kind, executed back to back."""
    out = C.c_double()
    _check(lib().qlstm_debug_barrier_latency(device, n_barriers, C.byref(out)), "qlstm_debug_barrier_latency")
    return out.value


# ---- calibration and quantization on the device (include/qlstm_calib.h): marshalling only

_GATES = ("i", "f", "z", "o")


def pack_float_layers(float_layers: Sequence, keep: list):
    """Marshals float layers (objects with the fields of workloads.float_lstm.FloatLayer) into a C array."""
    arr = (FloatLayer * len(float_layers))()
    for d, fl in zip(arr, float_layers):
        d.n_input, d.n_cell, d.n_output = fl.n_input, fl.n_cell, fl.n_output
        d.flags = (1 if fl.projection else 0) | (2 if fl.peephole else 0) | (4 if fl.layernorm else 0) | (8 if fl.cifg else 0)
        for gi, g in enumerate(_GATES):
            if fl.cifg and g == "i":
                continue
            d.W[gi] = _ptr(fl.W[g], np.float64, keep)
            d.R[gi] = _ptr(fl.R[g], np.float64, keep)
            d.b[gi] = _ptr(fl.b[g], np.float64, keep)
            if fl.layernorm:
                d.L[gi] = _ptr(fl.L[g], np.float64, keep)
            if fl.peephole and g != "z":
                d.P[gi] = _ptr(fl.P[g], np.float64, keep)
        if fl.projection:
            d.W_proj = _ptr(fl.W_proj, np.float64, keep)
            d.b_proj = _ptr(fl.b_proj, np.float64, keep)
    return arr


def calibrate(float_layers: Sequence, x: np.ndarray, device: int = 0):
    """qlstm_calibrate: float forward pass on the device; returns one dict of logged ranges per layer."""
    keep: list = []
    arr = pack_float_layers(float_layers, keep)
    x = np.ascontiguousarray(x, np.float64)
    T, B, _ = x.shape
    out = (Ranges * len(float_layers))()
    _check(lib().qlstm_calibrate(arr, len(float_layers), x.ctypes.data, T, B, device, out), "qlstm_calibrate")
    return [{"x_min": r.x_min, "x_max": r.x_max, "h_min": r.h_min, "h_max": r.h_max, "m_min": r.m_min, "m_max": r.m_max,
             "c_absmax": r.c_absmax, "g_absmax": dict(zip(_GATES, r.g_absmax))} for r in out]


class QuantizedLayer:
    """One layer as qlstm_quantize_model produced it: the fields of qlstm_layer_t as numpy copies, plus real scales."""


def quantize_model(float_layers: Sequence, ranges: Sequence[dict], device: int = 0):
    """qlstm_quantize_model: Table 2 with the reductions and roundings on the device; returns QuantizedLayer objects
    (usable wherever a layer description is expected)."""
    keep: list = []
    arr = pack_float_layers(float_layers, keep)
    rg = (Ranges * len(float_layers))()
    for d, r in zip(rg, ranges):
        for k in ("x_min", "x_max", "h_min", "h_max", "m_min", "m_max", "c_absmax"):
            setattr(d, k, float(r[k]))
        for gi, g in enumerate(_GATES):
            d.g_absmax[gi] = float(r["g_absmax"][g])
    h = C.c_void_p()
    _check(lib().qlstm_quantize_model(arr, rg, len(float_layers), device, C.byref(h)), "qlstm_quantize_model")
    try:
        ptr = lib().qlstm_quantized_layers(h)
        out = []
        for l in range(len(float_layers)):
            d = ptr[l]
            q = QuantizedLayer()
            q.n_input, q.n_cell, q.n_output, q.flags = d.n_input, d.n_cell, d.n_output, d.flags
            q.cell_int_bits, q.zp_x, q.zp_m, q.zp_h = d.cell_int_bits, d.zp_x, d.zp_m, d.zp_h

            def grab(addr, dtype, shape):
                if not addr:
                    return None
                n = int(np.prod(shape))
                buf = (C.c_char * (n * np.dtype(dtype).itemsize)).from_address(addr)
                return np.frombuffer(buf, dtype=dtype).reshape(shape).copy()
            q.W = [grab(d.W[g], np.int8, (d.n_cell, d.n_input)) for g in range(4)]
            q.R = [grab(d.R[g], np.int8, (d.n_cell, d.n_output)) for g in range(4)]
            q.P = [grab(d.P[g], np.int16, (d.n_cell,)) for g in range(4)]
            q.b = [grab(d.b[g], np.int32, (d.n_cell,)) for g in range(4)]
            q.L = [grab(d.L[g], np.int16, (d.n_cell,)) for g in range(4)]
            q.W_proj = grab(d.W_proj, np.int8, (d.n_output, d.n_cell))
            q.b_proj = grab(d.b_proj, np.int32, (d.n_output,))
            for name in ("eff_x", "eff_h", "eff_c", "eff_ln"):
                setattr(q, name, [(getattr(d, name)[g].multiplier, getattr(d, name)[g].shift) for g in range(4)])
            q.eff_m = (d.eff_m.multiplier, d.eff_m.shift)
            q.eff_proj = (d.eff_proj.multiplier, d.eff_proj.shift)
            sc = (C.c_double * 4)()
            _check(lib().qlstm_quantized_scales(h, l, sc), "qlstm_quantized_scales")
            q.s_x, q.s_h, q.s_m, q.s_c = sc[0], sc[1], sc[2], sc[3]
            out.append(q)
        return out
    finally:
        lib().qlstm_quantized_destroy(h)
