#!/usr/bin/env python
"""Benchmark of the integer LSTM forward pass.

  python bench.py --gpus N --steps K --warmup W            # this library (CUDA, sm_100a)
  python bench.py --impl reference --steps K --warmup W    # the CPU oracle, as a reported baseline

A "step" is one pass of the whole hot path (input projection + recurrent steps of every layer)
over one batch: the production-shaped configuration 5 (8 layers, layer norm + projection,
input 640, cell 2048, projection 640, T = 300) at batch 256.  The metric is batch*timesteps/s.
With N > 1 (torchrun) every rank runs the same workload on its own GPU: batch rows are
independent, there is no collective on the data path, scaling is weak.  Rank 0 prints one JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "quantized LSTM batch*timesteps/sec"
UNIT = "batch*timesteps/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [v.strip() for v in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1]))
                    mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


# DRAM traffic of the recurrent kernel from one ncu capture of full-size launches (three counters, one pass; its
# summary is kept with the other profile summaries): dram__bytes_read.sum + dram__bytes_write.sum = 1269.9 + 52.8 MB
# per launch (one layer, 300 steps) of config 5 at batch 256, against 1309.9 MB algorithmic (X read once, y written
# once).  Valid only for the kernel sources the counters were taken from and for that launch shape: otherwise null.
NCU_RECURRENT = {"bytes": 1322.7e6, "steps": 300, "config": 5, "batch": 256, "source_sha": "41be06a06a9b908e"}

# DRAM traffic of the input-projection kernel from one ncu capture of a full-size launch (three counters, one pass):
# dram__bytes_read.sum + dram__bytes_write.sum = 54.5 + 1204.1 MB at 76800 rows of config 5 (algorithmic: 49.2 MB of x,
# 5.2 MB of W, 1258.3 MB of int16 output, part of which is still in L2 when the kernel ends).  Valid only for the
# kernel sources the counters were taken from and for that launch shape: otherwise reported as null.
NCU_PROJECTION = {"bytes": 1258.6e6, "rows": 76800, "config": 5, "source_sha": "b04867077a26bd59"}

# The recurrent kernel is bound by plain integer arithmetic (the fixed-point epilogues), not by its matmuls or by
# memory.  Peak: 148 SMs x 64 int32 lanes (4 schedulers x 16-lane integer pipe) x the SM clock; a microbenchmark of
# this very arithmetic saturates at 64-68 thread instructions per clock per SM.  Algorithmic integer operations per
# unit, counted as machine integer instructions of the leanest exact form of each step (measured in isolation):
INT_LANES_PER_SM = 64
OPS_ACTIVATION = 53          # integer sigmoid / tanh: polynomial of degree 6 + one exact division
OPS_ACTIVATION_LOOKUP = 11   # the same value read from the kernel's memoised table (|x|, clamp, load, decode, sign)
OPS_LAYERNORM = 38           # one layer-norm value: exact quotient, multiply-add, rescale
OPS_GATE_SUM = 20            # one gate pre-activation: + bias, rescale, + X, saturate
OPS_CELL = 30                # cell update, hidden state product, rescale, requantize
OPS_PEEPHOLE = 15            # one peephole term
OPS_PROJ_OUT = 12            # one projection output: + bias, rescale, requantize


def algorithmic_int_ops(layers, B, T, ops_activation=OPS_ACTIVATION):
    """Integer operations of the recurrent part per pass over the whole stack (see the constants above)."""
    total = 0
    for q in layers:
        G = 3 if (q.flags & 8) else 4
        per_cell = (G + 1) * ops_activation + OPS_CELL + G * OPS_GATE_SUM
        if q.flags & 4:
            per_cell += G * OPS_LAYERNORM
        if q.flags & 2:
            per_cell += (G - 1) * OPS_PEEPHOLE
        per_row = q.n_cell * per_cell + (q.n_output * OPS_PROJ_OUT if (q.flags & 1) else 0)
        total += per_row * B * T
    return total


def _source_sha(files):
    import hashlib
    m = hashlib.sha256()
    for f in files:
        with open(os.path.join(ROOT, "paper_2101_05453_b200", "csrc", f), "rb") as fh:
            m.update(fh.read())
    return m.hexdigest()[:16]


def recurrent_source_sha():
    return _source_sha(("recurrent_sm100.cu", "act_table.cuh", "qmath.cuh", "sm100_ptx.cuh"))


def projection_source_sha():
    return _source_sha(("proj_gemm_sm100.cu", "qmath.cuh", "sm100_ptx.cuh"))


def algorithmic_ops(layers, B, T):
    """int8 multiply-accumulates counted as 2 ops, per pass: (projection GEMMs, recurrent + projection matmuls)."""
    gemm = rec = 0
    for q in layers:
        G = 3 if (q.flags & 8) else 4
        gemm += 2 * T * B * G * q.n_cell * q.n_input
        rec += 2 * T * B * G * q.n_cell * q.n_output
        if q.flags & 1:
            rec += 2 * T * B * q.n_output * q.n_cell
    return gemm, rec


def oracle_sample(w_full_index, threads_hint, T_sample, rows_n):
    """Times the CPU oracle, as it stands, on `rows_n` batch rows x T_sample steps of the workload."""
    from oracle import qlstm_ref
    from workloads import make_workload
    rows = list(range(rows_n))
    w = make_workload(w_full_index, rows=rows, T=T_sample)
    h0, c0 = w.initial_state()
    t0 = time.perf_counter()
    qlstm_ref.run(w.layers, w.x, h0, c0)
    dt = time.perf_counter() - t0
    return rows_n * T_sample / dt, dt, qlstm_ref.num_threads()


def run_reference(args):
    """The reference arm: the oracle on the host cores, each step a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import qlstm_ref
    cores = qlstm_ref.num_threads()
    rows_n, T_s = max(1, min(args.batch, cores)), 8
    for _ in range(args.warmup):
        oracle_sample(args.config, cores, 2, rows_n)
    times = []
    for _ in range(args.steps):
        v, dt, _ = oracle_sample(args.config, cores, T_s, rows_n)
        times.append(dt)
    total = sum(times)
    value = rows_n * T_s * args.steps / total
    sample = f"{rows_n} batch rows x {T_s} timesteps of config {args.config} per step"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": {"workload": f"config5-ln-proj-8x2048 batch {args.batch} T {args.T}", "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--config", type=int, default=5)
    ap.add_argument("--batch", type=int, default=256)
    ap.add_argument("--T", type=int, default=None)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-latency", action="store_true")
    args = ap.parse_args()

    from workloads import CONFIGS, make_workload
    if args.T is None:
        args.T = CONFIGS[args.config].T
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import paper_2101_05453_b200 as qlstm

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    w = make_workload(args.config, batch=args.batch, T=args.T)
    T, B = w.T, w.B
    O = w.layers[-1].n_output
    peaks = measured_peaks()

    q = qlstm.QLSTM(w.layers, T, B, device=local)
    stream = torch.cuda.current_stream().cuda_stream
    h0, c0 = w.initial_state()
    x = torch.from_numpy(w.x).to(dev)
    h_init = torch.from_numpy(h0).to(dev)
    c_init = torch.from_numpy(c0).to(dev)
    h = h_init.clone()
    c = c_init.clone()
    y = torch.zeros((T, B, O), dtype=torch.int8, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)     # > L2 (126 MB)

    def one_step(profile=False):
        h.copy_(h_init)
        c.copy_(c_init)
        flush.zero_()                                                  # evict L2 between timed passes
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        q.run(x, T, B, h, c, y, stream=stream)
        b.record()
        return a, b

    for _ in range(max(args.warmup, 3)):
        one_step()
    q.last_status()
    torch.cuda.synchronize()
    q.set_profiling(1)                    # per-kernel event times only: the device phase timers slow the kernel
    q.get_profile(reset=True)

    sampler = ClockSampler(local)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    events = [one_step() for _ in range(args.steps)]
    torch.cuda.synchronize()
    q.last_status()
    if dist is not None:
        dist.barrier()
    clocks = sampler.stop()
    step_ms = [a.elapsed_time(b) for a, b in events]
    total_ms = sum(step_ms)
    prof = q.get_profile(reset=True)
    # phase breakdown of the recurrent kernel: a separate untimed pass with the device phase timers on
    q.set_profiling(2)
    one_step()
    torch.cuda.synchronize()
    prof_phase = q.get_profile(reset=True)
    q.set_profiling(0)
    if dist is not None:
        t = torch.tensor([total_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    value = world * B * T * args.steps / (total_ms * 1e-3)

    # ---- end to end through the host-buffer entry point: H2D of x, h, c and D2H of y, h, c inside the timed region
    xh = torch.from_numpy(w.x).pin_memory()
    hh = torch.from_numpy(h0.copy()).pin_memory()
    ch = torch.from_numpy(c0.copy()).pin_memory()
    yh = torch.empty((T, B, O), dtype=torch.int8).pin_memory()
    h0t, c0t = torch.from_numpy(h0), torch.from_numpy(c0)
    e2e_times = []
    for i in range(2 + min(args.steps, 5)):
        hh.copy_(h0t)
        ch.copy_(c0t)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        q.run_host_raw(xh.data_ptr(), T, B, hh.data_ptr(), ch.data_ptr(), yh.data_ptr())
        dt = time.perf_counter() - t0
        if i >= 2:
            e2e_times.append(dt)
    e2e_t = sum(e2e_times) / len(e2e_times)
    if dist is not None:
        t = torch.tensor([e2e_t], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_t = float(t.item())
    h2d = xh.numel() + hh.numel() + ch.numel() * 2
    d2h = yh.numel() + hh.numel() + ch.numel() * 2
    e2e = {"value": world * B * T / e2e_t, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}
    e2e_matches = bool(np.array_equal(yh.numpy(), y.cpu().numpy()))

    # ---- rooflines.  Input projection: dense int8 contraction on the tensor cores.  Recurrent kernel: the slower of
    # its int8 matmuls at tensor peak and its per-step bytes are both far below the time it takes, which is
    # integer-ALU and barrier time; its headline fraction is against the integer-pipe peak, with the matmul and byte
    # fractions beside it.
    gemm_ops, rec_ops = algorithmic_ops(w.layers, B, T)
    int8_sustained = 2.0 * peaks["bf16_tflops_sustained"]     # TOP/s: bf16 measured x nominal int8:bf16 ratio of 2
    int8_burst = 2.0 * peaks["bf16_tflops"]
    n_l = len(w.layers)
    proj_ms = prof["projection_ms"] / max(args.steps, 1)
    rec_ms = prof["recurrent_ms"] / max(args.steps, 1)
    proj_tops = gemm_ops / (proj_ms * 1e-3) / 1e12 if proj_ms > 0 else 0.0
    rec_tops = rec_ops / (rec_ms * 1e-3) / 1e12 if rec_ms > 0 else 0.0
    sm_mhz = clocks.get("sm_mhz") or clocks.get("sm_max_mhz") or 1965.0
    sm_max = clocks.get("sm_max_mhz") or 1965.0
    mma_peak = None
    if rank == 0:
        try:
            from paper_2101_05453_b200 import binding
            mma_peak = binding.mma_i8_peak(local, 20000)
        except Exception:
            mma_peak = None
    roof_proj = {"kernel": "input_projection", "bound": "tensor", "achieved": proj_tops, "peak": int8_sustained,
                 "unit": "TOP/s", "frac": proj_tops / int8_sustained, "traffic": None,
                 "peak_source": f"2 x bf16 sustained ({peaks['source']}): the kernel is timed inside the long pass",
                 "frac_vs_2x_bf16_burst": proj_tops / int8_burst,
                 "measured_mma_i8_issue_peak_tops": mma_peak,
                 "frac_vs_measured_mma_issue_peak": (proj_tops / mma_peak) if mma_peak else None,
                 "achieved_at_max_clock": proj_tops * sm_max / sm_mhz,
                 "ms_per_launch": proj_ms / n_l}
    if (args.config == NCU_PROJECTION["config"] and B * T == NCU_PROJECTION["rows"]
            and projection_source_sha() == NCU_PROJECTION["source_sha"]):
        roof_proj["traffic"] = NCU_PROJECTION["bytes"]                                   # bytes per launch (one layer)
    q0 = w.layers[0]
    G0 = 3 if (q0.flags & 8) else 4
    roof_proj["algorithmic_hbm_bytes"] = B * T * q0.n_input + q0.n_input * q0.n_cell * G0 + 2 * B * T * q0.n_cell * G0
    roof_proj["hbm_frac"] = roof_proj["algorithmic_hbm_bytes"] / (proj_ms / n_l * 1e-3) / 1e9 / peaks["hbm_gbs"] if proj_ms > 0 else None
    int_ops = algorithmic_int_ops(w.layers, B, T)
    sm_ghz = sm_mhz / 1e3
    alu_peak = 148 * INT_LANES_PER_SM * sm_ghz / 1e3                     # T int-op/s at the clock seen during the run
    rec_alu = int_ops / (rec_ms * 1e-3) / 1e12 if rec_ms > 0 else 0.0
    rec_bytes = T * B * (q0.n_cell * G0 * 2 + q0.n_output) + 2 * B * (q0.n_output + 2 * q0.n_cell)
    roof_rec = {"kernel": "recurrent", "bound": "alu", "achieved": rec_alu, "peak": alu_peak, "unit": "Tint-op/s",
                "frac": rec_alu / alu_peak, "traffic": None,
                "peak_source": f"148 SMs x {INT_LANES_PER_SM} int32 lanes x {sm_ghz:.3f} GHz (SM clock sampled during the run); "
                               "a derived model: the per-unit operation counts are this library's own leanest forms",
                "frac_vs_issue_peak_128_per_clk": rec_alu / (2 * alu_peak),
                "frac_counting_activations_as_lookups": (algorithmic_int_ops(w.layers, B, T, OPS_ACTIVATION_LOOKUP) /
                                                         (rec_ms * 1e-3) / 1e12 / alu_peak) if rec_ms > 0 else 0.0,
                "activation_note": "achieved / frac count a sigmoid or tanh as the arithmetic of its fixed-point definition "
                                   f"({OPS_ACTIVATION} operations: the unit of work of the method); the kernel reads memoised "
                                   f"values instead ({OPS_ACTIVATION_LOOKUP} operations), which the second fraction counts",
                "algorithmic_int_ops_per_launch": int_ops / n_l,
                "matmul_tops": rec_tops, "matmul_frac_of_int8_peak": rec_tops / int8_sustained,
                "matmul_frac_of_2x_bf16_burst": rec_tops / int8_burst,
                "hbm_frac": rec_bytes / (rec_ms / n_l * 1e-3) / 1e9 / peaks["hbm_gbs"] if rec_ms > 0 else None,
                "ms_per_launch": rec_ms / n_l,
                "us_per_layer_step": 1e3 * rec_ms / (n_l * T),
                "phase_us_per_layer_step": {k: 1e3 * prof_phase[k] / (n_l * T) for k in
                                            ("phase_a_ms", "matmul_a_ms", "wait_a_ms", "phase_b_ms", "wait_b_ms", "phase_c_ms", "wait_c_ms")},
                "phase_note": "separate pass with the device phase timers on (they slow the kernel: "
                              f"{1e3 * prof_phase['recurrent_ms'] / (n_l * T):.2f} us per layer-step in that pass)"}
    if (args.config == NCU_RECURRENT["config"] and B == NCU_RECURRENT["batch"] and T == NCU_RECURRENT["steps"]
            and recurrent_source_sha() == NCU_RECURRENT["source_sha"]):
        roof_rec["traffic"] = NCU_RECURRENT["bytes"]                                     # bytes per launch (one layer)
    # algorithmic HBM bytes of the recurrent kernel per launch: X read once, y written once, state in and out
    roof_rec["algorithmic_hbm_bytes"] = rec_bytes
    dominant = roof_rec if rec_ms >= proj_ms else roof_proj

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": {"workload": f"config{args.config}-{w.config.name} batch {B} T {T}",
                       "layers": n_l, "n_input": w.layers[0].n_input, "n_cell": w.layers[0].n_cell,
                       "n_output": O, "l2": "256 MiB buffer written between timed passes; X workspace "
                       f"{T * B * w.layers[0].n_cell * 8 / 1e6:.0f} MB per layer exceeds L2"},
            "clocks": clocks, "e2e": e2e, "e2e_matches_device_run": e2e_matches,
            "gpu_launches": prof["projection_launches"] + prof["recurrent_launches"] + prof["other_launches"],
            "roofline": dominant, "roofline_projection": roof_proj, "roofline_recurrent": roof_rec}

    def time_passes(qh, wl, n_warm=3, n_timed=3, impl=None, profile=False):
        """Median pass time (ms) of workload wl on handle qh with everything resident; optionally the per-kernel profile."""
        if impl is not None:
            qh.set_impl(*impl)
        xs = torch.from_numpy(wl.x).to(dev)
        hs0, cs0 = wl.initial_state()
        hs, cs = torch.from_numpy(hs0).to(dev), torch.from_numpy(cs0).to(dev)
        ys = torch.zeros((wl.T, wl.B, wl.layers[-1].n_output), dtype=torch.int8, device=dev)
        ts = []
        qh.set_profiling(1 if profile else 0)
        for i in range(n_warm + n_timed):
            if i == n_warm and profile:
                qh.get_profile(reset=True)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            qh.run(xs, wl.T, wl.B, hs, cs, ys, stream=stream)
            b.record()
            torch.cuda.synchronize()
            if i >= n_warm:
                ts.append(a.elapsed_time(b))
        qh.last_status()
        pr = qh.get_profile(reset=True) if profile else None
        qh.set_profiling(0)
        return statistics.median(ts), pr, n_timed

    def streaming_us(qh, wl, n_calls=60):
        """One time step per call on the default stream, state carried by the caller: microseconds per call."""
        xs1 = torch.from_numpy(wl.x[:1]).to(dev).contiguous()
        hs0, cs0 = wl.initial_state()
        hs, cs = torch.from_numpy(hs0).to(dev), torch.from_numpy(cs0).to(dev)
        ys1 = torch.zeros((1, wl.B, wl.layers[-1].n_output), dtype=torch.int8, device=dev)
        for _ in range(10):
            qh.run(xs1, 1, wl.B, hs, cs, ys1, stream=stream)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(n_calls):
            qh.run(xs1, 1, wl.B, hs, cs, ys1, stream=stream)
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        qh.last_status()
        return 1e6 * dt / n_calls

    def config_entry(index, Bc, with_oracle=True):
        """One row of the per-configuration table: whole pass, its two kernels, and the oracle on a bounded sample."""
        wl = make_workload(index, batch=Bc)
        qh = qlstm.QLSTM(wl.layers, wl.T, wl.B, device=local)
        ms, pr, n = time_passes(qh, wl, profile=True)
        nl = len(wl.layers)
        g_ops, _ = algorithmic_ops(wl.layers, wl.B, wl.T)
        ent = {"workload": f"config{index}-{wl.config.name} batch {wl.B} T {wl.T}", "value": wl.B * wl.T / (ms * 1e-3), "unit": UNIT,
               "ms_per_pass": ms, "us_per_timestep_whole_stack": 1e3 * ms / wl.T}
        if pr["projection_launches"] > 0:
            p_ms = pr["projection_ms"] / n
            tops = g_ops / (p_ms * 1e-3) / 1e12
            ent.update(path="per layer: projection GEMM + persistent recurrent kernel", projection_us_per_launch=1e3 * p_ms / nl,
                       projection_tops=tops, projection_frac_of_2x_bf16_sustained=tops / int8_sustained,
                       projection_frac_of_2x_bf16_burst=tops / int8_burst,
                       recurrent_us_per_layer_step=1e3 * pr["recurrent_ms"] / (n * nl * wl.T))
        else:
            ent.update(path="whole-stack kernel (layers as a wavefront, input projection inside the step)",
                       us_per_layer_step=1e3 * ms / (nl * wl.T))
        if wl.B <= 4:
            ent["streaming_us_per_call_T1"] = streaming_us(qh, wl)
        qh.close()
        if with_oracle and not args.no_cpu_baseline:
            from oracle import qlstm_ref
            cores = qlstm_ref.num_threads()
            rows_n = max(1, min(wl.B, cores))
            v0, dt0, _ = oracle_sample(index, cores, 2, rows_n)
            T_s = int(max(2, min(wl.T, 2.5 / max(dt0 / 2, 1e-6))))
            v, dt, cores = oracle_sample(index, cores, T_s, rows_n)
            ent["cpu_oracle"] = {"value": v, "unit": UNIT, "cores": cores, "sample": f"{rows_n} rows x {T_s} steps, {dt:.1f} s"}
        return ent

    if rank == 0:
        if not args.no_latency and args.config == 5:
            # batch-1 latency on the same model: whole-stack kernel, against the layer-after-layer path
            w1 = make_workload(5, batch=1, T=T)
            q1 = qlstm.QLSTM(w1.layers, T, 1, device=local)
            ms, _, _ = time_passes(q1, w1)
            ms_layers, pr_l, n = time_passes(q1, w1, impl=(0, 2), profile=True)
            q1.set_impl(0, 0)
            line["latency_batch1"] = {"us_per_timestep_whole_stack": 1e3 * ms / T, "us_per_layer_step": 1e3 * ms / (T * n_l),
                                      "ms_per_pass": ms, "kernel": "whole-stack kernel, one launch for all layers and steps",
                                      "layer_after_layer_us_per_timestep": 1e3 * ms_layers / T,
                                      "layer_after_layer_recurrent_us_per_layer_step": 1e3 * pr_l["recurrent_ms"] / (n * n_l * T),
                                      "streaming_us_per_call_T1": streaming_us(q1, w1)}
            q1.close()
            try:
                from paper_2101_05453_b200 import binding
                bar_us = binding.barrier_latency_us(local, 3000)
                phases = 3 if (w.layers[0].flags & 1) else 2
                line["barrier_floor"] = {"us_per_grid_barrier": bar_us, "barriers_per_layer_step": phases,
                                         "us_per_layer_step": bar_us * phases,
                                         "how": "3000 grid-wide barriers back to back, one block per SM, nothing in between"}
            except Exception as exc:                                   # reported, never fatal
                line["barrier_floor"] = {"error": str(exc)}
            # the other batch sizes of the configuration's sweep, then the other configurations
            per = {}
            for Bs in (1, 8, 16, 64):
                per[f"config5_batch{Bs}"] = config_entry(5, Bs, with_oracle=False)
            line["batch_sweep"] = {k.split("batch")[1]: {"value": v["value"], "unit": UNIT, "ms_per_pass": v["ms_per_pass"],
                                                         "us_per_layer_step": 1e3 * v["ms_per_pass"] / (T * n_l)}
                                   for k, v in per.items()}
        if not args.no_cpu_baseline:
            from oracle import qlstm_ref
            cores = qlstm_ref.num_threads()
            rows_n = max(1, min(B, cores))
            v0, dt0, _ = oracle_sample(args.config, cores, 2, rows_n)
            T_s = int(max(2, min(T, 15.0 / (dt0 / 2))))
            v, dt, cores = oracle_sample(args.config, cores, T_s, rows_n)
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": f"{rows_n} batch rows x {T_s} timesteps of the same workload, {dt:.1f} s"}
        if not args.no_latency and args.config == 5:
            for index in (1, 2, 3, 4):
                per[f"config{index}"] = config_entry(index, None)
            per["config1"]["us_per_step_batch1"] = per["config1"]["us_per_timestep_whole_stack"]
            line["per_config"] = per
        print(json.dumps(line))
    q.close()
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
