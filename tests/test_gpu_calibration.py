"""Calibration (Section 4) and the Table 2 quantizer on the device, against the host recipe (needs a B200)."""
import numpy as np
import pytest

from oracle import qlstm_ref as R
from workloads import make_workload, random_layer_stack
from workloads.float_lstm import LayerStats, run_sequence
from workloads.quantize import quantize_asym_int8, quantize_model

pytestmark = pytest.mark.gpu

VARIANTS = [dict(), dict(projection=True, layernorm=True), dict(peephole=True, cifg=True),
            dict(projection=True, peephole=True, layernorm=True), dict(layernorm=True, cifg=True)]


def host_ranges(float_layers, x):
    stats = [LayerStats() for _ in float_layers]
    run_sequence(float_layers, x, stats)
    return stats, [{"x_min": s.x_min, "x_max": s.x_max, "h_min": s.h_min, "h_max": s.h_max, "m_min": s.m_min, "m_max": s.m_max,
                    "c_absmax": s.c_absmax, "g_absmax": dict(s.g_absmax)} for s in stats]


@pytest.mark.parametrize("kw", VARIANTS, ids=lambda k: "+".join(sorted(k)) or "basic")
def test_device_calibration_logs_the_same_ranges(kw):
    from paper_2101_05453_b200 import binding
    w = random_layer_stack(900 + len(kw), 2, 24, 56, 40, T=9, B=5, **kw)
    _, want = host_ranges(w.float_layers, w.x_float)
    got = binding.calibrate(w.float_layers, w.x_float)
    for l, (g, r) in enumerate(zip(got, want)):
        for k in ("x_min", "x_max", "h_min", "h_max", "m_min", "m_max", "c_absmax"):
            assert g[k] == pytest.approx(r[k], rel=1e-9, abs=1e-12), (l, k)       # fp64 sums in another order
        if w.float_layers[l].layernorm:
            for gate in w.float_layers[l].gates:
                assert g["g_absmax"][gate] == pytest.approx(r["g_absmax"][gate], rel=1e-9), (l, gate)


@pytest.mark.parametrize("kw", VARIANTS, ids=lambda k: "+".join(sorted(k)) or "basic")
def test_device_quantizer_equals_the_host_recipe(kw):
    """Same ranges in, so every integer and every (multiplier, shift) must be identical: the device does the same
    IEEE operations in the same order."""
    from paper_2101_05453_b200 import binding
    w = random_layer_stack(910 + len(kw), 2, 24, 56, 40, T=6, B=4, **kw)
    stats, ranges = host_ranges(w.float_layers, w.x_float)
    want = quantize_model(w.float_layers, stats)
    got = binding.quantize_model(w.float_layers, ranges)
    for l, (g, r) in enumerate(zip(got, want)):
        for k in ("n_input", "n_cell", "n_output", "flags", "cell_int_bits", "zp_x", "zp_m", "zp_h"):
            assert getattr(g, k) == getattr(r, k), (l, k)
        for k in ("W", "R", "P", "b", "L"):
            for gi in range(4):
                a, b = getattr(g, k)[gi], getattr(r, k)[gi]
                assert (a is None) == (b is None), (l, k, gi)
                if a is not None:
                    assert np.array_equal(a, b), (l, k, gi)
        for k in ("eff_x", "eff_h", "eff_c", "eff_ln"):
            assert [tuple(v) for v in getattr(g, k)] == [tuple(map(int, v)) for v in getattr(r, k)], (l, k)
        assert tuple(g.eff_m) == tuple(map(int, r.eff_m)) and tuple(g.eff_proj) == tuple(map(int, r.eff_proj))
        if r.W_proj is not None:
            assert np.array_equal(g.W_proj, r.W_proj) and np.array_equal(g.b_proj, r.b_proj)
        assert (g.s_x, g.s_h, g.s_m, g.s_c) == (r.s_x, r.s_h, r.s_m, r.s_c)


def test_float_model_to_integer_run_entirely_on_the_device():
    """Calibrate and quantize on the GPU, run the integer path on what came out, and compare with the oracle on the
    same layers (bit exact) and with the float LSTM (within the quantization error bound of the float pins)."""
    import torch
    import paper_2101_05453_b200 as qlstm
    from paper_2101_05453_b200 import binding
    w = make_workload(2, batch=4, T=40)
    ranges = binding.calibrate(w.float_layers, w.x_float)
    layers = binding.quantize_model(w.float_layers, ranges)
    x = quantize_asym_int8(w.x_float, layers[0].s_x, layers[0].zp_x)
    h0 = np.concatenate([np.full(w.B * q.n_output, q.zp_h, np.int8) for q in layers])
    c0 = np.concatenate([np.zeros(w.B * q.n_cell, np.int16) for q in layers])
    want_y, want_h, want_c, _ = R.run(layers, x, h0, c0)
    with qlstm.QLSTM(layers, w.T, w.B) as hnd:
        dev = torch.device("cuda:0")
        xd, hd, cd = (torch.from_numpy(a.copy()).to(dev) for a in (x, h0, c0))
        y = torch.zeros((w.T, w.B, layers[-1].n_output), dtype=torch.int8, device=dev)
        hnd.run(xd, w.T, w.B, hd, cd, y, stream=torch.cuda.current_stream().cuda_stream)
        hnd.last_status()
        assert np.array_equal(y.cpu().numpy(), want_y) and np.array_equal(hd.cpu().numpy(), want_h)
        assert np.array_equal(cd.cpu().numpy(), want_c)
    yf, _, _ = run_sequence(w.float_layers, w.x_float)
    q = layers[-1]
    err = np.abs(q.s_h * (want_y.astype(float) - q.zp_h) - yf)
    assert err.max() <= 0.05 and err.mean() <= 1.0 * q.s_h


def test_calibration_argument_checks():
    import paper_2101_05453_b200 as qlstm
    from paper_2101_05453_b200 import binding
    w = random_layer_stack(930, 1, 16, 32, 32, T=3, B=2)
    fl = w.float_layers[0]
    bad = type(fl)(**{**fl.__dict__})
    bad.n_output = 7                                       # no projection but n_output != n_cell
    with pytest.raises(qlstm.QlstmError) as e:
        binding.calibrate([bad], w.x_float)
    assert e.value.code == qlstm.ERR_DIM
