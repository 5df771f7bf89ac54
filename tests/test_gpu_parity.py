"""Parity of the CUDA path against the CPU oracle, bit for bit, through the C ABI (needs a B200)."""
import copy

import numpy as np
import pytest

from oracle import qlstm_ref as R
from tests.gpu_util import assert_trace_equal, run_gpu
from workloads import make_workload, random_layer_stack

pytestmark = pytest.mark.gpu

SIMPLE, FAST, AUTO = 1, 2, 0
STACK = 5            # recurrent_impl: the whole-stack kernel for small batches, forced (schedule chosen by the call's length)
STACK_WAVEFRONT, STACK_SEQUENTIAL = 6, 7          # ... with one of its two schedules forced


def oracle(w, trace=False, x=None, h0=None, c0=None):
    hh, cc = w.initial_state()
    if h0 is not None:
        hh, cc = h0, c0
    return R.run(w.layers, w.x if x is None else x, hh, cc, trace=trace)


def check_equal(got, want, what):
    for name, g, r in zip(("y", "h", "c"), got[:3], want[:3]):
        if not np.array_equal(g, r):
            bad = np.argwhere(g != r)
            raise AssertionError(f"{what}: {name} differs at {len(bad)} places, first {bad[0]}: "
                                 f"gpu {g[tuple(bad[0])]} oracle {r[tuple(bad[0])]}")


# ------------------------------------------------------------------ every tensor at every step

@pytest.mark.parametrize("index", [1, 2])
def test_trace_parity_small_configs(index):
    w = make_workload(index)
    want = oracle(w, trace=True)
    got = run_gpu(w, impl=(SIMPLE, SIMPLE), trace=True)
    assert_trace_equal(got[3], want[3], f"config {index}")
    check_equal(got, want, f"config {index}")


VARIANTS = [
    dict(),
    dict(projection=True),
    dict(peephole=True),
    dict(layernorm=True),
    dict(cifg=True),
    dict(projection=True, peephole=True, layernorm=True),
    dict(projection=True, layernorm=True),
    dict(peephole=True, cifg=True),
    dict(layernorm=True, cifg=True, projection=True),
    dict(peephole=True, layernorm=True, cifg=True, projection=True),
]


@pytest.mark.parametrize("kw", VARIANTS, ids=lambda k: "+".join(sorted(k)) or "basic")
def test_trace_parity_variants_ragged_shapes(kw):
    # odd widths: nothing is a multiple of a tile, a warp or a vector
    w = random_layer_stack(40 + len(kw), 2, 19, 37, 23, T=7, B=5, **kw)
    want = oracle(w, trace=True)
    got = run_gpu(w, impl=(SIMPLE, SIMPLE), trace=True)
    assert_trace_equal(got[3], want[3], str(kw))
    check_equal(got, want, str(kw))


@pytest.mark.parametrize("kw", VARIANTS, ids=lambda k: "+".join(sorted(k)) or "basic")
def test_auto_path_parity_variants(kw):
    # shapes that span several tiles of the fast kernels plus a ragged tail
    w = random_layer_stack(60 + len(kw), 2, 48, 176, 80, T=9, B=11, **kw)
    want = oracle(w)
    got = run_gpu(w, impl=(AUTO, AUTO))
    check_equal(got, want, str(kw))


@pytest.mark.parametrize("kw", VARIANTS, ids=lambda k: "+".join(sorted(k)) or "basic")
def test_fast_kernels_forced_parity_variants(kw):
    """Tensor-core projection and persistent recurrent kernel forced on (an unsupported shape would raise)."""
    w = random_layer_stack(90 + len(kw), 2, 64, 208, 96, T=8, B=37, **kw)
    want = oracle(w)
    got = run_gpu(w, impl=(FAST, FAST))
    check_equal(got, want, str(kw))


@pytest.mark.parametrize("B", [1, 2, 31, 128, 129, 200, 256])
def test_fast_kernels_batch_sizes(B):
    w = random_layer_stack(7, 1, 32, 64, 48, projection=True, layernorm=True, T=5, B=B)
    want = oracle(w)
    got = run_gpu(w, impl=(FAST, FAST))
    check_equal(got, want, f"B={B}")


@pytest.mark.parametrize("B", [1, 2, 3, 4, 8, 16])
@pytest.mark.parametrize("kw", [dict(projection=True, layernorm=True), dict(cifg=True), dict(peephole=True, projection=True),
                                dict(peephole=True, layernorm=True)], ids=lambda k: "+".join(sorted(k)))
def test_small_batch_both_matmul_paths(B, kw):
    """At batch <= 4 the recurrent kernel uses dp4a mat-vecs by default; impl 3 forces the tensor-core path, impl 4
    the dp4a path up to batch 16."""
    w = random_layer_stack(300 + B, 2, 32, 112, 48, T=6, B=B, **kw)
    want = oracle(w)
    check_equal(run_gpu(w, impl=(FAST, FAST)), want, f"default path B={B} {kw}")
    check_equal(run_gpu(w, impl=(FAST, 3)), want, f"tcgen05 B={B} {kw}")
    check_equal(run_gpu(w, impl=(FAST, 4)), want, f"dp4a B={B} {kw}")


# ------------------------------------------------------------------ whole-stack kernel (batch <= 16)

@pytest.mark.parametrize("B", [1, 2, 3, 4, 7, 16])
@pytest.mark.parametrize("kw", VARIANTS, ids=lambda k: "+".join(sorted(k)) or "basic")
def test_stack_kernel_parity_variants(B, kw):
    """All layers and steps in one launch: three layers so that the wavefront is deeper than one hand-over, widths that
    leave ragged shares to the last block of a group; both schedules (one group of blocks per layer / every layer on
    all blocks)."""
    w = random_layer_stack(500 + B, 3, 48, 112, 64, T=7, B=B, **kw)
    want = oracle(w)
    check_equal(run_gpu(w, impl=(AUTO, STACK_WAVEFRONT)), want, f"stack kernel, wavefront, B={B} {kw}")
    check_equal(run_gpu(w, impl=(AUTO, STACK_SEQUENTIAL)), want, f"stack kernel, sequential, B={B} {kw}")


@pytest.mark.parametrize("index,kw", [(1, {}), (2, {}), (3, dict(batch=2, T=12)), (4, dict(batch=3, T=12)),
                                      (5, dict(batch=1, T=24)), (5, dict(batch=4, T=8)), (5, dict(batch=8, T=12)),
                                      # one cell per thread instead of four lanes per cell (batch x cells of a block above
                                      # 128), with layer norm + peephole and its second statistics exchange
                                      (3, dict(batch=16, T=6)), (3, dict(batch=8, T=3)), (4, dict(batch=16, T=6))])
@pytest.mark.parametrize("impl", [STACK_WAVEFRONT, STACK_SEQUENTIAL])
def test_stack_kernel_parity_configs(index, kw, impl):
    w = make_workload(index, **kw)
    check_equal(run_gpu(w, impl=(AUTO, impl)), oracle(w), f"stack kernel config {index} {kw}")


@pytest.mark.parametrize("index,kw", [(1, {}), (2, dict(batch=2, T=20)), (5, dict(batch=1, T=10))])
def test_streaming_one_step_per_call(index, kw):
    """One time step per call, the state carried by the caller (Section 3.2.2): y, h and c of every call against
    the oracle's trace - bit for bit, and through the default kernel selection."""
    import paper_2101_05453_b200 as qlstm
    w = make_workload(index, **kw)
    want = oracle(w, trace=True)
    tr = want[3]
    h, c = w.initial_state()
    with qlstm.QLSTM(w.layers, 1, w.B) as hnd:
        for t in range(w.T):
            y, h, c, _ = run_gpu(w, handle=hnd, x=w.x[t:t + 1], h0=h, c0=c)
            assert np.array_equal(y[0], want[0][t]), f"y differs at step {t}"
            off_h = off_c = 0
            for l, q in enumerate(w.layers):
                assert np.array_equal(c[off_c:off_c + w.B * q.n_cell].reshape(w.B, q.n_cell), tr[l]["c"][t]), (l, t)
                assert np.array_equal(h[off_h:off_h + w.B * q.n_output].reshape(w.B, q.n_output), tr[l]["h"][t]), (l, t)
                off_h += w.B * q.n_output
                off_c += w.B * q.n_cell
    check_equal((want[0], h, c), want, "state after the last call")


def test_stack_kernel_bounded_wait_reports_timeout():
    """Every counter of the whole-stack kernel waits for an arrival nobody makes: the waits run into their 3 ms limit,
    all blocks leave, the status is QLSTM_ERR_TIMEOUT and the next run on the handle is correct."""
    import paper_2101_05453_b200 as qlstm
    w = random_layer_stack(58, 2, 32, 64, 48, projection=True, layernorm=True, T=4, B=2)
    want = oracle(w)
    with qlstm.QLSTM(w.layers, w.T, w.B) as hnd:
        for impl in (STACK_WAVEFRONT, STACK_SEQUENTIAL):
            hnd.debug_barrier_timeout(1, 3_000_000)
            with pytest.raises(qlstm.QlstmError) as e:
                run_gpu(w, handle=hnd, impl=(AUTO, impl))
            assert e.value.code == qlstm.ERR_TIMEOUT
            hnd.debug_barrier_timeout(0)
            check_equal(run_gpu(w, handle=hnd, impl=(AUTO, impl)), want, "after timeout")


def test_stack_kernel_refuses_what_it_cannot_run():
    import paper_2101_05453_b200 as qlstm
    w = random_layer_stack(59, 1, 32, 64, 64, T=3, B=17)
    with qlstm.QLSTM(w.layers, w.T, w.B) as hnd:
        with pytest.raises(qlstm.QlstmError) as e:
            run_gpu(w, handle=hnd, impl=(AUTO, STACK))          # batch 17 > 16
        assert e.value.code == qlstm.ERR_DIM


def test_trace_parity_config3_slice():
    w = make_workload(3, batch=3, T=6)
    want = oracle(w, trace=True)
    got = run_gpu(w, impl=(SIMPLE, SIMPLE), trace=True)
    assert_trace_equal(got[3], want[3], "config 3")


# ------------------------------------------------------------------ the five configurations

@pytest.mark.parametrize("index,kw", [
    (1, {}), (2, {}),
    (3, dict(batch=32, T=24)),
    (4, dict(batch=64, T=24)),
    (5, dict(batch=1, T=24)),
    (5, dict(batch=8, T=24)),
    (5, dict(batch=64, T=6)),
])
def test_config_parity(index, kw):
    w = make_workload(index, **kw)
    want = oracle(w)
    got = run_gpu(w)
    check_equal(got, want, f"config {index} {kw}")


@pytest.mark.parametrize("index,rows", [(3, [0, 13, 31]), (4, [0, 40, 63]), (5, [0, 100, 255])])
def test_full_size_parity_on_sampled_rows(index, rows):
    """Full T and full batch on the GPU in the launch configuration the benchmark times; the oracle
    recomputes sampled batch rows one by one (rows never interact)."""
    w = make_workload(index)
    got = run_gpu(w)
    ws = make_workload(index, rows=rows)
    want = oracle(ws)
    y = got[0][:, rows]
    assert np.array_equal(y, want[0]), f"config {index}: y differs on sampled rows"
    off_h = off_c = 0
    offs_h = offs_c = 0
    for q in w.layers:
        hg = got[1][off_h:off_h + w.B * q.n_output].reshape(w.B, q.n_output)[rows]
        cg = got[2][off_c:off_c + w.B * q.n_cell].reshape(w.B, q.n_cell)[rows]
        hr = want[1][offs_h:offs_h + len(rows) * q.n_output].reshape(len(rows), q.n_output)
        cr = want[2][offs_c:offs_c + len(rows) * q.n_cell].reshape(len(rows), q.n_cell)
        assert np.array_equal(hg, hr) and np.array_equal(cg, cr)
        off_h += w.B * q.n_output
        off_c += w.B * q.n_cell
        offs_h += len(rows) * q.n_output
        offs_c += len(rows) * q.n_cell


@pytest.mark.parametrize("batch,rows", [(1, [0]), (8, [0, 7]), (64, [0, 63])])
def test_full_length_parity_config5_batch_sweep(batch, rows):
    """The production-shaped stack over all 300 steps at the smaller batch sizes of its sweep (the launch
    configurations whose latency the benchmark reports), against the oracle on sampled rows."""
    w = make_workload(5, batch=batch)
    got = run_gpu(w)
    want = oracle(make_workload(5, rows=rows))
    assert np.array_equal(got[0][:, rows], want[0]), f"config 5 batch {batch}: y differs on sampled rows"
    off_h = off_c = offs_h = offs_c = 0
    for q in w.layers:
        hg = got[1][off_h:off_h + w.B * q.n_output].reshape(w.B, q.n_output)[rows]
        cg = got[2][off_c:off_c + w.B * q.n_cell].reshape(w.B, q.n_cell)[rows]
        hr = want[1][offs_h:offs_h + len(rows) * q.n_output].reshape(len(rows), q.n_output)
        cr = want[2][offs_c:offs_c + len(rows) * q.n_cell].reshape(len(rows), q.n_cell)
        assert np.array_equal(hg, hr) and np.array_equal(cg, cr)
        off_h += w.B * q.n_output
        off_c += w.B * q.n_cell
        offs_h += len(rows) * q.n_output
        offs_c += len(rows) * q.n_cell


@pytest.mark.parametrize("kw,B", [(dict(projection=True, layernorm=True), 37), (dict(peephole=True, layernorm=True), 20),
                                  (dict(cifg=True), 130), (dict(projection=True, peephole=True), 3)],
                         ids=lambda v: "+".join(sorted(v)) if isinstance(v, dict) else str(v))
def test_persistent_kernel_cell_state_every_step(kw, B):
    """The persistent kernel hands back c only at the end of a call, so it is called one step at a time on one
    handle and c^t, h^t of every layer are compared with the oracle's trace at every step."""
    import paper_2101_05453_b200 as qlstm
    w = random_layer_stack(123, 2, 32, 96, 48, T=9, B=B, **kw)
    _, _, _, tr = oracle(w, trace=True)
    h, c = w.initial_state()
    with qlstm.QLSTM(w.layers, 1, w.B) as hnd:
        for t in range(w.T):
            y, h, c, _ = run_gpu(w, handle=hnd, impl=(FAST, FAST), x=w.x[t:t + 1], h0=h, c0=c)
            off_h = off_c = 0
            for l, q in enumerate(w.layers):
                ct = c[off_c:off_c + w.B * q.n_cell].reshape(w.B, q.n_cell)
                ht = h[off_h:off_h + w.B * q.n_output].reshape(w.B, q.n_output)
                assert np.array_equal(ct, tr[l]["c"][t]), f"{kw}: c of layer {l} differs at step {t}"
                assert np.array_equal(ht, tr[l]["h"][t]), f"{kw}: h of layer {l} differs at step {t}"
                off_h += w.B * q.n_output
                off_c += w.B * q.n_cell
            assert np.array_equal(y[0], tr[-1]["h"][t])


# ------------------------------------------------------------------ pieces and edge cases

@pytest.mark.parametrize("impl", [SIMPLE, AUTO])
def test_input_projection_matches_oracle(impl):
    import torch
    import paper_2101_05453_b200 as qlstm
    w = random_layer_stack(77, 1, 96, 200, 200, T=5, B=70, peephole=True)
    _, _, _, tr = oracle(w, trace=True)
    q = w.layers[0]
    rows = w.T * w.B
    with qlstm.QLSTM(w.layers, w.T, w.B) as hnd:
        hnd.set_impl(impl, impl)
        xd = torch.from_numpy(w.x).cuda()
        out = torch.zeros((rows, q.n_cell, 4), dtype=torch.int16, device="cuda")
        hnd.input_projection(0, xd, rows, out, stream=torch.cuda.current_stream().cuda_stream)
        hnd.last_status()
        got = out.cpu().numpy().reshape(w.T, w.B, q.n_cell, 4).transpose(0, 3, 1, 2)
    assert np.array_equal(got, tr[0]["xg"])


@pytest.mark.parametrize("cifg", [False, True], ids=["four-gates", "three-gates"])
def test_input_projection_many_tiles_per_block(cifg):
    """6000 rows x 600 cells: several output tiles per block, a ragged last m-tile and a ragged last panel; with four
    gates the blocks take equal contiguous tile ranges, with three (CIFG) one panel per block and shared m-tile ranges."""
    import torch
    import paper_2101_05453_b200 as qlstm
    from paper_2101_05453_b200.binding import projection_plan
    w = random_layer_stack(78, 1, 96, 600, 600, T=40, B=150, cifg=cifg)
    q = w.layers[0]
    G = 3 if cifg else 4
    rows = w.T * w.B
    pl = projection_plan(rows, q.n_cell * G, q.n_input)
    assert pl["per_cta"] > 1 and (pl["m_ranges"] > 0) == cifg
    _, _, _, tr = oracle(w, trace=True)
    with qlstm.QLSTM(w.layers, w.T, w.B) as hnd:
        xd = torch.from_numpy(w.x).cuda()
        out = torch.zeros((rows, q.n_cell, G), dtype=torch.int16, device="cuda")
        hnd.input_projection(0, xd, rows, out, stream=torch.cuda.current_stream().cuda_stream)
        hnd.last_status()
        got = out.cpu().numpy().reshape(w.T, w.B, q.n_cell, G).transpose(0, 3, 1, 2)
    assert np.array_equal(got, tr[0]["xg"][:, 4 - G:])


def test_streaming_equivalence_and_state_carry():
    import paper_2101_05453_b200 as qlstm
    w = random_layer_stack(81, 2, 32, 64, 48, projection=True, layernorm=True, T=10, B=6)
    want = oracle(w)
    with qlstm.QLSTM(w.layers, w.T, w.B) as hnd:
        y1, h1, c1, _ = run_gpu(w, handle=hnd, x=w.x[:3])
        y2, h2, c2, _ = run_gpu(w, handle=hnd, x=w.x[3:], h0=h1, c0=c1)
    check_equal((np.concatenate([y1, y2]), h2, c2), want, "streaming")


def test_run_host_matches_device_run():
    import paper_2101_05453_b200 as qlstm
    w = make_workload(2)
    want = oracle(w)
    h0, c0 = w.initial_state()
    with qlstm.QLSTM(w.layers, w.T, w.B) as hnd:
        got = hnd.run_host(w.x, h0, c0)
    check_equal(got, want, "run_host")


def test_deterministic_run_to_run():
    w = make_workload(3, batch=16, T=10)
    a = run_gpu(w)
    b = run_gpu(w)
    check_equal(a, b, "determinism")


def test_empty_inputs_and_limits():
    import torch
    import paper_2101_05453_b200 as qlstm
    w = make_workload(1)
    with qlstm.QLSTM(w.layers, 4, 2) as hnd:
        x = torch.zeros((4, 2, 16), dtype=torch.int8, device="cuda")
        h = torch.full((64,), 5, dtype=torch.int8, device="cuda")
        c = torch.full((64,), 9, dtype=torch.int16, device="cuda")
        y = torch.zeros((4, 2, 32), dtype=torch.int8, device="cuda")
        hnd.run(x, 0, 2, h, c, y)          # T = 0: no-op
        hnd.run(x, 4, 0, h, c, y)          # B = 0: no-op
        hnd.last_status()
        assert int(h[0]) == 5 and int(c[0]) == 9
        with pytest.raises(qlstm.QlstmError) as e:
            hnd.run(x, 5, 2, h, c, y)      # beyond max_T
        assert e.value.code == qlstm.ERR_ARG
        with pytest.raises(qlstm.QlstmError) as e:
            hnd.run(None, 4, 2, h, c, y)
        assert e.value.code == qlstm.ERR_ARG


def test_misaligned_device_pointers_are_rejected_before_any_launch():
    """x, c, y (and the projection's output) are accessed with 16- / 32-byte vectors; a sliced pointer is an
    argument error, not a device fault.  h may sit anywhere."""
    import torch
    import paper_2101_05453_b200 as qlstm
    w = random_layer_stack(57, 1, 32, 64, 64, T=3, B=4)
    want = oracle(w)
    h0, c0 = w.initial_state()
    with qlstm.QLSTM(w.layers, w.T, w.B) as hnd:
        pad = 64
        xb = torch.zeros(w.x.size + pad, dtype=torch.int8, device="cuda")
        yb = torch.zeros(w.T * w.B * 64 + pad, dtype=torch.int8, device="cuda")
        hb = torch.zeros(h0.size + pad, dtype=torch.int8, device="cuda")
        cb = torch.zeros(c0.size + pad, dtype=torch.int16, device="cuda")
        ok = dict(x=xb.data_ptr(), h=hb.data_ptr(), c=cb.data_ptr(), y=yb.data_ptr())
        for name, off in (("x", 4), ("y", 8), ("c", 2)):
            args = dict(ok)
            args[name] += off
            with pytest.raises(qlstm.QlstmError) as e:
                hnd.run(args["x"], w.T, w.B, args["h"], args["c"], args["y"])
            assert e.value.code == qlstm.ERR_ARG, name
        out = torch.zeros(w.T * w.B * 256 + pad, dtype=torch.int16, device="cuda")
        with pytest.raises(qlstm.QlstmError) as e:
            hnd.input_projection(0, ok["x"], w.T * w.B, out.data_ptr() + 16)
        assert e.value.code == qlstm.ERR_ARG
        # an odd h pointer is fine
        xb[:w.x.size] = torch.from_numpy(w.x.reshape(-1)).cuda()
        hb[3:3 + h0.size] = torch.from_numpy(h0).cuda()
        cb[:c0.size] = torch.from_numpy(c0).cuda()
        hnd.run(ok["x"], w.T, w.B, ok["h"] + 3, ok["c"], ok["y"], stream=torch.cuda.current_stream().cuda_stream)
        hnd.last_status()
        got = (yb[:w.T * w.B * 64].cpu().numpy().reshape(w.T, w.B, 64), hb[3:3 + h0.size].cpu().numpy(), cb[:c0.size].cpu().numpy())
        check_equal(got, want, "odd h pointer")


def test_bounded_wait_reports_timeout_and_handle_stays_usable():
    """A grid barrier that waits for an arrival nobody makes runs into its (here 3 ms) limit: the kernel returns
    by itself, the status is QLSTM_ERR_TIMEOUT, and the next run on the same handle is correct again."""
    import paper_2101_05453_b200 as qlstm
    w = random_layer_stack(55, 1, 32, 64, 48, projection=True, layernorm=True, T=4, B=20)
    want = oracle(w)
    with qlstm.QLSTM(w.layers, w.T, w.B) as hnd:
        hnd.set_impl(FAST, FAST)
        hnd.debug_barrier_timeout(1, 3_000_000)
        with pytest.raises(qlstm.QlstmError) as e:
            run_gpu(w, handle=hnd, impl=(FAST, FAST))
        assert e.value.code == qlstm.ERR_TIMEOUT
        hnd.debug_barrier_timeout(0)
        check_equal(run_gpu(w, handle=hnd, impl=(FAST, FAST)), want, "after timeout")


def test_batch_beyond_the_persistent_kernel_limit_uses_the_simple_path():
    w = random_layer_stack(56, 1, 16, 32, 32, T=3, B=300)
    check_equal(run_gpu(w), oracle(w), "B=300")


def test_folded_bias_out_of_range_is_rejected():
    import paper_2101_05453_b200 as qlstm
    w = make_workload(1)
    bad = copy.deepcopy(w.layers[0])
    bad.R[1][:] = 127
    bad.zp_h = bad.zp_m = -128
    bad.b[1][:] = 2 ** 31 - 1              # b - zp_h * sum(R) leaves int32
    with pytest.raises(qlstm.QlstmError) as e:
        qlstm.QLSTM([bad], 4, 1)
    assert e.value.code == qlstm.ERR_RANGE


def test_saturating_extremes_match_oracle():
    """Hand-built layer whose every clamp engages: accumulator + bias, gate sum, cell update."""
    from workloads.quantize import QLayer
    C = 8
    q = QLayer(4, C, C, 0, 0, -128, -128, -128)
    for g in range(4):
        q.W[g] = np.full((C, 4), 127, np.int8)
        q.R[g] = np.full((C, C), 127 if g != 2 else -127, np.int8)
        q.b[g] = np.full(C, 2 ** 31 - 1 - 127 * 128 * C, np.int32)
        q.eff_x[g] = (1 << 30, 5)
        q.eff_h[g] = ((1 << 31) - 1, -10)
    q.eff_m = (1 << 30, -21)
    x = np.full((3, 2, 4), 127, np.int8)

    class W:
        layers = [q]
        B, T = 2, 3

        def initial_state(self):
            return np.full(2 * C, 127, np.int8), np.full(2 * C, 32767, np.int16)
    w = W()
    w.x = x
    want = oracle(w, trace=True)
    got = run_gpu(w, impl=(SIMPLE, SIMPLE), trace=True)
    assert_trace_equal(got[3], want[3], "extremes")
    got2 = run_gpu(w)
    check_equal(got2, want, "extremes auto")


# ------------------------------------------------------------------ building blocks over their whole domain

@pytest.mark.parametrize("m", [0, 1, 2, 3, 4, 5, 6, 9, 15])
def test_device_activations_exhaustive(m):
    """Every int16 input of the kernels' integer sigmoid / tanh, on the device, against the oracle."""
    import torch
    from paper_2101_05453_b200 import binding
    sig = torch.zeros(65536, dtype=torch.int16, device="cuda")
    tnh = torch.zeros(65536, dtype=torch.int16, device="cuda")
    binding.eval_activations(m, sig, tnh, stream=torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert np.array_equal(sig.cpu().numpy().astype(np.int32), R.sigmoid_all(m))
    assert np.array_equal(tnh.cpu().numpy().astype(np.int32), R.tanh_all(m))


@pytest.mark.parametrize("m,room", [(0, 128), (1, 128), (2, 128), (2, 96), (3, 128), (3, 64), (4, 128), (5, 128), (5, 96),
                                    (6, 128), (9, 128), (15, 128)])
def test_device_activation_tables_exhaustive(m, room):
    """The memoised nonlinearities of the persistent kernel (tables built as at create time for `room` KB of idle shared
    memory, the kernel's own lookup code) on every int16 input against the oracle: sigmoid and tanh of the gates
    (Q3.12), tanh of a Q_{m.15-m} cell."""
    import torch
    from paper_2101_05453_b200 import binding
    out = [torch.full((65536,), 12345, dtype=torch.int16, device="cuda") for _ in range(3)]
    lay = binding.eval_activation_tables(m, room * 1024, *out, stream=torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    nbytes, tz_off, tc_off, tz_amax, tc_amax, tc_mode, sig_packed = lay
    assert 0 < nbytes <= room * 1024 and nbytes % 16 == 0, lay         # the definition passes the formats' checks
    assert tz_off % 16 == 0 and tc_off % 16 == 0
    assert tc_mode == (0 if m == 3 else (1 if m < 3 else 2)), lay      # steps of 2^m fit the 5-bit offsets up to m = 3
    assert sig_packed == (1 if room < 128 else 0), lay                 # the plain sigmoid table alone is 64 KB
    assert 0 < tz_amax <= 32768 and 0 < tc_amax <= 32768
    sig, tz, tc = (o.cpu().numpy().astype(np.int32) for o in out)
    assert np.array_equal(sig, R.sigmoid_all(3))
    assert np.array_equal(tz, R.tanh_all(3))
    assert np.array_equal(tc, R.tanh_all(m))


def test_device_activation_tables_that_do_not_fit():
    import torch
    from paper_2101_05453_b200 import binding
    out = [torch.full((65536,), 12345, dtype=torch.int16, device="cuda") for _ in range(3)]
    lay = binding.eval_activation_tables(2, 48 * 1024, *out, stream=torch.cuda.current_stream().cuda_stream)
    assert lay[0] == 0
    assert all(int(o.min()) == 12345 and int(o.max()) == 12345 for o in out)


@pytest.mark.parametrize("idx,B", [(5, 256), (5, 40), (4, 64), (3, 32), (2, 8)])
def test_tables_and_arithmetic_agree(idx, B):
    """The same call with the memoised nonlinearities and with the definition evaluated in the kernel: identical
    outputs and state, both equal to the oracle (which the other parity tests compare the default path with)."""
    import torch
    import paper_2101_05453_b200 as qlstm
    T = 6
    w = make_workload(idx, batch=B, T=T)
    O = w.layers[-1].n_output
    dev = torch.device("cuda:0")
    q = qlstm.QLSTM(w.layers, T, B, device=0)
    q.set_impl(2, 2)
    res = []
    for enable in (1, 0, 2):                  # tables; definition evaluated; general instantiation (any scale)
        n_tab = q.activation_tables(enable)
        assert n_tab == len(w.layers)                 # every layer of these configurations has room for its tables
        h0, c0 = w.initial_state()
        h, c = torch.from_numpy(h0).to(dev), torch.from_numpy(c0).to(dev)
        y = torch.zeros((T, B, O), dtype=torch.int8, device=dev)
        q.run(torch.from_numpy(w.x).to(dev), T, B, h, c, y)
        torch.cuda.synchronize()
        q.last_status()
        res.append((y.cpu().numpy(), h.cpu().numpy(), c.cpu().numpy()))
    q.close()
    check_equal(res[0], res[1], f"config {idx} batch {B}: tables against arithmetic")
    check_equal(res[0], res[2], f"config {idx} batch {B}: tables against the general instantiation")
    if B <= 64:
        check_equal(res[0], oracle(w), f"config {idx} batch {B}: tables against the oracle")


@pytest.mark.parametrize("kw", VARIANTS, ids=lambda k: "+".join(sorted(k)) or "basic")
@pytest.mark.parametrize("B", [2, 40])
def test_scales_with_a_left_shift(B, kw):
    """Effective scales of 1 and above (shift > 0, Section 3.2.4's rescale with its saturating left shift) in every
    place the recurrent part rescales: the layers then take the general instantiation of the persistent kernel and the
    general epilogue of the projection GEMM.  Everything saturates early; the result is still the oracle's, bit for bit."""
    w = random_layer_stack(900 + B, 2, 32, 112, 48, T=5, B=B, **kw)
    for q in w.layers:
        for g in range(4):
            if q.eff_h[g] is not None and q.eff_h[g][0]:
                q.eff_h[g] = (q.eff_h[g][0], 1)
            if g == 1 and q.eff_x[g] is not None and q.eff_x[g][0]:
                q.eff_x[g] = (q.eff_x[g][0], 2)
            if getattr(q, "eff_c", None) and q.eff_c[g] is not None and q.eff_c[g][0]:
                q.eff_c[g] = (q.eff_c[g][0], 1)
            if getattr(q, "eff_ln", None) and q.eff_ln[g] is not None and q.eff_ln[g][0] and g == 2:
                q.eff_ln[g] = (q.eff_ln[g][0], 1)
        q.eff_m = (q.eff_m[0], 1)
        if q.eff_proj[0]:
            q.eff_proj = (q.eff_proj[0], 1)
    want = oracle(w)
    check_equal(run_gpu(w, impl=(FAST, FAST)), want, f"left shifts, fast kernels, B={B} {kw}")
    check_equal(run_gpu(w, impl=(SIMPLE, SIMPLE)), want, f"left shifts, simple kernels, B={B} {kw}")


@pytest.mark.parametrize("seed", range(10))
def test_device_layernorm_rows(seed):
    import torch
    from paper_2101_05453_b200 import binding
    rng = np.random.default_rng(700 + seed)
    n = int(rng.integers(1, 8191)) if seed else 8191
    q = (rng.integers(-32768, 32768, n) // int(rng.integers(1, 60))).astype(np.int16)
    if seed == 1:
        q[:] = 123                                   # sigma = 0
    if seed == 2:
        q[:] = 0
        q[n // 2] = 32767                            # one outlier: the largest z-score
    if seed == 3:
        q = np.where(np.arange(n) % 2 == 0, 32767, -32768).astype(np.int16)
    L = rng.integers(-32767, 32768, n).astype(np.int16)
    b = (rng.integers(-2 ** 31 + 1, 2 ** 31, n) // int(rng.integers(1, 3000))).astype(np.int32)
    eff = (int(rng.integers(1 << 30, 1 << 31)), int(rng.integers(-14, 2)))
    qd, Ld, bd = (torch.from_numpy(a).cuda() for a in (q, L, b))
    out = torch.zeros(n, dtype=torch.int16, device="cuda")
    binding.eval_layernorm_row(qd, n, Ld, bd, eff, out, stream=torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy(), R.layernorm_row(q, L, b, eff))
