"""The allocation-free layer-norm entry point against the existing per-row one (needs a B200).

Collected last on purpose: a failure here must not hide any other test from a run that stops at the
first failure.  qlstm_layernorm_rows_static serves callers that cannot allocate device memory when they
need a result (a real-time per-frame loop, a process whose own arena owns the whole GPU, a plug-in
callback); its only scratch is a fixed array inside the library, shared by all calls.  The test calls it
twice in a row - the second time with fewer rows, a different width and different data, so that anything
wrongly carried over in that array from the first call would show - and checks every row bit for bit
against qlstm_eval_layernorm_row, and against the CPU oracle's layer norm as well.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _rows(rng, rows, n):
    q = (rng.integers(-32768, 32768, (rows, n)) // rng.integers(1, 40, (rows, 1))).astype(np.int16)
    q[0] = 77                                         # a constant row: sigma = 0
    L = rng.integers(-32767, 32768, n).astype(np.int16)
    b = (rng.integers(-2 ** 31 + 1, 2 ** 31, n) // 997).astype(np.int32)
    eff = (int(rng.integers(1 << 30, 1 << 31)), int(rng.integers(-13, -8)))
    return q, L, b, eff


def _run_static(binding, torch, q, L, b, eff):
    rows, n = q.shape
    qd, Ld, bd = (torch.from_numpy(a).cuda() for a in (q, L, b))
    out = torch.zeros((rows, n), dtype=torch.int16, device="cuda")
    binding.layernorm_rows_static(qd, rows, n, Ld, bd, eff, out, stream=torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def _run_per_row(binding, torch, q, L, b, eff):
    rows, n = q.shape
    Ld, bd = torch.from_numpy(L).cuda(), torch.from_numpy(b).cuda()
    res = np.empty_like(q)
    for r in range(rows):
        qd = torch.from_numpy(q[r].copy()).cuda()
        out = torch.zeros(n, dtype=torch.int16, device="cuda")
        binding.eval_layernorm_row(qd, n, Ld, bd, eff, out, stream=torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        res[r] = out.cpu().numpy()
    return res


def test_static_scratch_layernorm_matches_per_row_entry_point_twice():
    import torch
    from paper_2101_05453_b200 import binding
    rng = np.random.default_rng(2101)
    first = _rows(rng, 37, 2048)
    second = _rows(rng, 5, 1000)
    for q, L, b, eff in (first, second):
        got = _run_static(binding, torch, q, L, b, eff)
        want = _run_per_row(binding, torch, q, L, b, eff)
        assert np.array_equal(got, want)                 # integer arithmetic: bit exact
        from oracle import qlstm_ref
        for r in range(q.shape[0]):
            assert np.array_equal(got[r], qlstm_ref.layernorm_row(q[r], L, b, eff)), r


def test_static_scratch_size_limit_is_reported():
    import torch
    import paper_2101_05453_b200 as qlstm
    from paper_2101_05453_b200 import binding
    q = torch.zeros((1, 16), dtype=torch.int16, device="cuda")
    L = torch.ones(16, dtype=torch.int16, device="cuda")
    b = torch.zeros(16, dtype=torch.int32, device="cuda")
    with pytest.raises(qlstm.QlstmError) as e:
        binding.layernorm_rows_static(q, 4097, 16, L, b, (1 << 30, -10), q)
    assert e.value.code == qlstm.ERR_DIM


def test_static_scratch_rejects_scales_outside_the_encodable_window():
    import torch
    import paper_2101_05453_b200 as qlstm
    from paper_2101_05453_b200 import binding
    q = torch.zeros((1, 16), dtype=torch.int16, device="cuda")
    L = torch.ones(16, dtype=torch.int16, device="cuda")
    b = torch.zeros(16, dtype=torch.int32, device="cuda")
    for eff in ((1 << 30, -32), (1 << 29, -5), (1 << 30, 31)):
        with pytest.raises(qlstm.QlstmError) as e:
            binding.layernorm_rows_static(q, 1, 16, L, b, eff, q)
        assert e.value.code == qlstm.ERR_ARG
        with pytest.raises(qlstm.QlstmError) as e:
            binding.eval_layernorm_row(q, 16, L, b, eff, q)
        assert e.value.code == qlstm.ERR_ARG
