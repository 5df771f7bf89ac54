"""Bidirectional stacks (Section 7) through the C ABI against the oracle run once per direction (needs a B200)."""
import numpy as np
import pytest

from oracle import qlstm_ref as R
from workloads import random_layer_stack

pytestmark = pytest.mark.gpu


def two_directions(seed, n_layers, I, C, O, T, B, **kw):
    f = random_layer_stack(seed, n_layers, I, C, O, T=T, B=B, **kw)
    b = random_layer_stack(seed + 1000, n_layers, I, C, O, T=T, B=B, **kw)
    b.layers[0].zp_x = f.layers[0].zp_x                 # both directions read the same int8 input
    return f, b


@pytest.mark.parametrize("kw,B,T", [(dict(), 3, 9), (dict(projection=True, layernorm=True), 20, 6),
                                    (dict(cifg=True, peephole=True), 130, 5), (dict(projection=True), 1, 12)],
                         ids=lambda v: "+".join(sorted(v)) or "basic" if isinstance(v, dict) else str(v))
def test_bidirectional_matches_two_oracle_runs(kw, B, T):
    import torch
    import paper_2101_05453_b200 as qlstm
    f, b = two_directions(70, 2, 32, 96, 48, T, B, **kw)
    x = f.x
    hf0, cf0 = f.initial_state()
    hb0, cb0 = b.initial_state()
    yf, hf, cf, _ = R.run(f.layers, x, hf0, cf0)
    yb, hb, cb, _ = R.run(b.layers, x[::-1], hb0, cb0)          # the backward stack walks the sequence from its end
    want = np.concatenate([yf, yb[::-1]], axis=2)               # at step t: forward h^t | backward state after x_{T-1}..x_t
    with qlstm.BiQLSTM(f.layers, b.layers, T, B) as q:
        dev = torch.device("cuda:0")
        xd = torch.from_numpy(np.ascontiguousarray(x)).to(dev)
        st = [torch.from_numpy(a.copy()).to(dev) for a in (hf0, cf0, hb0, cb0)]
        y = torch.zeros((T, B, q.n_output), dtype=torch.int8, device=dev)
        for _ in range(2):                                      # a second call on the same handle: workspaces are reused
            for t_, a in zip(st, (hf0, cf0, hb0, cb0)):
                t_.copy_(torch.from_numpy(a))
            q.run(xd, T, B, st[0], st[1], st[2], st[3], y, stream=torch.cuda.current_stream().cuda_stream)
            q.last_status()
            assert np.array_equal(y.cpu().numpy(), want)
            for got, ref in zip(st, (hf, cf, hb, cb)):
                assert np.array_equal(got.cpu().numpy(), ref)


def test_bidirectional_argument_checks():
    import paper_2101_05453_b200 as qlstm
    f, b = two_directions(71, 1, 32, 64, 64, 4, 2)
    b.layers[0].zp_x = f.layers[0].zp_x + 1                     # the two directions disagree about their input
    with pytest.raises(qlstm.QlstmError) as e:
        qlstm.BiQLSTM(f.layers, b.layers, 4, 2)
    assert e.value.code == qlstm.ERR_ARG
