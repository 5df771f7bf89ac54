"""GPU-side helpers for the parity tests: run a workload through the C ABI on cuda:0."""
import numpy as np

import paper_2101_05453_b200 as qlstm
from paper_2101_05453_b200.binding import parse_trace


def run_gpu(w, impl=(0, 0), trace=False, h0=None, c0=None, handle=None, x=None):
    import torch
    x_np = w.x if x is None else x
    T, B = x_np.shape[0], x_np.shape[1]
    q = handle or qlstm.QLSTM(w.layers, max(T, 1), max(B, 1))
    q.set_impl(*impl)
    hh, cc = w.initial_state()
    if h0 is not None:
        hh, cc = h0, c0
    dev = torch.device("cuda:0")
    xd = torch.from_numpy(np.ascontiguousarray(x_np)).to(dev)
    hd = torch.from_numpy(np.array(hh, copy=True)).to(dev)
    cd = torch.from_numpy(np.array(cc, copy=True)).to(dev)
    yd = torch.zeros((T, B, w.layers[-1].n_output), dtype=torch.int8, device=dev)
    td = None
    if trace:
        td = torch.zeros(max(q.trace_bytes(T, B), 1), dtype=torch.uint8, device=dev)
    q.run(xd, T, B, hd, cd, yd, td, stream=torch.cuda.current_stream().cuda_stream)
    q.last_status()
    tr = parse_trace(td.cpu().numpy(), q.dims, T, B) if trace and T > 0 and B > 0 else None
    out = (yd.cpu().numpy(), hd.cpu().numpy(), cd.cpu().numpy(), tr)
    if handle is None:
        q.close()
    return out


def assert_trace_equal(got, want, what=""):
    for l, (g, r) in enumerate(zip(got, want)):
        for k in r:
            if not np.array_equal(g[k], r[k]):
                bad = np.argwhere(g[k] != r[k])
                raise AssertionError(f"{what} layer {l} tensor {k}: {len(bad)} mismatches, first at {bad[0]}: "
                                     f"gpu {g[k][tuple(bad[0])]} oracle {r[k][tuple(bad[0])]}")
