"""Multi-process (gloo, world size 2, CPU) check of the batch sharding: every rank runs its shard of the
batch, and the gathered shards equal the full-batch result.  The per-rank compute here is the CPU oracle
(no GPU in this test); the sharding arithmetic is the package's own."""
import os
import socket

import numpy as np
import pytest

from paper_2101_05453_b200.sharding import shard_bounds, state_slices


def test_shard_bounds_partition():
    for n in (0, 1, 7, 8, 256, 257):
        for world in (1, 2, 3, 8):
            spans = [shard_bounds(n, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
            sizes = [e - b for b, e in spans]
            assert max(sizes) - min(sizes) <= 1


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out_path):
    import torch
    import torch.distributed as dist
    from oracle import qlstm_ref
    from workloads import random_layer_stack
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = random_layer_stack(123, 2, 12, 24, 16, projection=True, layernorm=True, T=6, B=5)
    h0, c0 = w.initial_state()
    b0, b1 = shard_bounds(w.B, rank, world)
    hi, ci = state_slices(w.layers, w.B, b0, b1)
    y, _, _, _ = qlstm_ref.run(w.layers, w.x[:, b0:b1], h0[hi], c0[ci])
    # gather variable-sized shards: pad to the largest
    width = max(shard_bounds(w.B, r, world)[1] - shard_bounds(w.B, r, world)[0] for r in range(world))
    pad = np.zeros((w.T, width, y.shape[2]), np.int8)
    pad[:, :y.shape[1]] = y
    bufs = [torch.zeros(pad.shape, dtype=torch.int8) for _ in range(world)]
    dist.all_gather(bufs, torch.from_numpy(pad))
    t = torch.tensor([float(rank + 1)])
    dist.all_reduce(t, op=dist.ReduceOp.MAX)            # the timing reduction bench.py does
    if rank == 0:
        parts = []
        for r in range(world):
            e0, e1 = shard_bounds(w.B, r, world)
            parts.append(bufs[r].numpy()[:, :e1 - e0])
        full, _, _, _ = qlstm_ref.run(w.layers, w.x, h0, c0)
        ok = np.array_equal(np.concatenate(parts, axis=1), full) and float(t) == world
        with open(out_path, "w") as f:
            f.write("ok" if ok else "mismatch")
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_shards_concatenate_to_full_batch(tmp_path):
    import torch.multiprocessing as mp
    out = str(tmp_path / "result.txt")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    assert open(out).read() == "ok"
