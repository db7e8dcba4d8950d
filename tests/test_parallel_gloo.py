"""World-size-2 CPU test (gloo) of the token-sharded path: shards cover the tokens exactly once and the
weight gradient is the all-reduced sum of the per-shard gradients (computed here with the oracle)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import layer as olay, split as osp
from paper_2509_00404_b200 import parallel, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _shard_wgrad(x, d, start, stop):
    xq = olay.quantize_operand(x[start:stop], 0, 0, osp.MODE_FULL, 1)
    dq = olay.quantize_operand(d[start:stop], 0, 0, osp.MODE_FULL, 2)
    return olay.linear_wgrad(dq, xq)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    x, _ = synth.planted(256, 128, 4, 60.0, 6.0, 1.0, 5)
    d, _ = synth.planted(256, 64, 4, 6e-3, 6e-4, 1e-4, 6)
    start, stop = parallel.shard_rows(256, rank, world)
    dw = torch.from_numpy(_shard_wgrad(x, d, start, stop))
    parallel.allreduce_weight_grad_(dw)
    out[rank] = (start, stop, dw.numpy().copy())
    dist.destroy_process_group()


def test_two_rank_token_sharding_and_weight_gradient_sum():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    (s0, e0, dw0), (s1, e1, dw1) = res[0], res[1]
    assert (s0, e0, s1, e1) == (0, 128, 128, 256)
    assert np.array_equal(dw0, dw1)                                    # every rank holds the same sum
    x, _ = synth.planted(256, 128, 4, 60.0, 6.0, 1.0, 5)
    d, _ = synth.planted(256, 64, 4, 6e-3, 6e-4, 1e-4, 6)
    want = _shard_wgrad(x, d, 0, 128) + _shard_wgrad(x, d, 128, 256)
    assert np.allclose(dw0, want, rtol=1e-12, atol=1e-15)
    exact = d.astype(np.float64).T @ x.astype(np.float64)
    assert np.linalg.norm(dw0 - exact) / np.linalg.norm(exact) < 0.2      # NVFP4-level agreement with the unsharded product


def test_shard_ranges_cover_rows_once():
    for total, world in ((4096, 2), (4096, 8), (1000, 3), (64, 4)):
        ranges = [parallel.shard_rows(total, r, world) for r in range(world)]
        covered = np.zeros(total, dtype=int)
        for a, b in ranges:
            assert 0 <= a <= b <= total
            covered[a:b] += 1
        assert np.all(covered == 1)
        assert all((b - a) % 64 == 0 for a, b in ranges[:-1] if b < total)
