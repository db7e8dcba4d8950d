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


def _shard_wgrad(x, d, start, stop, k=0, p=0):
    """Each shard is its own matrix: it samples, splits and quantizes its own rows (no exchange), seeds offset by the shard."""
    mode = osp.MODE_SAMPLED if k else osp.MODE_FULL
    xq = olay.quantize_operand(x[start:stop], k, p, mode, 1 + start)
    dq = olay.quantize_operand(d[start:stop], k, p, mode, 2 + start)
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


def _worker_uneven(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    x, _ = synth.planted(1040, 128, 4, 60.0, 6.0, 1.0, 5)
    d, _ = synth.planted(1040, 64, 4, 6e-3, 6e-4, 1e-4, 6)
    start, stop = parallel.shard_rows(1040, rank, world)
    dw = torch.from_numpy(_shard_wgrad(x, d, start, stop, k=4, p=4)) if stop > start else torch.zeros((64, 128), dtype=torch.float64)
    parallel.allreduce_weight_grad_(dw)
    out[rank] = (start, stop, dw.numpy().copy())
    dist.destroy_process_group()


def test_uneven_shards_with_the_split_path():
    """1040 tokens over 3 and over 4 ranks (shards of 384, 384, 272 rows, and one rank with the short remainder), every
    shard split with k > 0 in SAMPLED mode on its own rows: all ranks end with the same sum of the per-shard gradients."""
    x, _ = synth.planted(1040, 128, 4, 60.0, 6.0, 1.0, 5)
    d, _ = synth.planted(1040, 64, 4, 6e-3, 6e-4, 1e-4, 6)
    exact = d.astype(np.float64).T @ x.astype(np.float64)
    for world in (3, 4):
        port = _free_port()
        with mp.Manager() as mgr:
            out = mgr.dict()
            mp.spawn(_worker_uneven, args=(world, port, out), nprocs=world, join=True)
            res = dict(out)
        ranges = [(res[r][0], res[r][1]) for r in range(world)]
        assert ranges[0][0] == 0 and ranges[-1][1] == 1040 and all(ranges[i][1] == ranges[i + 1][0] for i in range(world - 1))
        assert all((b - a) % 64 == 0 for a, b in ranges[:-1])
        want = sum(_shard_wgrad(x, d, a, b, k=4, p=4) for a, b in ranges if b > a)
        for r in range(world):
            assert np.allclose(res[r][2], want, rtol=1e-12, atol=1e-18)
        assert np.linalg.norm(want - exact) / np.linalg.norm(exact) < 0.25


def test_shard_ranges_cover_rows_once():
    for total, world in ((4096, 2), (4096, 8), (1000, 3), (64, 4)):
        ranges = [parallel.shard_rows(total, r, world) for r in range(world)]
        covered = np.zeros(total, dtype=int)
        for a, b in ranges:
            assert 0 <= a <= b <= total
            covered[a:b] += 1
        assert np.all(covered == 1)
        assert all((b - a) % 64 == 0 for a, b in ranges[:-1] if b < total)
