"""Sharded gradient exchange on CPU ranks (gloo): the movement and ordering logic of paper_2609_17380_b200.dist with the
oracle's accumulator plugged in as the arithmetic.  The folded, gathered gradient must equal, bit for bit, the
single-process fold of the same micro-batch gradients (Sec. 6 / Appendix A: the exchange is movement only)."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2609_17380_b200.dist import PeerReducer, ShardPlan, ShardedReducer


def _grad(m, n):
    g = np.random.default_rng(1000 + m).standard_normal(n).astype(np.float32) * np.float32(1e-3)
    g[::7] *= np.float32(2.0 ** -20)      # a few tiny magnitudes so that rounding order matters
    return g


def _single(mesh, n):
    acc = oracle.Accum(mesh[0], mesh[1], mesh[2], n)
    for m in range(mesh[0] * mesh[1] * mesh[2]):
        acc.push(_grad(m, n))
    return acc.result()


def _worker(rank, world, port, mesh, n, outdir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        M = mesh[0] * mesh[1] * mesh[2]
        plan = ShardPlan(M, world, n)
        red = ShardedReducer(plan, rank, "cpu")
        stage = torch.empty(n, dtype=torch.float32)
        for j, m in enumerate(plan.local_microbatches(rank)):
            red.wait()                                  # the staging buffer is free again
            stage.copy_(torch.from_numpy(_grad(m, n)))
            red.scatter(j, stage)

        def fold(slices, out):
            acc = oracle.Accum(mesh[0], mesh[1], mesh[2], out.numel())
            for s in slices:
                acc.push(s.numpy())
            out.copy_(torch.from_numpy(acc.result()))

        out = torch.full((plan.padded,), float("nan"))
        got = red.fold_and_gather(fold, out).numpy()
        np.save(os.path.join(outdir, "rank%d.npy" % rank), got)
    finally:
        dist.destroy_process_group()


def _peer_worker(rank, world, port, mesh, n, outdir, stashes):
    """The peer-memory variant: `stashes` are shared-memory tensors standing in for the ranks' symmetric buffers."""
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        M = mesh[0] * mesh[1] * mesh[2]
        plan = ShardPlan(M, world, n)
        red = PeerReducer(plan, rank, stashes[rank], lambda owner, j, lo, hi: stashes[owner][j, lo:hi], dist.barrier)
        for j, m in enumerate(plan.local_microbatches(rank)):
            red.scatter(j, torch.from_numpy(_grad(m, n)))

        def fold(slices, out):
            acc = oracle.Accum(mesh[0], mesh[1], mesh[2], out.numel())
            for s in slices:
                acc.push(s.numpy())
            out.copy_(torch.from_numpy(acc.result()))

        out = torch.full((plan.padded,), float("nan"))
        np.save(os.path.join(outdir, "rank%d.npy" % rank), red.fold_and_gather(fold, out).numpy())
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world,mesh,n", [(2, (2, 2, 2), 1000), (4, (2, 2, 2), 300), (3, (1, 2, 3), 5000)])
def test_peer_fold_equals_single_process(tmp_path, world, mesh, n):
    M = mesh[0] * mesh[1] * mesh[2]
    stashes = [torch.zeros((M // world, n), dtype=torch.float32).share_memory_() for _ in range(world)]
    mp.spawn(_peer_worker, args=(world, _free_port(), mesh, n, str(tmp_path), stashes), nprocs=world, join=True)
    want = _single(mesh, n)
    for r in range(world):
        got = np.load(tmp_path / ("rank%d.npy" % r))
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), "rank %d differs" % r


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


@pytest.mark.parametrize("world,mesh,n", [(2, (2, 2, 2), 1000), (4, (2, 2, 2), 1000), (4, (2, 2, 2), 300),
                                          (2, (1, 2, 3), 777), (3, (1, 2, 3), 5000), (8, (2, 2, 2), 4099)])
def test_sharded_fold_equals_single_process(tmp_path, world, mesh, n):
    mp.spawn(_worker, args=(world, _free_port(), mesh, n, str(tmp_path)), nprocs=world, join=True)
    want = _single(mesh, n)
    for r in range(world):
        got = np.load(tmp_path / ("rank%d.npy" % r))
        assert got.shape == want.shape
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), "rank %d differs" % r


def test_shard_plan():
    p = ShardPlan(8, 4, 1000)
    assert [p.owner(m) for m in range(8)] == [0, 0, 1, 1, 2, 2, 3, 3]
    assert list(p.local_microbatches(2)) == [4, 5]
    b = [p.bounds(c) for c in range(4)]
    assert b[0][0] == 0 and b[-1][1] == 1000 and all(b[i][1] == b[i + 1][0] for i in range(3))
    assert all(lo % 4 == 0 for lo, _ in b) and p.padded >= 1000 and p.chunk % 256 == 0
    q = ShardPlan(8, 4, 300)                      # fewer elements than ranks x alignment: trailing slices are empty
    assert [q.bounds(c) for c in range(4)] == [(0, 256), (256, 300), (300, 300), (300, 300)]
    with pytest.raises(ValueError):
        ShardPlan(8, 3, 1000)
