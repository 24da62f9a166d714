"""Column sharding over ranks, on CPU: two gloo ranks each take their column range of every
[W, d] tensor, run the step on it (the oracle's column view stands in for def_step_columns,
which takes the same j0 / n arguments), and the pieces put together must equal the unsharded
step exactly -- with no exchange between the ranks during the steps."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2004_05298_b200 import workloads as WL


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, d, steps, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl = WL.get(2).scaled(d, W=3)
        j0, j1 = WL.shard_columns(wl.d, world, rank)
        n = j1 - j0
        cols = np.arange(j0, j1, dtype=np.int64)
        x = WL.initial_params(wl, "cpu").numpy()[j0:j1].copy()
        e = np.zeros((wl.W, n), np.float32)
        m = np.zeros((wl.W, n), np.float32)
        for t in range(steps):
            g = np.ascontiguousarray(WL.gradients(wl, t, "cpu").numpy()[:, j0:j1])
            s = oracle.block_start(wl.rbgs_seed, t, wl.d)       # drawn over the global d on every rank
            oracle.step(x, g, e, m, d=wl.d, k=wl.k, s=s, eta=wl.lr, mu=wl.momentum, cols=cols)
        # the only communication: collecting the shards afterwards, to compare
        sizes = [torch.zeros(1, dtype=torch.int64) for _ in range(world)]
        dist.all_gather(sizes, torch.tensor([n]))
        np.savez(os.path.join(out_dir, "rank%d.npz" % rank), x=x, e=e, m=m, j0=j0, j1=j1)
        dist.barrier()
        # time reduction used by the benchmark: max over ranks
        tmax = torch.tensor([float(rank + 1)], dtype=torch.float64)
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        assert float(tmax) == float(world)
        assert sum(int(v) for v in sizes) == wl.d
    finally:
        dist.destroy_process_group()


def test_two_ranks_column_sharding(tmp_path):
    world, d, steps = 2, 50_002, 5                      # d % 4 == 2: the shard boundary gets rounded
    mp.spawn(_rank_main, args=(world, _free_port(), d, steps, str(tmp_path)), nprocs=world, join=True)
    wl = WL.get(2).scaled(d, W=3)
    x = WL.initial_params(wl, "cpu").numpy().copy()
    e = np.zeros((wl.W, wl.d), np.float32)
    m = np.zeros((wl.W, wl.d), np.float32)
    for t in range(steps):
        g = WL.gradients(wl, t, "cpu").numpy()
        oracle.step(x, g, e, m, d=wl.d, k=wl.k, s=oracle.block_start(wl.rbgs_seed, t, wl.d), eta=wl.lr, mu=wl.momentum)
    covered = 0
    for rank in range(world):
        part = np.load(tmp_path / ("rank%d.npz" % rank))
        j0, j1 = int(part["j0"]), int(part["j1"])
        assert j0 == covered and j0 % 4 == 0
        covered = j1
        assert np.array_equal(part["x"], x[j0:j1])
        assert np.array_equal(part["e"], e[:, j0:j1]) and np.array_equal(part["m"], m[:, j0:j1])
    assert covered == wl.d


def test_shard_columns_partition():
    for d in (1, 3, 4, 10, 855_770, 138_357_544):
        for world in (1, 2, 3, 4, 8):
            edges = [WL.shard_columns(d, world, r) for r in range(world)]
            assert edges[0][0] == 0 and edges[-1][1] == d
            for (a0, a1), (b0, b1) in zip(edges[:-1], edges[1:]):
                assert a1 == b0 and a0 <= a1
            assert all(j0 % 4 == 0 or j0 == d for j0, _ in edges)      # empty trailing shards sit at d
