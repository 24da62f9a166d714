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


# ---------------------------------------------------------------------------
# Row sharding: workers cut across ranks, Algorithm 1's ring-allreduce step as an all-reduce (gloo, CPU).
# Each rank gets the sum of its own workers' sparsified vectors from the oracle (a step from
# x = 0 with eta-scaled inputs moves x by minus their mean; two workers per rank keep the
# mean's scaling exact), the ranks all-reduce those sums, and every rank applies the average.
# ---------------------------------------------------------------------------
def _rows_rank_main(rank, world, port, d, k, steps, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        W_local, lr, mu = 2, 0.1, 0.9
        rng = np.random.default_rng(77)                               # same stream on every rank
        x = (0.05 * rng.standard_normal(d)).astype(np.float32)
        e = np.zeros((W_local, d), np.float32); m = np.zeros((W_local, d), np.float32)
        for t in range(steps):
            g_all = (0.1 * rng.standard_normal((W_local * world, d))).astype(np.float32)
            g = np.ascontiguousarray(g_all[rank * W_local:(rank + 1) * W_local])
            s = oracle.block_start(4, t, d)
            moved = np.zeros(d, np.float32)
            oracle.step(moved, g, e, m, d=d, k=k, s=s, eta=lr, mu=mu)  # moved = -(local sum) / W_local
            local_sum = torch.from_numpy(-moved * W_local)
            dist.all_reduce(local_sum, op=dist.ReduceOp.SUM)            # the k block values (zeros elsewhere)
            x = x - local_sum.numpy() / np.float32(W_local * world)
        np.savez(os.path.join(out_dir, "rows%d.npz" % rank), x=x, e=e, m=m)
    finally:
        dist.destroy_process_group()


def test_two_ranks_row_sharding(tmp_path):
    world, d, k, steps = 2, 5_003, 700, 6
    mp.spawn(_rows_rank_main, args=(world, _free_port(), d, k, steps, str(tmp_path)), nprocs=world, join=True)
    rng = np.random.default_rng(77)
    x = (0.05 * rng.standard_normal(d)).astype(np.float32)
    W = 2 * world
    e = np.zeros((W, d), np.float32); m = np.zeros((W, d), np.float32)
    for t in range(steps):
        g = (0.1 * rng.standard_normal((W, d))).astype(np.float32)
        oracle.step(x, g, e, m, d=d, k=k, s=oracle.block_start(4, t, d), eta=0.1, mu=0.9)
    parts = [np.load(tmp_path / ("rows%d.npz" % r)) for r in range(world)]
    assert np.array_equal(parts[0]["x"], parts[1]["x"]), "replicas diverged"
    assert np.array_equal(np.concatenate([p["e"] for p in parts]), e)
    assert np.array_equal(np.concatenate([p["m"] for p in parts]), m)
    assert np.max(np.abs(parts[0]["x"] - x)) <= 1e-6 * np.max(np.abs(x))
