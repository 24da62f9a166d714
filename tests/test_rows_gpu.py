"""The row-sharded step (workers cut across GPUs, Algorithm 1's ring-allreduce step as a real all-reduce) on
ONE GPU: with a one-rank NCCL group it must equal def_step bit for bit; with two ranks'
halves run one after the other and their block sums added, it must equal the oracle's step
over all workers up to the order in which the workers' values are added."""
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist

import oracle
from paper_2004_05298_b200 import workloads as WL

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    from paper_2004_05298_b200 import binding
    return binding


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.mark.parametrize("pair", [True, False], ids=["pair", "general"])
def test_one_rank_nccl_group_equals_def_step(B, pair):
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    created = not dist.is_initialized()
    if created:
        dist.init_process_group("nccl", init_method="tcp://127.0.0.1:%d" % _free_port(), rank=0, world_size=1,
                                device_id=dev)
    try:
        wl = WL.get(1).scaled(300_004, W=5)
        ctx = B.def_create(wl.d, wl.W, wl.k, 0, wl.lr, wl.momentum)
        B.def_set_small_step_bytes(ctx, 0 if pair else 1 << 60)
        x1 = WL.initial_params(wl, dev); e1, m1 = WL.zeros_state(wl, dev)
        x2 = x1.clone(); e2, m2 = WL.zeros_state(wl, dev)
        block = torch.full((wl.k,), 7.0, device=dev)
        steps = [0, 1, 2] + [t for t in range(3, 4000) if oracle.block_start(3, t, wl.d) + wl.k > wl.d][:1]
        for t in steps:
            g = WL.gradients(wl, t, dev)
            B.def_step(ctx, x1, g, e1, m1, t, 3)
            B.def_step_rows(ctx, x2, g, e2, m2, block, t, 3)
        torch.cuda.synchronize()
        assert torch.equal(x1, x2) and torch.equal(e1, e2) and torch.equal(m1, m2)
        B.def_destroy(ctx)
    finally:
        if created:
            dist.destroy_process_group()


def test_two_ranks_emulated_in_sequence(B):
    dev = torch.device("cuda", 0)
    d, W_local, ranks, k, lr, mu = 200_003, 3, 2, 9_000, 0.1, 0.9       # odd d: general kernel, V = 1
    W = W_local * ranks
    rng = np.random.default_rng(5)
    x0 = (0.05 * rng.standard_normal(d)).astype(np.float32)
    xo = x0.copy(); eo = np.zeros((W, d), np.float32); mo = np.zeros((W, d), np.float32)
    xs = [torch.from_numpy(x0).to(dev) for _ in range(ranks)]           # every rank holds a replica of x
    es = [torch.zeros(W_local, d, device=dev) for _ in range(ranks)]
    ms = [torch.zeros(W_local, d, device=dev) for _ in range(ranks)]
    bs = [torch.zeros(k, device=dev) for _ in range(ranks)]
    ctxs = [B.def_create(d, W_local, k, 0, lr, mu) for _ in range(ranks)]
    for t in range(5):
        gh = (0.1 * rng.standard_normal((W, d))).astype(np.float32)
        for r in range(ranks):
            g = torch.from_numpy(gh[r * W_local:(r + 1) * W_local]).to(dev)
            B.def_step_rows_local(ctxs[r], g, es[r], ms[r], bs[r], t, 8)
        total = bs[0] + bs[1]                                           # what the all-reduce returns
        for r in range(ranks):
            B.def_step_rows_apply(ctxs[r], xs[r], total, W, t, 8)
        oracle.step(xo, gh, eo, mo, d=d, k=k, s=oracle.block_start(8, t, d), eta=lr, mu=mu)
    torch.cuda.synchronize()
    assert torch.equal(xs[0], xs[1]), "replicas diverged"
    got_e = torch.cat(es).cpu().numpy(); got_m = torch.cat(ms).cpu().numpy()
    assert np.array_equal(got_e, eo) and np.array_equal(got_m, mo)      # per-worker state: no cross-rank arithmetic
    err = np.max(np.abs(xs[0].cpu().numpy() - xo)) / np.max(np.abs(xo))
    assert err <= 1e-6, err                                             # only the order of the sum differs
    assert B.lib.def_step_rows_apply(ctxs[0].handle, xs[0].data_ptr(), total.data_ptr(), 2, 0, 8) == B.DEF_ERR_ARG
    for c in ctxs:
        B.def_destroy(c)
