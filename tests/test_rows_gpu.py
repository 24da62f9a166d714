"""The row-sharded step (workers cut across GPUs, Algorithm 1's ring-allreduce step as a real all-reduce) on
ONE GPU: with a one-rank NCCL group it must equal def_step bit for bit -- for every d mod 4, with
and without the side stream that takes the all-reduce off the critical path, with and without the
fused detach output; with two ranks' halves run one after the other and their block sums added,
it must equal the oracle's step over all workers up to the order in which the workers' values are
added."""
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


@pytest.fixture(scope="module")
def one_rank_group():
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    created = not dist.is_initialized()
    if created:
        dist.init_process_group("nccl", init_method="tcp://127.0.0.1:%d" % _free_port(), rank=0, world_size=1,
                                device_id=dev)
    yield dev
    if created:
        dist.destroy_process_group()


@pytest.mark.parametrize("side_stream", [False, True], ids=["one_stream", "side_stream"])
@pytest.mark.parametrize("detach", [False, True], ids=["plain", "detach"])
@pytest.mark.parametrize("pair", [True, False], ids=["pair", "general"])
@pytest.mark.parametrize("d", [300_004, 300_005, 300_006, 300_007])
def test_one_rank_nccl_group_equals_def_step(B, one_rank_group, d, pair, detach, side_stream):
    """d % 4 in {0, 1, 2, 3}: the 128-bit kernel pair, and the flat stream with the block-columns kernel."""
    dev = one_rank_group
    wl = WL.get(1).scaled(d, W=5)
    ctx = B.def_create(wl.d, wl.W, wl.k, 0, wl.lr, wl.momentum, (0.4, 0.0))
    B.def_set_small_step_bytes(ctx, 0 if pair else 1 << 60)
    side = torch.cuda.Stream() if side_stream else None
    if side_stream:
        B.def_set_rows_stream(ctx, side)
    x1 = WL.initial_params(wl, dev); e1, m1 = WL.zeros_state(wl, dev)
    x2 = x1.clone(); e2, m2 = WL.zeros_state(wl, dev)
    z1 = torch.full((wl.W, wl.d), -3.0, device=dev); z2 = torch.full((wl.W, wl.d), -4.0, device=dev)
    block = torch.full((wl.k,), 7.0, device=dev)
    steps = [0, 1, 2] + [t for t in range(3, 4000) if oracle.block_start(3, t, wl.d) + wl.k > wl.d][:1]
    gs = [WL.gradients(wl, t, dev) for t in steps]
    torch.cuda.synchronize()
    for t, g in zip(steps, gs):                      # nothing between the calls waits for the GPU
        if detach:
            B.def_step_detach(ctx, x1, g, e1, m1, z1, t, 3)
        else:
            B.def_step(ctx, x1, g, e1, m1, t, 3)
        B.def_step_rows(ctx, x2, g, e2, m2, block, t, 3, detached_out=z2 if detach else None)
    torch.cuda.synchronize()
    assert torch.equal(x1, x2) and torch.equal(e1, e2) and torch.equal(m1, m2)
    if detach:
        assert torch.equal(z1, z2)
    if pair and d % 4 != 0:
        # the flat path: the general kernel is not needed for contiguous rows with aligned bases
        B.def_set_kernel_timing(ctx, True)
        B.def_step_rows_local(ctx, gs[0], e2, m2, block, 0, 3)
        torch.cuda.synchronize()
        assert B.def_kernel_time(ctx, B.DEF_KERNEL_GENERAL)[1] == 0
        assert B.def_kernel_time(ctx, B.DEF_KERNEL_STREAM)[1] == 1 and B.def_kernel_time(ctx, B.DEF_KERNEL_BLOCK)[1] == 1
    if side_stream:
        B.def_set_rows_stream(ctx, None)
    B.def_destroy(ctx)


def test_block_sums_are_complete_when_the_side_stream_reads_them(B):
    """k = d on the pair path: the block kernel does all the work and the stream kernel none.  A
    reader on the side stream (standing in for the all-reduce) must see every block sum, and the
    next step on the context's stream must see the update."""
    dev = torch.device("cuda", 0)
    d, W, lr, mu, seed = 1_000_000, 6, 0.1, 0.9, 5
    rng = np.random.default_rng(3)
    ctx = B.def_create(d, W, d, 0, lr, mu)
    B.def_set_small_step_bytes(ctx, 0)
    side = torch.cuda.Stream()
    B.def_set_rows_stream(ctx, side)
    x = torch.from_numpy((0.05 * rng.standard_normal(d)).astype(np.float32)).to(dev)
    e = torch.zeros(W, d, device=dev); m = torch.zeros(W, d, device=dev)
    xo = x.cpu().numpy().copy(); eo = np.zeros((W, d), np.float32); mo = np.zeros((W, d), np.float32)
    ghs = [(0.1 * rng.standard_normal((W, d))).astype(np.float32) for _ in range(6)]
    gs = [torch.from_numpy(g).to(dev) for g in ghs]
    block = torch.zeros(d, device=dev)
    seen = torch.zeros(len(gs), d, device=dev)
    torch.cuda.synchronize()
    for t, g in enumerate(gs):
        B.def_step_rows_local(ctx, g, e, m, block, t, seed)
        with torch.cuda.stream(side):
            seen[t].copy_(block)                     # ordered only by the side stream
        B.def_step_rows_apply(ctx, x, block, W, t, seed)
    torch.cuda.synchronize()
    for t, gh in enumerate(ghs):
        before = xo.copy()
        s = oracle.block_start(seed, t, d)
        oracle.step(xo, gh, eo, mo, d=d, k=d, s=s, eta=lr, mu=mu)
        # block_sum[i] belongs to coordinate (s + i) mod d; x_t - x_{t+1} = sum / W up to two roundings
        sums = np.roll(seen[t].cpu().numpy(), s)
        assert np.allclose(sums / np.float32(W), before - xo, rtol=0, atol=1e-6)
    assert np.array_equal(x.cpu().numpy(), xo) and np.array_equal(m.cpu().numpy(), mo)
    assert not e.any()
    B.def_destroy(ctx)


@pytest.mark.parametrize("detach", [False, True], ids=["plain", "detach"])
@pytest.mark.parametrize("d", [200_003, 200_004], ids=["odd_d", "aligned_d"])
def test_two_ranks_emulated_in_sequence(B, d, detach):
    dev = torch.device("cuda", 0)
    W_local, ranks, k, lr, mu, lam = 3, 2, 9_000, 0.1, 0.9, 0.3
    W = W_local * ranks
    rng = np.random.default_rng(5)
    x0 = (0.05 * rng.standard_normal(d)).astype(np.float32)
    xo = x0.copy(); eo = np.zeros((W, d), np.float32); mo = np.zeros((W, d), np.float32)
    xs = [torch.from_numpy(x0).to(dev) for _ in range(ranks)]           # every rank holds a replica of x
    es = [torch.zeros(W_local, d, device=dev) for _ in range(ranks)]
    ms = [torch.zeros(W_local, d, device=dev) for _ in range(ranks)]
    zs = [torch.full((W_local, d), -5.0, device=dev) for _ in range(ranks)]
    bs = [torch.zeros(k, device=dev) for _ in range(ranks)]
    ctxs = [B.def_create(d, W_local, k, 0, lr, mu, (lam, 0.0)) for _ in range(ranks)]
    for c in ctxs:
        B.def_set_small_step_bytes(c, 0)
    for t in range(5):
        gh = (0.1 * rng.standard_normal((W, d))).astype(np.float32)
        for r in range(ranks):
            g = torch.from_numpy(gh[r * W_local:(r + 1) * W_local]).to(dev)
            if detach:
                B.def_step_rows_local_detach(ctxs[r], xs[r], g, es[r], ms[r], bs[r], zs[r], t, 8)
            else:
                B.def_step_rows_local(ctxs[r], g, es[r], ms[r], bs[r], t, 8)
        total = bs[0] + bs[1]                                           # what the all-reduce returns
        for r in range(ranks):
            if detach:
                B.def_step_rows_apply_detach(ctxs[r], xs[r], total, W, zs[r], t, 8)
            else:
                B.def_step_rows_apply(ctxs[r], xs[r], total, W, t, 8)
        oracle.step(xo, gh, eo, mo, d=d, k=k, s=oracle.block_start(8, t, d), eta=lr, mu=mu)
        if detach:
            # the detach points follow from the GPU's own x_{t+1} (which differs from the oracle's in
            # the last bits: the ranks' sums were added in another order) and the oracle's errors
            xg = xs[0].cpu().numpy()
            zg = torch.cat(zs).cpu().numpy()
            for w in range(W):
                assert np.array_equal(zg[w], oracle.detach(xg, np.ascontiguousarray(eo[w]), lam)), (t, w)
    torch.cuda.synchronize()
    assert torch.equal(xs[0], xs[1]), "replicas diverged"
    got_e = torch.cat(es).cpu().numpy(); got_m = torch.cat(ms).cpu().numpy()
    assert np.array_equal(got_e, eo) and np.array_equal(got_m, mo)      # per-worker state: no cross-rank arithmetic
    err = np.max(np.abs(xs[0].cpu().numpy() - xo)) / np.max(np.abs(xo))
    assert err <= 1e-6, err                                             # only the order of the sum differs
    assert B.lib.def_step_rows_apply(ctxs[0].handle, xs[0].data_ptr(), total.data_ptr(), 2, 0, 8) == B.DEF_ERR_ARG
    for c in ctxs:
        B.def_destroy(c)


def test_rows_argument_checks(B):
    dev = torch.device("cuda", 0)
    d, W, k = 4096, 2, 100
    ctx = B.def_create(d, W, k, 0, 0.1, 0.9)
    x = torch.zeros(d, device=dev); g = torch.zeros(W, d, device=dev); e = torch.zeros(W, d, device=dev)
    m = torch.zeros(W, d, device=dev); z = torch.zeros(W, d, device=dev); b = torch.zeros(k, device=dev)
    f = B.lib.def_step_rows_local_detach
    assert f(ctx.handle, None, g.data_ptr(), e.data_ptr(), m.data_ptr(), b.data_ptr(), z.data_ptr(), 0, 0) == B.DEF_ERR_NULL
    assert f(ctx.handle, x.data_ptr(), g.data_ptr(), e.data_ptr(), m.data_ptr(), b.data_ptr(), None, 0, 0) == B.DEF_ERR_NULL
    assert f(ctx.handle, x.data_ptr(), g.data_ptr(), e.data_ptr(), m.data_ptr(), b.data_ptr(), e.data_ptr(), 0, 0) == B.DEF_ERR_ALIAS
    assert f(ctx.handle, e.data_ptr(), g.data_ptr(), e.data_ptr(), m.data_ptr(), b.data_ptr(), z.data_ptr(), 0, 0) == B.DEF_ERR_ALIAS
    fa = B.lib.def_step_rows_apply_detach
    assert fa(ctx.handle, x.data_ptr(), b.data_ptr(), W, None, 0, 0) == B.DEF_ERR_NULL
    assert fa(ctx.handle, x.data_ptr(), b.data_ptr(), W, x.data_ptr(), 0, 0) == B.DEF_ERR_ALIAS
    # the side stream must not be the context's own stream
    s = torch.cuda.Stream()
    B.def_set_stream(ctx, s)
    assert B.lib.def_set_rows_stream(ctx.handle, s.cuda_stream) == B.DEF_ERR_ARG
    B.def_set_stream(ctx, None)
    B.def_set_rows_stream(ctx, s)
    assert B.lib.def_set_stream(ctx.handle, s.cuda_stream) == B.DEF_ERR_ARG
    B.def_set_rows_stream(ctx, None)
    B.def_destroy(ctx)


def test_random_shapes_rows_halves_equal_def_step(B):
    """Seeded sweep: the two halves of the row-sharded step with all workers on one rank (no
    collective between them) against def_step / def_step_detach -- any d, k from 1 to d, both launch
    strategies, with and without momentum, the detach output and the side stream -- bit for bit,
    with nothing between the calls that waits for the GPU."""
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(20261201)
    side = torch.cuda.Stream()
    for case in range(150):
        d = int(rng.choice([rng.integers(1, 3000), rng.integers(3000, 300000)]))
        W = int(rng.choice([1, 2, 3, 5, 8]))
        k = int(rng.choice([1, d, max(1, d - 1), max(1, d // 2), int(rng.integers(1, d + 1))]))
        mom = float(rng.choice([0.0, 0.9])); detach = bool(rng.integers(0, 2)); use_side = bool(rng.integers(0, 2))
        pair = 0 if rng.random() < 0.8 else 1 << 60
        what = dict(case=case, d=d, W=W, k=k, mom=mom, detach=detach, side=use_side, pair=pair)
        ctx1 = B.def_create(d, W, k, 0, 0.1, mom, (0.4, 0.0)); ctx2 = B.def_create(d, W, k, 0, 0.1, mom, (0.4, 0.0))
        B.def_set_small_step_bytes(ctx1, pair); B.def_set_small_step_bytes(ctx2, pair)
        if use_side:
            B.def_set_rows_stream(ctx2, side)
        x1 = torch.randn(d, device=dev) * 0.05; x2 = x1.clone()
        e1 = torch.zeros(W, d, device=dev); e2 = torch.zeros(W, d, device=dev)
        m1 = torch.zeros(W, d, device=dev) if mom else None; m2 = torch.zeros(W, d, device=dev) if mom else None
        z1 = torch.full((W, d), -1.0, device=dev); z2 = torch.full((W, d), -2.0, device=dev)
        blk = torch.full((k,), 5.0, device=dev)
        gs = [torch.randn(W, d, device=dev) * 0.1 for _ in range(4)]
        torch.cuda.synchronize()
        for t, g in zip((int(v) for v in rng.integers(0, 10 ** 6, size=4)), gs):
            if detach:
                B.def_step_detach(ctx1, x1, g, e1, m1, z1, t, 3)
                B.def_step_rows_local_detach(ctx2, x2, g, e2, m2, blk, z2, t, 3)
                B.def_step_rows_apply_detach(ctx2, x2, blk, W, z2, t, 3)
            else:
                B.def_step(ctx1, x1, g, e1, m1, t, 3)
                B.def_step_rows_local(ctx2, g, e2, m2, blk, t, 3)
                B.def_step_rows_apply(ctx2, x2, blk, W, t, 3)
        torch.cuda.synchronize()
        assert torch.equal(x1, x2) and torch.equal(e1, e2), what
        assert not mom or torch.equal(m1, m2), what
        assert not detach or torch.equal(z1, z2), what
        if use_side:
            B.def_set_rows_stream(ctx2, None)
        B.def_destroy(ctx1); B.def_destroy(ctx2)
