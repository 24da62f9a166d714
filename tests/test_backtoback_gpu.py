"""Steps enqueued back to back with nothing between them that waits for the GPU.

A step on 16-byte aligned tensors is a pair of kernels that may run side by side: the kernel of
the tiles that touch the block, and the stream kernel of all the others, which is allowed to
start before the first has finished.  The next step (Algorithm 1's update feeding the next
iteration's error-feedback step) is ordered behind the stream kernel only, so the stream kernel
must not complete before the block kernel has.  The cases below make the block kernel carry all
or most of the work (k = d, k = d - 1, k about d / 2, many workers) while the stream kernel has
little or none, run 24 steps without any host synchronisation or copy in between, and only then
read the state and the returned model: bit for bit the oracle's."""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    from paper_2004_05298_b200 import binding
    return binding


CASES = [
    # d, W, k
    (1_048_576, 8, 1_048_576),        # k = d: the stream kernel has nothing to do
    (1_048_576, 8, 1_048_575),        # k = d - 1: one tile is shared by both ends of the block
    (1_000_000, 8, 500_123),          # half and half
    (262_144, 64, 262_144),           # many workers: the longest block kernel per coordinate
    (1_000_002, 8, 1_000_002),        # d % 4 = 2: block-columns kernel and flat stream
    (1_000_003, 5, 999_000),
]


@pytest.mark.parametrize("d,W,k", CASES)
@pytest.mark.parametrize("momentum", [0.9, 0.0])
def test_pair_back_to_back_without_host_sync(B, d, W, k, momentum):
    dev = torch.device("cuda")
    steps, seed, lr = 24, 17, 0.1
    rng = np.random.default_rng(d + W + k)
    n_g = 4                                               # a few gradient buffers, reused in turn
    ghs = [(0.1 * rng.standard_normal((W, d))).astype(np.float32) for _ in range(n_g)]
    gs = [torch.from_numpy(g).to(dev) for g in ghs]
    x = torch.from_numpy((0.05 * rng.standard_normal(d)).astype(np.float32)).to(dev)
    e = torch.zeros(W, d, device=dev)
    m = torch.zeros(W, d, device=dev) if momentum else None
    y = torch.empty(d, device=dev)
    xo = x.cpu().numpy().copy(); eo = np.zeros((W, d), np.float32)
    mo = np.zeros((W, d), np.float32) if momentum else None
    ctx = B.def_create(d, W, k, B.DEF_VARIANT_DEF, lr, momentum)
    B.def_set_small_step_bytes(ctx, 0)                    # always the pair
    B.def_step(ctx, x, gs[0], e, m, 10_000, seed)         # first call (device query) and warm-up
    torch.cuda.synchronize()
    oracle.step(xo, ghs[0], eo, mo, d=d, k=k, s=oracle.block_start(seed, 10_000, d), eta=lr, mu=momentum)
    launches = B.def_launch_count(ctx)
    for t in range(steps):                                # nothing here waits for the GPU
        B.def_step(ctx, x, gs[t % n_g], e, m, t, seed)
    B.def_output(ctx, x, e, y)
    assert B.def_launch_count(ctx) - launches == 2 * steps + 1
    torch.cuda.synchronize()
    for t in range(steps):
        oracle.step(xo, ghs[t % n_g], eo, mo, d=d, k=k, s=oracle.block_start(seed, t, d), eta=lr, mu=momentum)
    assert np.array_equal(x.cpu().numpy(), xo), "params"
    assert np.array_equal(e.cpu().numpy(), eo), "errors"
    if momentum:
        assert np.array_equal(m.cpu().numpy(), mo), "mom"
    assert np.array_equal(y.cpu().numpy(), oracle.output(oracle.VARIANT_DEF, xo, eo)), "returned model"
    B.def_destroy(ctx)


def test_pair_back_to_back_with_detach_output(B):
    """The same with the fused detach output: z of the last step against the oracle's detach points."""
    dev = torch.device("cuda")
    d, W, k, steps, seed, lr, mu, lam = 1_048_576, 8, 1_048_000, 12, 4, 0.1, 0.9, 0.3
    rng = np.random.default_rng(99)
    ghs = [(0.1 * rng.standard_normal((W, d))).astype(np.float32) for _ in range(3)]
    gs = [torch.from_numpy(g).to(dev) for g in ghs]
    x = torch.from_numpy((0.05 * rng.standard_normal(d)).astype(np.float32)).to(dev)
    e = torch.zeros(W, d, device=dev); m = torch.zeros(W, d, device=dev); z = torch.zeros(W, d, device=dev)
    xo = x.cpu().numpy().copy(); eo = np.zeros((W, d), np.float32); mo = np.zeros((W, d), np.float32)
    ctx = B.def_create(d, W, k, B.DEF_VARIANT_DEF, lr, mu, (lam, 0.0))
    B.def_set_small_step_bytes(ctx, 0)
    B.def_step_detach(ctx, x, gs[0], e, m, z, 777, seed)
    torch.cuda.synchronize()
    oracle.step(xo, ghs[0], eo, mo, d=d, k=k, s=oracle.block_start(seed, 777, d), eta=lr, mu=mu)
    for t in range(steps):
        B.def_step_detach(ctx, x, gs[t % 3], e, m, z, t, seed)
    torch.cuda.synchronize()
    for t in range(steps):
        oracle.step(xo, ghs[t % 3], eo, mo, d=d, k=k, s=oracle.block_start(seed, t, d), eta=lr, mu=mu)
    assert np.array_equal(x.cpu().numpy(), xo) and np.array_equal(e.cpu().numpy(), eo) and np.array_equal(m.cpu().numpy(), mo)
    zh = z.cpu().numpy()
    for w in range(W):
        assert np.array_equal(zh[w], oracle.detach(xo, np.ascontiguousarray(eo[w]), lam)), w
    B.def_destroy(ctx)


@pytest.mark.parametrize("mode", ["never", "always"])
def test_pair_overlap_modes_give_the_same_bits(B, mode):
    """The second kernel of the pair started beside the first, or strictly after it: same results."""
    dev = torch.device("cuda")
    d, W, k, seed, lr, mu = 700_000, 6, 200_000, 9, 0.1, 0.9
    rng = np.random.default_rng(17)
    gh = (0.1 * rng.standard_normal((W, d))).astype(np.float32)
    g = torch.from_numpy(gh).to(dev)
    x = torch.from_numpy((0.05 * rng.standard_normal(d)).astype(np.float32)).to(dev)
    e = torch.zeros(W, d, device=dev); m = torch.zeros(W, d, device=dev)
    xo = x.cpu().numpy().copy(); eo = np.zeros((W, d), np.float32); mo = np.zeros((W, d), np.float32)
    ctx = B.def_create(d, W, k, B.DEF_VARIANT_DEF, lr, mu)
    B.def_set_small_step_bytes(ctx, 0)
    B.def_set_pair_overlap(ctx, B.DEF_OVERLAP_NEVER if mode == "never" else B.DEF_OVERLAP_ALWAYS)
    for t in range(8):
        B.def_step(ctx, x, g, e, m, t, seed)
    torch.cuda.synchronize()
    for t in range(8):
        oracle.step(xo, gh, eo, mo, d=d, k=k, s=oracle.block_start(seed, t, d), eta=lr, mu=mu)
    assert np.array_equal(x.cpu().numpy(), xo) and np.array_equal(e.cpu().numpy(), eo) and np.array_equal(m.cpu().numpy(), mo)
    assert B.lib.def_set_pair_overlap(ctx.handle, 7) == B.DEF_ERR_ARG
    B.def_destroy(ctx)
