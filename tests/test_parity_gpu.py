"""GPU parity: the CUDA library, called through its C boundary, against the CPU oracle
on the same seeded inputs.

Bars: block starts and masks bit-exact; params, errors and momentum within a maximum
relative error of 1e-5 of the fp32 oracle (zeros must be zeros) after the workload's
steps -- the library performs the same roundings in the same order as the oracle, so
the difference is expected to be exactly 0 and the tests also report whether it is --
and within 1e-5 of the tensor's scale of the fp64 shadow.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2004_05298_b200 import workloads as WL

pytestmark = pytest.mark.gpu

REL_TOL = 1e-5          # maximum element-wise relative error vs the fp32 oracle
SHADOW_TOL = 1e-5       # maximum error vs the fp64 shadow, relative to the tensor's scale


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device (run with -m 'not gpu' on a CPU box)")
    from paper_2004_05298_b200 import binding
    return binding


def compare(a, b, what, rel_tol=REL_TOL):
    """a: library result, b: fp32 oracle result (numpy float32 arrays of one shape)."""
    a = np.asarray(a); b = np.asarray(b)
    assert a.shape == b.shape, what
    if a.dtype == np.float32 and b.dtype == np.float32 and a.flags.c_contiguous and b.flags.c_contiguous \
            and np.array_equal(a.view(np.uint32), b.view(np.uint32)):
        return True                                    # the same bits: every bar below holds trivially
    both_nan = np.isnan(a) & np.isnan(b)
    a = np.where(both_nan, 0, a); b = np.where(both_nan, 0, b)
    assert np.array_equal(a == 0, b == 0), "%s: zero pattern differs" % what
    nz = b != 0
    if nz.any():
        with np.errstate(invalid="ignore", over="ignore"):
            rel = np.abs(a[nz].astype(np.float64) - b[nz].astype(np.float64)) / np.abs(b[nz].astype(np.float64))
        rel = np.where(a[nz] == b[nz], 0.0, rel)       # equal infinities
        m1 = float(np.max(rel))
        assert m1 <= rel_tol, "%s: max relative error %.3e > %.1e" % (what, m1, rel_tol)
    return bool(np.array_equal(a, b))


def compare_shadow(a, b64, what, tol=SHADOW_TOL):
    scale = float(np.max(np.abs(b64)))
    if scale == 0.0:
        assert not np.any(a), what
        return
    err = float(np.max(np.abs(a.astype(np.float64) - b64)))
    assert err <= tol * scale, "%s: %.3e of scale vs the fp64 shadow" % (what, err / scale)


def guarded(shape, device, fill=-12345.0, guard=64, offset=0):
    """A tensor of `shape` inside a larger sentinel-filled buffer; `offset` floats shift its
    start off the buffer's 16-byte grid.  Returns (view, check) where check() asserts that
    nothing outside the view was written."""
    n = int(np.prod(shape))
    buf = torch.full((n + 2 * guard + 8,), fill, dtype=torch.float32, device=device)
    start = guard + offset
    view = buf[start:start + n].view(*shape)

    def check():
        assert bool((buf[:start] == fill).all()) and bool((buf[start + n:] == fill).all()), \
            "a write landed outside the tensor"
    return view, check


def find_steps(d, k, seed, want):
    """Steps whose block start satisfies want(s), by scanning the oracle's sampler."""
    out = []
    t = 0
    while len(out) < 2 and t < 200000:
        if want(oracle.block_start(seed, t, d)):
            out.append(t)
        t += 1
    return out


# ---------------------------------------------------------------------------
# a1: the sampler, bit for bit
# ---------------------------------------------------------------------------
def test_block_start_device_matches_oracle(B):
    n = 1 << 20
    rng = np.random.default_rng(2024)
    seeds = rng.integers(0, 2 ** 64, size=n, dtype=np.uint64)
    steps = rng.integers(0, 2 ** 64, size=n, dtype=np.uint64)
    seeds[: n // 2] %= 8                      # the small seeds and steps real runs use
    steps[: n // 2] %= 100000
    choices = np.array([1, 2, 3, 855770, 1000000, 11689512, 25557032, 138357544, 2 ** 40 + 7, 2 ** 62],
                       dtype=np.int64)
    ds = choices[rng.integers(0, len(choices), size=n)]
    dev = torch.device("cuda")
    out = torch.empty(n, dtype=torch.int64, device=dev)
    B.def_block_start_device(torch.from_numpy(seeds.view(np.int64)).to(dev),
                             torch.from_numpy(steps.view(np.int64)).to(dev),
                             torch.from_numpy(ds).to(dev), out)
    got = out.cpu().numpy()
    f = oracle.default().lib.def_oracle_block_start
    want = np.fromiter((f(int(a), int(b), int(c)) for a, b, c in zip(seeds, steps, ds)), dtype=np.int64, count=n)
    assert np.array_equal(got, want)


# ---------------------------------------------------------------------------
# whole-tensor parity on shapes chosen to hit every code path
# ---------------------------------------------------------------------------
def run_whole(B, d, W, k, steps, momentum, seed, lr=0.1, offsets=(0, 0, 0, 0), sigma=0.1,
              variant=0, special=None, pair=True):
    dev = torch.device("cuda")
    rng = np.random.default_rng(d * 31 + W * 7 + k)
    x, cx = guarded((d,), dev, offset=offsets[0])
    g, cg = guarded((W, d), dev, offset=offsets[1])
    e, ce = guarded((W, d), dev, offset=offsets[2])
    x.copy_(torch.from_numpy((0.05 * rng.standard_normal(d)).astype(np.float32)))
    e.zero_()
    m = cm = None
    if momentum:
        m, cm = guarded((W, d), dev, offset=offsets[3])
        m.zero_()
    xo = x.cpu().numpy().copy(); eo = np.zeros((W, d), np.float32)
    mo = np.zeros((W, d), np.float32) if momentum else None
    x64 = xo.astype(np.float64); e64 = eo.astype(np.float64)
    m64 = mo.astype(np.float64) if momentum else None
    ctx = B.def_create(d, W, k, variant, lr, momentum)
    B.def_set_small_step_bytes(ctx, 0 if pair else 1 << 60)   # the kernel pair, or one launch of the general kernel
    exact = True
    for t in steps:
        gh = (sigma * rng.standard_normal((W, d))).astype(np.float32)
        if special is not None:
            special(gh, t)
        g.copy_(torch.from_numpy(gh))
        B.def_step(ctx, x, g, e, m, t, seed)
        s = oracle.block_start(seed, t, d)
        assert B.def_block_start(ctx, t, seed) == s
        oracle.step(xo, gh, eo, mo, d=d, k=k, s=s, eta=lr, mu=momentum)
        oracle.step(x64, gh.astype(np.float64), e64, m64, d=d, k=k, s=s, eta=lr, mu=momentum)
        # the mask, bit-exact: e' is +0 on the block, and nowhere the oracle's is not
        mask = oracle.block_mask(d, k, s)
        eg = e.cpu().numpy()
        if special is None:
            assert not eg[:, mask].any() and not np.signbit(eg[:, mask]).any(), "block not zeroed at step %d" % t
            assert np.array_equal(eg == 0, eo == 0), "zero pattern of the new error differs at step %d" % t
            assert np.count_nonzero(eg[:, ~mask] == 0) <= 2, "coordinates outside the block were zeroed"
        assert np.array_equal(g.cpu().numpy(), gh, equal_nan=True), "grads must not be written"
    torch.cuda.synchronize()
    for chk in (cx, cg, ce, cm):
        if chk:
            chk()
    exact &= compare(x.cpu().numpy(), xo, "params")
    exact &= compare(e.cpu().numpy(), eo, "errors")
    if momentum:
        exact &= compare(m.cpu().numpy(), mo, "mom")
    if special is None:
        compare_shadow(x.cpu().numpy(), x64, "params")
        compare_shadow(e.cpu().numpy(), e64, "errors")
        if momentum:
            compare_shadow(m.cpu().numpy(), m64, "mom")
    B.def_destroy(ctx)
    return exact


SHAPES = [
    # d, W, k
    (1, 1, 1), (2, 3, 1), (5, 3, 2), (8, 2, 3), (1023, 3, 1), (1024, 4, 1024), (1025, 5, 1024),
    (4099, 7, 100), (4100, 16, 4099), (100003, 9, 3125), (65536, 64, 777), (300000, 13, 150000),
]


@pytest.mark.parametrize("d,W,k", SHAPES)
@pytest.mark.parametrize("momentum", [0.9, 0.0])
@pytest.mark.parametrize("pair", [True, False], ids=["pair", "general"])
def test_small_shapes(B, d, W, k, momentum, pair):
    seed = 11
    wrap = find_steps(d, k, seed, lambda s: s + k > d)          # block wraps past the end
    tail = find_steps(d, k, seed, lambda s: s >= d - 1)          # starts on the last coordinate
    steps = sorted(set([0, 1, 2, 3] + wrap + tail))
    exact = run_whole(B, d, W, k, steps, momentum, seed, pair=pair)
    assert exact, "expected bit-identical results (same roundings in the same order)"


@pytest.mark.parametrize("offsets", [(0, 0, 0, 0), (1, 0, 0, 0), (0, 2, 2, 2), (0, 1, 2, 3), (2, 2, 2, 2), (3, 1, 0, 0)])
@pytest.mark.parametrize("d", [4096, 4098, 4099])
def test_alignment_classes(B, d, offsets):
    """16-, 8- and 4-byte aligned bases with d % 4 in {0, 2, 3}: every access width."""
    assert run_whole(B, d, 5, 333, [0, 1, 2, 5], 0.9, 3, offsets=offsets)


def test_ieee_specials_propagate(B):
    def special(gh, t):
        if t == 0:
            gh[0, 3] = np.inf; gh[1, 5] = np.nan; gh[0, 7] = -np.inf; gh[1, 7] = np.inf
            gh[0, 11] = -0.0; gh[1, 11] = -0.0
    d, W, k = 64, 2, 64                                            # k = d: every coordinate is sent
    run_whole(B, d, W, k, [0, 1], 0.9, 1, special=special)
    run_whole(B, d, W, 8, [0, 1, 2], 0.0, 1, special=special)


# ---------------------------------------------------------------------------
# the workloads at full size
# ---------------------------------------------------------------------------
def run_workload_whole(B, wl, steps):
    dev = torch.device("cuda")
    x = WL.initial_params(wl, dev)
    e, m = WL.zeros_state(wl, dev)
    col_sigma = WL.column_sigma(wl, dev) if wl.grad == "per_tensor" else None
    xo = x.cpu().numpy().copy()
    eo = np.zeros((wl.W, wl.d), np.float32); mo = np.zeros((wl.W, wl.d), np.float32)
    x64 = xo.astype(np.float64); e64 = eo.astype(np.float64); m64 = mo.astype(np.float64)
    ctx = B.def_create(wl.d, wl.W, wl.k, wl.variant, wl.lr, wl.momentum, (wl.lam, 0.0))
    g = torch.empty(wl.W, wl.d, dtype=torch.float32, device=dev)
    after10 = None
    for t in range(steps):
        WL.gradients(wl, t, dev, out=g, col_sigma=col_sigma)
        B.def_step(ctx, x, g, e, m, t, wl.rbgs_seed)
        gh = g.cpu().numpy()
        s = oracle.block_start(wl.rbgs_seed, t, wl.d)
        oracle.step(xo, gh, eo, mo, d=wl.d, k=wl.k, s=s, eta=wl.lr, mu=wl.momentum)
        oracle.step(x64, gh.astype(np.float64), e64, m64, d=wl.d, k=wl.k, s=s, eta=wl.lr, mu=wl.momentum)
        zeros = (e == 0).sum(dim=1)          # k per worker, plus the rare p that is exactly 0
        assert bool((zeros >= wl.k).all()) and int(zeros.sum()) - wl.W * wl.k <= 8 + wl.W * wl.d // 10 ** 6
        assert np.array_equal(e.cpu().numpy() == 0, eo == 0), "zero pattern of the new error differs"
        if t + 1 == 10 or t + 1 == steps:
            exact = compare(x.cpu().numpy(), xo, "params after %d steps" % (t + 1))
            exact &= compare(e.cpu().numpy(), eo, "errors after %d steps" % (t + 1))
            exact &= compare(m.cpu().numpy(), mo, "mom after %d steps" % (t + 1))
            compare_shadow(x.cpu().numpy(), x64, "params")
            compare_shadow(e.cpu().numpy(), e64, "errors")
            compare_shadow(m.cpu().numpy(), m64, "mom")
            after10 = exact if after10 is None else (after10 and exact)
    assert B.def_launch_count(ctx) >= steps
    B.def_destroy(ctx)
    return after10


def test_config1_whole(B):
    wl = WL.get(1)
    assert run_workload_whole(B, wl, wl.steps)


def test_config2_whole(B):
    wl = WL.get(2)                                   # d % 4 == 2: 8-byte aligned rows
    assert run_workload_whole(B, wl, wl.steps)


def host_memory_available():
    try:
        with open("/proc/meminfo") as fh:
            for line in fh:
                if line.startswith("MemAvailable:"):
                    return int(line.split()[1]) * 1024
    except OSError:
        pass
    return None


def run_workload_every_element(B, wl, steps, check_at, detach=False):
    """Full-size run in the launch configuration the benchmark times, with the fp32 oracle stepping
    the WHOLE tensors beside it (its all-cores build: the same source and the same bits as the
    plain build, see test_oracle_parallel.py; no fp64 shadow at this size).  After the steps in
    check_at, params, errors and mom are compared on every element: the stated bar (relative
    error <= 1e-5, equal zero patterns) and bit-identity."""
    dev = torch.device("cuda")
    o = oracle.all_cores()
    x = WL.initial_params(wl, dev)
    e, m = WL.zeros_state(wl, dev)
    col_sigma = WL.column_sigma(wl, dev) if wl.grad == "per_tensor" else None
    xo = x.cpu().numpy().copy()
    eo = np.zeros((wl.W, wl.d), np.float32); mo = np.zeros((wl.W, wl.d), np.float32)
    ctx = B.def_create(wl.d, wl.W, wl.k, wl.variant, wl.lr, wl.momentum, (wl.lam, 0.0))
    g = torch.empty(wl.W, wl.d, dtype=torch.float32, device=dev)
    g_host = torch.empty(wl.W, wl.d, dtype=torch.float32).pin_memory()
    back = torch.empty(wl.W, wl.d, dtype=torch.float32).pin_memory()
    exact = True
    z = torch.empty(wl.W, wl.d, dtype=torch.float32, device=dev) if detach else None
    for t in range(steps):
        WL.gradients(wl, t, dev, out=g, col_sigma=col_sigma)
        if detach:
            B.def_step_detach(ctx, x, g, e, m, z, t, wl.rbgs_seed)
        else:
            B.def_step(ctx, x, g, e, m, t, wl.rbgs_seed)
        g_host.copy_(g)
        s = o.block_start(wl.rbgs_seed, t, wl.d)
        assert B.def_block_start(ctx, t, wl.rbgs_seed) == s
        o.step(xo, g_host.numpy(), eo, mo, d=wl.d, k=wl.k, s=s, eta=wl.lr, mu=wl.momentum)
        if t + 1 in check_at:
            exact &= compare(x.cpu().numpy(), xo, "params after %d steps" % (t + 1))
            for dev_t, host_t, name in ((e, eo, "errors"), (m, mo, "mom")):
                back.copy_(dev_t)
                exact &= compare(back.numpy(), host_t, "%s after %d steps" % (name, t + 1))
            if detach:                                    # every worker's next detach point, every coordinate
                back.copy_(z)
                zh = back.numpy()
                for w in range(wl.W):
                    assert np.array_equal(zh[w], o.detach(xo, eo[w], wl.lam)), "detach point of worker %d" % w
    assert B.def_launch_count(ctx) == 2 * steps, "the kernel pair the benchmark times"
    B.def_destroy(ctx)
    del g, e, m, x, z, g_host, back
    torch.cuda.empty_cache()
    return exact


@pytest.mark.parametrize("cfg", [3, 4])
def test_config_full_size_every_element(B, cfg):
    """Configs 3 and 4 whole, all their steps, every element of every tensor."""
    wl = WL.get(cfg)
    assert run_workload_every_element(B, wl, wl.steps, {10, wl.steps})


def _config5_needs_host_memory():
    need = 80 << 30
    avail = host_memory_available()
    if avail is not None and avail < need:
        pytest.skip("host has %.0f GB available; a whole-tensor run of config 5 needs about 60 GB "
                    "(the sampled tests cover this configuration)" % (avail / 2 ** 30))


@pytest.mark.parametrize("ratio", [32, 8, 1000])
def test_config5_full_size_every_element(B, ratio):
    """Config 5 whole for its 10 steps at the default ratio and at both ends of its sweep: 2.2e9
    elements per tensor.  The oracle's state, its temporaries and the pinned staging buffers need
    about 60 GB of host memory."""
    _config5_needs_host_memory()
    wl = WL.get(5).with_ratio(ratio)
    assert run_workload_every_element(B, wl, wl.steps, {wl.steps})


def test_config5_detach_output_every_element(B):
    """Config 5 with the fused detach output, 3 steps: z of every worker on every coordinate."""
    _config5_needs_host_memory()
    assert run_workload_every_element(B, WL.get(5), 3, {3}, detach=True)


def sample_columns(wl, steps, n_random=20000, halo=48):
    """Coordinates the oracle follows on a full-size run: random ones, both ends of the
    vector, and a halo around both ends of every step's block (where a wrong mask shows)."""
    rng = np.random.default_rng(wl.cfg * 17 + wl.ratio)
    cols = set(int(v) for v in rng.integers(0, wl.d, size=n_random))
    cols.update(range(0, halo)); cols.update(range(wl.d - halo, wl.d))
    for t in range(steps):
        s = oracle.block_start(wl.rbgs_seed, t, wl.d)
        for edge in (s, s + wl.k):
            for j in range(edge - halo, edge + halo):
                cols.add(j % wl.d)
    return np.array(sorted(cols), dtype=np.int64)


def run_workload_sampled(B, wl, steps):
    """Full-size run in the launch configuration the benchmark times; the oracle follows a
    sample of coordinates (a column view), and whole-tensor properties are checked on the GPU."""
    dev = torch.device("cuda")
    cols = sample_columns(wl, steps)
    cols_dev = torch.from_numpy(cols).to(dev)
    x = WL.initial_params(wl, dev)
    x0 = x.clone()
    e, m = WL.zeros_state(wl, dev)
    col_sigma = WL.column_sigma(wl, dev) if wl.grad == "per_tensor" else None
    xo = x[cols_dev].cpu().numpy().copy()
    n = len(cols)
    eo = np.zeros((wl.W, n), np.float32); mo = np.zeros((wl.W, n), np.float32)
    x64 = xo.astype(np.float64); e64 = eo.astype(np.float64); m64 = mo.astype(np.float64)
    ctx = B.def_create(wl.d, wl.W, wl.k, wl.variant, wl.lr, wl.momentum, (wl.lam, 0.0))
    g = torch.empty(wl.W, wl.d, dtype=torch.float32, device=dev)
    touched = torch.zeros(wl.d, dtype=torch.bool, device=dev)
    y_expected = x0.double()                          # Eq. 8: y_{t+1} = y_t - eta * mean_k m_{k,t+1}
    M = torch.zeros(wl.W, wl.d, dtype=torch.float32, device=dev)
    exact = True
    for t in range(steps):
        WL.gradients(wl, t, dev, out=g, col_sigma=col_sigma)
        B.def_step(ctx, x, g, e, m, t, wl.rbgs_seed)
        s = oracle.block_start(wl.rbgs_seed, t, wl.d)
        assert B.def_block_start(ctx, t, wl.rbgs_seed) == s
        gh = np.ascontiguousarray(g[:, cols_dev].cpu().numpy())
        oracle.step(xo, gh, eo, mo, d=wl.d, k=wl.k, s=s, eta=wl.lr, mu=wl.momentum, cols=cols)
        oracle.step(x64, gh.astype(np.float64), e64, m64, d=wl.d, k=wl.k, s=s, eta=wl.lr, mu=wl.momentum, cols=cols)
        # whole-tensor properties that hold at any size
        expect = torch.zeros(wl.d, dtype=torch.bool, device=dev)        # the k coordinates from s
        expect[s:min(s + wl.k, wl.d)] = True
        if s + wl.k > wl.d:
            expect[: s + wl.k - wl.d] = True
        assert int(expect.sum()) == wl.k
        touched |= expect
        is_zero = (e == 0)
        assert bool(is_zero[:, expect].all()), "a block coordinate kept a non-zero error"
        # outside the block e' = p, which is exactly 0 only where a drawn gradient is (a few in 1e8)
        stray = int(is_zero.sum()) - wl.W * wl.k
        assert 0 <= stray <= 8 + wl.W * wl.d // 10 ** 6, "coordinates outside the block were zeroed: %d" % stray
        del is_zero
        M.mul_(wl.momentum).add_(g)
        y_expected -= wl.lr * (M.sum(dim=0, dtype=torch.float64) / wl.W)
        if t + 1 == 10 or t + 1 == steps:
            exact &= compare(x[cols_dev].cpu().numpy(), xo, "params after %d steps" % (t + 1))
            exact &= compare(e[:, cols_dev].cpu().numpy(), eo, "errors after %d steps" % (t + 1))
            exact &= compare(m[:, cols_dev].cpu().numpy(), mo, "mom after %d steps" % (t + 1))
            compare_shadow(x[cols_dev].cpu().numpy(), x64, "params")
            compare_shadow(e[:, cols_dev].cpu().numpy(), e64, "errors")
            compare_shadow(m[:, cols_dev].cpu().numpy(), m64, "mom")
    assert bool((x[~touched] == x0[~touched]).all()), "params moved outside every block"
    y = x.double() - e.sum(dim=0, dtype=torch.float64) / wl.W
    scale = float(y_expected.abs().max())
    assert float((y - y_expected).abs().max()) <= 2e-5 * scale, "Eq. 8 identity at full size"
    B.def_destroy(ctx)
    del g, e, m, M, x, touched
    torch.cuda.empty_cache()
    return exact


@pytest.mark.parametrize("cfg", [3, 4])
def test_config_full_size_sampled(B, cfg):
    wl = WL.get(cfg)
    assert run_workload_sampled(B, wl, wl.steps)


@pytest.mark.parametrize("ratio", WL.CFG5_RATIOS)
@pytest.mark.parametrize("variant", WL.CFG5_VARIANTS)
def test_config5_full_size_sampled(B, ratio, variant):
    wl = WL.get(5).with_ratio(ratio, variant)
    assert run_workload_sampled(B, wl, wl.steps)


# ---------------------------------------------------------------------------
# column ranges, host memory, streams, resume
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("ratio", [32, 2], ids=["k=d/32", "k=d/2"])
@pytest.mark.parametrize("pair", [True, False], ids=["pair", "general"])
def test_step_columns_equals_whole_step(B, pair, ratio):
    """Column ranges of the model stepped separately (aligned and unaligned cuts, padded rows) against
    the whole step, on steps whose block lies inside a range, straddles cuts, and wraps past d: every
    range has to find its own share of the block's tiles."""
    dev = torch.device("cuda")
    wl = WL.get(2).scaled(200_001, W=6).with_ratio(ratio)
    d, W, k = wl.d, wl.W, wl.k
    x = WL.initial_params(wl, dev); e, m = WL.zeros_state(wl, dev)
    cuts = [0, 4, 70_000, 70_003, 150_002, d]                     # aligned and unaligned pieces
    xs = [x[a:b].clone() for a, b in zip(cuts[:-1], cuts[1:])]
    ctx = B.def_create(d, W, k, wl.variant, wl.lr, wl.momentum)
    B.def_set_small_step_bytes(ctx, 0 if pair else 1 << 60)
    es = [torch.zeros(W, b - a + 5, device=dev) for a, b in zip(cuts[:-1], cuts[1:])]   # ld = n + 5
    ms = [torch.zeros(W, b - a + 5, device=dev) for a, b in zip(cuts[:-1], cuts[1:])]
    steps = sorted(set(list(range(5)) + find_steps(d, k, 9, lambda s: s + k > d) + find_steps(d, k, 9, lambda s: s < 70_000 < s + k)))
    for t in steps:
        g = WL.gradients(wl, t, dev)
        B.def_step(ctx, x, g, e, m, t, 9)
        for i, (a, b) in enumerate(zip(cuts[:-1], cuts[1:])):
            gl = torch.zeros(W, b - a + 5, device=dev)
            gl[:, : b - a] = g[:, a:b]
            B.def_step_columns(ctx, a, b - a, b - a + 5, xs[i], gl, es[i], ms[i], t, 9)
    for i, (a, b) in enumerate(zip(cuts[:-1], cuts[1:])):
        assert torch.equal(xs[i], x[a:b])
        assert torch.equal(es[i][:, : b - a], e[:, a:b]) and torch.equal(ms[i][:, : b - a], m[:, a:b])
        assert not es[i][:, b - a:].any() and not ms[i][:, b - a:].any(), "padding columns were written"
    B.def_destroy(ctx)


@pytest.mark.parametrize("ratio", [32, 3, 1], ids=["k=d/32", "k=d/3", "k=d"])
def test_column_shards_on_the_kernel_pair(B, ratio):
    """Column shards with 16-byte aligned rows run the kernel pair, each kernel with a grid for its
    own tiles of the shard only: shards that hold all, part or none of the block (one run or both,
    the block wrapping past d into the first shard) against the oracle on every element."""
    dev = torch.device("cuda")
    d, W, seed, lr, mu = 600_000, 5, 21, 0.1, 0.9
    k = max(1, d // ratio)
    cuts = [0, 1024, 100_004, 100_008, 333_336, 599_996, d]      # multiples of 4: every shard keeps 16-byte rows
    rng = np.random.default_rng(ratio)
    x0 = (0.05 * rng.standard_normal(d)).astype(np.float32)
    xo = x0.copy(); eo = np.zeros((W, d), np.float32); mo = np.zeros((W, d), np.float32)
    ctx = B.def_create(d, W, k, 0, lr, mu)
    B.def_set_small_step_bytes(ctx, 0)
    B.def_set_kernel_timing(ctx, True)
    shards = []
    for a, b in zip(cuts[:-1], cuts[1:]):
        n = b - a
        shards.append((a, n, torch.from_numpy(x0[a:b].copy()).to(dev), torch.zeros(W, n, device=dev), torch.zeros(W, n, device=dev)))
    steps = sorted(set([0, 1, 2] + find_steps(d, k, seed, lambda s: s + k > d) + find_steps(d, k, seed, lambda s: s < 100_006 < s + k)))
    for t in steps:
        gh = (0.1 * rng.standard_normal((W, d))).astype(np.float32)
        oracle.step(xo, gh, eo, mo, d=d, k=k, s=oracle.block_start(seed, t, d), eta=lr, mu=mu)
        for a, n, xs, es, ms in shards:
            g = torch.from_numpy(np.ascontiguousarray(gh[:, a:a + n])).to(dev)
            plan = B.def_tile_plan(ctx, a, n, t, seed)
            assert plan[1] + plan[2] + plan[3] == -(-n // 1024)
            B.def_step_columns(ctx, a, n, n, xs, g, es, ms, t, seed)
    assert B.def_kernel_time(ctx, B.DEF_KERNEL_GENERAL)[1] == 0
    assert B.def_kernel_time(ctx, B.DEF_KERNEL_STREAM)[1] == len(steps) * len(shards)
    for a, n, xs, es, ms in shards:
        assert np.array_equal(xs.cpu().numpy(), xo[a:a + n]), a
        assert np.array_equal(es.cpu().numpy(), eo[:, a:a + n]) and np.array_equal(ms.cpu().numpy(), mo[:, a:a + n]), a
    B.def_destroy(ctx)


@pytest.mark.parametrize("pair", [False, True], ids=["general", "pair"])
@pytest.mark.parametrize("momentum", [0.9, 0.0])
def test_step_host_matches_oracle(B, momentum, pair):
    """Every tensor in host memory, streamed through the staging slots in column pieces; with `pair`
    every piece runs the kernel pair on its column range (as the pieces of a large model do)."""
    wl = WL.get(1).scaled(3_000_001, W=5, momentum=momentum)      # odd d: unaligned host rows
    d, W, k = wl.d, wl.W, wl.k
    x = WL.initial_params(wl, "cpu").pin_memory()
    e = torch.zeros(W, d).pin_memory()
    m = torch.zeros(W, d).pin_memory() if momentum else None
    xo = x.numpy().copy(); eo = np.zeros((W, d), np.float32)
    mo = np.zeros((W, d), np.float32) if momentum else None
    ctx = B.def_create(d, W, k, wl.variant, wl.lr, momentum)
    if pair:
        B.def_set_small_step_bytes(ctx, 0)
    for t in range(3):
        g = WL.gradients(wl, t, "cpu").pin_memory()
        B.def_step_host(ctx, x, g, e, m, t, 4)
        oracle.step(xo, g.numpy(), eo, mo, d=d, k=k, s=oracle.block_start(4, t, d), eta=wl.lr, mu=momentum)
    assert compare(x.numpy(), xo, "params") and compare(e.numpy(), eo, "errors")
    if momentum:
        assert compare(m.numpy(), mo, "mom")
    B.def_destroy(ctx)


def test_stream_and_resume(B):
    dev = torch.device("cuda")
    wl = WL.get(1).scaled(500_000)
    ctx = B.def_create(wl.d, wl.W, wl.k, wl.variant, wl.lr, wl.momentum)
    side = torch.cuda.Stream()

    def run(step_list, state=None, stream=None):
        if state is None:
            x = WL.initial_params(wl, dev); e, m = WL.zeros_state(wl, dev)
        else:
            x, e, m = (t.clone() for t in state)
        B.def_set_stream(ctx, stream)
        for t in step_list:
            g = WL.gradients(wl, t, dev)
            if stream is not None:
                stream.wait_stream(torch.cuda.current_stream())
            B.def_step(ctx, x, g, e, m, t, 2)
            if stream is not None:
                torch.cuda.current_stream().wait_stream(stream)
        torch.cuda.synchronize()
        B.def_set_stream(ctx, None)
        return x, e, m

    straight = run(range(10))
    half = run(range(5), stream=side)
    resumed = run(range(5, 10), state=half)               # the sampler has no state to carry
    for a, b in zip(straight, resumed):
        assert torch.equal(a, b)
    B.def_destroy(ctx)


# ---------------------------------------------------------------------------
# the step with the fused detach output (Algorithm 1's detach step of the next iteration)
# ---------------------------------------------------------------------------
def run_detach(B, d, W, k, steps, momentum, lam, variant=0, offsets=(0, 0, 0, 0, 0), seed=7, pair=True):
    dev = torch.device("cuda")
    rng = np.random.default_rng(d + 13 * W + k)
    x, cx = guarded((d,), dev, offset=offsets[0])
    g, cg = guarded((W, d), dev, offset=offsets[1])
    e, ce = guarded((W, d), dev, offset=offsets[2])
    z, cz = guarded((W, d), dev, offset=offsets[4])
    x.copy_(torch.from_numpy((0.05 * rng.standard_normal(d)).astype(np.float32))); e.zero_(); z.fill_(-3.0)
    m = cm = None
    if momentum:
        m, cm = guarded((W, d), dev, offset=offsets[3]); m.zero_()
    xo = x.cpu().numpy().copy(); eo = np.zeros((W, d), np.float32)
    mo = np.zeros((W, d), np.float32) if momentum else None
    ctx = B.def_create(d, W, k, variant, 0.1, momentum, (lam, 0.0))
    B.def_set_small_step_bytes(ctx, 0 if pair else 1 << 60)
    lam_used = 0.0 if variant == B.DEF_VARIANT_EF else lam
    for t in steps:
        gh = (0.1 * rng.standard_normal((W, d))).astype(np.float32)
        g.copy_(torch.from_numpy(gh))
        B.def_step_detach(ctx, x, g, e, m, z, t, seed)
        oracle.step(xo, gh, eo, mo, d=d, k=k, s=oracle.block_start(seed, t, d), eta=0.1, mu=momentum)
        zh = z.cpu().numpy()
        for w in range(W):
            want = oracle.detach(xo, np.ascontiguousarray(eo[w]), lam_used)
            assert np.array_equal(zh[w], want), "detach point of worker %d differs at step %d" % (w, t)
    assert np.array_equal(x.cpu().numpy(), xo) and np.array_equal(e.cpu().numpy(), eo)
    if momentum:
        assert np.array_equal(m.cpu().numpy(), mo)
    for chk in (cx, cg, ce, cm, cz):
        if chk:
            chk()
    B.def_destroy(ctx)


@pytest.mark.parametrize("d,W,k", [(1, 1, 1), (8, 2, 3), (1025, 5, 1024), (4099, 7, 100), (65536, 64, 777),
                                   (300000, 13, 150000), (100003, 9, 3125), (2_000_000, 4, 62_500)])
@pytest.mark.parametrize("momentum", [0.9, 0.0])
@pytest.mark.parametrize("pair", [True, False], ids=["pair", "general"])
def test_step_detach_small_shapes(B, d, W, k, momentum, pair):
    wrap = find_steps(d, k, 7, lambda s: s + k > d)
    run_detach(B, d, W, k, sorted(set([0, 1, 2] + wrap)), momentum, 0.3, pair=pair)


@pytest.mark.parametrize("offsets", [(0, 0, 0, 0, 0), (0, 0, 0, 0, 1), (2, 2, 2, 2, 2), (0, 1, 2, 3, 0), (0, 0, 0, 0, 2)])
def test_step_detach_alignment_and_variants(B, offsets):
    for d in (4096, 4098, 4099):
        run_detach(B, d, 5, 333, [0, 1, 4], 0.9, 0.6, offsets=offsets)
    run_detach(B, 5000, 3, 100, [0, 1], 0.9, 0.6, variant=B.DEF_VARIANT_EF)         # lambda forced to 0: z = x
    run_detach(B, 5000, 3, 100, [0, 1], 0.9, 1.0, variant=B.DEF_VARIANT_DEF_A)


def test_step_detach_full_size_sampled(B):
    """Config 5 at full size: z on sampled coordinates against the oracle, and the step's own
    outputs identical to those of the plain step."""
    wl = WL.get(5)
    dev = torch.device("cuda")
    steps = 4
    cols = sample_columns(wl, steps)
    cols_dev = torch.from_numpy(cols).to(dev)
    x = WL.initial_params(wl, dev); e, m = WL.zeros_state(wl, dev)
    z = torch.empty(wl.W, wl.d, dtype=torch.float32, device=dev)
    xo = x[cols_dev].cpu().numpy().copy()
    n = len(cols)
    eo = np.zeros((wl.W, n), np.float32); mo = np.zeros((wl.W, n), np.float32)
    ctx = B.def_create(wl.d, wl.W, wl.k, wl.variant, wl.lr, wl.momentum, (wl.lam, 0.0))
    g = torch.empty(wl.W, wl.d, dtype=torch.float32, device=dev)
    for t in range(steps):
        WL.gradients(wl, t, dev, out=g)
        B.def_step_detach(ctx, x, g, e, m, z, t, wl.rbgs_seed)
        gh = np.ascontiguousarray(g[:, cols_dev].cpu().numpy())
        oracle.step(xo, gh, eo, mo, d=wl.d, k=wl.k, s=oracle.block_start(wl.rbgs_seed, t, wl.d), eta=wl.lr, mu=wl.momentum, cols=cols)
        zh = z[:, cols_dev].cpu().numpy()
        for w in range(wl.W):
            assert np.array_equal(zh[w], oracle.detach(xo, np.ascontiguousarray(eo[w]), wl.lam)), (t, w)
        # whole tensor: x - lambda e' in fp64, rounded to fp32.  That rounds twice where the kernel's
        # fused multiply-add rounds once, so a handful of elements in 2e9 may differ by one ulp.
        ref = (x.unsqueeze(0).double() - float(np.float32(wl.lam)) * e.double()).float()
        differ = ref != z
        assert int(differ.sum()) <= 256, "detach output differs in many places"
        assert float((ref - z).abs().max()) <= 2.0 ** -22 * float(x.abs().max())
        del differ
        del ref
    assert np.array_equal(x[cols_dev].cpu().numpy(), xo) and np.array_equal(e[:, cols_dev].cpu().numpy(), eo)
    B.def_destroy(ctx)


def test_padded_rows_keep_the_kernel_pair(B):
    """An odd d with rows padded to a multiple of 4 floats runs the 128-bit kernels (plus a
    one-float-wide launch for the last d % 4 coordinates) and still matches the oracle."""
    dev = torch.device("cuda")
    d, W, k = 300_003, 6, 20_000
    ld = (d + 3) // 4 * 4
    rng = np.random.default_rng(9)
    x = torch.from_numpy((0.05 * rng.standard_normal(d)).astype(np.float32)).to(dev)
    e = torch.zeros(W, ld, device=dev); m = torch.zeros(W, ld, device=dev)
    xo = x.cpu().numpy().copy(); eo = np.zeros((W, d), np.float32); mo = np.zeros((W, d), np.float32)
    ctx = B.def_create(d, W, k, 0, 0.1, 0.9)
    B.def_set_small_step_bytes(ctx, 0)
    B.def_set_kernel_timing(ctx, True)
    for t in range(4):
        gh = (0.1 * rng.standard_normal((W, d))).astype(np.float32)
        g = torch.zeros(W, ld, device=dev); g[:, :d] = torch.from_numpy(gh).to(dev)
        B.def_step_columns(ctx, 0, d, ld, x, g, e, m, t, 6)
        oracle.step(xo, gh, eo, mo, d=d, k=k, s=oracle.block_start(6, t, d), eta=0.1, mu=0.9)
    assert B.def_kernel_time(ctx, B.DEF_KERNEL_STREAM)[1] == 4 and B.def_kernel_time(ctx, B.DEF_KERNEL_BLOCK)[1] == 4
    assert B.def_kernel_time(ctx, B.DEF_KERNEL_GENERAL)[1] == 4          # the 3-coordinate tail
    assert np.array_equal(x.cpu().numpy(), xo)
    assert np.array_equal(e[:, :d].cpu().numpy(), eo) and np.array_equal(m[:, :d].cpu().numpy(), mo)
    assert not e[:, d:].any() and not m[:, d:].any()
    B.def_destroy(ctx)


def test_empty_ranges_are_no_ops(B):
    dev = torch.device("cuda")
    ctx = B.def_create(1000, 2, 10, 0, 0.1, 0.9)
    x = torch.ones(0, device=dev); t2 = torch.ones(2, 0, device=dev)
    before = B.def_launch_count(ctx)
    B.def_step_columns(ctx, 500, 0, 0, x, t2, t2.clone(), t2.clone(), 0, 0)
    B.def_step_columns(ctx, 1000, 0, 0, x, t2, t2.clone(), t2.clone(), 0, 0)
    assert B.def_launch_count(ctx) == before
    B.def_destroy(ctx)


@pytest.mark.parametrize("pair", [True, False], ids=["pair", "general"])
def test_step_replays_from_a_cuda_graph(B, pair):
    """def_step only enqueues kernels (no allocation, no synchronisation), so it can be recorded
    into a CUDA graph on the context's stream; replays redo the recorded (step, seed)."""
    dev = torch.device("cuda")
    d, W, k = 400_000, 4, 12_500
    rng = np.random.default_rng(21)
    x = torch.from_numpy((0.05 * rng.standard_normal(d)).astype(np.float32)).to(dev)
    gh = (0.1 * rng.standard_normal((W, d))).astype(np.float32)
    g = torch.from_numpy(gh).to(dev)
    e = torch.zeros(W, d, device=dev); m = torch.zeros(W, d, device=dev)
    xo = x.cpu().numpy().copy(); eo = np.zeros((W, d), np.float32); mo = np.zeros((W, d), np.float32)
    ctx = B.def_create(d, W, k, 0, 0.1, 0.9)
    B.def_set_small_step_bytes(ctx, 0 if pair else 1 << 60)
    B.def_step(ctx, x, g, e, m, 5, 3)                      # first call outside capture (device query)
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        B.def_set_stream(ctx, side)
        with torch.cuda.graph(graph, stream=side):
            B.def_step(ctx, x, g, e, m, 5, 3)
        B.def_set_stream(ctx, None)
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    s = oracle.block_start(3, 5, d)
    for _ in range(4):                                     # the eager call + three replays (capture runs nothing)
        oracle.step(xo, gh, eo, mo, d=d, k=k, s=s, eta=0.1, mu=0.9)
    assert np.array_equal(x.cpu().numpy(), xo) and np.array_equal(e.cpu().numpy(), eo) and np.array_equal(m.cpu().numpy(), mo)
    B.def_destroy(ctx)


@pytest.mark.parametrize("d", [5_000_001, 3_000_002, 2_051])
def test_unaligned_contiguous_rows_take_the_flat_path(B, d):
    """d % 4 != 0 with 16-byte aligned bases: block coordinates by one kernel, the rest as a flat
    stream over the W * d floats.  Whole tensors against the oracle, wrapped blocks included."""
    dev = torch.device("cuda")
    W, k, seed = 7, max(1, d // 16), 12
    rng = np.random.default_rng(d)
    x = torch.from_numpy((0.05 * rng.standard_normal(d)).astype(np.float32)).to(dev)
    e = torch.zeros(W, d, device=dev); m = torch.zeros(W, d, device=dev)
    xo = x.cpu().numpy().copy(); eo = np.zeros((W, d), np.float32); mo = np.zeros((W, d), np.float32)
    ctx = B.def_create(d, W, k, 0, 0.1, 0.9)
    B.def_set_small_step_bytes(ctx, 0)
    B.def_set_kernel_timing(ctx, True)
    steps = [0, 1] + find_steps(d, k, seed, lambda s: s + k > d)[:1]
    for t in steps:
        gh = (0.1 * rng.standard_normal((W, d))).astype(np.float32)
        g = torch.from_numpy(gh).to(dev)
        B.def_step(ctx, x, g, e, m, t, seed)
        oracle.step(xo, gh, eo, mo, d=d, k=k, s=oracle.block_start(seed, t, d), eta=0.1, mu=0.9)
        assert torch.equal(g.cpu(), torch.from_numpy(gh))
    assert B.def_kernel_time(ctx, B.DEF_KERNEL_STREAM)[1] == len(steps)
    assert B.def_kernel_time(ctx, B.DEF_KERNEL_BLOCK)[1] == len(steps)
    assert B.def_kernel_time(ctx, B.DEF_KERNEL_GENERAL)[1] == 0
    assert np.array_equal(x.cpu().numpy(), xo)
    assert np.array_equal(e.cpu().numpy(), eo) and np.array_equal(m.cpu().numpy(), mo)
    B.def_destroy(ctx)


@pytest.mark.parametrize("d,momentum", [(5_000_001, 0.9), (3_000_002, 0.9), (2_100_003, 0.0), (2_051, 0.9)])
def test_unaligned_rows_with_detach_take_the_flat_path(B, d, momentum):
    """The step with the fused detach output on contiguous rows with d % 4 != 0: the flat stream in
    its chunked order (several segments of coordinates, spare slots, ragged last CTA) and the
    block-columns kernel, every element of x, e', m' and z against the oracle, wrapped blocks included."""
    dev = torch.device("cuda")
    W, k, seed, lam = 6, max(1, d // 16), 12, 0.3
    rng = np.random.default_rng(d)
    x, cx = guarded((d,), dev)
    e, ce = guarded((W, d), dev); z, cz = guarded((W, d), dev)
    x.copy_(torch.from_numpy((0.05 * rng.standard_normal(d)).astype(np.float32))); e.zero_(); z.fill_(-7.0)
    m = cm = None
    if momentum:
        m, cm = guarded((W, d), dev); m.zero_()
    xo = x.cpu().numpy().copy(); eo = np.zeros((W, d), np.float32)
    mo = np.zeros((W, d), np.float32) if momentum else None
    ctx = B.def_create(d, W, k, 0, 0.1, momentum, (lam, 0.0))
    B.def_set_small_step_bytes(ctx, 0)
    B.def_set_kernel_timing(ctx, True)
    steps = [0, 1] + find_steps(d, k, seed, lambda s: s + k > d)[:1]
    for t in steps:
        gh = (0.1 * rng.standard_normal((W, d))).astype(np.float32)
        g = torch.from_numpy(gh).to(dev)
        B.def_step_detach(ctx, x, g, e, m, z, t, seed)
        oracle.step(xo, gh, eo, mo, d=d, k=k, s=oracle.block_start(seed, t, d), eta=0.1, mu=momentum)
        zh = z.cpu().numpy()
        for w in range(W):
            assert np.array_equal(zh[w], oracle.detach(xo, np.ascontiguousarray(eo[w]), lam)), (t, w)
    assert B.def_kernel_time(ctx, B.DEF_KERNEL_STREAM)[1] == len(steps)
    assert B.def_kernel_time(ctx, B.DEF_KERNEL_BLOCK)[1] == len(steps)
    assert B.def_kernel_time(ctx, B.DEF_KERNEL_GENERAL)[1] == 0
    assert np.array_equal(x.cpu().numpy(), xo) and np.array_equal(e.cpu().numpy(), eo)
    if momentum:
        assert np.array_equal(m.cpu().numpy(), mo)
    for chk in (cx, ce, cz, cm):
        if chk:
            chk()
    B.def_destroy(ctx)


def test_random_shapes_and_layouts(B):
    """Seeded sweep over shapes, alignments, launch strategies, momentum on/off and the fused
    detach output: every case bit-identical to the oracle, nothing written outside the tensors."""
    rng = np.random.default_rng(20260101)
    for case in range(60):
        d = int(rng.choice([rng.integers(1, 40), rng.integers(40, 5000), rng.integers(5000, 60000)]))
        W = int(rng.choice([1, 2, 3, 5, 8, 16, 33]))
        k = int(rng.choice([1, d, max(1, d // 2), int(rng.integers(1, d + 1))]))
        momentum = float(rng.choice([0.0, 0.5, 0.9]))
        offsets = tuple(int(v) for v in rng.integers(0, 4, size=5))
        if rng.random() < 0.5:
            offsets = (0, 0, 0, 0, 0)
        pair = bool(rng.integers(0, 2))
        seed = int(rng.integers(0, 1000))
        steps = [int(v) for v in rng.integers(0, 10 ** 6, size=3)]
        if rng.random() < 0.4:
            run_detach(B, d, W, k, steps, momentum, float(rng.choice([0.0, 0.3, 1.0])), offsets=offsets, seed=seed, pair=pair)
        else:
            assert run_whole(B, d, W, k, steps, momentum, seed, offsets=offsets[:4], pair=pair), (case, d, W, k)


def test_random_column_views(B):
    """Seeded sweep over column ranges of larger models (any j0 and n, padded or contiguous rows),
    block lengths from 1 to d, both launch strategies, momentum on / off and the fused detach
    output: every case bit-identical to the oracle's column view, padding columns untouched."""
    dev = torch.device("cuda")
    rng = np.random.default_rng(20261130)
    for case in range(250):
        d = int(rng.choice([rng.integers(2048, 20000), rng.integers(20000, 400000)]))
        W = int(rng.choice([1, 2, 3, 5, 8, 16]))
        k = int(rng.choice([1, d, d - 1, max(1, d // 2), max(1, d // 8), int(rng.integers(1, d + 1))]))
        mom = float(rng.choice([0.0, 0.9]))
        detach = bool(rng.integers(0, 2))
        lam, seed = 0.3, int(rng.integers(0, 1000))
        if rng.random() < 0.5:
            j0, n = 0, d
        else:
            j0 = int(rng.integers(0, d)); n = int(rng.integers(1, d - j0 + 1))
            if rng.random() < 0.5:
                j0 = j0 // 4 * 4
        ld = n if rng.random() < 0.5 else (n + 3) // 4 * 4 + int(rng.choice([0, 4]))
        x0 = (0.05 * rng.standard_normal(d)).astype(np.float32)
        cols = np.arange(j0, j0 + n, dtype=np.int64)
        xo = x0[j0:j0 + n].copy(); eo = np.zeros((W, n), np.float32)
        mo = np.zeros((W, n), np.float32) if mom else None
        x = torch.from_numpy(xo.copy()).to(dev)
        e = torch.zeros(W, ld, device=dev); m = torch.zeros(W, ld, device=dev) if mom else None
        z = torch.full((W, ld), -9.0, device=dev) if detach else None
        ctx = B.def_create(d, W, k, 0, 0.1, mom, (lam, 0.0))
        B.def_set_small_step_bytes(ctx, 0 if rng.random() < 0.8 else 1 << 60)
        what = dict(case=case, d=d, W=W, k=k, mom=mom, detach=detach, j0=j0, n=n, ld=ld, seed=seed)
        for t in (int(v) for v in rng.integers(0, 10 ** 6, size=3)):
            gh = (0.1 * rng.standard_normal((W, n))).astype(np.float32)
            g = torch.zeros(W, ld, device=dev); g[:, :n] = torch.from_numpy(gh).to(dev)
            if detach:
                B.def_step_columns_detach(ctx, j0, n, ld, x, g, e, m, z, t, seed)
            else:
                B.def_step_columns(ctx, j0, n, ld, x, g, e, m, t, seed)
            oracle.step(xo, gh, eo, mo, d=d, k=k, s=oracle.block_start(seed, t, d), eta=0.1, mu=mom,
                        cols=cols if n != d else None)
            if detach:
                zh = z[:, :n].cpu().numpy()
                for w in range(W):
                    assert np.array_equal(zh[w], oracle.detach(xo, np.ascontiguousarray(eo[w]), lam)), (what, t, w)
        assert np.array_equal(x.cpu().numpy(), xo) and np.array_equal(e[:, :n].cpu().numpy(), eo), what
        if mom:
            assert np.array_equal(m[:, :n].cpu().numpy(), mo), what
        assert not e[:, n:].any(), what
        if detach:
            assert bool((z[:, n:] == -9.0).all()), what
        B.def_destroy(ctx)
