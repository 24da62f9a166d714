"""GPU parity of the helpers around the step -- the detach point (Algorithm 1's detach step), the
returned model (Algorithm 1's Output) and the distances of Eq. 9 -- against the CPU
oracle, through the C boundary.  detach and output do the oracle's roundings in the oracle's
order (bit-identical expected, gate 1e-5 relative).  The distances are fp64 sums whose
order differs from the oracle's plain loop: for N = W * n summed terms the two can differ by
up to N * 2^-53 of the sum (1.1e-9 at the sizes used here), so the gate is 2e-9 of stats[0]."""
import numpy as np
import pytest
import torch

import oracle
from paper_2004_05298_b200 import workloads as WL

pytestmark = pytest.mark.gpu
STATS_TOL = 2e-9


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    from paper_2004_05298_b200 import binding
    return binding


def _state(d, W, steps, B, seed=3, momentum=0.9, variant=0, lam=0.3):
    """A few real steps so that x, e are what the helpers see in use (GPU and oracle copies)."""
    dev = torch.device("cuda")
    wl = WL.get(1).scaled(d, W=W, momentum=momentum)
    x = WL.initial_params(wl, dev); e, m = WL.zeros_state(wl, dev)
    ctx = B.def_create(d, W, wl.k, variant, wl.lr, momentum, (lam, 0.0))
    for t in range(steps):
        B.def_step(ctx, x, WL.gradients(wl, t, dev), e, m, t, seed)
    torch.cuda.synchronize()
    return ctx, x, e


def _offset_view(t, offset):
    """Copy of t whose storage starts `offset` floats off a 16-byte boundary."""
    buf = torch.empty(t.numel() + 8, dtype=t.dtype, device=t.device)
    v = buf[offset:offset + t.numel()].view(t.shape)
    v.copy_(t)
    return v


@pytest.mark.parametrize("d,W", [(1, 1), (7, 3), (4096, 4), (100_003, 5), (262_146, 16), (50_000, 64), (262_144, 16),
                                 (131_072, 3), (1_000_000, 5)])
@pytest.mark.parametrize("offset", [0, 1, 2])
def test_detach_and_output(B, d, W, offset):
    for variant, lam in ((B.DEF_VARIANT_DEF, 0.3), (B.DEF_VARIANT_DEF_A, 1.0), (B.DEF_VARIANT_EF, 0.7)):
        ctx, x, e = _state(d, W, 3, B, variant=variant, lam=lam)
        x, e = _offset_view(x, offset), _offset_view(e, offset)
        z = _offset_view(torch.full((W, d), -7.0, device="cuda"), offset)
        y = _offset_view(torch.full((d,), -7.0, device="cuda"), offset)
        B.def_detach(ctx, x, e, z)
        B.def_output(ctx, x, e, y)
        xh, eh = x.cpu().numpy(), e.cpu().numpy()
        lam_used = 0.0 if variant == B.DEF_VARIANT_EF else lam          # plain EF evaluates at x_t
        for w in range(W):
            assert np.array_equal(z[w].cpu().numpy(), oracle.detach(xh, np.ascontiguousarray(eh[w]), lam_used)), (variant, w)
        assert np.array_equal(y.cpu().numpy(), oracle.output(variant, xh, eh)), variant
        if variant != B.DEF_VARIANT_DEF:
            B.def_output(ctx, x, None, y)                               # errors are not needed for x_T
            assert torch.equal(y, x)
        B.def_destroy(ctx)


@pytest.mark.parametrize("d,n,ld", [(10_000, 3_001, 3_006), (400_000, 131_072, 131_080)])
def test_views_with_padding(B, d, n, ld):
    W = 4
    ctx, x, e = _state(d, W, 2, B)
    el = torch.full((W, ld), 9.0, device="cuda"); el[:, :n] = e[:, 100:100 + n]
    xl = x[100:100 + n].clone()
    z = torch.full((W, ld), -7.0, device="cuda"); y = torch.full((n,), -7.0, device="cuda")
    s = torch.zeros(3, dtype=torch.float64, device="cuda")
    B.def_detach(ctx, xl, el, z, n=n, ld=ld); B.def_output(ctx, xl, el, y, n=n, ld=ld); B.def_stats(ctx, el, s, n=n, ld=ld)
    eh = np.ascontiguousarray(el[:, :n].cpu().numpy()); xh = xl.cpu().numpy()
    assert np.array_equal(y.cpu().numpy(), oracle.output(0, xh, eh))
    for w in range(W):
        assert np.array_equal(z[w, :n].cpu().numpy(), oracle.detach(xh, np.ascontiguousarray(eh[w]), 0.3))
    assert bool((z[:, n:] == -7.0).all()), "padding columns were written"
    want = oracle.stats(eh, 0.3)
    assert np.allclose(s.cpu().numpy(), want, rtol=0, atol=STATS_TOL * want[0])
    B.def_destroy(ctx)


def test_bad_arguments(B):
    ctx, x, e = _state(1000, 2, 1, B)
    z = torch.empty_like(e); s = torch.zeros(3, dtype=torch.float64, device="cuda")
    assert B.lib.def_detach(ctx.handle, 1000, 1000, x.data_ptr(), e.data_ptr(), e.data_ptr()) == B.DEF_ERR_ALIAS
    assert B.lib.def_detach(ctx.handle, 1000, 999, x.data_ptr(), e.data_ptr(), z.data_ptr()) == B.DEF_ERR_ARG
    assert B.lib.def_output(ctx.handle, 1000, 1000, x.data_ptr(), None, z.data_ptr()) == B.DEF_ERR_NULL
    assert B.lib.def_output(ctx.handle, 1000, 1000, x.data_ptr(), e.data_ptr(), x.data_ptr()) == B.DEF_ERR_ALIAS
    assert B.lib.def_stats(ctx.handle, 1001, 1001, e.data_ptr(), s.data_ptr()) == B.DEF_ERR_ARG
    assert B.lib.def_stats(ctx.handle, 1000, 1000, e.data_ptr(), None) == B.DEF_ERR_NULL
    B.def_destroy(ctx)


@pytest.mark.parametrize("d,W", [(1, 1), (5, 2), (4099, 3), (1_000_000, 4), (300_001, 16), (600_000, 8)])
@pytest.mark.parametrize("offset", [0, 1, 2])
def test_stats_matches_oracle(B, d, W, offset):
    ctx, x, e = _state(d, W, 3, B, lam=0.3)
    e = _offset_view(e, offset)
    out = torch.zeros(3, dtype=torch.float64, device="cuda")
    B.def_stats(ctx, e, out)
    first = out.cpu().numpy().copy()
    want = oracle.stats(e.cpu().numpy(), 0.3)
    assert np.all(np.abs(first - want) <= STATS_TOL * want[0]), (first, want)
    B.def_stats(ctx, e, out)                                             # fixed order: identical bits
    assert np.array_equal(out.cpu().numpy(), first)
    B.def_destroy(ctx)


def test_stats_closed_form_at_full_size(B):
    """Every row constant (dyadic values): the three distances have exact closed forms at any n."""
    wl = WL.get(5)
    d, W, lam = wl.d, wl.W, 0.25
    a = np.array([(w % 5 - 2) * 0.5 for w in range(W)])                 # row constants
    e = torch.from_numpy(a.astype(np.float32)).cuda().unsqueeze(1).expand(W, d).contiguous()
    ctx = B.def_create(d, W, wl.k, 0, 0.1, 0.9, (lam, 0.0))
    out = torch.zeros(3, dtype=torch.float64, device="cuda")
    B.def_stats(ctx, e, out)
    got = out.cpu().numpy()
    want = np.array([d * np.mean(a * a), d * np.mean(a) ** 2, d * np.mean((np.mean(a) - lam * a) ** 2)])
    assert np.allclose(got, want, rtol=1e-12), (got, want)
    # column shards add up
    total = np.zeros(3)
    cuts = [0, 40_000_000, 40_000_004, 100_000_001, d]
    for j0, j1 in zip(cuts[:-1], cuts[1:]):
        part = e[:, j0:j1].contiguous()
        B.def_stats(ctx, part, out, n=j1 - j0, ld=j1 - j0)
        total += out.cpu().numpy()
    assert np.allclose(total, got, rtol=1e-12)
    B.def_destroy(ctx)


@pytest.mark.parametrize("d,W,offset", [(1, 1, 0), (4099, 3, 0), (100_000, 4, 0), (100_002, 8, 2), (65_537, 16, 1)])
@pytest.mark.parametrize("momentum", [0.9, 0.0])
def test_scaling_compressor_step(B, d, W, offset, momentum):
    """C(v) = delta v (the DEF-A paragraph, Eq. 11): the step and its fused detach output against
    the oracle's scaling compressor, bit for bit."""
    dev = torch.device("cuda")
    delta, lam, lr = 0.25, 1.0, 0.1
    rng = np.random.default_rng(d + W)
    x = _offset_view(torch.from_numpy((0.05 * rng.standard_normal(d)).astype(np.float32)).cuda(), offset)
    e = _offset_view(torch.zeros(W, d, device=dev), offset)
    m = _offset_view(torch.zeros(W, d, device=dev), offset) if momentum else None
    z = _offset_view(torch.zeros(W, d, device=dev), offset)
    xo = x.cpu().numpy().copy(); eo = np.zeros((W, d), np.float32)
    mo = np.zeros((W, d), np.float32) if momentum else None
    ctx = B.def_create(d, W, 1, B.DEF_VARIANT_DEF_A, lr, momentum, (lam, 0.0))
    B.def_set_compressor(ctx, B.DEF_COMPRESSOR_SCALE, delta)
    with pytest.raises(B.DefError):
        B.def_set_compressor(ctx, B.DEF_COMPRESSOR_SCALE, 1.0)
    for t in range(4):
        gh = (0.1 * rng.standard_normal((W, d))).astype(np.float32)
        g = _offset_view(torch.from_numpy(gh).cuda(), offset)
        if t % 2:
            B.def_step_detach(ctx, x, g, e, m, z, t, 0)
        else:
            B.def_step(ctx, x, g, e, m, t, 0)
        oracle.step(xo, gh, eo, mo, d=d, k=1, s=0, eta=lr, mu=momentum, compressor=oracle.COMPRESSOR_SCALE, delta=delta)
        assert np.array_equal(x.cpu().numpy(), xo) and np.array_equal(e.cpu().numpy(), eo), t
        if momentum:
            assert np.array_equal(m.cpu().numpy(), mo)
        if t % 2:
            for w in range(W):
                assert np.array_equal(z[w].cpu().numpy(), oracle.detach(xo, np.ascontiguousarray(eo[w]), lam))
    B.def_set_compressor(ctx, B.DEF_COMPRESSOR_RBGS)                     # and back: the block again
    gh = (0.1 * rng.standard_normal((W, d))).astype(np.float32)
    B.def_step(ctx, x, _offset_view(torch.from_numpy(gh).cuda(), offset), e, m, 9, 2)
    oracle.step(xo, gh, eo, mo, d=d, k=1, s=oracle.block_start(2, 9, d), eta=lr, mu=momentum)
    assert np.array_equal(x.cpu().numpy(), xo) and np.array_equal(e.cpu().numpy(), eo)
    B.def_destroy(ctx)
