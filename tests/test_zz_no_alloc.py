"""def_stats_static -- the distances of Eq. 9 for callers that are not allowed to allocate
device memory (a host framework that owns every byte through its own pool, a deployment
with a memory budget fixed at start-up, a path that cannot take cudaMalloc's implicit
synchronisation).  It must give what def_stats gives, call after call, although its scratch
is one fixed array in the library that every call shares and that keeps the previous call's
contents.

This file is named so that pytest collects it last: a run that stops at the first failure
has then already run every other test.  It passes alone in a fresh process (the first call
here then performs the one-time address look-up) and after the other tests."""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu

STATS_TOL = 2e-9      # of stats[0]; the tolerance tests/test_aux_gpu.py uses for the distances


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.fail("this test needs a CUDA device")
    from paper_2004_05298_b200 import binding
    return binding


def _errors(W, n, seed, offset=0):
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    buf = torch.empty(W * n + 8, dtype=torch.float32, device="cuda")
    e = buf[offset:offset + W * n].view(W, n)
    e.normal_(0.0, 0.05, generator=gen)
    return e


def _reference(B, e, lam):
    """The existing entry point (context-owned scratch from cudaMalloc)."""
    W, n = e.shape
    ctx = B.def_create(n, W, 1, B.DEF_VARIANT_DEF, 0.1, 0.9, (lam, 0.0))
    out = torch.zeros(3, dtype=torch.float64, device="cuda")
    B.def_stats(ctx, e, out)
    torch.cuda.synchronize()
    B.def_destroy(ctx)
    return out.cpu().numpy()


def test_two_calls_in_a_row_match_def_stats(B):
    lam = 0.3
    # first call: many CTAs (fills every scratch slot); second: a different, smaller input whose
    # few CTAs must not see what the first call left behind; third: the first input again
    big = _errors(8, 3_000_000, seed=1)
    small = _errors(3, 70_001, seed=2, offset=1)            # odd n, 4-byte aligned rows
    out = torch.full((3,), -1.0, dtype=torch.float64, device="cuda")
    host = torch.empty(3, dtype=torch.float64).pin_memory()
    B.def_stats_static(small, lam, out)                     # the one-time address look-up, if this process has not done it
    torch.cuda.synchronize()
    # From here on the device's free memory must not move: cudaMemGetInfo sees every allocation
    # of the process, the library's own included (torch's counters would only see torch's pool).
    pool_before = torch.cuda.memory_allocated()
    free_before = torch.cuda.mem_get_info()[0]
    results = []
    for e in (big, small, big):
        B.def_stats_static(e, lam, out)
        host.copy_(out, non_blocking=True)                  # into pinned memory allocated above: no new buffer
        torch.cuda.synchronize()
        results.append(host.numpy().copy())
        assert torch.cuda.mem_get_info()[0] >= free_before, "device memory was allocated during the call"
    assert torch.cuda.memory_allocated() == pool_before     # nothing was taken from torch's pool either
    for e, got in zip((big, small, big), results):
        want = _reference(B, e, lam)                        # the existing entry point
        assert np.all(np.abs(got - want) <= STATS_TOL * want[0]), (got, want)
        truth = np.array(oracle.stats(e.cpu().numpy(), lam))   # and the CPU oracle's plain loops
        assert np.all(np.abs(got - truth) <= STATS_TOL * truth[0]), (got, truth)
    assert np.array_equal(results[0], results[2]), "same input, same bits, whatever ran in between"


def test_on_a_side_stream_and_limits(B):
    e = _errors(4, 500_000, seed=3)
    out = torch.zeros(3, dtype=torch.float64, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    B.def_stats_static(e, 1.0, out, stream=side)
    side.synchronize()
    want = _reference(B, e, 1.0)
    assert np.all(np.abs(out.cpu().numpy() - want) <= STATS_TOL * want[0])
    # beyond the stated maximum: a clear error, nothing launched
    f = B.lib.def_stats_static
    assert f(e.data_ptr(), B.DEF_STATS_STATIC_MAX_N + 1, B.DEF_STATS_STATIC_MAX_N + 1, 4, 0.3, out.data_ptr(), None) == B.DEF_ERR_ARG
    assert "at most" in B.def_last_error()
    assert f(e.data_ptr(), 10, 10, 65, 0.3, out.data_ptr(), None) == B.DEF_ERR_ARG
    assert f(e.data_ptr(), 10, 9, 4, 0.3, out.data_ptr(), None) == B.DEF_ERR_ARG
    assert f(None, 10, 10, 4, 0.3, out.data_ptr(), None) == B.DEF_ERR_NULL
    assert f(e.data_ptr(), 10, 10, 4, 0.3, out.data_ptr() + 4, None) == B.DEF_ERR_ALIGN
