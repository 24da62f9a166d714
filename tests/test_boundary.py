"""The C boundary without a GPU: the library loads, exports what include/def.h declares,
and turns every bad argument into its error code before anything is launched."""
import ctypes
import os
import re

import numpy as np
import pytest
import torch

import oracle
from paper_2004_05298_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HAS_GPU = torch.cuda.is_available()


def _declared_symbols():
    names = set()
    for fname in sorted(os.listdir(os.path.join(ROOT, "include"))):
        text = open(os.path.join(ROOT, "include", fname)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names.update(re.findall(r"\b(def_[a-z_0-9]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol():
    declared = _declared_symbols()
    assert {"def_create", "def_step", "def_destroy"} <= declared
    raw = ctypes.CDLL(B.LIB_PATH)
    for name in declared:
        assert hasattr(raw, name), "libdef_b200.so does not export %s" % name
    assert declared == set(B.SIGNATURES), "binding and header disagree: %s" % (declared ^ set(B.SIGNATURES))


def test_library_is_in_tree():
    assert os.path.dirname(B.LIB_PATH) == os.path.join(ROOT, "paper_2004_05298_b200")


@pytest.mark.parametrize("args,needle", [
    ((0, 4, 1, 0, 0.1, 0.9), "d must"),
    ((100, 0, 10, 0, 0.1, 0.9), "W must"),
    ((100, B.DEF_MAX_WORKERS + 1, 10, 0, 0.1, 0.9), "W must"),
    ((100, 4, 0, 0, 0.1, 0.9), "k must"),
    ((100, 4, 101, 0, 0.1, 0.9), "k must"),
    ((100, 4, 10, 3, 0.1, 0.9), "variant"),
    ((100, 4, 10, 0, float("nan"), 0.9), "lr"),
    ((100, 4, 10, 0, float("inf"), 0.9), "lr"),
    ((100, 4, 10, 0, 0.1, 1.0), "momentum"),
    ((100, 4, 10, 0, 0.1, -0.1), "momentum"),
])
def test_create_rejects(args, needle):
    with pytest.raises(B.DefError) as info:
        B.def_create(*args)
    assert needle in str(info.value)


def test_create_coeffs():
    with pytest.raises(B.DefError) as info:
        B.def_create(100, 4, 10, 0, 0.1, 0.9, coeffs=(1.5, 0.0))
    assert "lambda" in str(info.value)
    with pytest.raises(B.DefError) as info:
        B.def_create(100, 4, 10, 0, 0.1, 0.9, coeffs=(0.3, 5e-4))
    assert info.value.code == B.DEF_ERR_UNSUPPORTED
    ctx = B.def_create(100, 4, 10, B.DEF_VARIANT_EF, 0.1, 0.9, coeffs=(0.3, 0.0))
    B.def_destroy(ctx)
    B.def_destroy(ctx)                         # second destroy is a no-op in the binding
    assert B.lib.def_destroy(None) == B.DEF_ERR_NULL


def _raw_step(ctx, x, g, e, m, step=0, seed=0):
    return B.lib.def_step(ctx.handle, x, g, e, m, step, seed)


def test_step_validation_happens_before_any_launch():
    d, W = 1000, 4
    ctx = B.def_create(d, W, 100, 0, 0.1, 0.9)
    row = d * W * 4
    base = 0x7000_0000_0000                   # never dereferenced: validation is arithmetic only
    x, g, e, m = base, base + 0x100000, base + 0x100000 + row, base + 0x100000 + 2 * row
    assert _raw_step(ctx, None, g, e, m) == B.DEF_ERR_NULL
    assert _raw_step(ctx, x, None, e, m) == B.DEF_ERR_NULL
    assert _raw_step(ctx, x, g, None, m) == B.DEF_ERR_NULL
    assert _raw_step(ctx, x, g, e, None) == B.DEF_ERR_NULL and "mom" in B.def_last_error()
    assert _raw_step(ctx, x + 2, g, e, m) == B.DEF_ERR_ALIGN and "params" in B.def_last_error()
    assert _raw_step(ctx, x, g + 1, e, m) == B.DEF_ERR_ALIGN
    assert _raw_step(ctx, x, g, g, m) == B.DEF_ERR_ALIAS
    assert _raw_step(ctx, x, g, e, e + row - 4) == B.DEF_ERR_ALIAS and "errors and mom" in B.def_last_error()
    assert _raw_step(ctx, g + 8, g, e, m) == B.DEF_ERR_ALIAS
    assert B.lib.def_step(None, x, g, e, m, 0, 0) == B.DEF_ERR_NULL
    if not HAS_GPU:                            # valid arguments get as far as the device check
        assert _raw_step(ctx, x, g, e, m) == B.DEF_ERR_DEVICE
    # column ranges
    f = B.lib.def_step_columns
    assert f(ctx.handle, -1, 10, 10, x, g, e, m, 0, 0) == B.DEF_ERR_ARG
    assert f(ctx.handle, 995, 10, 10, x, g, e, m, 0, 0) == B.DEF_ERR_ARG
    assert f(ctx.handle, 0, 10, 9, x, g, e, m, 0, 0) == B.DEF_ERR_ARG and "stride" in B.def_last_error()
    B.def_destroy(ctx)
    # no momentum: mom must be NULL
    ctx = B.def_create(d, W, 100, 0, 0.1, 0.0)
    assert _raw_step(ctx, x, g, e, m) == B.DEF_ERR_ARG
    if not HAS_GPU:
        assert _raw_step(ctx, x, g, e, None) == B.DEF_ERR_DEVICE
    B.def_destroy(ctx)


def test_set_lr_and_stream():
    ctx = B.def_create(10, 1, 1, 0, 0.1, 0.0)
    B.def_set_lr(ctx, 0.01)
    with pytest.raises(B.DefError):
        B.def_set_lr(ctx, float("nan"))
    B.def_set_stream(ctx, None)
    assert B.def_launch_count(ctx) == 0
    B.def_destroy(ctx)


def test_host_block_start_matches_oracle():
    rng = np.random.default_rng(5)
    for d in (1, 7, 855770, 1_000_000, 138_357_544, 2 ** 40 + 9):
        ctx = B.def_create(d, 1, 1, 0, 0.1, 0.0)
        for _ in range(200):
            seed, step = (int(v) for v in rng.integers(0, 2 ** 64, size=2, dtype=np.uint64))
            if _ % 2:
                seed, step = seed % 6, step % 128
            assert B.def_block_start(ctx, step, seed) == oracle.block_start(seed, step, d)
        B.def_destroy(ctx)


def test_tile_plan_against_brute_force():
    """The cut of a step's tiles between the two kernels of a pair (host arithmetic the grids are
    sized from): against the set of tiles that hold a block coordinate, found by enumeration, with
    the block start taken from the oracle's sampler."""
    import random
    rnd = random.Random(5)
    TILE = 1024
    cases = 0
    for _ in range(400):
        d = rnd.choice([rnd.randint(1, 50), rnd.randint(50, 5000), rnd.randint(5000, 40000)])
        k = rnd.choice([1, d, max(1, d - 1), rnd.randint(1, d)])
        ctx = B.def_create(d, 2, k, 0, 0.1, 0.9)
        for step in range(6):
            seed = rnd.randrange(100)
            j0 = rnd.choice([0, rnd.randrange(d)])
            n = rnd.choice([d - j0, rnd.randint(1, d - j0)])
            s = oracle.block_start(seed, step, d)
            block = {(s + i) % d for i in range(k)}
            want = sorted({(j - j0) // TILE for j in block if j0 <= j < j0 + n})
            a_first, a_count, b_count, rest = B.def_tile_plan(ctx, j0, n, step, seed)
            got = list(range(b_count)) + list(range(a_first, a_first + a_count))
            assert a_count == 0 or b_count <= a_first, (d, k, s, j0, n)
            assert got == want, (d, k, s, j0, n, got[:5], want[:5])
            assert rest == -(-n // TILE) - len(want)
            cases += 1
        B.def_destroy(ctx)
    assert cases == 2400
    ctx = B.def_create(100, 2, 10, 0, 0.1, 0.9)
    out = (ctypes.c_int64 * 4)()
    assert B.lib.def_tile_plan(ctx.handle, 0, 0, 0, 0, out) == B.DEF_ERR_ARG
    assert B.lib.def_tile_plan(ctx.handle, 50, 51, 0, 0, out) == B.DEF_ERR_ARG
    assert B.lib.def_tile_plan(ctx.handle, 0, 100, 0, 0, None) == B.DEF_ERR_NULL
    B.def_destroy(ctx)
