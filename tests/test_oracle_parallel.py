"""The all-cores build of the oracle (same source, loops over coordinates as OpenMP parallel-for
loops) must give the bits of the plain single-threaded build: only which thread handles a
coordinate changes, never the operations on it or their order.  The benchmark times both as CPU
baselines and the full-size parity tests use the fast one, so this identity is what lets them
stand in for the plain oracle."""
import numpy as np
import pytest

import oracle


@pytest.mark.parametrize("dtype", [np.float32, np.float64])
@pytest.mark.parametrize("momentum", [0.9, 0.0])
def test_all_cores_build_is_bit_identical(dtype, momentum):
    serial, fast = oracle.default(), oracle.all_cores()
    assert serial.threads() == 1 and fast.threads() >= 1
    d, W, k = 300_007, 5, 9_000
    rng = np.random.default_rng(11)
    x0 = (0.05 * rng.standard_normal(d)).astype(dtype)

    def run(o, cols=None):
        n = d if cols is None else len(cols)
        x = (x0 if cols is None else x0[cols]).copy()
        e = np.zeros((W, n), dtype); m = np.zeros((W, n), dtype) if momentum else None
        local = np.random.default_rng(5)
        for t in range(4):
            g = (0.1 * local.standard_normal((W, d))).astype(dtype)
            if cols is not None:
                g = np.ascontiguousarray(g[:, cols])
            s = o.block_start(3, t, d) if t < 3 else d - 5            # the last block wraps
            o.step(x, g, e, m, d=d, k=k, s=s, eta=0.1, mu=momentum, cols=cols)
        y = o.output(oracle.VARIANT_DEF, x, e)
        z = o.detach(x, np.ascontiguousarray(e[W - 1]), 0.3)
        return [x, e, y, z] + ([m] if momentum else [])

    for cols in (None, np.sort(rng.choice(d, size=20_000, replace=False)).astype(np.int64)):
        a, b = run(serial, cols), run(fast, cols)
        for p, q in zip(a, b):
            assert np.array_equal(p, q)


def test_all_cores_scaling_compressor_and_compress():
    serial, fast = oracle.default(), oracle.all_cores()
    rng = np.random.default_rng(2)
    d = 100_003
    v = rng.standard_normal(d).astype(np.float32)
    assert np.array_equal(serial.compress(v, d, 777, d - 100), fast.compress(v, d, 777, d - 100))
    xs = []
    for o in (serial, fast):
        x = v.copy(); e = np.zeros((1, d), np.float32)
        for t in range(3):
            o.step(x, v.reshape(1, d), e, None, d=d, k=1, s=0, eta=0.1, compressor=oracle.COMPRESSOR_SCALE, delta=0.25)
        xs.append((x, e))
    assert np.array_equal(xs[0][0], xs[1][0]) and np.array_equal(xs[0][1], xs[1][1])
