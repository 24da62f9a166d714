"""Pins of the CPU oracle: checks against what the paper and the mathematics fix.

Each pin takes a loaded oracle (oracle.Oracle) and raises AssertionError when the
oracle disagrees with a value, closed form, invariant or library routine that does
not come from the oracle itself.  tests/test_oracle_pins.py runs them on the
committed oracle; tests/test_oracle_mutants.py plants one mistake at a time in a
copy of the oracle's source and requires that some pin notices.

The reference computations in here are deliberately whole-vector numpy / Python
integer statements of textbook routines (plain SGD, heavy-ball momentum, set
arithmetic mod d), not a second copy of the oracle's loops.
"""
import ctypes
import os
import subprocess
import tempfile

import numpy as np

VARIANT_DEF, VARIANT_DEF_A, VARIANT_EF = 0, 1, 2
COMPRESSOR_RBGS, COMPRESSOR_SCALE = 0, 1

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _rng(seed):
    return np.random.default_rng(seed)


def _close(a, b, rel, what):
    scale = max(1.0, float(np.max(np.abs(b)))) if np.size(b) else 1.0
    err = float(np.max(np.abs(np.asarray(a, dtype=np.float64) - np.asarray(b, dtype=np.float64)))) \
        if np.size(b) else 0.0
    assert err <= rel * scale, "%s: max abs difference %.3e exceeds %.1e x %.3e" % (what, err, rel, scale)


# ---------------------------------------------------------------------------
# Hand-worked example (tests/golden/hand_example_d8.txt): d = 8, K = 2, k = 3,
# eta = 1/2, mu = 1/2, all values dyadic so every result is exact in fp32.
# ---------------------------------------------------------------------------
def _load_hand_example():
    vals = {}
    with open(os.path.join(GOLDEN, "hand_example_d8.txt")) as fh:
        for line in fh:
            line = line.split("#", 1)[0].strip()
            if not line:
                continue
            name, rest = line.split("=", 1)
            vals[name.strip()] = np.array([float(v) for v in rest.split()], dtype=np.float64)
    return vals


def pin_hand_example(o):
    h = _load_hand_example()
    for dtype in (np.float32, np.float64):
        x = h["x0"].astype(dtype)
        e = np.zeros((2, 8), dtype)
        m = np.zeros((2, 8), dtype)
        for t in (0, 1):
            g = np.stack([h["g%d_w0" % t], h["g%d_w1" % t]]).astype(dtype)
            o.step(x, g, e, m, d=8, k=3, s=int(h["s%d" % t][0]), eta=0.5, mu=0.5)
            assert np.array_equal(x, h["x%d" % (t + 1)].astype(dtype)), ("x after step %d" % t, x)
            for w in (0, 1):
                assert np.array_equal(e[w], h["e%d_w%d" % (t + 1, w)].astype(dtype)), \
                    ("e of worker %d after step %d" % (w, t), e[w])
                assert np.array_equal(m[w], h["m%d_w%d" % (t + 1, w)].astype(dtype)), \
                    ("m of worker %d after step %d" % (w, t), m[w])
        y = o.output(VARIANT_DEF, x, e)
        assert np.array_equal(y, h["y2"].astype(dtype)), ("DEF output", y)
        assert np.array_equal(o.output(VARIANT_DEF_A, x, e), x)
        assert np.array_equal(o.output(VARIANT_EF, x, e), x)


# ---------------------------------------------------------------------------
# Eq. 8: y_{t+1} = y_t - eta * (mean over workers of g_{k,t}), y = x - mean_k e_k,
# for any start sequence and any K; with Eq. 10 the mean gradient becomes the
# mean momentum buffer, which follows heavy-ball M <- mu M + G.
# ---------------------------------------------------------------------------
def pin_telescoping_identity(o):
    for seed, (d, W, k, T, mu) in enumerate([(37, 3, 5, 9, 0.0), (64, 4, 17, 12, 0.9),
                                             (101, 1, 100, 6, 0.5), (50, 5, 1, 15, 0.7)]):
        rng = _rng(100 + seed)
        x0 = rng.standard_normal(d)
        x = x0.copy()
        e = np.zeros((W, d))
        m = np.zeros((W, d)) if mu > 0 else None
        M = np.zeros((W, d))                       # textbook heavy-ball buffers
        eta = 0.05
        y_expected = x0.copy()
        for t in range(T):
            g = rng.standard_normal((W, d))
            s = int(rng.integers(0, d))
            if t == 2:
                s = d - 1                          # a block that wraps for k > 1
            o.step(x, g, e, m, d=d, k=k, s=s, eta=eta, mu=mu)
            M = mu * M + g
            y_expected = y_expected - eta * M.mean(axis=0)
            y = o.output(VARIANT_DEF, x, e)
            _close(y, y_expected, 1e-12, "Eq. 8 identity, case %d step %d" % (seed, t))
            if m is not None:
                _close(m, M, 1e-12, "Eq. 10 momentum buffers, case %d step %d" % (seed, t))
        # the iteration must actually have compressed something
        if k < d:
            assert np.count_nonzero(e) == W * (d - k)


# ---------------------------------------------------------------------------
# k = d: the compressor is the identity, the error stays zero and x follows
# uncompressed synchronous momentum SGD (Eq. 2 with the heavy-ball buffer).
# ---------------------------------------------------------------------------
def pin_full_block_is_momentum_sgd(o):
    rng = _rng(7)
    d, W, T, eta, mu = 29, 4, 8, 0.1, 0.9
    for dtype, rel in ((np.float64, 1e-13), (np.float32, 2e-6)):
        x = rng.standard_normal(d).astype(dtype)
        X = x.astype(np.float64)
        e = np.zeros((W, d), dtype)
        m = np.zeros((W, d), dtype)
        M = np.zeros((W, d))
        for t in range(T):
            g = rng.standard_normal((W, d)).astype(dtype)
            o.step(x, g, e, m, d=d, k=d, s=int(rng.integers(0, d)), eta=eta, mu=mu)
            M = mu * M + g.astype(np.float64)
            X = X - eta * M.mean(axis=0)
            assert not e.any(), "k = d must leave no compression error"
            assert not np.signbit(e).any(), "the zero error is +0"
            _close(x, X, rel, "k = d path vs momentum SGD (%s) step %d" % (np.dtype(dtype).name, t))


# ---------------------------------------------------------------------------
# Algorithm 1's new-error step: C(p) + e' = p, coordinate by coordinate and bit for bit.
# One worker, x_0 = 0, e_0 = 0, eta = 1, no momentum: then p = g exactly,
# C(p) = -x_1 and e' = e_1.
# ---------------------------------------------------------------------------
def pin_sparsified_plus_error_is_p(o):
    rng = _rng(11)
    for d, k, s in [(40, 7, 3), (40, 7, 36), (33, 33, 5), (17, 1, 16)]:
        g = rng.standard_normal((1, d)).astype(np.float32)
        x = np.zeros(d, np.float32)
        e = np.zeros((1, d), np.float32)
        o.step(x, g, e, None, d=d, k=k, s=s, eta=1.0)
        Cp = -x
        assert np.array_equal(Cp + e[0], g[0]), "C(p) + e' != p"
        assert np.all((Cp == 0) | (e[0] == 0)), "a coordinate is both sent and kept as error"
        assert int(np.count_nonzero(Cp)) == k, "the sparsified part must have k coordinates"
        assert int(np.count_nonzero(e[0])) == d - k
        in_block = sorted(int(j) for j in np.nonzero(Cp)[0])
        assert in_block == sorted((s + i) % d for i in range(k)), (in_block, s, k, d)


# ---------------------------------------------------------------------------
# The block: exactly k distinct coordinates {(s+i) mod d}, one run, or two when
# it wraps.
# ---------------------------------------------------------------------------
def pin_block_shape(o):
    for d, k in [(1, 1), (2, 1), (2, 2), (10, 3), (10, 10), (10, 9), (97, 31)]:
        for s in range(d):
            mask = o.block_mask(d, k, s)
            want = np.zeros(d, bool)
            for i in range(k):
                want[(s + i) % d] = True
            assert np.array_equal(mask, want), (d, k, s)
            assert int(mask.sum()) == k
            runs = int(np.count_nonzero(np.diff(np.concatenate(([0], mask.astype(np.int8), [0]))) == 1))
            wraps = s + k > d and k < d            # k = d covers everything: one run
            assert runs == (2 if wraps else 1), (d, k, s, runs)
            for j in range(d):
                assert o.in_block(j, s, k, d) == bool(want[j])
    # a view sees the same predicate at its own coordinates
    cols = np.array([99, 0, 5, 50, 98, 4], dtype=np.int64)
    mask = o.block_mask(100, 7, 98, cols)          # block = {98, 99, 0, 1, 2, 3, 4}
    assert mask.tolist() == [True, True, False, False, True, True]


# ---------------------------------------------------------------------------
# Assumption 3: C(a) + C(b) = C(a + b) for a fixed start, bit for bit.
# ---------------------------------------------------------------------------
def pin_additivity(o):
    rng = _rng(13)
    d, k = 61, 20
    for s in (0, 7, 50, 60):
        a = rng.standard_normal(d).astype(np.float32)
        b = rng.standard_normal(d).astype(np.float32)
        lhs = o.compress(a, d, k, s) + o.compress(b, d, k, s)
        rhs = o.compress(a + b, d, k, s)
        assert np.array_equal(lhs, rhs)
        assert int(np.count_nonzero(rhs)) == k


# ---------------------------------------------------------------------------
# Assumption 5 and its remark: over the d equally likely starts, E C(v) = (k/d) v
# and E ||C(v) - v||^2 = (1 - k/d) ||v||^2 -- exact sums on integer-valued v.
# ---------------------------------------------------------------------------
def pin_expectation_over_starts(o):
    rng = _rng(17)
    for d, k in [(12, 5), (9, 1), (16, 16), (7, 6)]:
        v = rng.integers(-9, 10, size=d).astype(np.float64)
        total = np.zeros(d)
        sq = 0.0
        for s in range(d):
            c = o.compress(v, d, k, s)
            total += c
            sq += float(np.sum((c - v) ** 2))
        assert np.array_equal(total, k * v), "sum over starts of C_s(v) must be k v"
        assert sq == (d - k) * float(np.sum(v ** 2)), "mean squared residual must be (1 - k/d)|v|^2"


# ---------------------------------------------------------------------------
# K = 1 and lambda = 1: {y_t} is the SGD path (remark after Eq. 8); and with the
# scaling compressor C(v) = delta v, {x_t} is the geometric iterate average of
# Eq. 11.  The objective is a least-squares problem whose gradient is known in
# closed form.
# ---------------------------------------------------------------------------
def _quadratic(rng, d):
    A = rng.standard_normal((2 * d, d)) / np.sqrt(2 * d)
    b = rng.standard_normal(2 * d)
    return lambda theta: A.T @ (A @ theta - b)


def pin_single_worker_lambda_one_is_sgd(o):
    rng = _rng(19)
    d, k, T, eta = 23, 6, 25, 0.2
    grad = _quadratic(rng, d)
    x = rng.standard_normal(d)
    e = np.zeros((1, d))
    theta = x.copy()                               # plain SGD iterate
    for t in range(T):
        z = o.detach(x, e[0], 1.0)                 # Algorithm 1's detach step with lambda = 1
        g = grad(z)[None, :]
        o.step(x, g, e, None, d=d, k=k, s=int(rng.integers(0, d)), eta=eta)
        theta = theta - eta * grad(theta)
        y = o.output(VARIANT_DEF, x, e)
        _close(y, theta, 1e-12, "K=1, lambda=1: y_t vs SGD, step %d" % t)
    assert np.max(np.abs(x - theta)) > 1e-3, "x_T itself is not the SGD iterate"


def pin_scaling_compressor_is_iterate_averaging(o):
    rng = _rng(23)
    d, T, eta, delta = 11, 20, 0.15, 0.25
    grad = _quadratic(rng, d)
    y0 = rng.standard_normal(d)
    x = y0.copy()
    e = np.zeros((1, d))
    ys = [y0.copy()]
    for t in range(1, T + 1):
        z = o.detach(x, e[0], 1.0)
        g = grad(z)[None, :]
        o.step(x, g, e, None, d=d, k=1, s=0, eta=eta, compressor=COMPRESSOR_SCALE, delta=delta)
        ys.append(ys[-1] - eta * grad(ys[-1]))     # SGD path y_t
        closed = (1 - delta) ** t * ys[0]
        for tp in range(1, t + 1):
            closed = closed + delta * (1 - delta) ** (t - tp) * ys[tp]
        _close(x, closed, 1e-12, "Eq. 11 closed form at t = %d" % t)
    v = rng.standard_normal(d)
    assert np.array_equal(o.compress(v, d, 1, 0, compressor=COMPRESSOR_SCALE, delta=delta), delta * v)


# ---------------------------------------------------------------------------
# Detach point and outputs on exact values.
# ---------------------------------------------------------------------------
def pin_detach_and_output(o):
    x = np.array([1.0, -2.0, 0.5, 8.0], np.float32)
    e0 = np.array([0.5, 4.0, -1.0, 0.0], np.float32)
    e1 = np.array([1.5, 0.0, 3.0, -2.0], np.float32)
    assert np.array_equal(o.detach(x, e0, 0.0), x)                              # plain EF
    assert np.array_equal(o.detach(x, e0, 1.0), x - e0)
    assert np.array_equal(o.detach(x, e0, 0.25), np.array([0.875, -3.0, 0.75, 8.0], np.float32))
    e = np.stack([e0, e1])
    assert np.array_equal(o.output(VARIANT_DEF, x, e), np.array([0.0, -4.0, -0.5, 9.0], np.float32))
    assert np.array_equal(o.output(VARIANT_DEF_A, x, e), x)
    assert np.array_equal(o.output(VARIANT_EF, x, e), x)


# ---------------------------------------------------------------------------
# K workers average: with identical workers the step equals the one-worker step;
# with workers (g, -g) and e = 0 the block cancels and x does not move.
# ---------------------------------------------------------------------------
def pin_average_over_workers(o):
    rng = _rng(29)
    d, k, s, eta, mu = 19, 8, 15, 0.5, 0.5
    g1 = rng.integers(-8, 9, size=(1, d)).astype(np.float32)
    x1 = np.arange(d, dtype=np.float32)
    e1 = np.zeros((1, d), np.float32)
    m1 = np.zeros((1, d), np.float32)
    o.step(x1, g1, e1, m1, d=d, k=k, s=s, eta=eta, mu=mu)
    for W in (2, 3, 4, 8):
        x = np.arange(d, dtype=np.float32)
        e = np.zeros((W, d), np.float32)
        m = np.zeros((W, d), np.float32)
        o.step(x, np.repeat(g1, W, axis=0), e, m, d=d, k=k, s=s, eta=eta, mu=mu)
        _close(x, x1, 1e-6, "identical workers, W = %d" % W)
        assert np.array_equal(e, np.repeat(e1, W, axis=0))
    x = np.arange(d, dtype=np.float32)
    e = np.zeros((2, d), np.float32)
    o.step(x, np.concatenate([g1, -g1]), e, None, d=d, k=k, s=s, eta=eta)
    assert np.array_equal(x, np.arange(d, dtype=np.float32))
    # a worker's gradient moves x by eta * g / W on the block only
    W = 4
    g = np.zeros((W, d), np.float32)
    g[2] = 8.0
    x = np.zeros(d, np.float32)
    e = np.zeros((W, d), np.float32)
    o.step(x, g, e, None, d=d, k=k, s=s, eta=eta)
    want = np.where(o.block_mask(d, k, s), -eta * 8.0 / W, 0.0).astype(np.float32)
    assert np.array_equal(x, want)
    assert not e[[0, 1, 3]].any() and np.array_equal(e[2], np.where(o.block_mask(d, k, s), 0, 4.0))


# ---------------------------------------------------------------------------
# fp32 path against the fp64 shadow on the same inputs.
# ---------------------------------------------------------------------------
def pin_f32_tracks_f64(o):
    rng = _rng(31)
    d, W, k, T, eta, mu = 500, 4, 60, 10, 0.1, 0.9
    x32 = (0.05 * rng.standard_normal(d)).astype(np.float32)
    x64 = x32.astype(np.float64)
    e32 = np.zeros((W, d), np.float32); m32 = np.zeros((W, d), np.float32)
    e64 = np.zeros((W, d)); m64 = np.zeros((W, d))
    for t in range(T):
        g = (0.1 * rng.standard_normal((W, d))).astype(np.float32)
        s = o.block_start(5, t, d)
        o.step(x32, g, e32, m32, d=d, k=k, s=s, eta=eta, mu=mu)
        o.step(x64, g.astype(np.float64), e64, m64, d=d, k=k, s=s, eta=eta, mu=mu)
    for a, b, what in ((x32, x64, "x"), (e32, e64, "e"), (m32, m64, "m")):
        scale = float(np.max(np.abs(b)))
        assert float(np.max(np.abs(a - b))) <= 2e-6 * scale, what


# ---------------------------------------------------------------------------
# A view of sampled coordinates follows the whole step at those coordinates.
# ---------------------------------------------------------------------------
def pin_column_view(o):
    rng = _rng(37)
    d, W, k, eta, mu = 120, 3, 25, 0.1, 0.9
    cols = np.array(sorted(rng.choice(d, size=40, replace=False)), dtype=np.int64)[::-1].copy()
    x = rng.standard_normal(d).astype(np.float32)
    e = np.zeros((W, d), np.float32); m = np.zeros((W, d), np.float32)
    xv = x[cols].copy(); ev = e[:, cols].copy(); mv = m[:, cols].copy()
    for t in range(6):
        g = rng.standard_normal((W, d)).astype(np.float32)
        s = [110, 3, 96, 119, 0, 57][t]
        o.step(x, g, e, m, d=d, k=k, s=s, eta=eta, mu=mu)
        o.step(xv, np.ascontiguousarray(g[:, cols]), ev, mv, d=d, k=k, s=s, eta=eta, mu=mu, cols=cols)
    assert np.array_equal(xv, x[cols]) and np.array_equal(ev, e[:, cols]) and np.array_equal(mv, m[:, cols])


# ---------------------------------------------------------------------------
# Philox4x32-10 and the start index.
# ---------------------------------------------------------------------------
_M32 = 0xFFFFFFFF


def philox4x32_bigint(ctr, key, rounds=10):
    """Philox4x32 written on Python integers from the generator's published description."""
    c = [int(v) for v in ctr]
    k = [int(v) for v in key]
    for r in range(rounds):
        p0 = 0xD2511F53 * c[0]
        p1 = 0xCD9E8D57 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k[0], p1 & _M32, (p0 >> 32) ^ c[3] ^ k[1], p0 & _M32]
        k = [(k[0] + 0x9E3779B9) & _M32, (k[1] + 0xBB67AE85) & _M32]
    return tuple(c)


_aten = None


def aten_philox():
    """PyTorch's header-only CPU Philox engine, compiled once per process (g++)."""
    global _aten
    if _aten is None:
        import importlib.util
        spec = importlib.util.find_spec("torch")          # located, not imported: only its headers
        inc = os.path.join(os.path.dirname(spec.origin), "include")
        src = os.path.join(os.path.dirname(os.path.abspath(__file__)), "aten_philox_ref.cpp")
        out = os.path.join(tempfile.mkdtemp(prefix="aten_philox_"), "aten_philox_ref.so")
        subprocess.run(["g++", "-O1", "-std=c++17", "-shared", "-fPIC", "-I", inc, src, "-o", out],
                       check=True)
        lib = ctypes.CDLL(out)
        lib.aten_philox4x32_10.argtypes = [ctypes.c_uint64] * 3 + [ctypes.c_void_p]
        lib.aten_philox4x32_10.restype = None
        lib.aten_philox4x32_10_batch.argtypes = [ctypes.c_int64] + [ctypes.c_void_p] * 4
        lib.aten_philox4x32_10_batch.restype = None
        _aten = lib
    return _aten


def _aten_words(seed, subsequence, offset):
    out = (ctypes.c_uint32 * 4)()
    aten_philox().aten_philox4x32_10(seed, subsequence, offset, out)
    return tuple(int(v) for v in out)


def pin_philox_against_library_engine(o):
    rng = _rng(41)
    cases = [(0, 0, 0), (2 ** 64 - 1, 2 ** 64 - 1, 2 ** 64 - 1), (1, 0, 0), (0, 1, 0), (0, 0, 1),
             (0, 0, 2 ** 32), (0, 2 ** 32, 0), (2 ** 32, 0, 0)]
    cases += [tuple(int(v) for v in rng.integers(0, 2 ** 64, size=3, dtype=np.uint64)) for _ in range(3000)]
    for seed, subseq, offset in cases:
        ctr = (offset & _M32, offset >> 32, subseq & _M32, subseq >> 32)
        key = (seed & _M32, seed >> 32)
        got = o.philox4x32(ctr, key)
        assert got == _aten_words(seed, subseq, offset), (seed, subseq, offset)
        assert got == philox4x32_bigint(ctr, key), (seed, subseq, offset)
    # fewer rounds are a different bijection (guards the round count)
    assert o.philox4x32((1, 2, 3, 4), (5, 6), 7) == philox4x32_bigint((1, 2, 3, 4), (5, 6), 7)
    assert o.philox4x32((1, 2, 3, 4), (5, 6), 7) != o.philox4x32((1, 2, 3, 4), (5, 6), 10)


def philox4x32_numpy(ctr, key, rounds=10):
    """The same bijection on whole arrays: ctr [n, 4] and key [n, 2] as uint64 holding 32-bit words."""
    c0, c1, c2, c3 = (ctr[:, i].astype(np.uint64) for i in range(4))
    k0, k1 = key[:, 0].astype(np.uint64), key[:, 1].astype(np.uint64)
    mask, sh = np.uint64(_M32), np.uint64(32)
    for _ in range(rounds):
        p0 = np.uint64(0xD2511F53) * c0
        p1 = np.uint64(0xCD9E8D57) * c2
        c0, c1, c2, c3 = (p1 >> sh) ^ c1 ^ k0, p1 & mask, (p0 >> sh) ^ c3 ^ k1, p0 & mask
        k0, k1 = (k0 + np.uint64(0x9E3779B9)) & mask, (k1 + np.uint64(0xBB67AE85)) & mask
    return np.stack([c0, c1, c2, c3], axis=1).astype(np.uint32)


def pin_philox_million_pairs(o):
    """2^20 random (counter, key) pairs: the oracle's generator against the library engine and
    against the array statement above, word for word."""
    n = 1 << 20
    rng = _rng(53)
    seeds = rng.integers(0, 2 ** 64, size=n, dtype=np.uint64)
    subs = rng.integers(0, 2 ** 64, size=n, dtype=np.uint64)
    offs = rng.integers(0, 2 ** 64, size=n, dtype=np.uint64)
    seeds[: n // 4] %= 8; offs[: n // 4] %= 100000; subs[: n // 4] = 0x52424753   # what the steps really draw from
    lo, hi = (lambda v: v & np.uint64(_M32)), (lambda v: v >> np.uint64(32))
    ctr = np.ascontiguousarray(np.stack([lo(offs), hi(offs), lo(subs), hi(subs)], axis=1).astype(np.uint32))
    key = np.ascontiguousarray(np.stack([lo(seeds), hi(seeds)], axis=1).astype(np.uint32))
    got = np.empty((n, 4), np.uint32)
    f = o.lib.def_oracle_philox4x32
    c0, k0, g0 = ctr.ctypes.data, key.ctypes.data, got.ctypes.data
    for i in range(n):
        f(c0 + 16 * i, k0 + 8 * i, 10, g0 + 16 * i)
    want = np.empty((n, 4), np.uint32)
    aten_philox().aten_philox4x32_10_batch(n, seeds.ctypes.data, subs.ctypes.data, offs.ctypes.data, want.ctypes.data)
    assert np.array_equal(got, want)
    assert np.array_equal(got, philox4x32_numpy(ctr, key))


def pin_block_start(o):
    rng = _rng(43)
    tag = 0x52424753
    ds = [1, 2, 3, 1000, 855770, 1000000, 11689512, 25557032, 138357544, 2 ** 40 + 7, 2 ** 62]
    for _ in range(400):
        seed, step = (int(v) for v in rng.integers(0, 2 ** 64, size=2, dtype=np.uint64))
        if _ % 3 == 0:
            seed, step = seed % 7, step % 200          # the small seeds and steps real runs use
        for d in ds:
            words = _aten_words(seed, tag, step)
            r = words[0] | (words[1] << 32)
            assert o.block_start(seed, step, d) == (r * d) >> 64, (seed, step, d)
    # uniform over [0, d): chi-square on 64 bins, 64000 consecutive steps
    for d in (1000000, 855770, 138357544):
        starts = np.array([o.block_start(3, t, d) for t in range(64000)])
        assert starts.min() >= 0 and starts.max() < d
        counts = np.bincount(starts * 64 // d, minlength=64)
        chi2 = float(np.sum((counts - 1000.0) ** 2 / 1000.0))
        assert chi2 < 120.0, (d, chi2)                 # 63 dof: P(chi2 > 120) < 2e-5
        assert len(np.unique(starts)) > 60000 or d < 10 ** 6 + 1


# ---------------------------------------------------------------------------
# The distances of Eq. 9: an exact small case, the special cases the text names,
# and the expansion (1/K) sum_k |e_t - l e_k|^2 = (1 - 2l)|e_t|^2 + l^2 (1/K) sum_k |e_k|^2,
# whose minimiser l* = |e_t|^2 / ((1/K) sum_k |e_k|^2) is the paper's lambda*(t).
# ---------------------------------------------------------------------------
def pin_distances(o):
    e = np.array([[2.0, 0.0, -4.0], [0.0, 2.0, 4.0]], np.float32)       # e_t = (1, 1, 0)
    got = o.stats(e, 0.5)
    # (1/2)(20 + 20) = 20; |e_t|^2 = 2; e_t - e_k/2 = (0,1,2), (1,0,-2): (5 + 5)/2 = 5
    assert got == (20.0, 2.0, 5.0), got
    rng = _rng(47)
    for W, n in [(1, 50), (4, 33), (7, 200)]:
        e = rng.standard_normal((W, n)).astype(np.float32)
        a, b, _ = o.stats(e, 0.3)
        assert b <= a * (1 + 1e-12)                                     # |mean|^2 <= mean of squares
        assert abs(o.stats(e, 0.0)[2] - b) <= 1e-12 * a                 # lambda = 0 is plain EF
        if W == 1:
            assert abs(a - b) <= 1e-12 * a and o.stats(e, 1.0)[2] <= 1e-20 * a   # K = 1, lambda = 1 vanishes
        for lam in (0.1, 0.3, 0.8, 1.0):
            c = o.stats(e, lam)[2]
            lam = float(np.float32(lam))                                # the fp32 entry point takes lambda as a float
            assert abs(c - ((1 - 2 * lam) * b + lam * lam * a)) <= 1e-12 * a, (W, n, lam)
        best = b / a                                                    # lambda*(t)
        if best <= 1.0:
            at = o.stats(e, best)[2]
            assert at <= o.stats(e, best * 0.9)[2] and at <= o.stats(e, min(1.0, best * 1.1))[2]
        e64 = e.astype(np.float64)
        assert np.allclose(o.stats(e64, 0.25), o.stats(e, 0.25), rtol=1e-12)


ALL_PINS = [
    ("hand_example", pin_hand_example),
    ("telescoping_identity", pin_telescoping_identity),
    ("full_block_is_momentum_sgd", pin_full_block_is_momentum_sgd),
    ("sparsified_plus_error_is_p", pin_sparsified_plus_error_is_p),
    ("block_shape", pin_block_shape),
    ("additivity", pin_additivity),
    ("expectation_over_starts", pin_expectation_over_starts),
    ("single_worker_lambda_one_is_sgd", pin_single_worker_lambda_one_is_sgd),
    ("scaling_compressor_is_iterate_averaging", pin_scaling_compressor_is_iterate_averaging),
    ("detach_and_output", pin_detach_and_output),
    ("average_over_workers", pin_average_over_workers),
    ("f32_tracks_f64", pin_f32_tracks_f64),
    ("column_view", pin_column_view),
    ("philox_against_library_engine", pin_philox_against_library_engine),
    ("philox_million_pairs", pin_philox_million_pairs),
    ("block_start", pin_block_start),
    ("distances", pin_distances),
]
