"""ctypes front end of oracle/libdef_oracle.so (numpy arrays in, numpy arrays out).

Test infrastructure only: the tests, the smoke check and the benchmark's CPU
baseline call this; the CUDA library never does.  All the arithmetic is in
def_oracle.c; this file only marshals arguments.
"""
import ctypes
import numpy as np

from . import build as _build

COMPRESSOR_RBGS = 0
COMPRESSOR_SCALE = 1
VARIANT_DEF = 0
VARIANT_DEF_A = 1
VARIANT_EF = 2

__all__ = [
    "COMPRESSOR_RBGS", "COMPRESSOR_SCALE", "VARIANT_DEF", "VARIANT_DEF_A", "VARIANT_EF",
    "Oracle", "default", "all_cores", "philox4x32", "block_start", "in_block", "block_mask", "compress",
    "step", "detach", "output", "stats",
]

_i64 = ctypes.c_int64
_u64 = ctypes.c_uint64
_ptr = ctypes.c_void_p


def _real(dtype):
    dtype = np.dtype(dtype)
    if dtype == np.float32:
        return "f32", ctypes.c_float
    if dtype == np.float64:
        return "f64", ctypes.c_double
    raise TypeError("the oracle computes in float32 or float64, got %s" % dtype)


def _p(a):
    return None if a is None else a.ctypes.data_as(_ptr)


def _check(a, dtype, shape, name, writable=False):
    if not isinstance(a, np.ndarray) or a.dtype != dtype or not a.flags.c_contiguous:
        raise TypeError("%s must be a C-contiguous numpy array of %s" % (name, dtype))
    if tuple(a.shape) != tuple(shape):
        raise ValueError("%s has shape %s, expected %s" % (name, a.shape, tuple(shape)))
    if writable and not a.flags.writeable:
        raise ValueError("%s must be writable" % name)


class Oracle:
    """One loaded copy of the oracle library (the default one, or a variant a test built)."""

    def __init__(self, lib_path=None):
        path = lib_path or _build.build()
        self.lib = lib = ctypes.CDLL(path)
        lib.def_oracle_philox4x32.argtypes = [_ptr, _ptr, ctypes.c_int, _ptr]
        lib.def_oracle_philox4x32.restype = None
        lib.def_oracle_block_start.argtypes = [_u64, _u64, _i64]
        lib.def_oracle_block_start.restype = _i64
        lib.def_oracle_in_block.argtypes = [_i64, _i64, _i64, _i64]
        lib.def_oracle_in_block.restype = ctypes.c_int
        lib.def_oracle_block_mask.argtypes = [_i64, _i64, _i64, _i64, _ptr, _ptr]
        lib.def_oracle_block_mask.restype = None
        lib.def_oracle_threads.argtypes = []
        lib.def_oracle_threads.restype = ctypes.c_int
        for sfx, real in (("f32", ctypes.c_float), ("f64", ctypes.c_double)):
            f = getattr(lib, "def_oracle_compress_" + sfx)
            f.argtypes = [ctypes.c_int, _i64, _i64, _i64, real, _i64, _ptr, _ptr, _ptr]
            f.restype = None
            f = getattr(lib, "def_oracle_step_" + sfx)
            f.argtypes = [ctypes.c_int, _i64, _i64, _i64, _i64, real, real, real, _i64, _ptr,
                          _ptr, _ptr, _ptr, _ptr]
            f.restype = ctypes.c_int
            f = getattr(lib, "def_oracle_detach_" + sfx)
            f.argtypes = [real, _i64, _ptr, _ptr, _ptr]
            f.restype = None
            f = getattr(lib, "def_oracle_output_" + sfx)
            f.argtypes = [ctypes.c_int, _i64, _i64, _ptr, _ptr, _ptr]
            f.restype = None
            f = getattr(lib, "def_oracle_stats_" + sfx)
            f.argtypes = [real, _i64, _i64, _ptr, _ptr]
            f.restype = None

    def threads(self):
        """Host threads the loops over coordinates run on (1 unless this is the all-cores build)."""
        return int(self.lib.def_oracle_threads())

    # ---- block start ------------------------------------------------------
    def philox4x32(self, ctr, key, rounds=10):
        c = (ctypes.c_uint32 * 4)(*[int(v) & 0xFFFFFFFF for v in ctr])
        k = (ctypes.c_uint32 * 2)(*[int(v) & 0xFFFFFFFF for v in key])
        out = (ctypes.c_uint32 * 4)()
        self.lib.def_oracle_philox4x32(c, k, int(rounds), out)
        return tuple(int(v) for v in out)

    def block_start(self, seed, step, d):
        return int(self.lib.def_oracle_block_start(int(seed), int(step), int(d)))

    def in_block(self, j, s, k, d):
        return bool(self.lib.def_oracle_in_block(int(j), int(s), int(k), int(d)))

    def _cols(self, cols, n):
        if cols is None:
            return None
        cols = np.ascontiguousarray(cols, dtype=np.int64)
        if cols.shape != (n,):
            raise ValueError("cols has shape %s, expected (%d,)" % (cols.shape, n))
        return cols

    def block_mask(self, d, k, s, cols=None):
        n = int(d) if cols is None else len(cols)
        cols = self._cols(cols, n)
        mask = np.empty(n, dtype=np.uint8)
        self.lib.def_oracle_block_mask(int(d), int(k), int(s), n, _p(cols), _p(mask))
        return mask.astype(bool)

    # ---- the method -------------------------------------------------------
    def compress(self, v, d, k, s, cols=None, compressor=COMPRESSOR_RBGS, delta=0.0):
        sfx, _ = _real(v.dtype)
        n = v.shape[0]
        _check(v, v.dtype, (n,), "v")
        if cols is None and compressor == COMPRESSOR_RBGS and n != d:
            raise ValueError("a whole vector has n == d; pass cols for a view")
        cols = self._cols(cols, n)
        out = np.empty_like(v)
        getattr(self.lib, "def_oracle_compress_" + sfx)(
            int(compressor), int(d), int(k), int(s), float(delta), n, _p(cols), _p(v), _p(out))
        return out

    def step(self, x, g, e, m, *, d, k, s, eta, mu=0.0, cols=None,
             compressor=COMPRESSOR_RBGS, delta=0.0):
        """One iteration in place on x[n], e[W,n], m[W,n] (m may be None); g[W,n] is read."""
        sfx, _ = _real(x.dtype)
        W, n = g.shape
        _check(x, x.dtype, (n,), "x", writable=True)
        _check(g, x.dtype, (W, n), "g")
        _check(e, x.dtype, (W, n), "e", writable=True)
        if m is not None:
            _check(m, x.dtype, (W, n), "m", writable=True)
        if cols is None and n != d:
            raise ValueError("a whole step has n == d; pass cols for a view")
        if not (1 <= k <= d) or not (0 <= s < d) or W < 1:
            raise ValueError("need 1 <= k <= d, 0 <= s < d, W >= 1")
        cols = self._cols(cols, n)
        rc = getattr(self.lib, "def_oracle_step_" + sfx)(
            int(compressor), int(d), int(W), int(k), int(s), float(delta), float(eta), float(mu),
            int(n), _p(cols), _p(x), _p(g), _p(e), _p(m))
        if rc != 0:
            raise MemoryError("oracle step could not allocate its temporaries")

    def detach(self, x, e_w, lam):
        sfx, _ = _real(x.dtype)
        n = x.shape[0]
        _check(x, x.dtype, (n,), "x")
        _check(e_w, x.dtype, (n,), "e_w")
        out = np.empty_like(x)
        getattr(self.lib, "def_oracle_detach_" + sfx)(float(lam), n, _p(x), _p(e_w), _p(out))
        return out

    def output(self, variant, x, e):
        sfx, _ = _real(x.dtype)
        W, n = e.shape
        _check(x, x.dtype, (n,), "x")
        _check(e, x.dtype, (W, n), "e")
        out = np.empty_like(x)
        getattr(self.lib, "def_oracle_output_" + sfx)(int(variant), int(W), n, _p(x), _p(e),
                                                      _p(out))
        return out

    def stats(self, e, lam):
        """(mean_k |e_k|^2, |mean_k e_k|^2, mean_k |mean e - lam e_k|^2) as Python floats."""
        sfx, _ = _real(e.dtype)
        W, n = e.shape
        _check(e, e.dtype, (W, n), "e")
        out = (ctypes.c_double * 3)()
        getattr(self.lib, "def_oracle_stats_" + sfx)(float(lam), int(W), int(n), _p(e), out)
        return tuple(float(v) for v in out)


_default = None


def default():
    """The oracle built from the committed source (compiled on first use)."""
    global _default
    if _default is None:
        _default = Oracle()
    return _default


_all_cores = None


def all_cores():
    """The same source built with OpenMP: loops over coordinates run on every host core, with
    the operations on each coordinate and their order unchanged (same bits as default())."""
    global _all_cores
    if _all_cores is None:
        _all_cores = Oracle(_build.build_all_cores())
    return _all_cores


def philox4x32(ctr, key, rounds=10):
    return default().philox4x32(ctr, key, rounds)


def block_start(seed, step, d):
    return default().block_start(seed, step, d)


def in_block(j, s, k, d):
    return default().in_block(j, s, k, d)


def block_mask(d, k, s, cols=None):
    return default().block_mask(d, k, s, cols)


def compress(v, d, k, s, cols=None, compressor=COMPRESSOR_RBGS, delta=0.0):
    return default().compress(v, d, k, s, cols, compressor, delta)


def step(x, g, e, m, **kw):
    return default().step(x, g, e, m, **kw)


def detach(x, e_w, lam):
    return default().detach(x, e_w, lam)


def output(variant, x, e):
    return default().output(variant, x, e)


def stats(e, lam):
    return default().stats(e, lam)
