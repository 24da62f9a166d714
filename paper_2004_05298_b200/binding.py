"""Thin ctypes binding of libdef_b200.so: the same entry points as include/def.h, taking
torch tensors.  It checks dtype / contiguity / device / shape and passes data pointers;
every step of the method runs inside the library's CUDA kernels.  There is no CPU or
eager fallback: if the library cannot be built or loaded, importing fails loudly."""
import ctypes
import os

import torch

from . import build as _build

DEF_VARIANT_DEF, DEF_VARIANT_DEF_A, DEF_VARIANT_EF = 0, 1, 2
DEF_OK = 0
DEF_ERR_ARG, DEF_ERR_NULL, DEF_ERR_ALIGN, DEF_ERR_ALIAS = -1, -2, -3, -4
DEF_ERR_DEVICE, DEF_ERR_CUDA, DEF_ERR_UNSUPPORTED = -5, -6, -7
DEF_MAX_WORKERS = 64
DEF_KERNEL_STREAM, DEF_KERNEL_BLOCK, DEF_KERNEL_GENERAL = 0, 1, 2
DEF_COMPRESSOR_RBGS, DEF_COMPRESSOR_SCALE = 0, 1

_i64, _u64, _i32, _f32, _ptr = (ctypes.c_int64, ctypes.c_uint64, ctypes.c_int32, ctypes.c_float,
                                ctypes.c_void_p)

# name -> (restype, argtypes): every symbol include/def.h declares
SIGNATURES = {
    "def_create": (_ptr, [_i64, _i32, _i64, _i32, _f32, _f32, _ptr]),
    "def_destroy": (ctypes.c_int, [_ptr]),
    "def_step": (ctypes.c_int, [_ptr, _ptr, _ptr, _ptr, _ptr, _u64, _u64]),
    "def_step_columns": (ctypes.c_int, [_ptr, _i64, _i64, _i64, _ptr, _ptr, _ptr, _ptr, _u64, _u64]),
    "def_step_detach": (ctypes.c_int, [_ptr, _ptr, _ptr, _ptr, _ptr, _ptr, _u64, _u64]),
    "def_step_columns_detach": (ctypes.c_int, [_ptr, _i64, _i64, _i64, _ptr, _ptr, _ptr, _ptr, _ptr, _u64, _u64]),
    "def_step_rows_local": (ctypes.c_int, [_ptr, _ptr, _ptr, _ptr, _ptr, _u64, _u64]),
    "def_step_rows_apply": (ctypes.c_int, [_ptr, _ptr, _ptr, _i32, _u64, _u64]),
    "def_step_rows_local_detach": (ctypes.c_int, [_ptr, _ptr, _ptr, _ptr, _ptr, _ptr, _ptr, _u64, _u64]),
    "def_step_rows_apply_detach": (ctypes.c_int, [_ptr, _ptr, _ptr, _i32, _ptr, _u64, _u64]),
    "def_set_rows_stream": (ctypes.c_int, [_ptr, _ptr]),
    "def_step_host": (ctypes.c_int, [_ptr, _ptr, _ptr, _ptr, _ptr, _u64, _u64]),
    "def_step_columns_host": (ctypes.c_int, [_ptr, _i64, _i64, _i64, _ptr, _ptr, _ptr, _ptr, _u64, _u64]),
    "def_detach": (ctypes.c_int, [_ptr, _i64, _i64, _ptr, _ptr, _ptr]),
    "def_output": (ctypes.c_int, [_ptr, _i64, _i64, _ptr, _ptr, _ptr]),
    "def_stats": (ctypes.c_int, [_ptr, _i64, _i64, _ptr, _ptr]),
    "def_stats_static": (ctypes.c_int, [_ptr, _i64, _i64, _i32, _f32, _ptr, _ptr]),
    "def_set_stream": (ctypes.c_int, [_ptr, _ptr]),
    "def_set_lr": (ctypes.c_int, [_ptr, _f32]),
    "def_set_small_step_bytes": (ctypes.c_int, [_ptr, _i64]),
    "def_set_compressor": (ctypes.c_int, [_ptr, _i32, _f32]),
    "def_set_pair_overlap": (ctypes.c_int, [_ptr, _i32]),
    "def_block_start": (ctypes.c_int, [_ptr, _u64, _u64, _ptr]),
    "def_block_start_device": (ctypes.c_int, [_ptr, _ptr, _ptr, _i64, _ptr, _ptr]),
    "def_launch_count": (ctypes.c_int, [_ptr, _ptr]),
    "def_tile_plan": (ctypes.c_int, [_ptr, _i64, _i64, _u64, _u64, _ptr]),
    "def_set_kernel_timing": (ctypes.c_int, [_ptr, ctypes.c_int]),
    "def_kernel_time": (ctypes.c_int, [_ptr, ctypes.c_int, _ptr, _ptr]),
    "def_last_error": (ctypes.c_char_p, []),
}


class DefError(RuntimeError):
    def __init__(self, code, message):
        super().__init__("def error %d: %s" % (code, message))
        self.code = code


def _load():
    path = _build.build()
    if not os.path.exists(path):
        raise ImportError("libdef_b200.so is missing and could not be built")
    lib = ctypes.CDLL(path)
    for name, (restype, argtypes) in SIGNATURES.items():
        fn = getattr(lib, name)          # AttributeError if the library lacks a declared symbol
        fn.restype = restype
        fn.argtypes = argtypes
    return lib


lib = _load()
LIB_PATH = _build.LIB


def def_last_error():
    return lib.def_last_error().decode()


def _check(rc):
    if rc != DEF_OK:
        raise DefError(rc, def_last_error())


def _dev(t, name, shape=None, dtype=torch.float32, optional=False):
    if t is None:
        if optional:
            return None
        raise DefError(DEF_ERR_NULL, "%s is None" % name)
    if not isinstance(t, torch.Tensor) or t.dtype != dtype or not t.is_contiguous():
        raise TypeError("%s must be a contiguous %s torch tensor" % (name, dtype))
    if not t.is_cuda:
        raise TypeError("%s must live on the GPU" % name)
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError("%s has shape %s, expected %s" % (name, tuple(t.shape), tuple(shape)))
    return t.data_ptr()


def _host(t, name, shape, optional=False):
    if t is None:
        if optional:
            return None
        raise DefError(DEF_ERR_NULL, "%s is None" % name)
    if not isinstance(t, torch.Tensor) or t.dtype != torch.float32 or not t.is_contiguous() or t.is_cuda:
        raise TypeError("%s must be a contiguous float32 CPU tensor" % name)
    if tuple(t.shape) != tuple(shape):
        raise ValueError("%s has shape %s, expected %s" % (name, tuple(t.shape), tuple(shape)))
    return t.data_ptr()


class DefCtx:
    """Owner of one def_ctx handle (freed by def_destroy or when collected)."""

    def __init__(self, handle, d, W, k, variant, lr, momentum):
        self.handle = handle
        self.d, self.W, self.k, self.variant, self.lr, self.momentum = d, W, k, variant, lr, momentum

    def __del__(self):
        if getattr(self, "handle", None):
            lib.def_destroy(self.handle)
            self.handle = None


def def_create(d, W, k, variant, lr, momentum, coeffs=None):
    arr = None
    if coeffs is not None:
        arr = (ctypes.c_float * 2)(float(coeffs[0]), float(coeffs[1]))
    handle = lib.def_create(int(d), int(W), int(k), int(variant), float(lr), float(momentum), arr)
    if not handle:
        msg = def_last_error()
        raise DefError(DEF_ERR_UNSUPPORTED if "weight decay" in msg else DEF_ERR_ARG, msg)
    return DefCtx(handle, int(d), int(W), int(k), int(variant), float(lr), float(momentum))


def def_destroy(ctx):
    if ctx.handle:
        rc = lib.def_destroy(ctx.handle)
        ctx.handle = None
        _check(rc)


def def_set_stream(ctx, stream):
    """stream: a torch.cuda.Stream, a raw cudaStream_t integer, or None (legacy default)."""
    raw = stream.cuda_stream if isinstance(stream, torch.cuda.Stream) else (stream or 0)
    _check(lib.def_set_stream(ctx.handle, ctypes.c_void_p(raw)))


def def_set_lr(ctx, lr):
    _check(lib.def_set_lr(ctx.handle, float(lr)))
    ctx.lr = float(lr)


def def_step(ctx, params, grads, errors, mom, step, seed):
    d, W = ctx.d, ctx.W
    _check(lib.def_step(ctx.handle, _dev(params, "params", (d,)), _dev(grads, "grads", (W, d)),
                        _dev(errors, "errors", (W, d)), _dev(mom, "mom", (W, d), optional=True),
                        int(step), int(seed)))


def def_step_columns(ctx, j0, n, ld, params, grads, errors, mom, step, seed):
    """params: [n]; grads / errors / mom: [W, ld] (a rank's local column shard)."""
    W = ctx.W
    _check(lib.def_step_columns(ctx.handle, int(j0), int(n), int(ld), _dev(params, "params", (n,)),
                                _dev(grads, "grads", (W, ld)), _dev(errors, "errors", (W, ld)),
                                _dev(mom, "mom", (W, ld), optional=True), int(step), int(seed)))


def def_step_host(ctx, params, grads, errors, mom, step, seed):
    d, W = ctx.d, ctx.W
    _check(lib.def_step_host(ctx.handle, _host(params, "params", (d,)), _host(grads, "grads", (W, d)),
                             _host(errors, "errors", (W, d)), _host(mom, "mom", (W, d), optional=True),
                             int(step), int(seed)))


def def_step_columns_host(ctx, j0, n, ld, params, grads, errors, mom, step, seed):
    W = ctx.W
    _check(lib.def_step_columns_host(ctx.handle, int(j0), int(n), int(ld), _host(params, "params", (n,)),
                                     _host(grads, "grads", (W, ld)), _host(errors, "errors", (W, ld)),
                                     _host(mom, "mom", (W, ld), optional=True), int(step), int(seed)))


def def_block_start(ctx, step, seed):
    out = ctypes.c_int64(-1)
    _check(lib.def_block_start(ctx.handle, int(step), int(seed), ctypes.byref(out)))
    return int(out.value)


def def_block_start_device(seeds, steps, ds, starts_out, stream=None):
    """seeds, steps: uint64 bit patterns held in int64 CUDA tensors; ds, starts_out: int64."""
    n = seeds.numel()
    raw = stream.cuda_stream if isinstance(stream, torch.cuda.Stream) else (stream or 0)
    _check(lib.def_block_start_device(_dev(seeds, "seeds", (n,), torch.int64),
                                      _dev(steps, "steps", (n,), torch.int64),
                                      _dev(ds, "ds", (n,), torch.int64), n,
                                      _dev(starts_out, "starts_out", (n,), torch.int64),
                                      ctypes.c_void_p(raw)))


def def_tile_plan(ctx, j0, n, step, seed):
    """(first tile of run A, its tiles, tiles of run B from tile 0, tiles left to the stream kernel)."""
    out = (ctypes.c_int64 * 4)()
    _check(lib.def_tile_plan(ctx.handle, int(j0), int(n), int(step), int(seed), out))
    return tuple(int(v) for v in out)


def def_launch_count(ctx):
    out = ctypes.c_int64(0)
    _check(lib.def_launch_count(ctx.handle, ctypes.byref(out)))
    return int(out.value)


def def_set_kernel_timing(ctx, enable):
    _check(lib.def_set_kernel_timing(ctx.handle, 1 if enable else 0))


def def_kernel_time(ctx, kernel):
    """(total device milliseconds, launches) of one kernel kind since def_create."""
    ms, n = ctypes.c_double(0.0), ctypes.c_int64(0)
    _check(lib.def_kernel_time(ctx.handle, int(kernel), ctypes.byref(ms), ctypes.byref(n)))
    return float(ms.value), int(n.value)


def def_detach(ctx, params, errors, detached_out, n=None, ld=None):
    """detached_out[w] = params - lambda * errors[w]; whole model unless n / ld name a column view."""
    n = ctx.d if n is None else int(n)
    ld = n if ld is None else int(ld)
    _check(lib.def_detach(ctx.handle, n, ld, _dev(params, "params", (n,)), _dev(errors, "errors", (ctx.W, ld)),
                          _dev(detached_out, "detached_out", (ctx.W, ld))))


def def_output(ctx, params, errors, model_out, n=None, ld=None):
    """The model Algorithm 1 returns: y_T for DEF, x_T for DEF-A and EF."""
    n = ctx.d if n is None else int(n)
    ld = n if ld is None else int(ld)
    _check(lib.def_output(ctx.handle, n, ld, _dev(params, "params", (n,)),
                          _dev(errors, "errors", (ctx.W, ld), optional=True), _dev(model_out, "model_out", (n,))))


def def_stats(ctx, errors, stats_out, n=None, ld=None):
    """stats_out: 3 float64 on the GPU (see include/def.h)."""
    n = ctx.d if n is None else int(n)
    ld = n if ld is None else int(ld)
    _check(lib.def_stats(ctx.handle, n, ld, _dev(errors, "errors", (ctx.W, ld)),
                         _dev(stats_out, "stats_out", (3,), torch.float64)))


DEF_STATS_STATIC_SLOTS = 2048
DEF_STATS_STATIC_MAX_N = 1 << 31


def def_stats_static(errors, lam, stats_out, n=None, ld=None, stream=None):
    """def_stats without any allocation and without a context: the scratch is a fixed array in
    the library's device image (see include/def.h for who needs this and for its rules).
    errors: [W, ld] float32 on the GPU; stats_out: 3 float64 on the GPU."""
    W = errors.shape[0]
    ld = errors.shape[1] if ld is None else int(ld)
    n = ld if n is None else int(n)
    raw = stream.cuda_stream if isinstance(stream, torch.cuda.Stream) else (stream or 0)
    _check(lib.def_stats_static(_dev(errors, "errors", (W, ld)), n, ld, int(W), float(lam),
                                _dev(stats_out, "stats_out", (3,), torch.float64), ctypes.c_void_p(raw)))


def def_step_detach(ctx, params, grads, errors, mom, detached_out, step, seed):
    d, W = ctx.d, ctx.W
    _check(lib.def_step_detach(ctx.handle, _dev(params, "params", (d,)), _dev(grads, "grads", (W, d)),
                               _dev(errors, "errors", (W, d)), _dev(mom, "mom", (W, d), optional=True),
                               _dev(detached_out, "detached_out", (W, d)), int(step), int(seed)))


def def_step_columns_detach(ctx, j0, n, ld, params, grads, errors, mom, detached_out, step, seed):
    W = ctx.W
    _check(lib.def_step_columns_detach(ctx.handle, int(j0), int(n), int(ld), _dev(params, "params", (n,)),
                                       _dev(grads, "grads", (W, ld)), _dev(errors, "errors", (W, ld)),
                                       _dev(mom, "mom", (W, ld), optional=True),
                                       _dev(detached_out, "detached_out", (W, ld)), int(step), int(seed)))


def def_set_small_step_bytes(ctx, nbytes):
    _check(lib.def_set_small_step_bytes(ctx.handle, int(nbytes)))


DEF_OVERLAP_AUTO, DEF_OVERLAP_NEVER, DEF_OVERLAP_ALWAYS = 0, 1, 2


def def_set_pair_overlap(ctx, mode):
    _check(lib.def_set_pair_overlap(ctx.handle, int(mode)))


def def_set_compressor(ctx, compressor, delta=0.0):
    _check(lib.def_set_compressor(ctx.handle, int(compressor), float(delta)))


def def_step_rows_local(ctx, grads, errors, mom, block_sum_out, step, seed):
    d, W = ctx.d, ctx.W
    _check(lib.def_step_rows_local(ctx.handle, _dev(grads, "grads", (W, d)), _dev(errors, "errors", (W, d)),
                                   _dev(mom, "mom", (W, d), optional=True),
                                   _dev(block_sum_out, "block_sum_out", (ctx.k,)), int(step), int(seed)))


def def_step_rows_apply(ctx, params, block_sum, W_total, step, seed):
    _check(lib.def_step_rows_apply(ctx.handle, _dev(params, "params", (ctx.d,)),
                                   _dev(block_sum, "block_sum", (ctx.k,)), int(W_total), int(step), int(seed)))


def def_step_rows_local_detach(ctx, params, grads, errors, mom, block_sum_out, detached_out, step, seed):
    d, W = ctx.d, ctx.W
    _check(lib.def_step_rows_local_detach(ctx.handle, _dev(params, "params", (d,)), _dev(grads, "grads", (W, d)),
                                          _dev(errors, "errors", (W, d)), _dev(mom, "mom", (W, d), optional=True),
                                          _dev(block_sum_out, "block_sum_out", (ctx.k,)),
                                          _dev(detached_out, "detached_out", (W, d)), int(step), int(seed)))


def def_step_rows_apply_detach(ctx, params, block_sum, W_total, detached_out, step, seed):
    _check(lib.def_step_rows_apply_detach(ctx.handle, _dev(params, "params", (ctx.d,)),
                                          _dev(block_sum, "block_sum", (ctx.k,)), int(W_total),
                                          _dev(detached_out, "detached_out", (ctx.W, ctx.d)), int(step), int(seed)))


def def_set_rows_stream(ctx, stream):
    """Side stream of the row-sharded step (a torch.cuda.Stream, or None to switch it off): the
    block kernel, the all-reduce and the update run there, beside the streaming kernel."""
    raw = stream.cuda_stream if isinstance(stream, torch.cuda.Stream) else (stream or 0)
    _check(lib.def_set_rows_stream(ctx.handle, ctypes.c_void_p(raw)))
    ctx.rows_stream = stream if isinstance(stream, torch.cuda.Stream) else None


def def_step_rows(ctx, params, grads, errors, mom, block_sum, step, seed, group=None, detached_out=None):
    """One row-sharded step: local half, all-reduce of the k block sums over `group` (NCCL through
    torch.distributed), apply.  W_total = local W times the group size.  After def_set_rows_stream
    the all-reduce is issued on that side stream, where the library has put the block kernel and
    puts the update, so that it overlaps the streaming kernel on the context's stream."""
    import torch.distributed as dist
    if detached_out is None:
        def_step_rows_local(ctx, grads, errors, mom, block_sum, step, seed)
    else:
        def_step_rows_local_detach(ctx, params, grads, errors, mom, block_sum, detached_out, step, seed)
    side = getattr(ctx, "rows_stream", None)
    if side is not None:
        with torch.cuda.stream(side):
            dist.all_reduce(block_sum, op=dist.ReduceOp.SUM, group=group)
    else:
        dist.all_reduce(block_sum, op=dist.ReduceOp.SUM, group=group)
    W_total = ctx.W * dist.get_world_size(group)
    if detached_out is None:
        def_step_rows_apply(ctx, params, block_sum, W_total, step, seed)
    else:
        def_step_rows_apply_detach(ctx, params, block_sum, W_total, detached_out, step, seed)
