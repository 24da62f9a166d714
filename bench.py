#!/usr/bin/env python
"""Benchmark of the DEF / DEF-A / EF step on B200: gradient elements per second.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A step is one pass of the whole hot path (block start, momentum, error feedback,
sparsification, cross-worker average, update: two kernels that run side by side) over one batch
of synthetic gradients.  The timed workload is the VGG-16-sized one (d = 138,357,544,
W = 16, k = d/32, DEF, momentum 0.9): its 35 GB of state and gradients are far larger
than the L2, so no flush is needed between iterations.  Prints ONE JSON line on rank 0.

With N > 1 (launched by torch.distributed.run) the WORKERS are cut across the ranks, as in the
paper's own deployment: every rank holds W = 16 workers' rows of the full d-dimensional model and
a replica of x, so there are K = 16 N workers; a step is the local half (momentum, error feedback,
new error, the local workers' block sums), one NCCL all-reduce of the k block sums -- issued on a
side stream so that it overlaps the streaming kernel -- and the update.  Per-GPU work is fixed
("weak" scaling); the value is the elements all ranks processed divided by the slowest rank's
device time.  --sharding columns gives every rank a d-column shard of an N*d-dimensional model
instead (no exchange at all: the step is separate per coordinate).

--impl reference times the CPU oracle (plain C; the same source built with OpenMP for all host
cores, and the single-threaded build beside it) on a bounded sample of the same workload; it is a
deliberately slow program, reported as a baseline only.
"""
import argparse
import hashlib
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "DEF step gradient elements/s (W*d per step)"
UNIT = "elements/s"
FALLBACK_HBM_GBS = 6650.0

# DRAM traffic of one def_step_stream_kernel launch from ncu captures
# (dram__bytes_read.sum + dram__bytes_write.sum), as bytes per gradient element, per workload:
# config 5 from a one-pass capture of these two counters on the timed launch configuration itself,
# config 3 from the full-set capture.  Reported only for those workloads and only while the kernel
# source is the file the captures were taken on (hash below; see profiles/).
NCU_TRAFFIC_BYTES_PER_ELEMENT = {5: 19.97, 3: 19.43}
NCU_TRAFFIC_KERNEL_SHA256 = "7bd792a82d86626f0d3d101197064db994aa7a2dfb6136afe7df4003cd5af0ec"


def _measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def _kernel_hash():
    h = hashlib.sha256()
    with open(os.path.join(ROOT, "paper_2004_05298_b200", "csrc", "def_kernels.cuh"), "rb") as fh:
        h.update(fh.read())
    return h.hexdigest()


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while a region runs."""

    def __init__(self, device_index, period=0.02):
        super().__init__(daemon=True)
        self.period = period
        self.samples = []
        self.reasons = set()
        self.sm_max = None
        self.stop_flag = threading.Event()
        self.ok = False
        try:
            import pynvml
            import torch
            self.nv = pynvml
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            self.handle = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            self.sm_max = int(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception as exc:  # no NVML: report that, never guess
            self.error = repr(exc)

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            nv.nvmlClocksEventReasonHwSlowdown: "hw_slowdown",
            nv.nvmlClocksEventReasonHwThermalSlowdown: "hw_thermal_slowdown",
            nv.nvmlClocksEventReasonSwThermalSlowdown: "sw_thermal_slowdown",
            nv.nvmlClocksEventReasonSwPowerCap: "sw_power_cap",
            nv.nvmlClocksEventReasonHwPowerBrakeSlowdown: "hw_power_brake_slowdown",
            nv.nvmlClocksEventReasonApplicationsClocksSetting: "applications_clocks_setting",
        }
        while not self.stop_flag.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM)))
                bits = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle))
                for bit, name in names.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self.stop_flag.wait(self.period)

    def finish(self):
        self.stop_flag.set()
        if self.is_alive():
            self.join(timeout=2.0)
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": [], "samples": 0,
                    "note": "NVML unavailable" if not self.ok else "no sample fell in the region"}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.sm_max,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def _dist_setup(n_gpus):
    import torch
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        return dist, world, rank, local
    if n_gpus > 1:
        raise SystemExit("--gpus %d needs: python -m torch.distributed.run --nproc-per-node %d bench.py --gpus %d ..."
                         % (n_gpus, n_gpus, n_gpus))
    torch.cuda.set_device(0)
    return None, 1, 0, 0


def _barrier(dist):
    import torch
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()


def _max_over_ranks(dist, value):
    import torch
    if dist is None:
        return value
    t = torch.tensor([value], dtype=torch.float64, device="cuda")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def time_steps(B, ctx, shard, tensors, steps, warmup, seed, dist=None, flush=None, sample_clocks=None, step_fn=None,
               per_step_events=True):
    """Device time of `steps` steps, from CUDA events on the stream the steps are enqueued on.
    Without `flush`: an event before the first step and one after every step, launches back to
    back (the total is first event to last); with per_step_events off, one pair around the whole
    loop (an event between steps of a few microseconds would cost as much as the step).  With
    `flush` (a buffer larger than the L2 that is rewritten between iterations): one event pair per
    step, summed.  Returns (total ms, max over ranks; launches; this rank's per-step ms or None)."""
    import torch
    j0, n, ld = shard
    x, g, e, m = tensors
    if step_fn is None:
        def step_fn(t):
            B.def_step_columns(ctx, j0, n, ld, x, g, e, m, t, seed)
    for t in range(warmup):
        if flush is not None:
            flush.add_(1.0)                                # warm up the way the timed steps run
        step_fn(t)
    _barrier(dist)
    launches0 = B.def_launch_count(ctx)
    if sample_clocks is not None:
        sample_clocks.start()
    if flush is None and not per_step_events:
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record()
        for t in range(steps):
            step_fn(warmup + t)
        end.record()
        torch.cuda.synchronize()
        ms = start.elapsed_time(end)
        per_step = None
    elif flush is None:
        marks = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        marks[0].record()
        for t in range(steps):
            step_fn(warmup + t)
            marks[t + 1].record()
        torch.cuda.synchronize()
        ms = marks[0].elapsed_time(marks[-1])
        per_step = [marks[t].elapsed_time(marks[t + 1]) for t in range(steps)]
    else:
        pairs = []
        for t in range(steps):
            flush.add_(1.0)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            step_fn(warmup + t)
            b.record()
            pairs.append((a, b))
        torch.cuda.synchronize()
        per_step = [a.elapsed_time(b) for a, b in pairs]
        ms = sum(per_step)
    _barrier(dist)
    launches = B.def_launch_count(ctx) - launches0
    return _max_over_ranks(dist, ms), launches, per_step


def step_spread(per_step):
    """Median and minimum of the per-step device times (this rank's)."""
    if not per_step:
        return {}
    return {"ms_per_step_median": statistics.median(per_step), "ms_per_step_min": min(per_step)}


TILE = 1024   # coordinates per tile of the two step kernels (256 threads x 4)


def touched_columns(d, k, s, j0, n):
    """Local coordinates that lie in tiles touching the block {(s+i) mod d}: the block kernel's share."""
    runs = [(s, min(s + k, d))]
    if s + k > d:
        runs.append((0, s + k - d))
    tiles = set()
    for a, b in runs:
        a, b = max(a, j0), min(b, j0 + n)
        if b > a:
            tiles.update(range((a - j0) // TILE, (b - 1 - j0) // TILE + 1))
    return sum(min(TILE, n - t * TILE) for t in tiles)


def profile_kernels(B, ctx, shard, tensors, steps, first_step, seed, per_el, k_share, flush=None, step_fn=None):
    """Per-kernel device time over `steps` more steps (each launch bracketed by events inside the
    library, on the stream it is launched on, and waited for), with the algorithmic bytes each
    kernel had to move."""
    j0, n, ld = shard
    x, g, e, m = tensors
    W = ctx.W
    if step_fn is None:
        def step_fn(t):
            B.def_step_columns(ctx, j0, n, ld, x, g, e, m, t, seed)
    before = {kind: B.def_kernel_time(ctx, kind) for kind in (B.DEF_KERNEL_STREAM, B.DEF_KERNEL_BLOCK, B.DEF_KERNEL_GENERAL)}
    B.def_set_kernel_timing(ctx, True)
    bytes_stream = bytes_block = bytes_general = 0
    for t in range(steps):
        if flush is not None:
            flush.add_(1.0)
        step = first_step + t
        step_fn(step)
        cols = touched_columns(ctx.d, ctx.k, B.def_block_start(ctx, step, seed), j0, n)
        bytes_block += per_el * W * cols + 8 * k_share
        bytes_stream += per_el * W * (n - cols)
        bytes_general += per_el * W * n + 8 * k_share
    B.def_set_kernel_timing(ctx, False)
    out = []
    for kind, name, nbytes in ((B.DEF_KERNEL_STREAM, "def_step_stream_kernel", bytes_stream),
                               (B.DEF_KERNEL_BLOCK, "def_step_block_kernel", bytes_block),
                               (B.DEF_KERNEL_GENERAL, "def_step_kernel", bytes_general)):
        ms, cnt = B.def_kernel_time(ctx, kind)
        ms, cnt = ms - before[kind][0], cnt - before[kind][1]
        if cnt:
            out.append({"kernel": name, "launches": cnt, "ms_per_launch": ms / cnt,
                        "algorithmic_bytes_per_launch": nbytes / cnt if nbytes else None,
                        "GB/s": (nbytes / (ms * 1e-3) / 1e9) if nbytes else None})
    return out


def bench_rows(B, WL, wl, steps, warmup, dist, world, rank, sampler=None, side_stream=True, detach=False,
               profile=False):
    """Workers cut across ranks (the paper's deployment): every rank holds W rows of the full model and
    a replica of x; one step = local half, NCCL all-reduce of the k block sums (on a side stream,
    beside the streaming kernel, unless side_stream is off), apply.  With `detach` the step also
    writes the local workers' next detach points (24 instead of 20 bytes per gradient element)."""
    import torch
    dev = torch.device("cuda")
    ctx = B.def_create(wl.d, wl.W, wl.k, wl.variant, wl.lr, wl.momentum, (wl.lam, 0.0))
    side = torch.cuda.Stream() if side_stream else None
    if side is not None:
        B.def_set_rows_stream(ctx, side)
    x = WL.initial_params(wl, dev)
    e, m = WL.zeros_state(wl, dev)
    g = WL.gradients(wl, rank, dev)
    z = torch.empty(wl.W, wl.d, dtype=torch.float32, device=dev) if detach else None
    block = torch.zeros(wl.k, dtype=torch.float32, device=dev)

    def step_fn(t):
        B.def_step_rows(ctx, x, g, e, m, block, t, wl.rbgs_seed, detached_out=z)

    ms, launches, per_step = time_steps(B, ctx, (0, wl.d, wl.d), (x, g, e, m), steps, warmup, wl.rbgs_seed, dist, None,
                                        sampler, step_fn)
    per_el = 24 if detach else 20
    # local rows, the k block sums written, read and applied to x, and (detach) x read once
    alg_bytes = per_el * wl.W * wl.d + 16 * wl.k + (4 * wl.d if detach else 0)
    kernels = None
    if profile:
        kernels = profile_kernels(B, ctx, (0, wl.d, wl.d), (x, g, e, m), min(steps, 5), warmup + steps, wl.rbgs_seed,
                                  per_el, 0.5 * wl.k, None, step_fn)
    if side is not None:
        B.def_set_rows_stream(ctx, None)
    B.def_destroy(ctx)
    del x, g, e, m, z
    torch.cuda.empty_cache()
    return ms, launches, world * wl.W * wl.d, alg_bytes, kernels, per_step


def bench_rows_e2e(B, WL, wl, steps, warmup, dist, world, rank):
    """The row-sharded step with the step's input in host memory: every step copies the local
    workers' gradients [W, d] in from pinned host memory, runs def_step_rows, and copies the k
    updated block coordinates' sums out (what a training loop would log or checkpoint)."""
    import torch
    dev = torch.device("cuda")
    ctx = B.def_create(wl.d, wl.W, wl.k, wl.variant, wl.lr, wl.momentum, (wl.lam, 0.0))
    side = torch.cuda.Stream()
    B.def_set_rows_stream(ctx, side)
    x = WL.initial_params(wl, dev)
    e, m = WL.zeros_state(wl, dev)
    g = WL.gradients(wl, rank, dev)
    g_host = torch.empty(wl.W, wl.d, dtype=torch.float32, pin_memory=True)
    g_host.copy_(g)
    block = torch.zeros(wl.k, dtype=torch.float32, device=dev)
    block_host = torch.empty(wl.k, dtype=torch.float32, pin_memory=True)

    def step_fn(t):
        g.copy_(g_host, non_blocking=True)
        B.def_step_rows(ctx, x, g, e, m, block, t, wl.rbgs_seed)
        block_host.copy_(block, non_blocking=True)

    for t in range(warmup):
        step_fn(t)
    _barrier(dist)
    t0 = time.perf_counter()
    for t in range(steps):
        step_fn(warmup + t)
    torch.cuda.synchronize()
    sec = time.perf_counter() - t0
    _barrier(dist)
    sec = _max_over_ranks(dist, sec)
    B.def_set_rows_stream(ctx, None)
    B.def_destroy(ctx)
    del x, g, e, m
    torch.cuda.empty_cache()
    return {"value": world * wl.W * wl.d * steps / sec, "unit": UNIT,
            "h2d_bytes_per_step": 4 * wl.W * wl.d, "d2h_bytes_per_step": 4 * wl.k,
            "steps": steps, "ms_per_step": 1e3 * sec / steps,
            "api": "binding.def_step_rows; gradients copied in from pinned host memory and the k block sums copied "
                   "out every step (errors, momentum and the model stay on the GPU)"}


def bench_workload(B, WL, wl, steps, warmup, dist, world, rank, sampler=None, flush=None, profile=False):
    """Allocate a rank's column shard of the workload (the whole model on one rank), run, return
    (ms, launches, elements per step over all ranks, algorithmic bytes per step on this rank,
    per-kernel profile or None, this rank's per-step ms)."""
    import torch
    dev = torch.device("cuda")
    d_global = wl.d * world
    k_global = max(1, d_global // wl.ratio)
    j0, n = rank * wl.d, wl.d
    ctx = B.def_create(d_global, wl.W, k_global, wl.variant, wl.lr, wl.momentum, (wl.lam, 0.0))
    x = WL.initial_params(wl, dev)
    e, m = WL.zeros_state(wl, dev)
    if wl.momentum == 0.0:
        m = None
    col_sigma = WL.column_sigma(wl, dev) if wl.grad == "per_tensor" else None
    g = WL.gradients(wl, rank, dev, col_sigma=col_sigma)   # one gradient buffer, reused: values do not steer the kernel
    ms, launches, per_step = time_steps(B, ctx, (j0, n, n), (x, g, e, m), steps, warmup, wl.rbgs_seed, dist, flush, sampler,
                                        per_step_events=wl.algorithmic_bytes_per_step() >= 1e9)
    per_el = 20 if wl.momentum != 0.0 else 12
    alg_bytes = per_el * wl.W * n + 8 * k_global / world
    kernels = None
    if profile:
        kernels = profile_kernels(B, ctx, (j0, n, n), (x, g, e, m), steps, warmup + steps, wl.rbgs_seed, per_el,
                                  k_global / world, flush)
    B.def_destroy(ctx)
    del x, g, e, m
    torch.cuda.empty_cache()
    return ms, launches, wl.W * d_global, alg_bytes, kernels, per_step


def bench_graph_replay(B, WL, wl, replays=5):
    """The workload's whole loop of steps (each with its own step number) recorded once into a CUDA
    graph and replayed: what a launch-bound tiny model costs per step when the host is out of the way."""
    import torch
    dev = torch.device("cuda")
    ctx = B.def_create(wl.d, wl.W, wl.k, wl.variant, wl.lr, wl.momentum, (wl.lam, 0.0))
    x = WL.initial_params(wl, dev)
    e, m = WL.zeros_state(wl, dev)
    if wl.momentum == 0.0:
        m = None
    g = WL.gradients(wl, 0, dev)
    B.def_step(ctx, x, g, e, m, 0, wl.rbgs_seed)            # the first call (device query) stays outside the capture
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        B.def_set_stream(ctx, side)
        with torch.cuda.graph(graph, stream=side):
            for t in range(wl.steps):
                B.def_step(ctx, x, g, e, m, t, wl.rbgs_seed)
        B.def_set_stream(ctx, None)
    graph.replay()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(replays):
        graph.replay()
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / (replays * wl.steps)
    B.def_destroy(ctx)
    del graph, x, g, e, m
    torch.cuda.empty_cache()
    return ms


def bench_aux(B, WL, wl, reps=5):
    """Device time of the helpers around the step on the same workload: the detach point
    (Algorithm 1's detach step), DEF's returned model and the distances of Eq. 9."""
    import torch
    dev = torch.device("cuda")
    W, d = wl.W, wl.d
    ctx = B.def_create(d, W, wl.k, WL.VARIANT_DEF, wl.lr, wl.momentum, (wl.lam, 0.0))
    x = WL.initial_params(wl, dev)
    e = WL.gradients(wl, 0, dev)                      # any finite values
    z = torch.empty(W, d, dtype=torch.float32, device=dev)
    y = torch.empty(d, dtype=torch.float32, device=dev)
    st = torch.zeros(3, dtype=torch.float64, device=dev)
    g = WL.gradients(wl, 1, dev)
    m = torch.zeros(W, d, dtype=torch.float32, device=dev)
    counter = [0]

    def fused():
        counter[0] += 1
        B.def_step_detach(ctx, x, g, e, m, z, counter[0], wl.rbgs_seed)

    ops = [("def_step_detach", fused, 24 * W * d + 4 * d + 8 * wl.k),
           ("def_detach", lambda: B.def_detach(ctx, x, e, z), 8 * W * d + 4 * d),
           ("def_output", lambda: B.def_output(ctx, x, e, y), 4 * W * d + 8 * d),
           ("def_stats", lambda: B.def_stats(ctx, e, st), 4 * W * d)]
    out = []
    for name, fn, nbytes in ops:
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / reps
        out.append({"op": name, "ms": ms, "algorithmic_bytes": nbytes, "GB/s": nbytes / (ms * 1e-3) / 1e9})
    B.def_destroy(ctx)
    # Algorithm 1 as printed, without the momentum buffers: 12 B per gradient element
    ctx0 = B.def_create(d, W, wl.k, WL.VARIANT_DEF, wl.lr, 0.0, (wl.lam, 0.0))
    for t in range(3):
        B.def_step(ctx0, x, g, e, None, t, wl.rbgs_seed)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for t in range(reps):
        B.def_step(ctx0, x, g, e, None, 3 + t, wl.rbgs_seed)
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / reps
    nbytes = 12 * W * d + 8 * wl.k
    out.append({"op": "def_step without momentum", "ms": ms, "algorithmic_bytes": nbytes, "GB/s": nbytes / (ms * 1e-3) / 1e9})
    B.def_destroy(ctx0)
    del x, e, z, y, g, m
    torch.cuda.empty_cache()
    return out


def available_host_bytes():
    avail = None
    try:
        with open("/proc/meminfo") as fh:
            for line in fh:
                if line.startswith("MemAvailable:"):
                    avail = int(line.split()[1]) * 1024
    except OSError:
        pass
    for path in ("/sys/fs/cgroup/memory.max", "/sys/fs/cgroup/memory/memory.limit_in_bytes"):
        try:
            txt = open(path).read().strip()
            if txt != "max":
                lim = int(txt)
                cur = 0
                for cpath in ("/sys/fs/cgroup/memory.current", "/sys/fs/cgroup/memory/memory.usage_in_bytes"):
                    try:
                        cur = int(open(cpath).read().strip())
                        break
                    except OSError:
                        pass
                avail = min(avail, lim - cur) if avail is not None else lim - cur
        except (OSError, ValueError):
            pass
    return avail


def bench_e2e(B, WL, wl, steps, warmup, dist, world, rank):
    """The same step through def_step_columns_host: every tensor starts and ends in pinned host
    memory, host<->device copies inside the timed region (host wall clock around blocking calls)."""
    import torch
    need = 4 * (3 * wl.W + 1) * wl.d * 1.15
    avail = available_host_bytes()
    note = None
    cols = wl.d
    if avail is not None and need * max(1, world if dist is not None else 1) > 0.6 * avail:
        cols = int(0.6 * avail / max(1, world) / (4 * (3 * wl.W + 1) * 1.15)) // 4 * 4
        cols = max(4, min(cols, wl.d))
        note = "host memory holds %d of %d columns per rank; e2e measured on that column range" % (cols, wl.d)
    d_global = wl.d * world
    k_global = max(1, d_global // wl.ratio)
    ctx = B.def_create(d_global, wl.W, k_global, wl.variant, wl.lr, wl.momentum, (wl.lam, 0.0))
    x = torch.empty(cols, dtype=torch.float32, pin_memory=True)
    g = torch.empty(wl.W, cols, dtype=torch.float32, pin_memory=True)
    e = torch.empty(wl.W, cols, dtype=torch.float32, pin_memory=True)
    m = torch.empty(wl.W, cols, dtype=torch.float32, pin_memory=True)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(77 + rank)
    row = torch.empty(cols, dtype=torch.float32, device="cuda")
    x.copy_(row.normal_(0.0, 0.05, generator=gen))
    for w in range(wl.W):                       # inputs drawn on the device, then parked in host memory
        g[w].copy_(row.normal_(0.0, wl.sigma or 0.01, generator=gen))
    e.zero_()
    m.zero_()
    del row
    j0 = rank * wl.d
    for t in range(warmup):
        B.def_step_columns_host(ctx, j0, cols, cols, x, g, e, m, t, wl.rbgs_seed)
    _barrier(dist)
    t0 = time.perf_counter()
    for t in range(steps):
        B.def_step_columns_host(ctx, j0, cols, cols, x, g, e, m, warmup + t, wl.rbgs_seed)
    torch.cuda.synchronize()
    sec = time.perf_counter() - t0
    _barrier(dist)
    sec = _max_over_ranks(dist, sec)
    B.def_destroy(ctx)
    out = {"value": world * wl.W * cols * steps / sec, "unit": UNIT,
           "h2d_bytes_per_step": 4 * (3 * wl.W + 1) * cols, "d2h_bytes_per_step": 4 * (2 * wl.W + 1) * cols,
           "steps": steps, "ms_per_step": 1e3 * sec / steps, "api": "def_step_columns_host (pinned host tensors)"}
    if note:
        out["note"] = note
    return out


ORACLE_SAMPLE_COLUMNS = 8_000_000     # leading columns of the workload both CPU legs step over


def oracle_time(o, wl, steps, warmup, n):
    """Times one build of the CPU oracle (as it stands) on columns [0, n) of the workload, all W
    workers: `warmup` untimed steps (they also fault the pages in), then `steps` timed ones.
    Returns (elements/s, seconds, threads used)."""
    import numpy as np
    rng = np.random.default_rng(0)
    d, W, k = wl.d, wl.W, wl.k
    n = int(min(n, d))
    g = ((wl.sigma or 0.01) * rng.standard_normal((W, n), dtype=np.float32)).astype(np.float32)
    x, e, m = np.zeros(n, np.float32), np.zeros((W, n), np.float32), np.zeros((W, n), np.float32)
    cols = None if n == d else np.arange(n, dtype=np.int64)

    def run(t):
        o.step(x, g, e, m, d=d, k=k, s=o.block_start(wl.rbgs_seed, t, d), eta=wl.lr, mu=wl.momentum, cols=cols)

    for t in range(warmup):
        run(t)
    t0 = time.perf_counter()
    for t in range(steps):
        run(warmup + t)
    sec = time.perf_counter() - t0
    return W * n * steps / sec, sec, o.threads()


def cpu_baseline(wl, steps_all, warmup_all, steps_one=8, warmup_one=1, n=ORACLE_SAMPLE_COLUMNS):
    """The oracle on the host cores, both builds of the one source on the same sample with the
    same protocol: OpenMP over the coordinate loops (all cores; the headline figure) and the
    plain single-threaded build."""
    import oracle
    n = int(min(n, wl.d))
    v_all, sec_all, cores = oracle_time(oracle.all_cores(), wl, steps_all, warmup_all, n)
    v_one, sec_one, one = oracle_time(oracle.default(), wl, steps_one, warmup_one, n)
    sample = ("each step = one oracle step on columns [0, %d) of d = %d, all W = %d workers; %d warm-up + %d timed "
              "steps on %d threads (%.1f s), %d + %d on 1 thread (%.1f s)"
              % (n, wl.d, wl.W, warmup_all, steps_all, cores, sec_all, warmup_one, steps_one, sec_one))
    return {"value": v_all, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
            "seconds": sec_all, "steps": steps_all,
            "one_core": {"value": v_one, "unit": UNIT, "cores": one, "seconds": sec_one, "steps": steps_one},
            "host_cores": os.cpu_count()}


def run_reference(args):
    """The reference arm: the CPU oracle on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from paper_2004_05298_b200 import workloads as WL
    wl = WL.get(args.cfg)
    base = cpu_baseline(wl, args.steps, args.warmup, n=args.reference_columns)
    line = {
        "impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * base["seconds"] / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": workload_config(wl, 1, "single"),
        "cpu_baseline": base,
        "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(wl, world, sharding):
    from paper_2004_05298_b200 import workloads as WL
    big = wl.algorithmic_bytes_per_step() >= 1e9
    cfg = {"workload": "cfg%d %s: d=%d per GPU, W=%d per GPU, k=d/%d, %s, momentum %.1f, lr %.2f, fp32"
                       % (wl.cfg, wl.name, wl.d, wl.W, wl.ratio, WL.VARIANT_NAMES[wl.variant], wl.momentum, wl.lr),
           "variant": WL.VARIANT_NAMES[wl.variant],
           "l2": ("inputs larger than L2 (%.1f GB per GPU); no flush" % (wl.algorithmic_bytes_per_step() * 0.8 / 1e9))
           if big else "L2 flushed between steps (384 MB buffer rewritten)"}
    if sharding == "rows":
        cfg.update({"d": wl.d, "W": wl.W * world, "k": wl.k,
                    "parallelism": "workers (rows) sharded over %d GPU(s): W = %d per GPU, K = %d workers in all, NCCL "
                                   "all-reduce of the k = %d block sums per step on a side stream" % (world, wl.W, wl.W * world, wl.k)})
    elif sharding == "columns":
        cfg.update({"d": wl.d * world, "W": wl.W, "k": max(1, wl.d * world // wl.ratio),
                    "parallelism": "columns sharded over %d GPU(s), no collective" % world})
    else:
        cfg.update({"d": wl.d, "W": wl.W, "k": wl.k, "parallelism": "one GPU holds all W workers (no collective)"})
    return cfg


def roofline_of(kernels, step_gbs, alg_bytes, launches_per_step, peak, peak_kind, cfg=None):
    """The roofline object of the JSON line: the dominant kernel against the measured HBM peak."""
    top = max(kernels, key=lambda kk: kk["ms_per_launch"] * kk["launches"])
    achieved = top["GB/s"] if top["GB/s"] is not None else step_gbs
    traffic = None
    per_element = NCU_TRAFFIC_BYTES_PER_ELEMENT.get(cfg)
    if (per_element is not None and NCU_TRAFFIC_KERNEL_SHA256 == _kernel_hash()
            and top["algorithmic_bytes_per_launch"] and top["kernel"] == "def_step_stream_kernel"):
        traffic = per_element * top["algorithmic_bytes_per_launch"] / 20.0
    return {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "traffic": traffic, "peak_kind": "of %s" % peak_kind, "frac_of_8000_nominal": achieved / 8000.0,
            "kernel": top["kernel"], "algorithmic_bytes_per_launch": top["algorithmic_bytes_per_launch"],
            "launch_ms": top["ms_per_launch"],
            "whole_step": {"GB/s": step_gbs, "frac": step_gbs / peak, "frac_of_8000_nominal": step_gbs / 8000.0,
                           "algorithmic_bytes_per_step": alg_bytes, "launches_per_step": launches_per_step},
            "kernels": kernels,
            "note": "per-kernel times from a second pass of the same steps with each launch bracketed by "
                    "CUDA events on the launching stream; whole_step is the timed region itself"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cfg", type=int, default=5, choices=[1, 2, 3, 4, 5],
                    help="workload to time (default 5, the largest; smaller ones are for profiling)")
    ap.add_argument("--sharding", default="auto", choices=["auto", "single", "rows", "columns"],
                    help="auto (default): one GPU runs def_step on all W workers; N > 1 GPUs cut the workers (rows) across "
                         "ranks and all-reduce the k block sums (NCCL).  rows: that path, also on one GPU (a one-rank NCCL "
                         "group).  columns: each rank holds a column range of every tensor, no collective")
    ap.add_argument("--reference-columns", type=int, default=ORACLE_SAMPLE_COLUMNS,
                    help="--impl reference: leading columns of the workload every oracle step runs over")
    ap.add_argument("--no-side-stream", action="store_true",
                    help="rows: keep the all-reduce and the update on the context's stream, behind the streaming kernel")
    ap.add_argument("--aux", action="store_true",
                    help="with --no-extras: still time the helpers (detach, output, stats, step with fused detach)")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the other workloads, the end-to-end leg and the CPU baseline")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    from paper_2004_05298_b200 import binding as B
    from paper_2004_05298_b200 import workloads as WL

    dist, world, rank, local = _dist_setup(args.gpus)
    sharding = args.sharding
    if sharding == "auto":
        sharding = "single" if world == 1 else "rows"
    if sharding == "single" and world > 1:
        raise SystemExit("--sharding single needs one GPU")
    if sharding == "columns" and world == 1:
        sharding = "single"
    wl = WL.get(args.cfg)
    peak, peak_kind = _measured_peak()
    sampler = ClockSampler(local)
    line = {"metric": METRIC, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": workload_config(wl, world, sharding)}

    if sharding == "rows":
        import torch.distributed as tdist
        own_group = dist is None
        if own_group:                                      # one rank: still a real NCCL group
            tdist.init_process_group("nccl", init_method="tcp://127.0.0.1:29581", rank=0, world_size=1,
                                     device_id=torch.device("cuda", 0))
        side = not args.no_side_stream
        if not side:
            line["config"]["parallelism"] = line["config"]["parallelism"].replace("on a side stream", "on the step's own stream")
        ms, launches, elements, alg_bytes, kernels, per_step = bench_rows(B, WL, wl, args.steps, args.warmup, dist, world, rank,
                                                                          sampler, side_stream=side, profile=True)
        clocks = sampler.finish()
        step_gbs = alg_bytes * args.steps / (ms * 1e-3) / 1e9
        line.update({"value": elements * args.steps / (ms * 1e-3), "ms_per_step": ms / args.steps, **step_spread(per_step),
                     "gpu_launches": launches, "clocks": clocks,
                     "roofline": roofline_of(kernels, step_gbs, alg_bytes, launches / args.steps, peak, peak_kind,
                                            cfg=wl.cfg if wl.ratio == WL.get(wl.cfg).ratio and wl.momentum != 0.0 else None)})
        if args.aux or not args.no_extras:
            ms_z, _, _, bytes_z, _, per_z = bench_rows(B, WL, wl, min(args.steps, 10), 3, dist, world, rank, None,
                                                       side_stream=side, detach=True)
            n_z = min(args.steps, 10)
            line["aux"] = [{"op": "def_step_rows with the fused detach output", "ms": ms_z / n_z, "algorithmic_bytes": bytes_z,
                            "GB/s": bytes_z * n_z / (ms_z * 1e-3) / 1e9, **step_spread(per_z)}]
        if not args.no_extras:
            line["e2e"] = bench_rows_e2e(B, WL, wl, max(1, min(args.steps, 3)), 1, dist, world, rank)
            if world == 1:
                line["cpu_baseline"] = cpu_baseline(wl, 20, 1)
        if own_group or dist is not None:
            tdist.destroy_process_group()
        if rank == 0:                                      # last, after whatever the communicator logs on its way out
            print(json.dumps(line), flush=True)
        return

    small = wl.algorithmic_bytes_per_step() < 1e9          # fits the L2: flush it between steps
    main_flush = torch.zeros(96 * 1024 * 1024, dtype=torch.float32, device="cuda") if small else None
    ms, launches, elements, alg_bytes, kernels, per_step = bench_workload(B, WL, wl, args.steps, args.warmup, dist, world, rank,
                                                                          sampler, flush=main_flush, profile=True)
    del main_flush
    clocks = sampler.finish()
    step_gbs = alg_bytes * args.steps / (ms * 1e-3) / 1e9
    line.update({"value": elements * args.steps / (ms * 1e-3), "ms_per_step": ms / args.steps, **step_spread(per_step),
                 "gpu_launches": launches, "clocks": clocks,
                 "roofline": roofline_of(kernels, step_gbs, alg_bytes, launches / args.steps, peak, peak_kind,
                                            cfg=wl.cfg if wl.ratio == WL.get(wl.cfg).ratio and wl.momentum != 0.0 else None)})

    if args.no_extras and args.aux and world == 1:
        line["aux"] = bench_aux(B, WL, wl)
    if not args.no_extras:
        e2e_steps = max(1, min(args.steps, 3))
        line["e2e"] = bench_e2e(B, WL, wl, e2e_steps, 1, dist, world, rank)
        if world == 1:
            per = []
            flush = torch.zeros(96 * 1024 * 1024, dtype=torch.float32, device="cuda")  # 384 MB > L2
            todo = [WL.get(c) for c in (1, 2, 3, 4)]
            todo += [WL.get(5).with_ratio(r, v) for r in WL.CFG5_RATIOS for v in WL.CFG5_VARIANTS
                     if not (r == wl.ratio and v == wl.variant)]
            for w in todo:
                small = w.algorithmic_bytes_per_step() < 1e9
                ms_w, launches_w, el_w, bytes_w, _, per_w = bench_workload(B, WL, w, w.steps, 3, None, 1, 0,
                                                                           flush=flush if small else None)
                gbs = bytes_w * w.steps / (ms_w * 1e-3) / 1e9
                resident = None
                if small:      # the whole state fits the L2: also the back-to-back time without a flush ("effective")
                    ms_r, _, _, _, _, per_r = bench_workload(B, WL, w, w.steps, 3, None, 1, 0, flush=None)
                    resident = {"ms_per_step": ms_r / w.steps, **step_spread(per_r),
                                "effective_GB/s": bytes_w * w.steps / (ms_r * 1e-3) / 1e9,
                                "graph_replay_ms_per_step": bench_graph_replay(B, WL, w),
                                "note": "state stays in the 126 MB L2 between steps: not an HBM figure; graph_replay = the "
                                        "loop of steps recorded into one CUDA graph and replayed"}
                per.append({"cfg": w.cfg, "name": w.name, "ratio": w.ratio, "variant": WL.VARIANT_NAMES[w.variant],
                            "steps": w.steps, "ms_per_step": ms_w / w.steps, **step_spread(per_w),
                            "elements_per_s": el_w * w.steps / (ms_w * 1e-3),
                            "GB/s": gbs, "frac_of_measured_peak": gbs / peak, "frac_of_8000_nominal": gbs / 8000.0,
                            "launches_per_step": launches_w / w.steps, "l2_resident": resident,
                            "l2": "flushed between steps" if small else "inputs larger than L2"})
            del flush
            line["aux"] = bench_aux(B, WL, wl)
            line["per_config"] = per
            line["per_config_note"] = ("EF, DEF and DEF-A run the same kernels given the gradients: the variant changes only "
                                       "where the caller evaluates them and the returned model")
            line["cpu_baseline"] = cpu_baseline(wl, 20, 1)
    if dist is not None:
        dist.destroy_process_group()
    if rank == 0:                                          # last, after whatever the communicator logs on its way out
        print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()
