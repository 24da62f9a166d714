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

# DRAM traffic of one def_step_stream_kernel launch from an ncu capture
# (dram__bytes_read.sum + dram__bytes_write.sum), as bytes per gradient element, and the
# hash of the kernel source the capture was taken on.  Reported only while the source is
# unchanged (see profiles/).
NCU_TRAFFIC_BYTES_PER_ELEMENT = 19.42
NCU_TRAFFIC_KERNEL_SHA256 = "deb13c2113f9bab04b32bee152010e98657aa46f3d5ca502d764c15853436536"


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


def time_steps(B, ctx, shard, tensors, steps, warmup, seed, dist=None, flush=None, sample_clocks=None, step_fn=None):
    """Device time of `steps` steps.  Without `flush`: one event pair around the whole loop,
    launches back to back.  With `flush` (a buffer larger than the L2 that is rewritten
    between iterations): one event pair per step, summed."""
    import torch
    j0, n, ld = shard
    x, g, e, m = tensors
    if step_fn is None:
        def step_fn(t):
            B.def_step_columns(ctx, j0, n, ld, x, g, e, m, t, seed)
    for t in range(warmup):
        step_fn(t)
    _barrier(dist)
    launches0 = B.def_launch_count(ctx)
    if sample_clocks is not None:
        sample_clocks.start()
    if flush is None:
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record()
        for t in range(steps):
            step_fn(warmup + t)
        end.record()
        torch.cuda.synchronize()
        ms = start.elapsed_time(end)
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
        ms = sum(a.elapsed_time(b) for a, b in pairs)
    _barrier(dist)
    launches = B.def_launch_count(ctx) - launches0
    return _max_over_ranks(dist, ms), launches


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


def profile_kernels(B, ctx, shard, tensors, steps, first_step, seed, per_el, k_share, flush=None):
    """Per-kernel device time over `steps` more steps (each launch bracketed by events inside the
    library and waited for), with the algorithmic bytes each kernel had to move."""
    j0, n, ld = shard
    x, g, e, m = tensors
    W = ctx.W
    before = {kind: B.def_kernel_time(ctx, kind) for kind in (B.DEF_KERNEL_STREAM, B.DEF_KERNEL_BLOCK, B.DEF_KERNEL_GENERAL)}
    B.def_set_kernel_timing(ctx, True)
    bytes_stream = bytes_block = bytes_general = 0
    for t in range(steps):
        if flush is not None:
            flush.add_(1.0)
        step = first_step + t
        B.def_step_columns(ctx, j0, n, ld, x, g, e, m, step, seed)
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


def bench_rows(B, WL, wl, steps, warmup, dist, world, rank, sampler=None):
    """Workers cut across ranks (the paper's deployment): every rank holds W rows of the full model and
    a replica of x; one step = local half, NCCL all-reduce of the k block sums, apply."""
    import torch
    dev = torch.device("cuda")
    ctx = B.def_create(wl.d, wl.W, wl.k, wl.variant, wl.lr, wl.momentum, (wl.lam, 0.0))
    x = WL.initial_params(wl, dev)
    e, m = WL.zeros_state(wl, dev)
    g = WL.gradients(wl, rank, dev)
    block = torch.zeros(wl.k, dtype=torch.float32, device=dev)

    def step_fn(t):
        B.def_step_rows(ctx, x, g, e, m, block, t, wl.rbgs_seed)

    ms, launches = time_steps(B, ctx, (0, wl.d, wl.d), (x, g, e, m), steps, warmup, wl.rbgs_seed, dist, None, sampler, step_fn)
    B.def_destroy(ctx)
    del x, g, e, m
    torch.cuda.empty_cache()
    return ms, launches, world * wl.W * wl.d, 20 * wl.W * wl.d + 12 * wl.k


def bench_workload(B, WL, wl, steps, warmup, dist, world, rank, sampler=None, flush=None, profile=False):
    """Allocate a rank's shard of the workload, run, return (ms, launches, elements per step over
    all ranks, algorithmic bytes per step on this rank, per-kernel profile or None)."""
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
    ms, launches = time_steps(B, ctx, (j0, n, n), (x, g, e, m), steps, warmup, wl.rbgs_seed, dist, flush, sampler)
    per_el = 20 if wl.momentum != 0.0 else 12
    alg_bytes = per_el * wl.W * n + 8 * k_global / world
    kernels = None
    if profile:
        kernels = profile_kernels(B, ctx, (j0, n, n), (x, g, e, m), steps, warmup + steps, wl.rbgs_seed, per_el,
                                  k_global / world, flush)
    B.def_destroy(ctx)
    del x, g, e, m
    torch.cuda.empty_cache()
    return ms, launches, wl.W * d_global, alg_bytes, kernels


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


def oracle_sample_run(WL, wl, steps, warmup, budget_s):
    """Times the CPU oracle (as it stands, one thread) on a leading column range of the workload,
    sized from a short probe so that warmup + steps stay within budget_s."""
    import numpy as np
    import oracle
    rng = np.random.default_rng(0)
    d, W, k = wl.d, wl.W, wl.k

    def make(n):
        g = (wl.sigma or 0.01) * rng.standard_normal((W, n), dtype=np.float32)
        return (np.zeros(n, np.float32), g, np.zeros((W, n), np.float32), np.zeros((W, n), np.float32),
                np.arange(n, dtype=np.int64))

    def run(state, t):
        x, g, e, m, cols = state
        s = oracle.block_start(wl.rbgs_seed, t, d)
        oracle.step(x, g, e, m, d=d, k=k, s=s, eta=wl.lr, mu=wl.momentum, cols=cols if len(cols) != d else None)

    probe = make(min(d, 250_000))
    t0 = time.perf_counter(); run(probe, 0); rate = W * len(probe[4]) / (time.perf_counter() - t0)
    n = int(min(d, max(1000, rate * budget_s / (steps + warmup) / W)))
    state = make(n)
    for t in range(warmup):
        run(state, t)
    t0 = time.perf_counter()
    for t in range(steps):
        run(state, warmup + t)
    sec = time.perf_counter() - t0
    return W * n * steps / sec, sec, n


def run_reference(args):
    """The reference arm: the CPU oracle on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from paper_2004_05298_b200 import workloads as WL
    wl = WL.get(5)
    value, sec, n = oracle_sample_run(WL, wl, args.steps, args.warmup, budget_s=args.reference_budget_s)
    sample = "each step = one oracle step on columns [0, %d) of d = %d, all W = %d workers" % (n, wl.d, wl.W)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sec / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": workload_config(wl, 1),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(wl, world):
    from paper_2004_05298_b200 import workloads as WL
    return {"workload": "cfg%d %s: d=%d per GPU, W=%d, k=d/%d, %s, momentum %.1f, lr %.2f, fp32"
                        % (wl.cfg, wl.name, wl.d, wl.W, wl.ratio, WL.VARIANT_NAMES[wl.variant], wl.momentum, wl.lr),
            "d": wl.d * world, "W": wl.W, "k": max(1, wl.d * world // wl.ratio), "variant": WL.VARIANT_NAMES[wl.variant],
            "parallelism": "columns sharded over %d GPU(s), no collective" % world,
            "l2": ("inputs larger than L2 (%.1f GB per GPU); no flush" % (wl.algorithmic_bytes_per_step() * 0.8 / 1e9))
            if wl.algorithmic_bytes_per_step() >= 1e9 else "L2 flushed between steps (384 MB buffer rewritten)"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cfg", type=int, default=5, choices=[1, 2, 3, 4, 5],
                    help="workload to time (default 5, the largest; smaller ones are for profiling)")
    ap.add_argument("--sharding", default="columns", choices=["columns", "rows"],
                    help="columns (default): each rank holds a column range of every tensor, no collective; "
                         "rows: each rank holds W workers of the full model and the k block sums are all-reduced (NCCL)")
    ap.add_argument("--reference-budget-s", type=float, default=90.0,
                    help="--impl reference: CPU seconds the whole run (warm-up + steps) may take")
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
    wl = WL.get(args.cfg)
    if args.sharding == "rows":
        import torch.distributed as tdist
        if dist is None:                                   # one rank: still a real NCCL group
            tdist.init_process_group("nccl", init_method="tcp://127.0.0.1:29581", rank=0, world_size=1,
                                     device_id=torch.device("cuda", 0))
        sampler = ClockSampler(local)
        ms, launches, elements, alg_bytes = bench_rows(B, WL, wl, args.steps, args.warmup, dist, world, rank, sampler)
        clocks = sampler.finish()
        peak, peak_kind = _measured_peak()
        gbs = alg_bytes * args.steps / (ms * 1e-3) / 1e9
        cfg = workload_config(wl, world)
        cfg["parallelism"] = "workers (rows) sharded over %d GPU(s): W = %d per GPU, NCCL all-reduce of k = %d floats per step" % (world, wl.W, wl.k)
        cfg["d"], cfg["W"], cfg["k"] = wl.d, wl.W * world, wl.k
        if rank == 0:
            print(json.dumps({
                "metric": METRIC, "value": elements * args.steps / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": cfg,
                "gpu_launches": launches, "clocks": clocks,
                "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                             "traffic": None, "peak_kind": "of %s" % peak_kind, "kernel": "whole step (local half + all-reduce + apply)"}}))
        tdist.destroy_process_group()
        return
    sampler = ClockSampler(local)
    small = wl.algorithmic_bytes_per_step() < 1e9          # fits the L2: flush it between steps
    main_flush = torch.zeros(96 * 1024 * 1024, dtype=torch.float32, device="cuda") if small else None
    ms, launches, elements, alg_bytes, kernels = bench_workload(B, WL, wl, args.steps, args.warmup, dist, world, rank,
                                                                sampler, flush=main_flush, profile=True)
    del main_flush
    clocks = sampler.finish()
    peak, peak_kind = _measured_peak()
    value = elements * args.steps / (ms * 1e-3)
    step_gbs = alg_bytes * args.steps / (ms * 1e-3) / 1e9
    top = max(kernels, key=lambda kk: kk["ms_per_launch"] * kk["launches"])      # the dominant kernel
    achieved = top["GB/s"] if top["GB/s"] is not None else step_gbs
    traffic = None
    if (NCU_TRAFFIC_BYTES_PER_ELEMENT is not None and NCU_TRAFFIC_KERNEL_SHA256 == _kernel_hash()
            and top["algorithmic_bytes_per_launch"]):
        traffic = NCU_TRAFFIC_BYTES_PER_ELEMENT * top["algorithmic_bytes_per_launch"] / 20.0
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": workload_config(wl, world),
        "gpu_launches": launches, "clocks": clocks,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": traffic, "peak_kind": "of %s" % peak_kind, "frac_of_8000_nominal": achieved / 8000.0,
                     "kernel": top["kernel"], "algorithmic_bytes_per_launch": top["algorithmic_bytes_per_launch"],
                     "launch_ms": top["ms_per_launch"],
                     "whole_step": {"GB/s": step_gbs, "frac": step_gbs / peak, "frac_of_8000_nominal": step_gbs / 8000.0,
                                    "algorithmic_bytes_per_step": alg_bytes, "launches_per_step": launches / args.steps},
                     "kernels": kernels,
                     "note": "per-kernel times from a second pass of the same steps with each launch bracketed by "
                             "CUDA events on the launching stream; whole_step is the timed region itself"},
    }

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
                ms_w, launches_w, el_w, bytes_w, _ = bench_workload(B, WL, w, w.steps, 3, None, 1, 0,
                                                                    flush=flush if small else None)
                gbs = bytes_w * w.steps / (ms_w * 1e-3) / 1e9
                resident = None
                if small:      # the whole state fits the L2: also the back-to-back time without a flush ("effective")
                    ms_r, _, _, _, _ = bench_workload(B, WL, w, w.steps, 3, None, 1, 0, flush=None)
                    resident = {"ms_per_step": ms_r / w.steps, "effective_GB/s": bytes_w * w.steps / (ms_r * 1e-3) / 1e9,
                                "note": "state stays in the 126 MB L2 between steps: not an HBM figure"}
                per.append({"cfg": w.cfg, "name": w.name, "ratio": w.ratio, "variant": WL.VARIANT_NAMES[w.variant],
                            "steps": w.steps, "ms_per_step": ms_w / w.steps, "elements_per_s": el_w * w.steps / (ms_w * 1e-3),
                            "GB/s": gbs, "frac_of_measured_peak": gbs / peak, "frac_of_8000_nominal": gbs / 8000.0,
                            "launches_per_step": launches_w / w.steps, "l2_resident": resident,
                            "l2": "flushed between steps" if small else "inputs larger than L2"})
            del flush
            line["aux"] = bench_aux(B, WL, wl)
            line["per_config"] = per
            line["per_config_note"] = ("EF, DEF and DEF-A run the same kernels given the gradients: the variant changes only "
                                       "where the caller evaluates them and the returned model")
            v, sec, n = oracle_sample_run(WL, wl, 3, 1, budget_s=20.0)
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle",
                                    "sample": "3 oracle steps on columns [0, %d) of d = %d, W = %d (%.1f s)" % (n, wl.d, wl.W, sec)}
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
