"""Host-side pieces of bench.py that need no GPU: the split of a step's bytes between the two
kernels, and the reference arm (the CPU oracle timed on a bounded sample), which must print
the contract's JSON line."""
import importlib.util
import json
import os
import random
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _bench():
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_touched_columns_against_brute_force():
    bench = _bench()
    rnd = random.Random(1)
    for _ in range(1500):
        d = rnd.randint(1, 9000); k = rnd.randint(1, d); s = rnd.randrange(d)
        j0 = rnd.randrange(d); n = rnd.randint(1, d - j0)
        block = {(s + i) % d for i in range(k)}
        tiles = {(j - j0) // bench.TILE for j in range(j0, j0 + n) if j in block}
        want = sum(min(bench.TILE, n - t * bench.TILE) for t in tiles)
        assert bench.touched_columns(d, k, s, j0, n) == want, (d, k, s, j0, n)


def test_reference_arm_prints_the_contract_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2",
                          "--warmup", "3", "--reference-columns", "200000"], capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "elements/s" and line["higher_is_better"] is True
    assert line["value"] > 0 and line["steps"] == 2 and line["vs_baseline"] is None
    base = line["cpu_baseline"]
    assert base["kind"] == "oracle" and base["cores"] >= 1 and base["value"] == line["value"]
    assert base["one_core"]["cores"] == 1 and base["one_core"]["value"] > 0     # the plain build, same sample
    assert "[0, 200000)" in base["sample"]
    assert line["e2e"]["value"] == line["value"] and line["e2e"]["h2d_bytes_per_step"] == 0
    assert "cfg5" in line["config"]["workload"]
    # other ranks of a multi-process launch do no work and print nothing
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                         capture_output=True, text=True, timeout=120, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_config_names_the_sharding_that_ran():
    bench = _bench()
    from paper_2004_05298_b200 import workloads as WL
    wl = WL.get(5)
    one = bench.workload_config(wl, 1, "single")
    rows = bench.workload_config(wl, 8, "rows")
    cols = bench.workload_config(wl, 8, "columns")
    assert one["W"] == 16 and one["d"] == wl.d and "no collective" in one["parallelism"]
    assert rows["W"] == 128 and rows["d"] == wl.d and rows["k"] == wl.k          # K = 16 N workers, full model per GPU
    assert "NCCL all-reduce" in rows["parallelism"] and "8 GPU" in rows["parallelism"]
    assert cols["W"] == 16 and cols["d"] == 8 * wl.d and cols["k"] == 8 * wl.d // wl.ratio
    assert all("model" not in c for c in (one, rows, cols))                       # workload keys, no model keys
    assert "flushed" in bench.workload_config(WL.get(1), 1, "single")["l2"]


def test_roofline_object_and_step_spread():
    bench = _bench()
    kernels = [{"kernel": "def_step_stream_kernel", "launches": 4, "ms_per_launch": 6.0, "algorithmic_bytes_per_launch": 42e9, "GB/s": 7000.0},
               {"kernel": "def_step_block_kernel", "launches": 4, "ms_per_launch": 0.2, "algorithmic_bytes_per_launch": 1.4e9, "GB/s": 7000.0}]
    r = bench.roofline_of(kernels, 6900.0, 44e9, 2.0, 6550.0, "measured", cfg=5)
    assert bench.roofline_of(kernels, 6900.0, 44e9, 2.0, 6550.0, "measured", cfg=4)["traffic"] is None   # no capture for that workload
    assert r["bound"] == "hbm" and r["kernel"] == "def_step_stream_kernel" and r["unit"] == "GB/s"
    assert abs(r["frac"] - 7000.0 / 6550.0) < 1e-12 and r["peak_kind"] == "of measured"
    assert r["traffic"] is None or abs(r["traffic"] - bench.NCU_TRAFFIC_BYTES_PER_ELEMENT[5] * 42e9 / 20.0) < 1.0
    # the traffic figure is only reported for the kernel file it was captured on
    assert (r["traffic"] is not None) == (bench.NCU_TRAFFIC_KERNEL_SHA256 == bench._kernel_hash())
    assert bench.step_spread([3.0, 1.0, 2.0]) == {"ms_per_step_median": 2.0, "ms_per_step_min": 1.0}
    assert bench.step_spread(None) == {}
