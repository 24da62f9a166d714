"""Build and run csrc/design_variants.cu: device times of design alternatives for the step's
kernels (flat stream, cache hints, 256-bit accesses, persistent grid, column walk, bulk async
copies, ways of obtaining the block start, block-kernel register budgets) on one B200.

    python -m paper_2004_05298_b200.design_variants [--d D] [--W W] [--ratio R] [--reps N] [--only substring]

Prints a markdown table (CUDA-event times, GB/s from the bytes each variant has to move).
The program is a measuring aid beside the library, not part of it."""
import os
import subprocess
import sys

from . import build as _build

HERE = os.path.dirname(os.path.abspath(__file__))
SOURCE = os.path.join(_build.CSRC, "design_variants.cu")
BINARY = os.path.join(HERE, "design_variants.bin")


def build(force=False):
    """nvcc the program for sm_100a (cross-compiles without a GPU); returns the binary's path."""
    deps = [SOURCE, os.path.join(_build.CSRC, "def_kernels.cuh")]
    if not force and os.path.exists(BINARY) and all(os.path.getmtime(f) <= os.path.getmtime(BINARY) for f in deps):
        return BINARY
    tmp = BINARY + ".tmp.%d" % os.getpid()
    cmd = [_build._nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-cudart", "static", "-I", _build.INCLUDE, SOURCE, "-o", tmp]
    proc = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    if proc.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + proc.stdout)
    os.replace(tmp, BINARY)
    return BINARY


if __name__ == "__main__":
    sys.exit(subprocess.call([build()] + sys.argv[1:]))
