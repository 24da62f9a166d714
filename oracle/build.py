"""Compile the CPU oracle (plain C, gcc) into oracle/libdef_oracle.so.

Test infrastructure: building the checker is not using it.  The flags keep the
arithmetic exactly as written: no fast-math, no contraction of a*b+c into a fused
multiply-add by the compiler (the fused operations the oracle wants are spelled
fmaf / fma in the source).
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SOURCES = ["def_oracle.c"]
DEPENDS = ["def_oracle.c", "def_oracle_body.inc"]
LIB = os.path.join(HERE, "libdef_oracle.so")
LIB_ALL_CORES = os.path.join(HERE, "libdef_oracle_allcores.so")   # same source, coordinate loops as OpenMP parallel-for
CFLAGS = ["-O2", "-std=c11", "-fPIC", "-shared", "-ffp-contract=off", "-fno-fast-math",
          "-Wall", "-Wextra"]


def needs_build(lib=LIB):
    if not os.path.exists(lib):
        return True
    built = os.path.getmtime(lib)
    return any(os.path.getmtime(os.path.join(HERE, f)) > built for f in DEPENDS)


def build(force=False, lib=LIB, source_dir=HERE, extra_flags=()):
    """gcc the oracle; returns the path of the shared library."""
    if not force and lib in (LIB, LIB_ALL_CORES) and not needs_build(lib):
        return lib
    tmp = lib + ".tmp.%d" % os.getpid()
    cmd = ["gcc", *CFLAGS, *extra_flags, "-I", source_dir,
           *[os.path.join(source_dir, s) for s in SOURCES], "-o", tmp, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, lib)
    return lib


def build_all_cores(force=False):
    """The same source with -fopenmp: the loops over coordinates become parallel-for loops."""
    return build(force=force, lib=LIB_ALL_CORES, extra_flags=("-fopenmp",))


if __name__ == "__main__":
    print(build(force=True))
    print(build_all_cores(force=True))
