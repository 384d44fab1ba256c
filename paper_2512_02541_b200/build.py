"""Builds libavggt.so (the C-ABI library) in-tree with nvcc for sm_100a."""

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libavggt.so")
# A second library for one GPU test: the same sources with a 0.5 ms limit on device-side waits and one K tile
# left out by the first thread block of the attention kernel, so that the time-out path can be exercised
# without hanging or faulting anything.  The product library never contains that switch.
WAIT_TEST_LIB = os.path.join(HERE, "libavggt_waittest.so")
WAIT_TEST_DEFINES = ["-DAVGGT_TEST_SKIP_K_LOAD=1", "-DAVGGT_WAIT_LIMIT_NS=500000ull"]
SOURCES = ["api.cu", "build_kv.cu", "build_kv_noalloc.cu", "global_attn.cu", "project_kv.cu"]
HEADERS = ["internal.h", "plan.h", "ptx.cuh", "tmap.h", os.path.join("..", "..", "include", "avggt.h")]


def _nvcc():
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: libavggt.so cannot be built")


def needs_build(lib=None):
    lib = lib or LIB
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS] + [os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps)


def _compile(lib, defines, verbose):
    cmd = [
        _nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
        "-Xcompiler", "-fPIC", "-shared", "-cudart", "static",
        "-Xptxas", "-v" if verbose else "-warn-spills",
        "-o", lib,
    ] + list(defines) + [os.path.join(CSRC, s) for s in SOURCES]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if verbose:
        sys.stderr.write(res.stdout + res.stderr)
    return lib


def build(force=False, verbose=False):
    """Compile every CUDA source into one shared library.  Returns its path."""
    if not force and not needs_build():
        return LIB
    return _compile(LIB, [], verbose)


def build_wait_test(force=False, verbose=False):
    """The wait-limit test's library (see WAIT_TEST_LIB).  Returns its path."""
    if not force and not needs_build(WAIT_TEST_LIB):
        return WAIT_TEST_LIB
    return _compile(WAIT_TEST_LIB, WAIT_TEST_DEFINES, verbose)


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
    print(build_wait_test(force=True))
