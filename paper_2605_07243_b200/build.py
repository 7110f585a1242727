"""Build the C-ABI CUDA library in-tree with nvcc for sm_100a.

    python -m paper_2605_07243_b200.build [--force] [--verbose] [--variant test|checked] [--all]

The shared object lands beside this file (libspecblock.so); nothing is cached elsewhere.
Two more builds of the same sources exist for the tests (`--variant`, or `--all` for all three):
  test     libspecblock_test.so, -DSB_TEST_KERNELS: adds the mma.sync and one-warp-per-row attention
           kernels (independent cross-checks of the tcgen05 kernels), the environment switches that
           force a kernel variant, and a kernel that lets a bounded device wait run out;
  checked  libspecblock_checked.so, -DSB_CHECKED: every computed page id, cache slot, query/output row and
           workspace offset is verified before use and reported as SB_ERR_BOUNDS instead of touching memory
           (this pool has no compute-sanitizer; this build and canary-padded buffers stand in for it).
The library proper has one attention backend and reads no environment variable.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libspecblock.so")
VARIANTS = {
    None: (LIB, []),
    "test": (os.path.join(_HERE, "libspecblock_test.so"), ["-DSB_TEST_KERNELS"]),
    "checked": (os.path.join(_HERE, "libspecblock_checked.so"), ["-DSB_CHECKED", "-rdc=true"]),
}
INCLUDE = os.path.join(os.path.dirname(_HERE), "include")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
    "-Xcompiler", "-fPIC", "--shared", "-Xcompiler", "-Wall",
    "--threads", "0",   # source files compiled in parallel
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale(lib=None):
    lib = lib or LIB
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(INCLUDE, "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, variant=None) -> str:
    lib, defines = VARIANTS[variant]
    if not force and not _stale(lib):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = lib + ".tmp%d" % os.getpid()
    cmd = [nvcc] + NVCC_FLAGS + defines + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + sources()
    subprocess.check_call(cmd)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    _variant = sys.argv[sys.argv.index("--variant") + 1] if "--variant" in sys.argv else None
    for _v in (list(VARIANTS) if "--all" in sys.argv else [_variant]):
        print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, variant=_v))
