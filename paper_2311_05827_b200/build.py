"""Builds the CUDA library in-tree with nvcc for sm_100a (``libaccept.so`` beside this file).

Besides the product there are two tests-only variants of the same sources (never loaded by the binding
unless a test asks for them):
  bounds  -DACCEPT_BOUNDS_CHECK: every access of a kernel to caller memory is checked against the byte
          ranges of the call, counted and skipped when outside (``libaccept_bounds.so``);
  stall   -DACCEPT_TEST_COPY_STALL: the staged batch-group encoder announces bytes that never arrive, so
          its bounded waits run out after 2 ms (``libaccept_stall.so``).
"""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libaccept.so")
SOURCES = [os.path.join(CSRC, "accept_api.cu")]
DEPENDS = sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cu", ".cuh"))) + [
    os.path.join(os.path.dirname(HERE), "include", "accept.h")]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-fmad=false",            # no FMA contraction: every fp32 operation rounds on its own
    "-shared", "-Xcompiler", "-fPIC",
]

VARIANTS = {
    "bounds": (os.path.join(HERE, "libaccept_bounds.so"), ["-DACCEPT_BOUNDS_CHECK"]),
    "stall": (os.path.join(HERE, "libaccept_stall.so"), ["-DACCEPT_TEST_COPY_STALL"]),
}


def _stale(lib: str) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(s) > t for s in DEPENDS)


def needs_build() -> bool:
    return _stale(LIB)


def _command(lib: str, defines, verbose: bool):
    nvcc = os.environ.get("NVCC", "nvcc")
    return [nvcc] + NVCC_FLAGS + list(defines) + (["-Xptxas", "-v"] if verbose else []) + ["-o", lib] + SOURCES


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build():
        return LIB
    subprocess.run(_command(LIB, [], verbose), check=True)
    return LIB


def build_variant(name: str, force: bool = False) -> str:
    """Builds (if stale) and returns the path of a tests-only variant."""
    lib, defines = VARIANTS[name]
    if force or _stale(lib):
        subprocess.run(_command(lib, defines, False), check=True)
    return lib


def build_all(force: bool = False) -> None:
    """The product and the tests-only variants, compiled side by side."""
    jobs = []
    if force or needs_build():
        jobs.append(subprocess.Popen(_command(LIB, [], False)))
    for lib, defines in VARIANTS.values():
        if force or _stale(lib):
            jobs.append(subprocess.Popen(_command(lib, defines, False)))
    failed = [j.args for j in jobs if j.wait() != 0]
    if failed:
        raise subprocess.CalledProcessError(1, failed[0])


if __name__ == "__main__":
    import sys
    if "--all" in sys.argv:
        build_all(force="--force" in sys.argv)
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
