"""Build the CUDA library in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
SOURCES = [os.path.join(_HERE, "csrc", name) for name in (
    "table_q_top.cu", "table_q_high.cu", "table_q_mid.cu", "table_q_low.cu",
    "bcast_sweep.cu", "bcast_sched.cu", "bcast_simulate.cu")]
HEADERS = [os.path.join(_HERE, "csrc", name) for name in (
    "schedule_core.cuh", "schedule_fast.cuh", "schedule_tile.cuh", "table_kernel.cuh", "host_util.h")]
HEADERS.append(os.path.join(os.path.dirname(_HERE), "include", "bcast_sched.h"))
LIBRARY = os.path.join(_HERE, "libbcast_sched.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "--extended-lambda", "-Xcompiler", "-fPIC", "-cudart", "shared"]


def needs_build() -> bool:
    if not os.path.exists(LIBRARY):
        return True
    built = os.path.getmtime(LIBRARY)
    return any(os.path.getmtime(f) > built for f in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False) -> str:
    if force or needs_build():
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        tmp = LIBRARY + ".tmp.%d" % os.getpid()
        flags = NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else [])
        # one object per source, compiled side by side, then one link
        objects = [tmp + ".%d.o" % i for i in range(len(SOURCES))]
        procs = [subprocess.Popen([nvcc] + flags + ["-c", "-o", obj, src]) for src, obj in zip(SOURCES, objects)]
        codes = [proc.wait() for proc in procs]
        try:
            if any(codes):
                raise subprocess.CalledProcessError(max(codes), nvcc)
            subprocess.check_call([nvcc] + NVCC_FLAGS + ["-shared", "-o", tmp] + objects)
            os.replace(tmp, LIBRARY)
        finally:
            for obj in objects:
                if os.path.exists(obj):
                    os.remove(obj)
    return LIBRARY


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
