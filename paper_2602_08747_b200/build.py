"""Builds libpard.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libpard.so")
SOURCES = ["pard_pipeline.cu", "pard_plan.cu", "pard_policy.cu", "pard_goodput.cu", "pard_host.cu",
           "pard_static.cu", "pard_wait.cu", "pard_priority.cu", "pard_qdelay.cu", "pard_replay.cu"]
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
         "-Xcompiler", "-fPIC", "-shared", "-cudart", "static"]


def _inputs():
    files = [os.path.join(CSRC, s) for s in SOURCES]
    files.append(os.path.join(CSRC, "pard_internal.h"))
    files.append(os.path.join(CSRC, "pard_plan_internal.cuh"))
    files.append(os.path.join(ROOT, "include", "pard.h"))
    return files


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(f) > t for f in _inputs())


def build(force: bool = False, verbose: bool = False) -> str:
    if not (force or stale()):
        return LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = LIB + ".tmp%d" % os.getpid()
    cmd = [nvcc] + FLAGS + (["-Xptxas", "-v"] if verbose else []) + \
          ["-I", os.path.join(ROOT, "include"), "-I", CSRC, "-o", tmp] + \
          [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.check_call(cmd)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
