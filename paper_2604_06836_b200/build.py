"""Builds libstq.so (the C-ABI library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libstq.so")
SOURCES = ["stq_step_fast.cu", "stq_step_variants.cu", "stq_step_split.cu", "stq_kernels.cu", "stq_static_stats.cu",
           "stq_api.cu", "stq_policy.cpp"]
HEADERS = [os.path.join(CSRC, "stq_internal.h"), os.path.join(CSRC, "stq_step_fast.cuh"), os.path.join(os.path.dirname(HERE), "include", "stq.h")]

# -fmad=false: the code-deciding arithmetic must not be contracted; fused operations are written
# explicitly where they are wanted.
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo", "--threads", "0",
    "-fmad=false", "-Xcompiler", "-fPIC", "-shared", "-cudart", "static",
    "-diag-suppress", "177",     # unused members of the per-width constant tables
]


def nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    raise RuntimeError("nvcc not found")


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES] + HEADERS
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not stale():
        return LIB
    tmp = LIB + f".tmp{os.getpid()}"
    cmd = [nvcc(), *NVCC_FLAGS, *(["-Xptxas", "-v"] if verbose else []), "-o", tmp,
           *[os.path.join(CSRC, s) for s in SOURCES]]
    subprocess.check_call(cmd)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
