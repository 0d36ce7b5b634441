"""Builds libcorun.so (sm_100a) in-tree with nvcc.  ``python -m paper_2608_14376_b200.build``"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libcorun.so")
SOURCES = ["engine.cu", "gemm.cu", "ops.cu", "attention.cu", "attention_prefill.cu", "no_alloc.cu", "sched.cu", "moe.cu", "mla_paged.cu", "mla_layer.cu", "wait_probe.cu", "microbench.cu"]
HEADERS = ["gemm.cuh", "ops.cuh", "ptx.cuh", "launch.cuh", "checks.cuh", os.path.join("..", "..", "include", "corun.h"),
           os.path.join("..", "..", "include", "corun_sched.h"), os.path.join("..", "..", "include", "corun_moe.h"),
           os.path.join("..", "..", "include", "corun_mla.h"), os.path.join("..", "..", "include", "corun_debug.h"), "moe.cuh", "mla.cuh"]
# CORUN_BUILD_DEBUG=1 in the environment compiles the kernel timelines in (-DCORUN_BUILD_DEBUG; see
# include/corun_debug.h); a marker file remembers which kind the library on disk is.
DEBUG = os.environ.get("CORUN_BUILD_DEBUG", "0") == "1"
# CORUN_CHECKED=1 compiles the kernels' index checks in (-DCORUN_CHECKED; csrc/checks.cuh)
CHECKED = os.environ.get("CORUN_CHECKED", "0") == "1"
KIND = os.path.join(HERE, "csrc", ".build_kind")


def _kind() -> str:
    return ("debug" if DEBUG else "serving") + ("+checked" if CHECKED else "")


def _nvcc() -> str:
    for c in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if c and (os.path.isabs(c) and os.path.exists(c) or not os.path.isabs(c)):
            return c
    return "nvcc"


def _sources():
    return [s for s in SOURCES if os.path.exists(os.path.join(CSRC, s))]


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    if (open(KIND).read().strip() if os.path.exists(KIND) else "serving") != _kind():
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in _sources() + HEADERS] + [os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps if os.path.exists(d))


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not stale():
        return LIB
    objs = []
    # no fast-math: the sampler's integer weights rely on separately rounded fp32 operations
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
             "-Xcompiler", "-fPIC", "-Xptxas", "-v" if verbose else "-O3"] + (["-DCORUN_BUILD_DEBUG"] if DEBUG else []) + (["-DCORUN_CHECKED"] if CHECKED else [])
    for s in _sources():
        o = os.path.join(CSRC, s.replace(".cu", ".o"))
        cmd = [_nvcc()] + flags + ["-c", os.path.join(CSRC, s), "-o", o]
        subprocess.check_call(cmd)
        objs.append(o)
    subprocess.check_call([_nvcc(), "-shared", "-o", LIB] + objs + ["-gencode", "arch=compute_100a,code=sm_100a"])
    with open(KIND, "w") as f:
        f.write(_kind())
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
