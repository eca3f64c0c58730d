"""Builds libemaslice.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libemaslice.so")
SOURCES = ["slice.cpp", "copy_kernels.cu", "layer_kernel.cu", "noalloc.cu"]
HEADERS = ["kernels.h", "ptx.cuh", "attention_tiles.cuh", os.path.join("..", "..", "include", "emaslice.h")]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS] + [os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps)


RESOURCES = os.path.join(HERE, "libemaslice.resources.txt")   # ptxas' report of the last build (git-ignored)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build() and os.path.exists(RESOURCES):
        return LIB
    cmd = [_nvcc(), "-std=c++17", "-O3", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
           "-Xcompiler", "-fPIC,-Wall,-Wno-unused-function", "-Xptxas", "-v", "-shared", "-o", LIB]
    cmd += [os.path.join(CSRC, f) for f in SOURCES]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed building libemaslice.so")
    with open(RESOURCES, "w") as f:
        f.write(res.stdout + res.stderr)
    return LIB


def kernel_resources() -> dict:
    """What ptxas reported for every kernel of the last build: registers per thread, bytes of stack
    frame, bytes of spill stores and loads, keyed by the kernel's (mangled) name. The layer kernel runs
    352 threads per CTA at the register limit of one CTA per SM; a change that makes it spill, or
    that makes the compiler keep a copy of its 1 KB parameter block on every thread's stack, costs
    several per cent of its bandwidth, and this report is where that shows without a GPU."""
    import re
    build()
    out, name = {}, None
    with open(RESOURCES) as f:
        for line in f:
            m = re.search(r"Compiling entry function '([^']+)'", line)
            if m:
                name = m.group(1)
                out[name] = {}
                continue
            if name is None:
                continue
            m = re.search(r"(\d+) bytes stack frame, (\d+) bytes spill stores, (\d+) bytes spill loads", line)
            if m and "stack" not in out[name]:
                out[name].update(stack=int(m.group(1)), spill_stores=int(m.group(2)), spill_loads=int(m.group(3)))
            m = re.search(r"Used (\d+) registers", line)
            if m:
                out[name]["registers"] = int(m.group(1))
                name = None
    return out


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
